"""Lock-step comparison of the CUDA library with the CPU oracle, phase by phase.

Tolerances (stated by the target): integer outputs bit-exact; hidden states rel-L2 <= 1e-2; logits
max-abs <= 5e-2; argmax / top-k decisions must match wherever the oracle's gap to the neighbouring
logits exceeds 0.1.  After each draft the oracle's tokens are fed to both verifies; after each verify
the oracle's argmax is fed to both acceptances, so both sides commit identical tokens and their states
stay comparable.
"""
from dataclasses import dataclass, field
from typing import List, Optional

import torch

from oracle.hydra_oracle import HydraOracle, topk_desc
from synth import plant_row, planted_length

HID_TOL = 1e-2
LOGIT_TOL = 5e-2
GAP = 0.1


def split_hi_lo(x: torch.Tensor) -> torch.Tensor:
    """[2, ...] bfloat16: hi = bf16(x), lo = bf16(x - hi) of a float tensor (how the library stores bfloat16-path
    activations and cache rows)."""
    hi = x.to(torch.bfloat16)
    lo = (x.float() - hi.float()).to(torch.bfloat16)
    return torch.stack([hi, lo]).contiguous()


def split_f16(x: torch.Tensor) -> torch.Tensor:
    """[2, ...] float16: hi = f16(x), lo = f16(x - hi) of a float tensor (how the library stores q and cache rows)."""
    hi = x.to(torch.float16)
    lo = (x.float() - hi.float()).to(torch.float16)
    return torch.stack([hi, lo]).contiguous()


def kv_raw(g, which: str) -> torch.Tensor:
    """Raw view of a cache buffer in its element type (float32 on the float path, float16 hi / lo planes on the
    bfloat16 path): KV_BASE -> [layers][k,v][planes][batch][heads][seq][hd], KV_PREFIX without the layer axis."""
    m = g.model
    shape = (2, g.kv_planes, g.max_batch, m.n_heads, g.max_seq, m.head_dim)
    if which == "KV_BASE":
        shape = (m.n_layers,) + shape
    return g.get_buffer(which).view(shape)


def kv_values(g, which: str) -> torch.Tensor:
    """Cache values as float (the planes added)."""
    return kv_raw(g, which).float().sum(dim=-5)


def rel_l2(a: torch.Tensor, b: torch.Tensor) -> float:
    a, b = a.double().flatten(), b.double().flatten()
    return float((a - b).norm() / (b.norm() + 1e-30))


@dataclass
class Stats:
    steps: int = 0
    forced_amax: int = 0            # under-gap argmax differences replaced by the oracle's
    undergap_children: int = 0      # drafted children accepted through the gap rule rather than exactly
    max_logit_err: float = 0.0
    max_hidden_err: float = 0.0
    max_head_logit_err: float = 0.0
    max_kv_err: float = 0.0
    max_hprime_err: float = 0.0
    max_prefix_kv_err: float = 0.0
    n_acc: List[List[int]] = field(default_factory=list)


def check_children(o: HydraOracle, b: int, tok_g: torch.Tensor, hp: torch.Tensor, st: Stats):
    """Every drafted child of every parent against the oracle's head evaluated on the library's own inputs: its path
    tokens (so a legitimate under-gap difference upstream does not cascade) and its h' (which is compared with the
    oracle's on its own; the random-weight head MLPs amplify an input difference several times per layer, so feeding
    the oracle's h' would test that amplification, not the head kernels)."""
    t = o.tree
    for d in range(1, t.K + 1):
        for p in t.level_parents[d - 1]:
            lg = o.head_logits(d, hp, [int(tok_g[b, j]) for j in t.path[p]])
            k = len(t.children[p])
            ref = topk_desc(lg, k + 1)
            vals = [float(lg[r]) for r in ref]
            got = [int(tok_g[b, c]) for c in t.children[p]]
            assert len(set(got)) == k, "duplicate children"
            for j in range(k):
                gap_lo = vals[j - 1] - vals[j] if j > 0 else float("inf")
                gap_hi = vals[j] - vals[j + 1]
                if got[j] == ref[j]:
                    continue
                assert not (gap_lo > GAP and gap_hi > GAP), \
                    f"child {j} of parent {p} (seq {b}): {got[j]} != {ref[j]} although both gaps exceed {GAP}"
                assert abs(float(lg[got[j]]) - vals[j]) <= GAP, f"child {j} of parent {p}: token outside the gap window"
                st.undergap_children += 1


def lockstep(o: HydraOracle, g, prompts, steps: int, seed: int, plant: bool = True, kv_layers=(0,), check_heads=True,
             teacher_fn=None) -> Stats:
    """o: oracle, g: paper_2402_05109_b200.Hydra.  Runs prefill + `steps` decode steps on both."""
    st = Stats()
    B, T, K = len(prompts), o.tree.T, o.h.n_heads
    m = o.m
    o.prefill(prompts)
    g.prefill(prompts)
    g.poll_status()
    # the ancestor-or-self bitmask is an integer output: bit for bit
    mask_g = g.get_buffer("TREE_MASK")[:T].cpu().tolist()
    assert [v & ((1 << 64) - 1) for v in mask_g] == o.tree.anc_mask, "tree mask differs"
    lens = g.get_buffer("LEN")[:B].cpu().tolist()
    assert lens == o.len
    hn = g.get_buffer("H_NEW").view(g.max_batch, K + 1, m.d_model)
    for b in range(B):
        e = rel_l2(hn[b, 0].cpu(), o.h_new[b][-1])
        st.max_hidden_err = max(st.max_hidden_err, e)
        assert e <= HID_TOL, f"prefill hidden rel-L2 {e}"
        lg = o.h_new[b][-1] @ o.W("lm_head").T
        top2 = torch.topk(lg, 2).values
        root_g = int(g.get_buffer("ROOT_TOK")[b])
        if float(top2[0] - top2[1]) > GAP:
            assert root_g == o.root_tok[b]
        elif root_g != o.root_tok[b]:
            raise AssertionError("prefill root token differs under the gap; cannot continue in lock-step")
    for s in range(steps):
        tok_o = o.draft()
        tok_g = g.draft()
        g.poll_status()
        assert tok_g[:, 0].cpu().tolist() == o.root_tok
        # the hidden state the heads consumed, and (Hydra++) the extra layer's cache over the committed rows
        hp = g.get_buffer("H_PRIME").view(g.max_batch, m.d_model)
        for b in range(B):
            e = rel_l2(hp[b].cpu(), o.hprime[b])
            st.max_hprime_err = max(st.max_hprime_err, e)
            assert e <= HID_TOL, f"step {s}: h' rel-L2 {e}"
        if o.h.prefix_attn:
            pkv = kv_values(g, "KV_PREFIX")
            for b in range(B):
                L = o.len[b]
                for which, ref in ((0, o.pk[b]), (1, o.pv[b])):
                    e = rel_l2(pkv[which, b, :, :L].permute(1, 0, 2).cpu(), ref[:L])
                    st.max_prefix_kv_err = max(st.max_prefix_kv_err, e)
                    assert e <= HID_TOL, f"step {s}: prefix-layer cache rel-L2 {e}"
        if check_heads:
            tg = tok_g.cpu().long()
            hp_o = [hp[b].cpu().to(o.dtype) for b in range(B)]      # the library's h' as the oracle head's input
            for b in range(B):
                check_children(o, b, tg, hp_o[b], st)
            if o.tree.K > 0:                       # logits of the last drafted level, numerically
                d = o.tree.K
                P = o.tree.level_parents[d - 1]
                hl = g.get_buffer("HEAD_LOGITS").view(-1, m.vocab)
                shared = getattr(o.h, "medusa", False)             # sequentially independent heads: one logits row per sequence
                for b in range(B):
                    for j, p in enumerate(P):
                        ref = o.head_logits(d, hp_o[b], [int(tg[b, i]) for i in o.tree.path[p]])
                        e = float((hl[b if shared else b * len(P) + j].cpu().double() - ref.double()).abs().max())
                        st.max_head_logit_err = max(st.max_head_logit_err, e)
                        assert e <= LOGIT_TOL, f"head logits max-abs {e}"
        tok = tok_o.clone()
        if plant:
            for b in range(B):
                mlen = min(planted_length(s, b, K), o.tree.K)
                teacher = (teacher_fn or o.greedy_continuation)(b, mlen + 2)[1:]
                row = plant_row(o.tree.parent, teacher, mlen, seed, s, b, vocab=m.vocab)
                for i, v in enumerate(row):
                    if v >= 0:
                        tok[b, i] = v
        amax_o, logits_o = o.verify(tok)
        tok_dev = tok.to(torch.int32).cuda()
        amax_g, logits_g = g.verify(tok_dev, want_logits=True)
        g.poll_status()
        err = float((logits_g.cpu().double() - logits_o.double()).abs().max())
        st.max_logit_err = max(st.max_logit_err, err)
        assert err <= LOGIT_TOL, f"step {s}: logits max-abs {err}"
        h_g = g.get_buffer("H_TREE")[:B * T * m.d_model].view(B, T, m.d_model).cpu()
        for b in range(B):
            e = rel_l2(h_g[b], o.h_tree[b])
            st.max_hidden_err = max(st.max_hidden_err, e)
            assert e <= HID_TOL, f"step {s}: hidden rel-L2 {e}"
        top2 = torch.topk(logits_o, 2, dim=-1).values
        gap = top2[..., 0] - top2[..., 1]
        diff = amax_g.cpu().long() != amax_o
        assert not bool((diff & (gap > GAP)).any()), f"step {s}: argmax differs where the gap exceeds {GAP}"
        st.forced_amax += int(diff.sum())
        amax_dev = amax_o.to(torch.int32).cuda()
        n_o, path_o, out_o = o.accept_compact(tok, amax_o)
        n_g, path_g, out_g = g.accept_compact(tok_dev, amax_dev)
        g.poll_status()
        assert torch.equal(n_g.cpu().long(), n_o) and torch.equal(path_g.cpu().long(), path_o) \
            and torch.equal(out_g.cpu().long(), out_o), f"step {s}: acceptance differs"
        assert g.get_buffer("LEN")[:B].cpu().tolist() == o.len
        assert g.get_buffer("ROOT_TOK")[:B].cpu().tolist() == o.root_tok
        assert g.get_buffer("N_NEW")[:B].cpu().tolist() == [int(n) + 1 for n in n_o]
        st.n_acc.append(n_o.tolist())
        kv = kv_values(g, "KV_BASE")
        for l in kv_layers:
            for b in range(B):
                L = o.len[b]
                for which, ref in ((0, o.kc[l][b]), (1, o.vc[l][b])):
                    got = kv[l, which, b, :, :L].permute(1, 0, 2).float().cpu()          # [L, H, hd]
                    e = rel_l2(got, ref[:L])
                    st.max_kv_err = max(st.max_kv_err, e)
                    assert e <= HID_TOL, f"step {s}: KV layer {l} rel-L2 {e}"
        for b in range(B):
            n = int(n_o[b])
            e = rel_l2(hn[b, :n + 1].cpu(), o.h_new[b])
            assert e <= HID_TOL
        st.steps += 1
    return st

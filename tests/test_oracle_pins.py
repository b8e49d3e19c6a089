"""Pins of the CPU oracle against things other than itself: a library Llama implementation, library
routines, closed forms, brute force and the invariants of greedy speculative decoding."""
import copy
import itertools
import math

import pytest
import torch

from oracle.hydra_oracle import (HydraOracle, TreeTables, rmsnorm, rope, silu, topk_desc, argmax_lowest)
from synth import get_config, make_weights, make_prompts, load_tree, chain_tree, star_tree
from synth.configs import ModelCfg, HeadCfg

torch.set_num_threads(8)


def tiny(prefix=False, mlp=1, K=3, seed=0):
    m = ModelCfg(2, 64, 4, 16, 96, 97, dtype="fp32")
    h = HeadCfg(K, mlp, prefix)
    return m, h, make_weights(m, h, seed)


def c1():
    cfg = get_config("c1")
    return cfg, make_weights(cfg.model, cfg.head, cfg.seed)


# ------------------------------------------------------------------ P7: masks by brute force
def test_ancestor_mask_brute_force():
    parent = load_tree("tree63_d4")
    t = TreeTables(parent)

    def reach(i, j):               # j reachable from i by parent pointers (recursive, independent of the walk)
        return i == j or (parent[i] >= 0 and reach(parent[i], j))

    for i in range(t.T):
        for j in range(t.T):
            assert bool(t.allowed[i, j]) == reach(i, j)
            assert ((t.anc_mask[i] >> j) & 1) == int(reach(i, j))
    ch = TreeTables(chain_tree(5))
    assert torch.equal(ch.allowed, torch.tril(torch.ones(6, 6, dtype=torch.bool)))
    st = TreeTables(star_tree(4))
    for i in range(1, 5):
        assert st.allowed[i].nonzero().flatten().tolist() == [0, i]


def test_tree_validation_and_shapes():
    for bad in ([0], [-1, 1], [-1, 0, 0, 2, 1]):            # last: rows not ordered by rank path
        with pytest.raises(ValueError):
            TreeTables(bad)
    t = TreeTables(load_tree("tree15_d3"))
    assert [sum(1 for d in t.depth if d == k) for k in range(4)] == [1, 4, 7, 4]
    assert [len(p) for p in t.level_parents] == [1, 4, 4]
    t = TreeTables(load_tree("tree63_d4"))
    assert [sum(1 for d in t.depth if d == k) for k in range(5)] == [1, 6, 16, 26, 15]
    assert [len(p) for p in t.level_parents] == [1, 5, 11, 10]
    assert [max(len(t.children[p]) for p in lv) for lv in t.level_parents] == [6, 5, 4, 3]


# ------------------------------------------------------------------ P8: sub-blocks vs library routines
def test_subblocks_against_torch():
    g = torch.Generator().manual_seed(1)
    x = torch.randn(5, 64, dtype=torch.float64, generator=g)
    w = torch.randn(64, dtype=torch.float64, generator=g)
    assert torch.allclose(rmsnorm(x, w, 1e-6), torch.nn.functional.rms_norm(x, (64,), w, 1e-6), atol=1e-13)
    assert torch.allclose(silu(x), torch.nn.functional.silu(x), atol=1e-14)
    # rope: identity at position 0, norm preserving, inner products depend on the position difference only
    q = torch.randn(3, 2, 16, dtype=torch.float64, generator=g)
    k = torch.randn(3, 2, 16, dtype=torch.float64, generator=g)
    assert torch.allclose(rope(q, torch.zeros(3, dtype=torch.long), 1e4), q)
    p1, p2 = torch.tensor([3, 10, 100]), torch.tensor([1, 4, 60])
    a = (rope(q, p1, 1e4) * rope(k, p2, 1e4)).sum(-1)
    b = (rope(q, p1 + 17, 1e4) * rope(k, p2 + 17, 1e4)).sum(-1)
    assert torch.allclose(a, b, atol=1e-12)
    assert torch.allclose(rope(q, p1, 1e4).norm(dim=-1), q.norm(dim=-1), atol=1e-12)
    # rotation of the pair (x_0, x_half) by angle pos * theta^0 = pos
    e = torch.zeros(1, 1, 16, dtype=torch.float64)
    e[0, 0, 0] = 1.0
    r = rope(e, torch.tensor([2]), 1e4)
    assert abs(r[0, 0, 0] - math.cos(2.0)) < 1e-14 and abs(r[0, 0, 8] - math.sin(2.0)) < 1e-14


def test_topk_and_argmax_ties_against_stable_sort():
    g = torch.Generator().manual_seed(2)
    for _ in range(50):
        lg = torch.randint(0, 6, (40,), generator=g).double()          # many exact ties
        ref = torch.sort(lg, descending=True, stable=True).indices.tolist()
        for k in (1, 3, 7):
            assert topk_desc(lg, k) == ref[:k]
        assert int(argmax_lowest(lg[None])[0]) == ref[0]


# ------------------------------------------------------------------ whole base model vs transformers' Llama
def hf_model(m, w):
    tr = pytest.importorskip("transformers")
    cfg = tr.LlamaConfig(vocab_size=m.vocab, hidden_size=m.d_model, intermediate_size=m.d_ffn,
                         num_hidden_layers=m.n_layers, num_attention_heads=m.n_heads,
                         num_key_value_heads=m.n_heads, head_dim=m.head_dim, rms_norm_eps=m.rms_eps,
                         rope_theta=m.rope_theta, max_position_embeddings=512, attention_bias=False,
                         mlp_bias=False, tie_word_embeddings=False, attn_implementation="eager")
    try:
        cfg.rope_parameters = {"rope_type": "default", "rope_theta": m.rope_theta}
    except Exception:
        pass
    model = tr.LlamaForCausalLM(cfg).double().eval()
    d, f = m.d_model, m.d_ffn
    sd = {"model.embed_tokens.weight": w["embed"], "lm_head.weight": w["lm_head"], "model.norm.weight": w["final_norm"]}
    for l in range(m.n_layers):
        p = f"model.layers.{l}."
        q, k, v = w[f"L{l}.wqkv"].split(d, dim=0)
        gte, up = w[f"L{l}.w_gate_up"].split(f, dim=0)
        sd.update({p + "self_attn.q_proj.weight": q, p + "self_attn.k_proj.weight": k,
                   p + "self_attn.v_proj.weight": v, p + "self_attn.o_proj.weight": w[f"L{l}.wo"],
                   p + "mlp.gate_proj.weight": gte, p + "mlp.up_proj.weight": up,
                   p + "mlp.down_proj.weight": w[f"L{l}.w_down"],
                   p + "input_layernorm.weight": w[f"L{l}.attn_norm"],
                   p + "post_attention_layernorm.weight": w[f"L{l}.ffn_norm"]})
    missing = model.load_state_dict({k: v.double() for k, v in sd.items()}, strict=False)
    assert not [k for k in missing.missing_keys if "rotary" not in k]
    return model


def test_prefill_and_chain_tree_against_transformers_llama():
    cfg, w = c1()
    m = cfg.model
    model = hf_model(m, w)
    prompt = make_prompts(cfg.seed, [32], m.vocab)[0]
    K = 3
    o = HydraOracle(m, cfg.head, chain_tree(K), w, 128)
    o.prefill([prompt])
    with torch.no_grad():
        ref = model(prompt[None].long()).logits[0]
    mine = o.h_new[0] @ o.W("lm_head").T
    # the library builds its rotary tables in float32, which bounds the agreement near 1e-7
    assert (mine - ref).abs().max() < 2e-6
    assert o.root_tok[0] == int(ref[-1].argmax())
    # chain-shaped tree == ordinary causal decoding of root, c1..cK (P1), checked against the library model
    chain = torch.tensor([[o.root_tok[0], 5, 900, 33]])
    amax, logits = o.verify(chain)
    with torch.no_grad():
        ref2 = model(torch.cat([prompt.long(), chain[0]])[None]).logits[0, 32:]
    assert (logits[0] - ref2).abs().max() < 2e-6
    assert amax[0].tolist() == ref2.argmax(-1).tolist()


# ------------------------------------------------------------------ P1/P2/P4: invariants of greedy speculation
def committed_tokens(prompt, emitted):
    return torch.cat([prompt.long(), torch.tensor(emitted, dtype=torch.long)])


@pytest.mark.parametrize("prefix,mlp", [(False, 1), (True, 2)])
def test_spec_decode_equals_greedy_and_compaction_equals_sequential(prefix, mlp):
    m, h, w = tiny(prefix, mlp)
    parent = load_tree("tree15_d3")
    prompt = make_prompts(3, [9], m.vocab)[0]
    o = HydraOracle(m, h, parent, w, 96)
    o.prefill([prompt])
    ar = o.greedy_continuation(0, 30)                      # autoregressive greedy stream (first = root)
    # root-only tree == plain greedy decoding
    o1 = HydraOracle(m, h, [-1], w, 96)
    o1.prefill([prompt])
    em1 = [o1.root_tok[0]]
    for _ in range(6):
        n, _, out = o1.step()
        assert int(n[0]) == 0
        em1.append(int(out[0, 0]))
    assert em1 == ar[:7]
    # any candidates (drafted / random / planted teacher tokens) give the same stream
    emitted = [o.root_tok[0]]
    g = torch.Generator().manual_seed(5)
    seen = set()
    for s in range(8):
        tok = o.draft()
        if s % 2 == 1:
            tok[:, 1:] = torch.randint(0, m.vocab, (1, o.tree.T - 1), generator=g)
        mlen = s % 4
        node = [i for i in range(o.tree.T) if o.tree.depth[i] == mlen][-1]
        for j in o.tree.path[node][1:]:
            tok[0, j] = ar[len(emitted) - 1 + o.tree.depth[j]]
        if mlen == 0:                                       # rule out a chance match at depth 1
            for r, j in enumerate(o.tree.children[0]):
                tok[0, j] = (ar[len(emitted)] + 1 + r) % m.vocab
        amax, _ = o.verify(tok)
        n, path, out = o.accept_compact(tok, amax)
        assert int(n[0]) >= mlen
        seen.add(int(n[0]))
        emitted += [t for t in out[0].tolist() if t >= 0]
        assert emitted == ar[:len(emitted)]
    assert seen >= {0, 1, 2, 3}
    # compacted cache == cache of decoding the committed tokens in one plain causal pass (P4)
    o2 = HydraOracle(m, h, parent, w, 96)
    o2.prefill([committed_tokens(prompt, emitted[:-1])])
    L = o.len[0]
    assert L == o2.len[0] == 9 + len(emitted) - 1
    for l in range(m.n_layers):
        assert (o.kc[l][0][:L] - o2.kc[l][0][:L]).abs().max() < 1e-12
        assert (o.vc[l][0][:L] - o2.vc[l][0][:L]).abs().max() < 1e-12
    assert o.root_tok[0] == o2.root_tok[0]
    assert (o.h_new[0][-1] - o2.h_new[0][-1]).abs().max() < 1e-11
    if prefix:                                             # prefix-layer cache likewise, and the drafts agree
        ta, tb = o.draft(), o2.draft()
        assert torch.equal(ta, tb)
        assert (o.pk[0][:L] - o2.pk[0][:L]).abs().max() < 1e-12


def test_chain_tree_equals_token_by_token_decode():
    m, h, w = tiny()
    prompt = make_prompts(4, [7], m.vocab)[0]
    o = HydraOracle(m, h, chain_tree(3), w, 64)
    o.prefill([prompt])
    chain = torch.tensor([[o.root_tok[0], 11, 12, 13]])
    _, logits = o.verify(chain)
    for k in range(4):                                      # feed the same tokens one at a time
        ok = HydraOracle(m, h, [-1], w, 64)
        ok.prefill([committed_tokens(prompt, chain[0, :k].tolist())])
        _, lg = ok.verify(chain[:, k:k + 1])
        assert (lg[0, 0] - logits[0, k]).abs().max() < 1e-12


# ------------------------------------------------------------------ P3: acceptance by brute force
def brute_force_accept(t, tok, amax):
    leaves = [i for i in range(t.T) if not t.children[i]]
    best = (0, 0)
    for leaf in leaves:
        p = t.path[leaf]
        n = 0
        while n + 1 < len(p) and tok[p[n + 1]] == amax[p[n]]:
            n += 1
        cand = (n, -p[n])                                   # longest match, lowest row among equals
        if cand > best or (n == best[0] and p[n] < -best[1] and n > 0):
            best = cand
    return best[0], -best[1]


def test_acceptance_against_brute_force():
    m, h, w = tiny()
    parent = load_tree("tree15_d3")
    g = torch.Generator().manual_seed(7)
    o = HydraOracle(m, h, parent, w, 64)
    o.prefill([make_prompts(1, [5], m.vocab)[0]])
    t = o.tree
    for trial in range(300):
        tok = torch.randint(0, 3, (1, t.T), generator=g)    # tiny alphabet: many matches and sibling duplicates
        amax = torch.randint(0, 3, (1, t.T), generator=g)
        o.h_tree = [torch.zeros(t.T, m.d_model, dtype=torch.float64)]
        o.len = [5]
        n, path, out = o.accept_compact(tok, amax)
        bn, bnode = brute_force_accept(t, tok[0].tolist(), amax[0].tolist())
        assert int(n[0]) == bn
        p = [x for x in path[0].tolist() if x >= 0]
        assert p == t.path[bnode]
        assert out[0].tolist()[:bn + 1] == [int(tok[0, j]) for j in p[1:]] + [int(amax[0, bnode])]
        assert o.len[0] == 5 + bn + 1 and o.root_tok[0] == int(amax[0, bnode])


# ------------------------------------------------------------------ P5: closed-form head cases
def test_head_closed_forms():
    m, h, w = tiny(prefix=False, mlp=3)
    w = {k: v.clone() for k, v in w.items()}
    d = m.d_model
    o = HydraOracle(m, h, load_tree("tree15_d3"), w, 64)
    o.prefill([make_prompts(2, [6], m.vocab)[0]])
    hlast = o.h_new[0][-1]
    base_logits = o.W("lm_head") @ hlast
    # (a) all-zero MLP: every head reproduces the base logits of the last processed row
    for k in list(w):
        if k.startswith("H"):
            w[k].zero_()
    tok, lgs = o.draft(return_logits=True)
    for p, lg in lgs[0].items():
        assert (lg - base_logits).abs().max() < 1e-12
        assert tok[0, o.tree.children[p][0]] == o.root_tok[0]
    # (b) first layer selects one block of the concatenation: y = h + silu(block), checked with torch's silu
    E = o.W("embed")
    path_tok = [3, 50, 77]
    for blk in range(4):
        w["H3.w1"].zero_()
        w["H3.w1"][:, blk * d:(blk + 1) * d] = torch.eye(d)
        vec = hlast if blk == 0 else E[path_tok[blk - 1]]
        ref = o.W("lm_head") @ (hlast + torch.nn.functional.silu(vec))
        assert (o.head_logits(3, hlast, path_tok) - ref).abs().max() < 1e-12
    # (c) deeper layers and biases: W = 0 leaves y + silu(bias)
    w["H3.w1"].zero_()
    w["H3.b1"].fill_(0.5)
    w["H3.br"][0].fill_(-1.0)
    y = hlast + torch.nn.functional.silu(torch.tensor(0.5, dtype=torch.float64))
    y = y + torch.nn.functional.silu(torch.tensor(-1.0, dtype=torch.float64))
    assert (o.head_logits(3, hlast, path_tok) - o.W("lm_head") @ y).abs().max() < 1e-12


def test_zeroed_embedding_columns_give_sequentially_independent_heads():
    m, h, w = tiny()
    w = {k: v.clone() for k, v in w.items()}
    for i in range(1, 4):
        w[f"H{i}.w1"][:, m.d_model:] = 0                     # head ignores x_t and the speculated tokens
    o = HydraOracle(m, h, load_tree("tree15_d3"), w, 64)
    o.prefill([make_prompts(2, [6], m.vocab)[0]])
    tok = o.draft()[0]
    t = o.tree
    for lv in t.level_parents:
        first = [int(tok[c]) for c in t.children[lv[0]]]
        for p in lv:
            kids = [int(tok[c]) for c in t.children[p]]
            assert kids == first[:len(kids)]


def test_medusa_heads_equal_hydra_heads_with_zeroed_embedding_columns():
    """Sequentially independent heads (Background, "Medusa decoding") are the special case of Hydra heads whose
    first layer ignores the token embeddings: same children, same logits."""
    m, h, w = tiny(mlp=2)
    hm = HeadCfg(h.n_heads, h.n_mlp_layers, h.prefix_attn, h.has_bias, medusa=True)
    wm = make_weights(m, hm, 0)
    w = {k: v.clone() for k, v in w.items()}
    d = m.d_model
    for i in range(1, h.n_heads + 1):
        assert tuple(wm[f"H{i}.w1"].shape) == (d, d)
        w[f"H{i}.w1"].zero_()
        w[f"H{i}.w1"][:, :d] = wm[f"H{i}.w1"]
        for k in ("b1", "wr", "br"):
            w[f"H{i}.{k}"] = wm[f"H{i}.{k}"]
    parent = load_tree("tree15_d3")
    prompt = [make_prompts(2, [6], m.vocab)[0]]
    oh, om = HydraOracle(m, h, parent, w, 64), HydraOracle(m, hm, parent, wm, 64)
    oh.prefill(prompt); om.prefill(prompt)
    th, lh = oh.draft(return_logits=True)
    tm, lm = om.draft(return_logits=True)
    assert torch.equal(th, tm)
    for p in lh[0]:
        assert float((lh[0][p] - lm[0][p]).abs().max()) < 1e-12


def test_children_sorted_by_descending_head_probability():
    cfg, w = c1()
    o = HydraOracle(cfg.model, cfg.head, load_tree(cfg.tree), w, cfg.max_seq)
    o.prefill(make_prompts(cfg.seed, cfg.prompt_lens, cfg.model.vocab))
    tok, lgs = o.draft(return_logits=True)
    for p, lg in lgs[0].items():
        kids = [int(tok[0, c]) for c in o.tree.children[p]]
        vals = [float(lg[k]) for k in kids]
        assert vals == sorted(vals, reverse=True)
        assert min(vals) >= float(torch.topk(lg, len(kids)).values[-1])
        assert len(set(kids)) == len(kids)


# ------------------------------------------------------------------ P9 / P10
def test_batch_invariance_ragged():
    m, h, w = tiny(prefix=True, mlp=2)
    parent = load_tree("tree15_d3")
    prompts = make_prompts(8, [5, 11, 8], m.vocab)
    ob = HydraOracle(m, h, parent, w, 64)
    ob.prefill(prompts)
    singles = []
    for p in prompts:
        o = HydraOracle(m, h, parent, w, 64)
        o.prefill([p])
        singles.append(o)
    for s in range(3):
        nb, pb, outb = ob.step()
        for b, o in enumerate(singles):
            n, p_, out = o.step()
            assert torch.equal(out[0], outb[b]) and torch.equal(p_[0], pb[b])


def test_sibling_permutation_invariance():
    m, h, w = tiny()
    parent = load_tree("tree15_d3")
    o = HydraOracle(m, h, parent, w, 64)
    prompt = make_prompts(9, [6], m.vocab)[0]
    o.prefill([prompt])
    t = o.tree
    tok = o.draft()
    _, lg = o.verify(tok)
    # swap the subtrees of root children 1 and 2 (both have two children in this tree)
    a, b = t.children[0][0], t.children[0][1]
    assert len(t.children[a]) == len(t.children[b])

    def subtree(r):
        rows = [r]
        for c in t.children[r]:
            rows += subtree(c)
        return rows

    sa, sb = subtree(a), subtree(b)
    assert len(sa) == len(sb)
    perm = list(range(t.T))
    for x, y in zip(sa, sb):
        perm[x], perm[y] = y, x
    tok2 = tok[:, perm]
    _, lg2 = o.verify(tok2)
    assert (lg2[0][perm] - lg[0]).abs().max() < 1e-11


# ------------------------------------------------------------------ typical acceptance (Section "Typical acceptance sampling")
def _typical_setup(seed=3):
    m, h, w = tiny()
    parent = load_tree("tree15_d3")
    o = HydraOracle(m, h, parent, w, 64)
    o.prefill([make_prompts(1, [5], m.vocab)[0]])
    g = torch.Generator().manual_seed(seed)
    return m, o, g


def _reset(o, m):
    o.h_tree = [torch.zeros(o.tree.T, m.d_model, dtype=torch.float64)]
    o.len = [5]


def test_typical_row_against_library_entropy_and_closed_forms():
    from oracle.hydra_oracle import typical_row
    scipy_special = pytest.importorskip("scipy.special")
    scipy_stats = pytest.importorskip("scipy.stats")
    g = torch.Generator().manual_seed(1)
    for tau in (0.3, 0.7, 1.0, 2.5):
        lg = torch.randn(97, generator=g, dtype=torch.float64) * 3.0
        p, thr = typical_row(lg, tau, 0.3, 0.5)
        p_lib = scipy_special.softmax(lg.numpy() / tau)
        assert float((p - torch.from_numpy(p_lib)).abs().max()) < 1e-14
        H = float(scipy_stats.entropy(p_lib))                   # natural logarithm
        assert abs(thr - min(0.3, 0.5 * math.exp(-H))) < 1e-14
    # a uniform row: p = 1/V, entropy log V, so the threshold is min(eps, alpha / V)
    V = 64
    p, thr = typical_row(torch.full((V,), 1.7, dtype=torch.float64), 0.7, 0.2, 0.4)
    assert float((p - 1.0 / V).abs().max()) < 1e-15 and abs(thr - min(0.2, 0.4 / V)) < 1e-15
    # a one-hot row (huge gap): entropy 0, threshold min(eps, alpha)
    lg = torch.zeros(V, dtype=torch.float64); lg[5] = 1e4
    p, thr = typical_row(lg, 1.0, 0.25, 0.1)
    assert float(p[5]) == 1.0 and thr == 0.1
    # the posterior threshold caps it from above
    assert typical_row(lg, 1.0, 0.05, 0.9)[1] == 0.05


def test_typical_acceptance_limits_and_brute_force():
    """tau -> 0: the temperature distribution collapses on the argmax, the entropy goes to 0 and the criterion is the
    greedy one.  eps -> 0 (alpha = sqrt(eps)): every candidate of non-zero probability passes, so the deepest leaf
    with the lowest row index wins.  In between: brute force over all root-to-leaf paths with the pass bits taken
    straight from the inequality."""
    from oracle.hydra_oracle import typical_row
    m, o, g = _typical_setup()
    t = o.tree
    V = m.vocab
    for trial in range(60):
        logits = torch.randn(1, t.T, V, generator=g, dtype=torch.float64) * 2.0
        amax = argmax_lowest(logits[0])[None]
        tok = torch.randint(0, V, (1, t.T), generator=g)
        for i in range(1, t.T):                                  # plant the argmax of the parent on about half the rows
            if torch.rand(1, generator=g).item() < 0.5:
                tok[0, i] = amax[0, t.parent[i]]
        # tau -> 0 equals the greedy criterion (bonus token: argmax either way)
        _reset(o, m)
        n_t, path_t, out_t = o.typical_accept_compact(tok, logits, 1e-3, 0.3, 0.5)
        _reset(o, m)
        n_g, path_g, out_g = o.accept_compact(tok, amax)
        assert torch.equal(n_t, n_g) and torch.equal(path_t, path_g) and torch.equal(out_t, out_g)
        # eps -> 0 accepts everything: the first row of the deepest level
        _reset(o, m)
        n_e, path_e, _ = o.typical_accept_compact(tok, logits, 0.7, 1e-300, 1e-150)
        deepest = min(i for i in range(t.T) if t.depth[i] == t.K)
        assert int(n_e[0]) == t.K and [x for x in path_e[0].tolist() if x >= 0] == t.path[deepest]
        # brute force at the paper's temperature and a threshold in its range
        tau, eps = 0.7, 0.15
        alpha = math.sqrt(eps)
        bits = [True] * t.T
        for i in range(1, t.T):
            z = logits[0, t.parent[i]] / tau
            p = torch.softmax(z, dim=0)                          # library routine
            H = float(torch.distributions.Categorical(probs=p).entropy())
            bits[i] = float(p[int(tok[0, i])]) > min(eps, alpha * math.exp(-H))
        best, best_len = 0, 0
        for leaf in range(t.T):                                  # every root-to-node path, longest all-pass prefix
            path = t.path[leaf]
            k = 0
            while k + 1 < len(path) and bits[path[k + 1]]:
                k += 1
            if k > best_len or (k == best_len and path[k] < best):
                best, best_len = path[k], k
        _reset(o, m)
        n_b, path_b, out_b = o.typical_accept_compact(tok, logits, tau, eps, alpha)
        assert int(n_b[0]) == best_len and [x for x in path_b[0].tolist() if x >= 0] == t.path[best]
        assert out_b[0].tolist()[:best_len + 1] == [int(tok[0, j]) for j in t.path[best][1:]] + [int(amax[0, best])]
        ok, margin = o.typical_pass(tok, logits, tau, eps, alpha)
        assert ok[0].tolist() == bits and all((margin[0, i] > 0) == bits[i] for i in range(1, t.T))


def test_bonus_token_inverse_cdf():
    """The sampled token against numpy's cumulative sum and searchsorted, and its frequencies against the distribution."""
    import numpy as np
    from oracle.hydra_oracle import inverse_cdf
    g = torch.Generator().manual_seed(5)
    p = torch.softmax(torch.randn(50, generator=g, dtype=torch.float64), dim=0)
    c = np.cumsum(p.numpy())
    us = torch.rand(4000, generator=g, dtype=torch.float64).tolist() + [0.0, 0.999999999]
    draws = [inverse_cdf(p, u) for u in us]
    assert draws == [int(np.searchsorted(c, u * c[-1], side="right")) for u in us]
    freq = torch.bincount(torch.tensor(draws[:4000]), minlength=50).double() / 4000
    assert float((freq - p).abs().max()) < 0.03
    m, o, _ = _typical_setup()
    t = o.tree
    logits = torch.randn(1, t.T, m.vocab, generator=g, dtype=torch.float64)
    tok = torch.zeros(1, t.T, dtype=torch.int64)
    _reset(o, m)
    n, path, out = o.typical_accept_compact(tok, logits, 0.7, 1.0, 1.0 - 1e-12, u=[0.37])   # threshold ~ exp(-H) <= max p: mixed
    best = [x for x in path[0].tolist() if x >= 0][-1]
    want = inverse_cdf(torch.softmax(logits[0, best] / 0.7, dim=0), 0.37)
    assert o.root_tok[0] == want == out[0].tolist()[int(n[0])]

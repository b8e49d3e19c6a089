"""Typical acceptance (Section "Typical acceptance sampling") on the GPU against the oracle: the per-candidate pass
bits, the accepted path, the compaction and the sampled token after the path, one decode step from identical state
per parameter setting.

The pass decision is a floating-point comparison, so the bits are compared where the oracle's margin
|log p - log threshold| exceeds MARGIN; a setting is only compared further (path, lengths, tokens) when every bit
agrees, which the test requires for most settings.  The sampled token t must satisfy the inverse-CDF rule within a
window: cdf(t - 1) - DELTA <= u < cdf(t) + DELTA under the oracle's distribution."""
import math

import pytest
import torch

from oracle.hydra_oracle import HydraOracle, typical_row, argmax_lowest
from synth import make_weights, make_prompts, load_tree
from synth.configs import ModelCfg, HeadCfg

pytestmark = pytest.mark.gpu

MARGIN = 2e-2
DELTA = 2e-4


def _plant_from_parent_top(o, tok, gen):
    """Level by level, overwrite about two thirds of the candidates with one of their parent's five most likely
    tokens (so that the pass bits are a mix); returns the tokens and the oracle's logits for them."""
    t = o.tree
    for d in range(1, t.K + 1):
        _, logits = o.verify(tok)
        for b in range(o.B):
            for i in range(1, t.T):
                if t.depth[i] == d and torch.rand(1, generator=gen).item() < 0.66:
                    top = torch.topk(logits[b, t.parent[i]], 5).indices
                    tok[b, i] = int(top[int(torch.randint(0, 5, (1,), generator=gen))])
    amax, logits = o.verify(tok)
    return tok, amax, logits


@pytest.mark.parametrize("tree", ["tree15_d3", "tree63_d4"])
def test_typical_acceptance_matches_oracle(tree):
    from paper_2402_05109_b200 import Hydra
    m = ModelCfg(2, 256, 2, 128, 512, 1024, dtype="bf16")
    parent = load_tree(tree)
    h = HeadCfg(4 if tree == "tree63_d4" else 3, 1, False)
    T, K, B, max_seq = len(parent), h.n_heads, 2, 160
    w = make_weights(m, h, 23)
    prompts = make_prompts(23, [40, 17], m.vocab)
    gen = torch.Generator().manual_seed(11)
    g = Hydra(m, h, parent, {k: v.cuda() for k, v in w.items()}, B, max_seq)
    compared, settings = 0, 0
    tau = 0.7
    for eps in (0.002, 0.004, 0.008, 0.02, 0.05):
        for u_vals in (None, [0.0311, 0.7424], [0.9993, 0.25]):
            settings += 1
            alpha = math.sqrt(eps)
            o = HydraOracle(m, h, parent, w, max_seq)
            o.prefill(prompts)
            g.prefill(prompts)
            tok, amax_o, logits_o = _plant_from_parent_top(o, o.draft(), gen)
            u_dev = None if u_vals is None else torch.tensor(u_vals, dtype=torch.float32).cuda()
            g.set_acceptance(1, tau, eps, alpha, u_dev)
            g.draft()
            tok_dev = tok.to(torch.int32).cuda()
            amax_g, logits_g = g.verify(tok_dev, want_logits=True)
            g.poll_status()
            assert float((logits_g.cpu().double() - logits_o).abs().max()) <= 5e-2
            ok_o, margin = o.typical_pass(tok, logits_o, tau, eps, alpha)
            lens0 = list(o.len)
            n_o, path_o, out_o = o.typical_accept_compact(tok, logits_o, tau, eps, alpha, u=u_vals)
            n_g, path_g, out_g = g.accept_compact(tok_dev, amax_o.to(torch.int32).cuda())
            g.poll_status()
            bits = g.get_buffer("PASS_BITS")[:B].cpu().tolist()
            agree = True
            for b in range(B):
                for i in range(1, T):
                    got = bool((bits[b] >> i) & 1)
                    if got != bool(ok_o[b, i]):
                        assert abs(float(margin[b, i])) <= MARGIN, (eps, b, i, float(margin[b, i]))
                        agree = False
            if not agree:
                continue                                    # an under-margin flip: the two sides may commit different paths
            compared += 1
            assert torch.equal(n_g.cpu().long(), n_o) and torch.equal(path_g.cpu().long(), path_o), (eps, u_vals)
            assert g.get_buffer("LEN")[:B].cpu().tolist() == o.len == [lens0[b] + int(n_o[b]) + 1 for b in range(B)]
            for b in range(B):
                n = int(n_o[b])
                assert out_g[b, :n].cpu().tolist() == out_o[b, :n].tolist()
                best = int(path_o[b, n])
                bonus = int(out_g[b, n])
                assert int(g.get_buffer("ROOT_TOK")[b]) == bonus
                if u_vals is None:
                    assert bonus == int(argmax_lowest(logits_o[b, best:best + 1])[0]) == int(out_o[b, n])
                else:
                    p, _ = typical_row(logits_o[b, best], tau, eps, alpha)
                    cdf = torch.cumsum(p, dim=0)
                    lo = float(cdf[bonus - 1]) if bonus > 0 else 0.0
                    assert lo - DELTA <= u_vals[b] < float(cdf[bonus]) + DELTA, (bonus, int(out_o[b, n]), u_vals[b])
            assert {int(v) for v in n_o.tolist()} <= set(range(K + 1))
    g.set_acceptance(0)
    g.close()
    assert compared >= settings - 3, (compared, settings)


def test_small_temperature_is_the_greedy_criterion():
    """tau -> 0 collapses the temperature distribution on the argmax: the typical pass bits must equal the greedy
    match bits, computed by the same kernel in its other mode."""
    from paper_2402_05109_b200 import Hydra
    m = ModelCfg(2, 256, 2, 128, 512, 1024, dtype="bf16")
    h = HeadCfg(3, 1, False)
    parent = load_tree("tree15_d3")
    B, max_seq = 2, 128
    w = make_weights(m, h, 29)
    prompts = make_prompts(29, [21, 33], m.vocab)
    gen = torch.Generator().manual_seed(3)
    o = HydraOracle(m, h, parent, w, max_seq)
    o.prefill(prompts)
    tok, amax_o, logits_o = _plant_from_parent_top(o, o.draft(), gen)
    for i in range(1, len(parent)):                         # plant the argmax of the parent on half the rows
        if i % 2:
            tok[:, i] = amax_o[:, parent[i]]
    amax_o, logits_o = o.verify(tok)
    g = Hydra(m, h, parent, {k: v.cuda() for k, v in w.items()}, B, max_seq)
    top2 = torch.topk(logits_o, 2, dim=-1).values
    clear = (top2[..., 0] - top2[..., 1]) > 0.1            # parent rows whose argmax cannot flip with the arithmetic
    results = []
    for mode in (0, 1):
        g.prefill(prompts)
        g.set_acceptance(mode, 0.01, 0.3, 0.5, None)
        g.draft()
        tok_dev = tok.to(torch.int32).cuda()
        amax_g = g.verify(tok_dev)
        assert bool(((amax_g.cpu().long() == amax_o) | ~clear).all())
        n, path, out = g.accept_compact(tok_dev, amax_o.to(torch.int32).cuda())
        g.poll_status()
        results.append((g.get_buffer("PASS_BITS")[:B].cpu().tolist(), n.cpu().tolist(), path.cpu().tolist(), out.cpu().tolist()))
    g.set_acceptance(0)
    g.close()
    checked = 0
    for b in range(B):
        for i in range(1, len(parent)):
            if bool(clear[b, parent[i]]):
                checked += 1
                assert (results[0][0][b] >> i) & 1 == (results[1][0][b] >> i) & 1, (b, i)
    assert checked >= len(parent)                           # most parents have a clear argmax
    if bool(clear.all()):
        assert results[0][1:] == results[1][1:]
    assert any(n > 0 for n in results[0][1])

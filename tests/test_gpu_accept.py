"""The acceptance + compaction kernel driven directly through hydra_accept_compact with arbitrary candidate and
argmax arrays: a three-token alphabet makes equal-depth ties and duplicate siblings frequent (the cases the drafted
and planted trees of the step tests never produce).  Integer outputs are compared bit for bit with the oracle; a
move is a copy, so every moved cache row of every layer (and plane) must EQUAL the pre-move row."""
import pytest
import torch

from oracle.hydra_oracle import HydraOracle
from synth import make_weights, make_prompts, load_tree
from synth.configs import ModelCfg, HeadCfg
from tests.parity import kv_raw

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,hd", [("fp32", 64), ("bf16", 128)])
def test_accept_compact_kernel_on_ties_and_duplicates(dtype, hd):
    from paper_2402_05109_b200 import Hydra
    m = ModelCfg(2, 256, 256 // hd, hd, 512, 1024, dtype=dtype)
    h = HeadCfg(3, 1, False)
    parent = load_tree("tree15_d3")
    T, K, B, max_seq = len(parent), h.n_heads, 2, 96
    w = make_weights(m, h, 17)
    prompts = make_prompts(17, [9, 30], m.vocab)
    o = HydraOracle(m, h, parent, w, max_seq)
    o.prefill(prompts)
    lens0 = list(o.len)
    g = Hydra(m, h, parent, {k: v.cuda() for k, v in w.items()}, B, max_seq)
    g.prefill(prompts)
    tok_real = g.draft()
    g.verify(tok_real)                              # a real forward: tree rows' K,V now sit at slots len + i
    g.poll_status()
    snapshot = g.workspace.clone()
    gen = torch.Generator().manual_seed(7)
    seen_n = set()
    for trial in range(300):
        tok = torch.randint(0, 3, (B, T), generator=gen)
        amax = torch.randint(0, 3, (B, T), generator=gen)
        # oracle side: only its acceptance logic is used (its own caches are moved along, not compared)
        o.len = list(lens0)
        o.h_tree = [torch.zeros(T, m.d_model, dtype=torch.float64) for _ in range(B)]
        n_o, path_o, out_o = o.accept_compact(tok, amax)
        # CUDA side: same state every trial
        g.workspace.copy_(snapshot)
        g.verify(tok_real)                          # rewrites the same tree rows; puts the context into the verified state
        pre = kv_raw(g, "KV_BASE").clone()
        h_tree = g.get_buffer("H_TREE")[:B * T * m.d_model].view(B, T, m.d_model).clone()
        n_g, path_g, out_g = g.accept_compact(tok.to(torch.int32).cuda(), amax.to(torch.int32).cuda())
        g.poll_status()
        assert torch.equal(n_g.cpu().long(), n_o), trial
        assert torch.equal(path_g.cpu().long(), path_o), trial
        assert torch.equal(out_g.cpu().long(), out_o), trial
        assert g.get_buffer("LEN")[:B].cpu().tolist() == o.len
        assert g.get_buffer("ROOT_TOK")[:B].cpu().tolist() == o.root_tok
        assert g.get_buffer("N_NEW")[:B].cpu().tolist() == [int(n) + 1 for n in n_o]
        post = kv_raw(g, "KV_BASE")
        h_new = g.get_buffer("H_NEW").view(g.max_batch, K + 1, m.d_model)
        for b in range(B):
            n, L = int(n_o[b]), lens0[b]
            seen_n.add(n)
            path = path_o[b, :n + 1].tolist()
            want = pre[:, :, :, b].clone()                                  # [layers][k,v][planes][heads][seq][hd]
            for k in range(1, n + 1):
                want[..., L + k, :] = pre[:, :, :, b, :, L + path[k], :]
            assert torch.equal(post[:, :, :, b, :, :L + n + 1], want[..., :L + n + 1, :]), (trial, b)
            assert torch.equal(h_new[b, :n + 1], h_tree[b, path]), (trial, b)
    assert seen_n == {0, 1, 2, 3}
    g.close()

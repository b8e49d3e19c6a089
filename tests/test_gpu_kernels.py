"""Kernel-level parity through the C ABI: the tensor-core GEMM, the SIMT GEMM and tree attention against
their plain definitions evaluated by the oracle's routines / torch CPU float64."""
import pytest
import torch

from oracle.hydra_oracle import masked_attention, TreeTables
from synth import normal_, load_tree
from tests.parity import split_hi_lo

pytestmark = pytest.mark.gpu


def rnd(shape, seed, stream, dtype, std=1.0):
    return normal_(torch.empty(shape, dtype=dtype), seed, stream, std)


@pytest.mark.parametrize("m,n,k", [(64, 256, 512), (64, 12288, 4096), (5, 128, 256), (11, 256, 1280), (16, 128, 64),
                                   (100, 512, 704), (256, 256, 1024), (300, 384, 512), (64, 4096, 11008),
                                   (1, 1024, 256), (64, 32000, 1024), (512, 1024, 512)])
def test_gemm_tensor_core_matches_definition(m, n, k):
    from paper_2402_05109_b200 import gemm
    x = rnd((m, k), 11, m + k, torch.bfloat16)
    w = rnd((n, k), 12, n + k, torch.bfloat16, 0.02)
    ref = x.double() @ w.double().T
    out = gemm(x.cuda(), w.cuda(), mode=0).cpu().double()
    # products of bfloat16 values are exact in float; only the float accumulation order differs
    tol = 1e-5 * float(ref.abs().max()) + 1e-6 * k ** 0.5
    assert float((out - ref).abs().max()) <= tol
    simt = gemm(x.cuda(), w.cuda(), mode=1).cpu().double()
    assert float((simt - ref).abs().max()) <= tol


@pytest.mark.parametrize("m,n,k", [(64, 512, 4096), (11, 256, 1280), (300, 384, 704)])
def test_gemm_hi_lo_activation_planes(m, n, k):
    """Float activations passed as hi/lo bfloat16 planes: the product must match the float activations to ~2^-16."""
    from paper_2402_05109_b200 import gemm
    x = rnd((m, k), 15, m + k, torch.float32)
    w = rnd((n, k), 16, n + k, torch.bfloat16, 0.02)
    ref = x.double() @ w.double().T
    out = gemm(split_hi_lo(x.cuda()), w.cuda(), mode=0).cpu().double()
    scale = float(ref.abs().max())
    assert float((out - ref).abs().max()) <= 3e-5 * scale
    single = gemm(x.to(torch.bfloat16).cuda(), w.cuda(), mode=0).cpu().double()
    assert float((single - ref).abs().max()) > 10 * float((out - ref).abs().max())       # the lo plane matters


@pytest.mark.parametrize("m,n,k", [(16, 768, 256), (7, 1376, 256), (16, 256, 688), (4, 1024, 1024)])
def test_gemm_float(m, n, k):
    from paper_2402_05109_b200 import gemm
    x = rnd((m, k), 13, 1, torch.float32)
    w = rnd((n, k), 14, 2, torch.float32, 0.02)
    ref = x.double() @ w.double().T
    out = gemm(x.cuda(), w.cuda()).cpu().double()
    assert float((out - ref).abs().max()) <= 1e-5 * float(ref.abs().max()) + 1e-6


@pytest.mark.parametrize("dtype,planes", [(torch.float32, 1), (torch.bfloat16, 1), (torch.bfloat16, 2)])
@pytest.mark.parametrize("hd", [64, 128])
@pytest.mark.parametrize("case", ["few_chunks", "many_chunks"])
def test_tree_attention_matches_masked_softmax(dtype, planes, hd, case):
    """few_chunks: at most 8 KV chunks per (head, sequence), which the bfloat16 kernel merges inside a thread-block
    cluster; many_chunks: one long sequence with two heads, 12 chunks, merged through scratch by the last CTA."""
    from paper_2402_05109_b200 import tree_attention
    parent = load_tree("tree63_d4")
    t = TreeTables(parent)
    tc = t.T
    if case == "few_chunks":
        B, H, S = 3, 3, 700
        pos0 = [0, 333, 600]                # empty cache, a cache spanning several KV chunks with a ragged tail, long
        n_rows = [tc, tc, 17]               # ragged row counts (rows beyond n_rows are ignored)
    else:
        B, H, S = 1, 2, 1500
        pos0 = [1391]
        n_rows = [tc]
    src = torch.float32 if planes == 2 else dtype
    kc = rnd((B, H, S, hd), 21, 1, src)
    vc = rnd((B, H, S, hd), 21, 2, src)
    q = rnd((B * tc, H, hd), 21, 3, src)
    dev = (lambda x: split_hi_lo(x.cuda())) if planes == 2 else (lambda x: x.cuda())
    mask = torch.tensor([a - (1 << 64) if a >= (1 << 63) else a for a in t.anc_mask], dtype=torch.int64)
    out = tree_attention(dev(q), dev(kc), dev(vc), torch.tensor(pos0, dtype=torch.int32).cuda(),
                         torch.tensor(n_rows, dtype=torch.int32).cuda(), mask.cuda(), tc).float().cpu()
    out = (out.sum(0) if planes == 2 else out).view(B, tc, H, hd)
    for b in range(B):
        n, L = n_rows[b], pos0[b] + n_rows[b]
        allowed = torch.cat([torch.ones(n, pos0[b], dtype=torch.bool), t.allowed[:n, :n]], dim=1)
        k = kc[b, :, :L].permute(1, 0, 2).double()
        v = vc[b, :, :L].permute(1, 0, 2).double()
        ref = masked_attention(q.view(B, tc, H, hd)[b, :n].double(), k, v, allowed)   # q, k, v hold the stored values
        err = float((out[b, :n].double() - ref).abs().max())
        tol = 2e-5 if dtype == torch.float32 else (2e-4 if planes == 2 else 2e-2)
        assert err <= tol, err


def test_bounded_wait_gives_up_and_the_context_stays_usable():
    """A one-CTA GEMM whose third weight tile is never requested: the tensor-core lane's bounded wait for it (or the
    epilogue's wait for the accumulator that then never completes) runs out, the kernel reports TIMEOUT with the place
    it gave up and returns.  Through a context's status buffer hydra_poll_status turns that into an error and clears
    it; the next ordinary GEMM is exact."""
    from paper_2402_05109_b200 import Hydra, HydraError, gemm, gemm_bounded_wait_probe
    from synth import make_weights
    from synth.configs import ModelCfg, HeadCfg
    m, n, k = 16, 128, 256                           # 4 k-blocks: the stream-K plan is a single CTA
    x = rnd((m, k), 41, 1, torch.bfloat16).cuda()
    w = rnd((n, k), 41, 2, torch.bfloat16, 0.02).cuda()
    word, diag = gemm_bounded_wait_probe(x, w, skip_unit=2, wait_limit=1024)
    assert word & 2, word                            # TIMEOUT bit
    assert diag[0] in (3, 5), diag                   # gave up waiting for the weight tile / for the accumulator
    assert diag[1] == 0 and diag[3] == 4 and diag[4] == 1 and diag[5:8] == [m, n, 4], diag
    mc = ModelCfg(1, 256, 4, 64, 512, 1024, dtype="bf16")
    hc = HeadCfg(1, 1, False)
    g = Hydra(mc, hc, [-1, 0], {kk: v.cuda() for kk, v in make_weights(mc, hc, 8).items()}, 1, 32)
    gemm_bounded_wait_probe(x, w, skip_unit=1, wait_limit=512, status_words=g.get_buffer("STATUS"))
    with pytest.raises(HydraError, match="timed out"):
        g.poll_status()
    g.poll_status()                                  # cleared by the poll
    g.close()
    ref = x.double().cpu() @ w.double().cpu().T
    out = gemm(x, w, mode=0).cpu().double()          # the device and the library are fine afterwards
    assert float((out - ref).abs().max()) <= 1e-5 * float(ref.abs().max()) + 1e-6 * k ** 0.5

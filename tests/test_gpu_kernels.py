"""Kernel-level parity through the C ABI: the tensor-core GEMM, the SIMT GEMM and tree attention against
their plain definitions evaluated by the oracle's routines / torch CPU float64."""
import pytest
import torch

from oracle.hydra_oracle import masked_attention, TreeTables
from synth import normal_, load_tree
from tests.parity import split_hi_lo, split_f16

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


def _attention_case(case):
    if case == "ragged_batch":
        return 3, 3, 700, [0, 333, 600], None      # empty cache, a cache of several tiles with a ragged tail, long
    if case == "one_long":
        return 1, 2, 1500, [1391], None            # few pairs: the most chunks per pair
    return 2, 2, 400, [130, 64], None


def _dev(x, planes):
    """Operand tensor on the device: as is, or float values as float16 hi / lo planes; and the values the kernel sees."""
    if planes == 1:
        return x.cuda(), x
    sp = split_f16(x)
    return sp.cuda(), sp.float().sum(0)


@pytest.mark.parametrize("dtype,planes", [(torch.float32, 1), (torch.float16, 1), (torch.float16, 2)])
@pytest.mark.parametrize("hd", [64, 128])
@pytest.mark.parametrize("case", ["ragged_batch", "one_long"])
def test_tree_attention_matches_masked_softmax(dtype, planes, hd, case):
    """Tree attention against the plain masked softmax of the oracle on the stored operand values.  float32: the SIMT
    kernel.  float16: the tensor-core kernel (bfloat16 hi + lo result).  One plane: the error budget is the float16
    rounding of the softmax weights (2^-12 relative); two planes (hi + lo): the bfloat16 hi/lo rounding of the result
    (2^-17) and float accumulation."""
    from paper_2402_05109_b200 import tree_attention
    parent = load_tree("tree63_d4")
    t = TreeTables(parent)
    tc = t.T
    B, H, S, pos0, _ = _attention_case(case)
    n_rows = [tc, tc, 17][:B] if B == 3 else [tc] * B       # ragged row counts (rows beyond n_rows are ignored)
    src = torch.float32 if planes == 2 else dtype
    kc = rnd((B, H, S, hd), 21, 1, src)
    vc = rnd((B, H, S, hd), 21, 2, src)
    q = rnd((B * tc, H, hd), 21, 3, src)
    # slots past the end of a sequence hold non-finite garbage: it must not leak into the result
    for b in range(B):
        kc[b, :, pos0[b] + n_rows[b]:] = float("nan")
        vc[b, :, pos0[b] + n_rows[b]:] = float("inf")
    mask = torch.tensor([a - (1 << 64) if a >= (1 << 63) else a for a in t.anc_mask], dtype=torch.int64)
    out_planes = 2 if dtype == torch.float16 else 1
    (q_d, q), (k_d, kc), (v_d, vc) = _dev(q, planes), _dev(kc, planes), _dev(vc, planes)
    out = tree_attention(q_d, k_d, v_d, torch.tensor(pos0, dtype=torch.int32).cuda(),
                         torch.tensor(n_rows, dtype=torch.int32).cuda(), mask.cuda(), tc, out_planes=out_planes).float().cpu()
    out = (out.sum(0) if out_planes == 2 else out).view(B, tc, H, hd)
    for b in range(B):
        n, L = n_rows[b], pos0[b] + n_rows[b]
        allowed = torch.cat([torch.ones(n, pos0[b], dtype=torch.bool), t.allowed[:n, :n]], dim=1)
        k = kc[b, :, :L].permute(1, 0, 2).double()
        v = vc[b, :, :L].permute(1, 0, 2).double()
        ref = masked_attention(q.view(B, tc, H, hd)[b, :n].double(), k, v, allowed)   # q, k, v hold the stored values
        err = float((out[b, :n].double() - ref).abs().max())
        assert err <= (2e-5 if dtype == torch.float32 else (1.5e-3 if planes == 1 else 1e-4)), err
        assert torch.isfinite(out[b]).all()
        assert float(out[b, n:].abs().max()) == 0.0 if n < tc else True       # unused rows come back as zeros


@pytest.mark.parametrize("planes", [1, 2])
@pytest.mark.parametrize("hd", [64, 128])
def test_tree_attention_rescales_when_the_maximum_climbs(hd, planes):
    """Keys whose scores grow along the sequence (each 64-row tile's maximum exceeds the previous one's by more than the
    kernel's rescale step of 8 in the exp2 domain): the running reference maximum must move at every tile and the
    output accumulator in tensor memory must be rescaled on the way."""
    from paper_2402_05109_b200 import tree_attention
    B, H, S, tc = 1, 2, 600, 64
    pos0, n_rows = [500], [tc]
    # q = noise + 1, k = small noise + 1.5 * (tile index): a key of tile t scores about 1.5 t sqrt(hd) on every row
    src = torch.float32 if planes == 2 else torch.float16
    q = (rnd((B * tc, H, hd), 22, 3, torch.float32) + 1.0).to(src)
    ramp = (torch.arange(S, dtype=torch.float32) / 64.0).floor()
    kc = (rnd((B, H, S, hd), 22, 1, torch.float32) * 0.05 + 1.5 * ramp[None, None, :, None]).to(src)
    vc = rnd((B, H, S, hd), 22, 2, src)
    (q_d, q), (k_d, kc), (v_d, vc) = _dev(q, planes), _dev(kc, planes), _dev(vc, planes)
    mask = torch.tensor([(1 << (i + 1)) - 1 if i < 63 else -1 for i in range(tc)], dtype=torch.int64)     # chain
    out = tree_attention(q_d, k_d, v_d, torch.tensor(pos0, dtype=torch.int32).cuda(),
                         torch.tensor(n_rows, dtype=torch.int32).cuda(), mask.cuda(), tc, out_planes=2).float().cpu().sum(0)
    out = out.view(B, tc, H, hd)
    L = pos0[0] + tc
    allowed = torch.cat([torch.ones(tc, pos0[0], dtype=torch.bool), torch.tril(torch.ones(tc, tc, dtype=torch.bool))], dim=1)
    ref = masked_attention(q.view(B, tc, H, hd)[0].double(), kc[0, :, :L].permute(1, 0, 2).double(),
                           vc[0, :, :L].permute(1, 0, 2).double(), allowed)
    scores = torch.einsum("nhd,lhd->hnl", q.view(B, tc, H, hd)[0].double(), kc[0, :, :L].permute(1, 0, 2).double()) / hd ** 0.5
    tile_max = torch.stack([scores[..., i:i + 64].max(dim=-1).values for i in range(0, 448, 64)])          # [tiles][H][rows]
    assert float(((tile_max[1:] - tile_max[:-1]) * 1.4427).min()) > 8.0       # every tile forces a rescale on every row
    assert float((out[0].double() - ref).abs().max()) <= (1.5e-3 if planes == 1 else 1e-4)


@pytest.mark.parametrize("hd,tc,planes", [(128, 128, 1), (64, 100, 1), (64, 128, 2), (128, 64, 2), (128, 40, 1), (128, 128, 2), (128, 90, 2)])
def test_causal_chunk_attention(hd, tc, planes):
    """mask = NULL: a causal chunk of up to 128 rows on top of the committed slots (the prompt pass)."""
    from paper_2402_05109_b200 import tree_attention
    B, H, S = 2, 3, 400
    pos0, n_rows = [256, 0], [tc, max(1, tc - 37)]
    src = torch.float32 if planes == 2 else torch.float16
    (q_d, q), (k_d, kc), (v_d, vc) = (_dev(rnd(shape, 23, i, src), planes)
                                      for i, shape in ((3, (B * tc, H, hd)), (1, (B, H, S, hd)), (2, (B, H, S, hd))))
    out = tree_attention(q_d, k_d, v_d, torch.tensor(pos0, dtype=torch.int32).cuda(),
                         torch.tensor(n_rows, dtype=torch.int32).cuda(), None, tc, out_planes=2).float().cpu().sum(0)
    out = out.view(B, tc, H, hd)
    for b in range(B):
        n, L = n_rows[b], pos0[b] + n_rows[b]
        allowed = torch.cat([torch.ones(n, pos0[b], dtype=torch.bool), torch.tril(torch.ones(n, n, dtype=torch.bool))], dim=1)
        ref = masked_attention(q.view(B, tc, H, hd)[b, :n].double(), kc[b, :, :L].permute(1, 0, 2).double(),
                               vc[b, :, :L].permute(1, 0, 2).double(), allowed)
        assert float((out[b, :n].double() - ref).abs().max()) <= (1.5e-3 if planes == 1 else 1e-4)


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

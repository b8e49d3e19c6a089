"""hydra_gemm_noalloc: the split-K GEMM for callers that cannot allocate device memory (a serving loop that
must avoid the allocator's locks and implicit synchronisation, a plugin inside a fixed memory budget).
Its partial sums live in an 8 MiB array inside the library, shared by all calls, so the test runs two
different problems back to back and checks each against hydra_gemm, which takes a caller-supplied buffer."""
import pytest
import torch

from synth import normal_

pytestmark = pytest.mark.gpu


def _operands(m, n, k, seed):
    x = normal_(torch.empty(m, k, dtype=torch.bfloat16), seed, 1, 1.0).cuda()
    w = normal_(torch.empty(n, k, dtype=torch.bfloat16), seed, 2, 0.02).cuda()
    return x, w


def test_noalloc_gemm_matches_gemm_on_two_calls_in_a_row():
    from paper_2402_05109_b200 import gemm, gemm_noalloc, HydraError
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # second problem is smaller than the first, so stale partial sums of call 1 sit beside the ones call 2 uses
    for (m, n, k, seed) in [(64, 4096, 2048, 31), (11, 256, 1280, 32)]:
        x, w = _operands(m, n, k, seed)
        out = torch.full((m, n), float("nan"), dtype=torch.float32, device="cuda")
        gemm_noalloc(x, w, out, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        ref = gemm(x, w, mode=0)
        exact = x.double().cpu() @ w.double().cpu().T
        tol = 1e-5 * float(exact.abs().max()) + 1e-6 * k ** 0.5        # same bound as the GEMM parity tests
        assert float((out.double().cpu() - exact).abs().max()) <= tol
        assert torch.equal(out, ref)          # same kernels, same split order: bit-identical
    # a problem whose partial sums exceed the built-in scratch is refused with a clear error, nothing launched
    x, w = _operands(256, 16384, 256, 33)
    out = torch.zeros(256, 16384, dtype=torch.float32, device="cuda")
    with pytest.raises(HydraError, match="8 MiB"):
        gemm_noalloc(x, w, out, status)
    assert float(out.abs().max()) == 0.0

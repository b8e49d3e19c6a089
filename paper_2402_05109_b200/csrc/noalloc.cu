// Stream-K GEMM entry point for callers that cannot allocate device memory.
//
// Who needs it: code that runs where cudaMalloc is off limits -- inside a latency-critical serving loop that
// must not take the allocator's locks or trigger an implicit device synchronisation, in a plugin whose host
// gave it a fixed memory budget, or after the process has handed all free device memory to a pool it does not
// control.  hydra_gemm makes such a caller bring the partial-sum buffer itself; this variant keeps
// that buffer inside the library image instead.
#include "launch.h"

namespace {

// Partial sums of the stream-K GEMM: hydra_gemm_partial_floats(m, n, k, 1, 0) floats.  8 MiB per GPU that loads the library, held until
// the process exits.  Shared by every call (and every thread) on that GPU.
constexpr size_t NOALLOC_SCRATCH_BYTES = 8u << 20;
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_SCRATCH_BYTES];

// device address of the array, per device; 0 until the first call on that device has looked it up (any thread may
// make that call: the slot is an atomic, and two threads racing on it store the same address)
std::atomic<uintptr_t> g_scratch_ptr[hydra::MAX_DEVICES];

}  // namespace

extern "C" hydra_status hydra_gemm_noalloc(const void* x, const void* w, float* out, int m, int n, int k, int32_t* status,
                                           void* stream) {
  using namespace hydra;
  if (!x || !w || !out || !status || m < 1 || n < 1 || k < 1) return HYDRA_ERR_INVALID;
  if (n % 128 || k % 64) return HYDRA_ERR_UNSUPPORTED;
  int slots = 1;
  gemm_tc_plan(m, n, k, nullptr, &slots);
  if ((size_t)slots * (size_t)m * (size_t)n * sizeof(float) > NOALLOC_SCRATCH_BYTES) {
    set_last_error("hydra_gemm_noalloc: the partial sums exceed the 8 MiB built-in scratch", cudaErrorInvalidValue);
    return HYDRA_ERR_CAPACITY;
  }
  int dev = -1;
  HYDRA_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= MAX_DEVICES) return HYDRA_ERR_UNSUPPORTED;
  uintptr_t addr = g_scratch_ptr[dev].load(std::memory_order_acquire);
  if (!addr) {
    // The array's name is only a host-side handle here; the kernels need its address on the current device.
    void* p = nullptr;
    HYDRA_CUDA(cudaGetSymbolAddress(&p, g_noalloc_scratch));
    addr = reinterpret_cast<uintptr_t>(p);
    g_scratch_ptr[dev].store(addr, std::memory_order_release);
  }
  if (!gemm_tc_available()) { set_last_error("cuTensorMapEncodeTiled entry point", cudaErrorUnknown); return HYDRA_ERR_CUDA; }
  cudaStream_t st = (cudaStream_t)stream;
  float* part = reinterpret_cast<float*>(addr);
  // every partial element the reduction reads is written by the GEMM first, so nothing has to be cleared
  SplitDesc sd;
  HYDRA_TRY(gemm_tc((const bf16*)x, m, 1, (const bf16*)w, part, m, n, k, &sd, status, nullptr, nullptr, st));
  return reduce_splits(part, sd, out, m, n, st);
}

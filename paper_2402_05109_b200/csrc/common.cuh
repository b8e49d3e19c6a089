// Shared device/host helpers of libhydra (internal).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <atomic>
#include "../../include/hydra.h"

namespace hydra {

typedef __nv_bfloat16 bf16;

// Device status word bits (sticky until polled).
enum : int { ST_BOUNDS = 1, ST_TIMEOUT = 2 };

// Launch bookkeeping: every launcher reports through this so the library can count its kernels.
extern thread_local long long* g_launch_counter;
void set_last_error(const char* what, cudaError_t e);
inline void count_launch() { if (g_launch_counter) ++*g_launch_counter; }

// Per-device one-time set-up (function attributes, SM counts) is keyed by the current device, so that one process
// may drive several GPUs; the flags are atomics because any thread may make the first call on a device.
constexpr int MAX_DEVICES = 64;
inline int current_device() { int d = 0; return cudaGetDevice(&d) == cudaSuccess && d >= 0 && d < MAX_DEVICES ? d : 0; }
struct PerDeviceFlag {
  std::atomic<bool> done[MAX_DEVICES];
  bool get() const { return done[current_device()].load(std::memory_order_acquire); }
  void set() { done[current_device()].store(true, std::memory_order_release); }
};
inline int sm_count() {
  static std::atomic<int> n[MAX_DEVICES];
  const int dev = current_device();
  int v = n[dev].load(std::memory_order_relaxed);
  if (v > 0) return v;
  if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v < 1) v = 148;
  n[dev].store(v, std::memory_order_relaxed);
  return v;
}

#define HYDRA_CUDA(call)                                                        \
  do { cudaError_t e_ = (call);                                                 \
       if (e_ != cudaSuccess) { hydra::set_last_error(#call, e_); return HYDRA_ERR_CUDA; } } while (0)

#define HYDRA_LAUNCH_CHECK()                                                    \
  do { hydra::count_launch(); cudaError_t e_ = cudaGetLastError();              \
       if (e_ != cudaSuccess) { hydra::set_last_error("kernel launch", e_); return HYDRA_ERR_CUDA; } } while (0)

#define HYDRA_TRY(call) do { hydra_status s_ = (call); if (s_ != HYDRA_OK) return s_; } while (0)

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<bf16>(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
// Programmatic dependent launch: every kernel of the library starts with pdl_trigger() (lets the next kernel
// in the stream get resident early) and pdl_wait() (blocks until the preceding kernel has completed and its
// writes are visible) before it touches memory, so dependencies stay transitive along the stream.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ float silu_f(float x) { return x / (1.0f + __expf(-x)); }

// Where the partial sums of a GEMM output element live.  The tensor-core GEMM cuts the (tile, k-block) line
// into ranges of q units per CTA; tile t = (m / mt) * n_tiles + (n >> bn_shift) (weight tiles of 128 or 256 rows)
// owns units [t*kb, (t+1)*kb), so its
// partial sums sit in slots 0 .. split_count-1 (slot s at part + s*stride + m*N + n), one per CTA that
// touched the tile, in CTA order.  A single-slot output is described by q = kb = 1.
struct SplitDesc { int q, kb, n_tiles, mt, bn_shift; size_t stride; };
__host__ __device__ __forceinline__ int split_count(const SplitDesc& sd, int m, int n) {
  const int u0 = ((m / sd.mt) * sd.n_tiles + (n >> sd.bn_shift)) * sd.kb;   // tiles * kb stays far below 2^31
  return (u0 + sd.kb - 1) / sd.q - u0 / sd.q + 1;
}
// acc[u] = sum over the ns[u] slots of the four floats at element offset off[u] of a slot (all loads of a round in flight together)
template <int U, int PMAX = 6>
__device__ __forceinline__ void sum_slots_multi(const float* part, size_t stride, const size_t (&off)[U], const int (&ns)[U], float4 (&acc)[U]) {
  int mx = 0;
#pragma unroll
  for (int u = 0; u < U; ++u) { acc[u] = make_float4(0.f, 0.f, 0.f, 0.f); mx = max(mx, ns[u]); }
#pragma unroll
  for (int p = 0; p < PMAX; ++p) {
    float4 v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) v[u] = p < ns[u] ? __ldcg(reinterpret_cast<const float4*>(part + p * stride + off[u])) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int u = 0; u < U; ++u) { acc[u].x += v[u].x; acc[u].y += v[u].y; acc[u].z += v[u].z; acc[u].w += v[u].w; }
  }
  for (int p = PMAX; p < mx; ++p)
#pragma unroll
    for (int u = 0; u < U; ++u)
      if (p < ns[u]) {
        const float4 v = __ldcg(reinterpret_cast<const float4*>(part + p * stride + off[u]));
        acc[u].x += v.x; acc[u].y += v.y; acc[u].z += v.z; acc[u].w += v.w;
      }
}
// one float: the slots of element `idx` summed in slot order, the first PMAX loads in flight together
template <int PMAX = 12>
__device__ __forceinline__ float sum_slots_scalar(const float* part, size_t stride, size_t idx, int ns) {
  float v[PMAX];
#pragma unroll
  for (int p = 0; p < PMAX; ++p) v[p] = p < ns ? __ldcg(part + p * stride + idx) : 0.f;
  float acc = 0.f;
#pragma unroll
  for (int p = 0; p < PMAX; ++p) acc += v[p];
  for (int p = PMAX; p < ns; ++p) acc += __ldcg(part + p * stride + idx);
  return acc;
}
inline SplitDesc single_slot(size_t stride) { return SplitDesc{1, 1, 1, 1 << 30, 7, stride}; }

// Launch with programmatic stream serialisation allowed (see pdl_wait).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Rows of one forward call: `batch` sequences with `tc` row slots each; sequence b uses its first
// n_rows[b] slots (all tc when n_rows is null).  Row i of b has KV slot pos0[b]+i, rotary position
// pos0[b]+depth[i] and may attend to cache slots < pos0[b] and to slot pos0[b]+j iff bit j of mask[i].
struct RowSet {
  int batch, tc;
  const int* n_rows;      // device [batch] or null
  const int* pos0;        // device [batch]
  const int* depth;       // device [tc]
  const uint64_t* mask;   // device [tc]; null: a causal chunk (row i sees new slots 0..i), bfloat16 model path only
};

}  // namespace hydra

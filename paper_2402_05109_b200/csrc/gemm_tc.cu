// Weight-streaming bfloat16 GEMM on the sm_100a tensor cores.
//
//   out[split][m][n] = sum_{k in split} x[m][k] * w[n][k]        (float accumulate, float out)
//
// The weight matrix is the large operand (read once from HBM), the activation slab is small (tree rows
// x batch) and L2 resident, so the roles are swapped with respect to the usual GEMM: a 128-row weight
// tile [128 n][64 k] is the MMA "A" operand (M = 128 TMEM lanes), the activation tile [MT rows][64 k] is
// the "B" operand (N = MT columns).  Both are K-major and land in shared memory through TMA with the
// 128-byte swizzle; accumulators live in tensor memory.  One CTA computes one [128 n] x [MT m] tile for
// one K range (split-K; partial sums are reduced by the consumer kernel, in fixed order).
//
// Warp roles (192 threads): warp 0 = TMA producer (one lane), warp 1 = TMEM allocation + MMA issue
// (one lane), warps 2..5 = epilogue (TMEM -> registers -> global, coalesced along n).
// Every mbarrier wait is bounded: when it runs out the CTA raises ST_TIMEOUT in the status word,
// skips its stores, lets its copies settle, frees its tensor memory and returns.
#include "launch.h"
#include <cuda.h>
#include <map>
#include <mutex>
#include <tuple>

namespace hydra {

namespace {

constexpr int BLOCK_N = 128;             // weight rows per tile (MMA M)
constexpr int BLOCK_K = 64;              // 64 bf16 = 128 bytes = one swizzle row
constexpr int A_BYTES = BLOCK_N * BLOCK_K * 2;
constexpr int SMEM_BUDGET = 200 * 1024;
constexpr uint32_t WAIT_LIMIT = 1u << 24;   // try_wait attempts before giving up

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
  }
  return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major tile stored with the 128-byte swizzle: rows are 128 bytes,
// groups of 8 rows are 1024 bytes apart (stride byte offset), descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFF) >> 4);          // start address
  d |= (uint64_t)1 << 16;                          // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset
  d |= (uint64_t)1 << 46;                          // version
  d |= (uint64_t)2 << 61;                          // SWIZZLE_128B
  return d;
}

// Instruction descriptor: D = f32, A = B = bf16, both K-major, M = 128, N = MT.
__host__ __device__ constexpr uint32_t instr_desc(int mt) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(mt >> 3) << 17) | ((uint32_t)(BLOCK_N >> 4) << 24);
}

template <int MT> struct TileCfg {
  static constexpr int B_BYTES = MT * BLOCK_K * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = (SMEM_BUDGET / STAGE_BYTES) > 10 ? 10 : (SMEM_BUDGET / STAGE_BYTES);
  static constexpr int TMEM_COLS = MT < 32 ? 32 : MT;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

template <int MT>
__global__ void __launch_bounds__(192, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, float* __restrict__ out,
               size_t split_stride, int m, int n, int kblocks, int splits, int* status) {
  using C = TileCfg<MT>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bars = tiles + C::STAGES * C::STAGE_BYTES;          // full[S], empty[S], tmem_full, tmem slot
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (C::STAGES + s); };
  const uint32_t tmem_full_bar = bars + 8u * (2 * C::STAGES);
  const uint32_t tmem_slot = bars + 8u * (2 * C::STAGES + 1);
  __shared__ int s_abort;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * BLOCK_N;
  const int split = blockIdx.y;
  const int m0 = blockIdx.z * MT;
  const int kb_begin = (int)(((long long)split * kblocks) / splits);
  const int kb_end = (int)(((long long)(split + 1) * kblocks) / splits);
  const int nkb = kb_end - kb_begin;

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(tmem_full_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmX) : "memory");
  }
  if (warp == 1) tmem_alloc(tmem_slot, C::TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  uint32_t tmem_base;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

  if (warp == 0) {
    if (lane == 0) {
      for (int kb = 0; kb < nkb; ++kb) {
        const int s = kb % C::STAGES;
        const uint32_t ph = (kb / C::STAGES) & 1;
        if (!mbar_wait(empty_bar(s), ph ^ 1u)) { atomicOr(status, ST_TIMEOUT); s_abort = 1; break; }
        const uint32_t a_dst = tiles + s * C::STAGE_BYTES;
        mbar_arrive_expect_tx(full_bar(s), C::STAGE_BYTES);
        tma_load_2d(a_dst, &tmW, (kb_begin + kb) * BLOCK_K, n0, full_bar(s));
        tma_load_2d(a_dst + A_BYTES, &tmX, (kb_begin + kb) * BLOCK_K, m0, full_bar(s));
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc(MT);
      for (int kb = 0; kb < nkb; ++kb) {
        const int s = kb % C::STAGES;
        const uint32_t ph = (kb / C::STAGES) & 1;
        if (!mbar_wait(full_bar(s), ph)) { atomicOr(status, ST_TIMEOUT); s_abort = 1; break; }
        tc_fence_after();
        const uint32_t a_addr = tiles + s * C::STAGE_BYTES;
        const uint64_t adesc = smem_desc_sw128(a_addr);
        const uint64_t bdesc = smem_desc_sw128(a_addr + A_BYTES);
#pragma unroll
        for (int k = 0; k < BLOCK_K / 16; ++k)           // 16 bf16 = 32 bytes per MMA: +2 in 16-byte units
          umma_bf16(tmem_base, adesc + 2u * k, bdesc + 2u * k, idesc, (uint32_t)((kb | k) != 0));
        umma_commit(empty_bar(s));                       // frees the stage once these MMAs have read it
      }
      umma_commit(tmem_full_bar);
    }
  } else {
    const int quarter = warp & 3;                        // TMEM lanes this warp may read
    bool ok = nkb > 0 && mbar_wait(tmem_full_bar, 0);
    if (!ok && lane == 0) atomicOr(status, ST_TIMEOUT);
    tc_fence_after();
    if (ok && !s_abort) {
      const int col_n = n0 + quarter * 32 + lane;
      float* dst = out + (size_t)split * split_stride + col_n;
#pragma unroll 1
      for (int c = 0; c < MT; c += 16) {
        if (m0 + c >= m) break;
        uint32_t r[16];
        tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c, r);
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (m0 + c + j < m) dst[(size_t)(m0 + c + j) * n] = __uint_as_float(r[j]);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (s_abort) {                                         // let copies in flight land before the CTA retires
    for (int i = 0; i < 2000; ++i) __nanosleep(100);
  }
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, C::TMEM_COLS); }
}

// ---- tensor maps -------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    return (EncodeTiledFn)p;
  }();
  return fn;
}

// 2-D bf16 row-major [rows][cols] tensor, box = [box_rows][64 cols], 128-byte swizzle.
bool get_tensor_map(const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows, CUtensorMap* out) {
  typedef std::tuple<const void*, uint64_t, uint64_t, uint32_t> Key;
  static std::map<Key, CUtensorMap> cache;
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  Key key(ptr, rows, cols, box_rows);
  auto it = cache.find(key);
  if (it != cache.end()) { *out = it->second; return true; }
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {BLOCK_K, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUtensorMap tm;
  CUresult r = fn(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (cache.size() > 4096) cache.clear();
  cache[key] = tm;
  *out = tm;
  return true;
}

template <int MT>
hydra_status launch(const CUtensorMap& tw, const CUtensorMap& tx, float* out, size_t split_stride, int m, int n, int k,
                    int splits, int* status, cudaStream_t st) {
  using C = TileCfg<MT>;
  static bool attr_done = false;
  if (!attr_done) {
    HYDRA_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
    attr_done = true;
  }
  dim3 grid(n / BLOCK_N, splits, (m + MT - 1) / MT);
  gemm_tc_kernel<MT><<<grid, 192, C::SMEM_BYTES, st>>>(tw, tx, out, split_stride, m, n, k / BLOCK_K, splits, status);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

}  // namespace

bool gemm_tc_available() { return encode_fn() != nullptr; }

hydra_status gemm_tc(const bf16* x, int x_rows_alloc, const bf16* w, float* out, size_t split_stride, int m, int n, int k,
                     int splits, int* status, cudaStream_t st) {
  if (m <= 0 || n <= 0 || k <= 0 || n % BLOCK_N || k % BLOCK_K || splits < 1) return HYDRA_ERR_UNSUPPORTED;
  if (((uintptr_t)x | (uintptr_t)w) & 15) return HYDRA_ERR_INVALID;
  if (splits > k / BLOCK_K) return HYDRA_ERR_INVALID;
  int mt = m <= 16 ? 16 : m <= 32 ? 32 : m <= 64 ? 64 : m <= 128 ? 128 : 256;
  if (x_rows_alloc < m) x_rows_alloc = m;
  CUtensorMap tw, tx;
  if (!get_tensor_map(w, (uint64_t)n, (uint64_t)k, BLOCK_N, &tw) ||
      !get_tensor_map(x, (uint64_t)x_rows_alloc, (uint64_t)k, (uint32_t)mt, &tx)) {
    set_last_error("cuTensorMapEncodeTiled", cudaErrorUnknown);
    return HYDRA_ERR_CUDA;
  }
  switch (mt) {
    case 16: return launch<16>(tw, tx, out, split_stride, m, n, k, splits, status, st);
    case 32: return launch<32>(tw, tx, out, split_stride, m, n, k, splits, status, st);
    case 64: return launch<64>(tw, tx, out, split_stride, m, n, k, splits, status, st);
    case 128: return launch<128>(tw, tx, out, split_stride, m, n, k, splits, status, st);
    default: return launch<256>(tw, tx, out, split_stride, m, n, k, splits, status, st);
  }
}

}  // namespace hydra

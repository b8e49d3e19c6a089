// Weight-streaming bfloat16 GEMM on the sm_100a tensor cores: persistent, stream-K, TMA + tcgen05 + TMEM.
//
//   part[slot][m][n] = sum over one K range of x[m][k] * w[n][k]        (float accumulate, float out)
//
// The weight matrix is the large operand (read once from HBM); the activation slab is small (tree rows x
// batch) and L2 resident.  So the roles are swapped with respect to the usual GEMM: a 128-row weight tile
// [128 n][64 k] is the MMA "A" operand (M = 128 TMEM lanes), the activation tile [MT rows][64 k] is the "B"
// operand (N = MT columns).  Both are K-major and land in shared memory through TMA with the 128-byte
// swizzle; accumulators live in tensor memory.
//
// Work decomposition (stream-K): the (tile, k-block) pairs of the whole GEMM are laid out in one line,
// tile-major, and cut into equal contiguous ranges, one per CTA (at most one CTA per SM), so that every SM
// streams the same number of weight bytes without interruption.  A CTA's range covers the tail of one tile,
// possibly whole tiles, and the head of another; each such run is a "segment" whose partial sum goes to
// slot (cta - first cta of the tile) of the partial buffer.  The consumer kernel adds the slots of a tile in
// fixed order (SplitDesc), so results are deterministic.
//
// A unit carries NH = 1 or 2 such weight tiles (256 weight rows in one TMA box) that share the unit's activation
// tile and accumulate side by side in tensor memory: wide outputs use 2.
//
// Warp roles (192 threads): warp 0 = TMA producer (one lane), warp 1 = TMEM allocation + MMA issue (one
// lane), warps 2..5 = epilogue (TMEM -> registers -> global, coalesced along n).  Two accumulator sets in
// TMEM (where 512 columns allow) let the epilogue of one segment overlap the main loop of the next.  The kernel is launched with
// programmatic stream serialisation: weight tiles (which never depend on the preceding kernel) are requested
// before griddepcontrol.wait, activations and all global writes after it.
// Precision: weights are bfloat16 (exact: the reference model's weights are the same bfloat16 values).  The
// activation operand comes as TWO bfloat16 planes, hi = bf16(v) and lo = bf16(v - hi), i.e. about 16 mantissa
// bits; each weight tile is multiplied with both planes into the same accumulator.  This doubles the MMA work
// (irrelevant while the kernel is HBM-bound) and the L2-resident activation traffic, not the HBM traffic, and
// keeps the hidden states within 1e-2 of a float reference over 32+ layers (plain bfloat16 operands drift to
// 4e-2).  x_lo_rows = 0 selects a single plane.
// Every mbarrier wait is bounded: when one runs out the CTA raises ST_TIMEOUT in the status word, stops
// storing, lets its copies settle, frees its tensor memory and returns.
#include "tc.cuh"
#include <map>
#include <mutex>
#include <tuple>

namespace hydra {

// ---- tensor maps -------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
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

bool tensor_map_encoder_available() { return encode_fn() != nullptr; }

bool get_tensor_map(const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows, bool half, CUtensorMap* out) {
  typedef std::tuple<const void*, uint64_t, uint64_t, uint32_t, bool> Key;
  static std::map<Key, CUtensorMap> cache;
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  Key key(ptr, rows, cols, box_rows, half);
  auto it = cache.find(key);
  if (it != cache.end()) { *out = it->second; return true; }
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUtensorMap tm;
  CUresult r = fn(&tm, half ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (cache.size() > 4096) cache.clear();
  cache[key] = tm;
  *out = tm;
  return true;
}

namespace {

using namespace tc;

constexpr int BLOCK_N = 128;             // weight rows per tile (MMA M)
constexpr int BLOCK_K = 64;              // 64 bf16 = 128 bytes = one swizzle row
constexpr int A_BYTES = BLOCK_N * BLOCK_K * 2;

// Instruction descriptor: D = f32, A = B = bf16, both K-major, M = 128, N = MT.
__host__ __device__ constexpr uint32_t instr_desc(int mt) { return instr_desc_f16(1, BLOCK_N, mt, 0); }

// One accumulator buffer (MT columns, plus MT more holding W*lo when `cat`) of this thread's lane -> partial-sum rows
// m0.. of column dst; 64 columns per batch of tensor-memory loads when the tile has that many.
template <int MT>
__device__ __forceinline__ void store_accumulator(uint32_t taddr, bool cat, float* dst, int m0, int m, int n) {
  if constexpr (MT >= 64) {
#pragma unroll 1
    for (int c = 0; c < MT; c += 64) {
      if (m0 + c >= m) break;
      uint32_t r[64];
      if (cat) {
        uint32_t r2[64];
        tmem_ld64x2(taddr + (uint32_t)c, taddr + (uint32_t)(MT + c), r, r2);
#pragma unroll
        for (int j = 0; j < 64; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(r2[j]));
      } else {
        tmem_ld64(taddr + (uint32_t)c, r);
      }
#pragma unroll
      for (int j = 0; j < 64; ++j)
        if (m0 + c + j < m) __stcg(dst + (size_t)(m0 + c + j) * n, __uint_as_float(r[j]));
    }
  } else {
#pragma unroll 1
    for (int c = 0; c < MT; c += 16) {
      if (m0 + c >= m) break;
      uint32_t r[16];
      tmem_ld16(taddr + (uint32_t)c, r);
      if (cat) {                                         // add the W*lo columns
        uint32_t r2[16];
        tmem_ld16(taddr + (uint32_t)(MT + c), r2);
#pragma unroll
        for (int j = 0; j < 16; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(r2[j]));
      }
#pragma unroll
      for (int j = 0; j < 16; ++j)
        if (m0 + c + j < m) __stcg(dst + (size_t)(m0 + c + j) * n, __uint_as_float(r[j]));
    }
  }
}

template <int MT, int BUDGET_KB, int NH = 1> struct TileCfg {        // NH: 128-row weight tiles per unit (they share the activation tile)
  static constexpr int SMEM_BUDGET = BUDGET_KB * 1024;
  static constexpr int B_PLANE = MT * BLOCK_K * 2;               // one activation plane of a stage
  static constexpr int B_BYTES = 2 * B_PLANE;                    // hi + lo
  static constexpr int W_BYTES = NH * A_BYTES;                   // weight rows of a unit: NH * 128
  static constexpr int STAGE_BYTES = W_BYTES + B_BYTES;
  static constexpr int STAGES = (SMEM_BUDGET / STAGE_BYTES) > 10 ? 10 : ((SMEM_BUDGET / STAGE_BYTES) < 2 ? 2 : (SMEM_BUDGET / STAGE_BYTES));
  // Two planes, MT <= 128: the hi and lo activation tiles sit back to back in shared memory and form ONE MMA B
  // operand of 2*MT rows, so each weight tile is read from shared memory once; accumulator columns [0, MT) hold
  // W*hi, [MT, 2MT) hold W*lo and the epilogue adds them.  MT = 256: two accumulating passes over the weight tile.
  static constexpr bool CAT = MT <= 128;
  static constexpr int ACC_COLS = CAT ? (2 * MT < 32 ? 32 : 2 * MT) : MT;   // columns of one accumulator buffer
  static constexpr int NBUF = 2 * NH * ACC_COLS <= 512 ? 2 : 1;   // accumulator sets: two when tensor memory allows
  static constexpr int TMEM_COLS = NBUF * NH * ACC_COLS;          // power of two, <= 512
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 512 /*barriers*/;
};

struct GemmArgs {
  float* part; size_t slot_stride;
  int m, n, kb, n_tiles, total_units, q;
  int x_lo_rows;                 // row offset of the lo plane inside the activation tensor map (0: single plane)
  int* status;
  int* diag;                     // optional int[8]: where the first bounded wait gave up (site, cta, unit, units, grid, m, n, kb)
  uint32_t wait_limit;           // polls before a barrier wait gives up
  int skip_unit;                 // >= 0: CTA 0 leaves out the weight-tile request of this unit (a test of the bounded waits), else -1
};

// Records the first wait that ran out (site: 1 producer/empty, 2 mma/acc-empty, 3 mma/full-w, 4 mma/full-x, 5 epilogue/acc-full).
#define GIVE_UP(site, unit) do { atomicOr(a.status, ST_TIMEOUT); \
    if (a.diag && atomicCAS(a.diag, 0, (site)) == 0) { a.diag[1] = blockIdx.x; a.diag[2] = (unit); a.diag[3] = n_units; \
      a.diag[4] = gridDim.x; a.diag[5] = a.m; a.diag[6] = a.n; a.diag[7] = a.kb; } } while (0)

template <int MT, int BUDGET_KB, int NH>
__global__ void __launch_bounds__(192, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, const GemmArgs a) {
  using C = TileCfg<MT, BUDGET_KB, NH>;
  constexpr int BN = NH * BLOCK_N;                       // weight rows of a unit
  extern __shared__ uint8_t smem_raw[];
  const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bars = tiles + C::STAGES * C::STAGE_BYTES;
  auto fullw_bar = [&](int s) { return bars + 8u * s; };
  auto fullx_bar = [&](int s) { return bars + 8u * (C::STAGES + s); };
  auto empty_bar = [&](int s) { return bars + 8u * (2 * C::STAGES + s); };
  auto accfull_bar = [&](int i) { return bars + 8u * (3 * C::STAGES + i); };
  auto accempty_bar = [&](int i) { return bars + 8u * (3 * C::STAGES + 2 + i); };
  const uint32_t tmem_slot = bars + 8u * (3 * C::STAGES + 4);
  __shared__ int s_abort;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int u_begin = blockIdx.x * a.q;
  const int u_end = min(u_begin + a.q, a.total_units);
  const int n_units = u_end - u_begin;

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(fullw_bar(s), 1); mbar_init(fullx_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(accfull_bar(i), 1); mbar_init(accempty_bar(i), 4); }
    mbar_init_fence();
    prefetch_tensormap(&tmW);
    prefetch_tensormap(&tmX);
    // weights do not depend on the preceding kernel: request the first ring of weight tiles right away, before the
    // CTA-wide set-up (TMEM allocation, barrier hand-over) and before griddepcontrol.wait
    const uint64_t pol_w0 = policy_evict_first();
    const int pre0 = n_units < C::STAGES ? n_units : C::STAGES;
    for (int i = 0; i < pre0; ++i) {
      const int u = u_begin + i, tile = u / a.kb;
      if (u == a.skip_unit) continue;
      mbar_arrive_expect_tx(fullw_bar(i), C::W_BYTES);
      tma_load_2d(tiles + i * C::STAGE_BYTES, &tmW, (u - tile * a.kb) * BLOCK_K, (tile % a.n_tiles) * BN, fullw_bar(i), pol_w0);
    }
  }
  if (warp == 1) tmem_alloc(tmem_slot, C::TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  grid_dep_launch();                       // all CTAs of this grid are resident: let the next kernel get ready
  uint32_t tmem_base;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

  if (warp == 0) {
    if (lane == 0) {
      const uint64_t pol_w = policy_evict_first(), pol_x = policy_evict_last();
      const int pre = n_units < C::STAGES ? n_units : C::STAGES;      // weight tiles already requested in the prologue
      // (k column, weight row, activation row) of the unit being issued, advanced without divisions
      int kcol = 0, nrow = 0, mrow = 0;
      if (n_units > 0) {
        const int tile = u_begin / a.kb;
        kcol = (u_begin - tile * a.kb) * BLOCK_K; nrow = (tile % a.n_tiles) * BN; mrow = (tile / a.n_tiles) * MT;
      }
      const int kend = a.kb * BLOCK_K, nend = a.n_tiles * BN, lo_rows = a.x_lo_rows;
      const uint32_t x_bytes = lo_rows ? C::B_BYTES : C::B_PLANE;
      int s = 0; uint32_t eph = 1;                       // ring stage, parity of its empty barrier
      grid_dep_wait();                     // activations are the preceding kernel's output
      for (int i = 0; i < n_units; ++i) {
        const uint32_t a_dst = tiles + s * C::STAGE_BYTES;
        if (i >= pre) {
          if (!mbar_wait(empty_bar(s), eph, a.wait_limit)) { GIVE_UP(1, i); s_abort = 1; break; }
          if (u_begin + i != a.skip_unit) {
            mbar_arrive_expect_tx(fullw_bar(s), C::W_BYTES);
            tma_load_2d(a_dst, &tmW, kcol, nrow, fullw_bar(s), pol_w);
          }
        }
        mbar_arrive_expect_tx(fullx_bar(s), x_bytes);
        tma_load_2d(a_dst + C::W_BYTES, &tmX, kcol, mrow, fullx_bar(s), pol_x);
        if (lo_rows) tma_load_2d(a_dst + C::W_BYTES + C::B_PLANE, &tmX, kcol, lo_rows + mrow, fullx_bar(s), pol_x);
        if (++s == C::STAGES) { s = 0; eph ^= 1u; }
        if ((kcol += BLOCK_K) == kend) { kcol = 0; if ((nrow += BN) == nend) { nrow = 0; mrow += MT; } }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const bool cat = C::CAT && a.x_lo_rows != 0;
      const uint32_t idesc = cat ? instr_desc(2 * MT) : instr_desc(MT);
      int seg = 0, s = 0;
      uint32_t ph = 0;                                   // ring stage, parity of its full barriers
      bool ok = true;
      const bool two_pass = a.x_lo_rows && !cat;
      int seg_len = n_units > 0 ? min((u_begin / a.kb + 1) * a.kb, u_end) - u_begin : 0;      // first segment: the tail of a tile
      for (int i = 0; i < n_units && ok;) {
        const int acc = seg % C::NBUF;
        const uint32_t acc_ph = (seg / C::NBUF) & 1;
        if (!mbar_wait(accempty_bar(acc), acc_ph ^ 1u, a.wait_limit)) { GIVE_UP(2, i); ok = false; break; }      // epilogue has drained this buffer
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * NH * C::ACC_COLS);
        for (int j = 0; j < seg_len; ++j, ++i) {
          if (!mbar_wait(fullw_bar(s), ph, a.wait_limit)) { GIVE_UP(3, i); ok = false; break; }
          if (!mbar_wait(fullx_bar(s), ph, a.wait_limit)) { GIVE_UP(4, i); ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = tiles + s * C::STAGE_BYTES;
          const uint64_t bdesc = smem_desc_sw128(a_addr + C::W_BYTES);
#pragma unroll
          for (int hh = 0; hh < NH; ++hh) {              // the unit's weight tiles, one accumulator each, same activation tile
            const uint64_t adesc = smem_desc_sw128(a_addr + hh * A_BYTES);
            const uint32_t d_h = tmem_d + (uint32_t)(hh * C::ACC_COLS);
#pragma unroll
            for (int k = 0; k < BLOCK_K / 16; ++k)       // 16 bf16 = 32 bytes per MMA: +2 in 16-byte units
              umma_f16(d_h, adesc + 2u * k, bdesc + 2u * k, idesc, (uint32_t)((j | k) != 0));
            if (two_pass) {                              // the low-order plane of the activations, same weights
              const uint64_t ldesc = smem_desc_sw128(a_addr + C::W_BYTES + C::B_PLANE);
#pragma unroll
              for (int k = 0; k < BLOCK_K / 16; ++k) umma_f16(d_h, adesc + 2u * k, ldesc + 2u * k, idesc, 1u);
            }
          }
          umma_commit(empty_bar(s));                     // frees the stage once these MMAs have read it
          if (++s == C::STAGES) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        umma_commit(accfull_bar(acc));                   // segment complete: hand the accumulator to the epilogue
        ++seg;
        seg_len = min(a.kb, n_units - i);                // every later segment starts a tile
      }
      if (!ok) { atomicOr(a.status, ST_TIMEOUT); s_abort = 1; }
    }
  } else {
    const int quarter = warp & 3;                        // TMEM lanes this warp may read
    const int epi_tid = quarter * 32 + lane;             // column of the tile this thread owns
    grid_dep_wait();                                     // the partial buffer may still be read by the preceding kernel
    int seg = 0;
    for (int i = 0; i < n_units;) {
      const int u = u_begin + i;
      const int tile = u / a.kb;
      const int seg_len = min((tile + 1) * a.kb, u_end) - u;
      const int acc = seg % C::NBUF;
      const uint32_t acc_ph = (seg / C::NBUF) & 1;
      if (!mbar_wait(accfull_bar(acc), acc_ph, a.wait_limit)) { if (lane == 0) GIVE_UP(5, i); break; }
      tc_fence_after();
      const int slot = blockIdx.x - (int)(((long long)tile * a.kb) / a.q);
      const int n0 = (tile % a.n_tiles) * BN, m0 = (tile / a.n_tiles) * MT;
      float* dst = a.part + (size_t)slot * a.slot_stride + n0 + epi_tid;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * NH * C::ACC_COLS);
#pragma unroll
      for (int hh = 0; hh < NH; ++hh)
        store_accumulator<MT>(taddr + (uint32_t)(hh * C::ACC_COLS), C::CAT && a.x_lo_rows != 0, dst + hh * BLOCK_N, m0, a.m, a.n);
      tc_fence_before();
      if (lane == 0) mbar_arrive(accempty_bar(acc));     // the MMA warp may reuse this accumulator
      i += seg_len;
      ++seg;
    }
  }
  __syncwarp();                                          // the one-lane roles rejoin their warps before the block-wide barrier
  tc_fence_before();
  __syncthreads();
  if (s_abort) {                                         // let copies in flight land before the CTA retires
    for (int i = 0; i < 2000; ++i) __nanosleep(100);
  }
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, C::TMEM_COLS); }
}

template <int MT, int BUDGET_KB, int NH>
hydra_status launch_b(const CUtensorMap& tw, const CUtensorMap& tx, const GemmArgs& a, int grid, cudaStream_t st) {
  using C = TileCfg<MT, BUDGET_KB, NH>;
  static PerDeviceFlag attr_done;
  if (!attr_done.get()) {
    HYDRA_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<MT, BUDGET_KB, NH>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
    attr_done.set();
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(192); cfg.dynamicSmemBytes = C::SMEM_BYTES; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  HYDRA_CUDA(cudaLaunchKernelEx(&cfg, gemm_tc_kernel<MT, BUDGET_KB, NH>, tw, tx, a));
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

// Shared memory per CTA: a deep ring, one CTA per SM (a 100 KB ring that lets the CTAs of two consecutive,
// programmatically overlapped GEMMs share an SM measured no faster).
template <int MT, int NH>
hydra_status launch(const CUtensorMap& tw, const CUtensorMap& tx, const GemmArgs& a, int grid, cudaStream_t st) {
  return launch_b<MT, 200, NH>(tw, tx, a, grid, st);
}

}  // namespace

bool gemm_tc_available() { return tensor_map_encoder_available(); }

int gemm_tile_rows(int m) { return m <= 16 ? 16 : m <= 32 ? 32 : m <= 64 ? 64 : m <= 128 ? 128 : 256; }

// Stream-K plan: equal contiguous unit ranges, one per CTA, at most one CTA per SM and at least 4 k-blocks each.
// 128-row weight tiles per unit: outputs of 4096 columns and more take two (half the activation-tile traffic and half
// the issue work per weight byte, a third more weight bytes in flight: -5 % step time at the 7B shape).  Above 64
// activation rows tensor memory holds one set of two accumulators only (the epilogue no longer overlaps the next
// segment), still a small gain.
int gemm_tile_halves(int m, int n) {
  return n % (2 * BLOCK_N) == 0 && n >= 4096 ? 2 : 1;
}

SplitDesc gemm_tc_plan(int m, int n, int k, int* grid, int* max_slots, int force_nh) {
  SplitDesc sd{};
  const int mt = gemm_tile_rows(m);
  const int nh = force_nh ? force_nh : gemm_tile_halves(m, n);
  sd.mt = mt; sd.n_tiles = n / (nh * BLOCK_N); sd.bn_shift = nh == 2 ? 8 : 7; sd.kb = k / BLOCK_K; sd.stride = (size_t)m * n;
  const int tiles = sd.n_tiles * ((m + mt - 1) / mt);
  const long long total = (long long)tiles * sd.kb;
  long long g = sm_count();
  if (g > total / 4) g = total / 4 > 0 ? total / 4 : 1;
  sd.q = (int)((total + g - 1) / g);
  if (grid) *grid = (int)((total + sd.q - 1) / sd.q);
  if (max_slots) {
    int mx = 1;
    for (int t = 0; t < tiles; ++t) {
      long long u0 = (long long)t * sd.kb;
      int ns = (int)((u0 + sd.kb - 1) / sd.q - u0 / sd.q) + 1;
      mx = ns > mx ? ns : mx;
    }
    *max_slots = mx;
  }
  return sd;
}

hydra_status gemm_tc(const bf16* x, int x_rows_alloc, int x_planes, const bf16* w, float* part, int m, int n, int k,
                     SplitDesc* sd_out, int* status, int* diag, const GemmDebug* dbg, cudaStream_t st) {
  if (m <= 0 || n <= 0 || k <= 0 || n % BLOCK_N || k % BLOCK_K || (x_planes != 1 && x_planes != 2)) return HYDRA_ERR_UNSUPPORTED;
  if (((uintptr_t)x | (uintptr_t)w) & 15) return HYDRA_ERR_INVALID;
  int grid = 1;
  SplitDesc sd = gemm_tc_plan(m, n, k, &grid, nullptr, 0);
  if (x_rows_alloc < m) x_rows_alloc = m;
  CUtensorMap tw, tx;
  const int nh = sd.bn_shift == 8 ? 2 : 1;
  if (!get_tensor_map(w, (uint64_t)n, (uint64_t)k, (uint32_t)(nh * BLOCK_N), false, &tw) ||
      !get_tensor_map(x, (uint64_t)x_rows_alloc * x_planes, (uint64_t)k, (uint32_t)sd.mt, false, &tx)) {
    set_last_error("cuTensorMapEncodeTiled", cudaErrorUnknown);
    return HYDRA_ERR_CUDA;
  }
  GemmArgs a{};
  a.part = part; a.slot_stride = sd.stride; a.m = m; a.n = n; a.kb = sd.kb; a.n_tiles = sd.n_tiles;
  a.total_units = sd.n_tiles * ((m + sd.mt - 1) / sd.mt) * sd.kb; a.q = sd.q; a.status = status;
  a.x_lo_rows = x_planes == 2 ? x_rows_alloc : 0; a.diag = diag;
  a.wait_limit = dbg && dbg->wait_limit ? dbg->wait_limit : WAIT_LIMIT; a.skip_unit = dbg ? dbg->skip_unit : -1;
  if (sd_out) *sd_out = sd;
  if (nh == 2) {
    switch (sd.mt) {
      case 16: return launch<16, 2>(tw, tx, a, grid, st);
      case 32: return launch<32, 2>(tw, tx, a, grid, st);
      case 64: return launch<64, 2>(tw, tx, a, grid, st);
      case 128: return launch<128, 2>(tw, tx, a, grid, st);
      default: return launch<256, 2>(tw, tx, a, grid, st);
    }
  }
  switch (sd.mt) {
    case 16: return launch<16, 1>(tw, tx, a, grid, st);
    case 32: return launch<32, 1>(tw, tx, a, grid, st);
    case 64: return launch<64, 1>(tw, tx, a, grid, st);
    case 128: return launch<128, 1>(tw, tx, a, grid, st);
    default: return launch<256, 1>(tw, tx, a, grid, st);
  }
}

}  // namespace hydra

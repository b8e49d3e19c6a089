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
#include "launch.h"
#include <cuda.h>
#include <cstdlib>
#include <map>
#include <mutex>
#include <tuple>

namespace hydra {

namespace {

constexpr int BLOCK_N = 128;             // weight rows per tile (MMA M)
constexpr int BLOCK_K = 64;              // 64 bf16 = 128 bytes = one swizzle row
constexpr int A_BYTES = BLOCK_N * BLOCK_K * 2;
constexpr uint32_t WAIT_LIMIT = 1u << 24;   // try_wait attempts before giving up

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(bar), "l"(policy)
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
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// 64 consecutive accumulator columns of this thread's lane (one wait for the whole batch)
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, uint32_t (&r)[64]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32,%33,%34,%35,%36,%37,%38,%39,%40,%41,%42,%43,%44,%45,%46,%47,%48,%49,%50,%51,%52,%53,%54,%55,%56,%57,%58,%59,%60,%61,%62,%63}, [%64];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
      : "r"(taddr)
      : "memory");
}
// the same for two column ranges at once (the W*hi and W*lo halves of a concatenated accumulator)
__device__ __forceinline__ void tmem_ld64x2(uint32_t taddr0, uint32_t taddr1, uint32_t (&r)[64], uint32_t (&q)[64]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32,%33,%34,%35,%36,%37,%38,%39,%40,%41,%42,%43,%44,%45,%46,%47,%48,%49,%50,%51,%52,%53,%54,%55,%56,%57,%58,%59,%60,%61,%62,%63}, [%128];\n\t"
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%64,%65,%66,%67,%68,%69,%70,%71,%72,%73,%74,%75,%76,%77,%78,%79,%80,%81,%82,%83,%84,%85,%86,%87,%88,%89,%90,%91,%92,%93,%94,%95,%96,%97,%98,%99,%100,%101,%102,%103,%104,%105,%106,%107,%108,%109,%110,%111,%112,%113,%114,%115,%116,%117,%118,%119,%120,%121,%122,%123,%124,%125,%126,%127}, [%129];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63]), "=r"(q[0]), "=r"(q[1]), "=r"(q[2]), "=r"(q[3]), "=r"(q[4]), "=r"(q[5]), "=r"(q[6]), "=r"(q[7]), "=r"(q[8]), "=r"(q[9]), "=r"(q[10]), "=r"(q[11]), "=r"(q[12]), "=r"(q[13]), "=r"(q[14]), "=r"(q[15]), "=r"(q[16]), "=r"(q[17]), "=r"(q[18]), "=r"(q[19]), "=r"(q[20]), "=r"(q[21]), "=r"(q[22]), "=r"(q[23]), "=r"(q[24]), "=r"(q[25]), "=r"(q[26]), "=r"(q[27]), "=r"(q[28]), "=r"(q[29]), "=r"(q[30]), "=r"(q[31]), "=r"(q[32]), "=r"(q[33]), "=r"(q[34]), "=r"(q[35]), "=r"(q[36]), "=r"(q[37]), "=r"(q[38]), "=r"(q[39]), "=r"(q[40]), "=r"(q[41]), "=r"(q[42]), "=r"(q[43]), "=r"(q[44]), "=r"(q[45]), "=r"(q[46]), "=r"(q[47]), "=r"(q[48]), "=r"(q[49]), "=r"(q[50]), "=r"(q[51]), "=r"(q[52]), "=r"(q[53]), "=r"(q[54]), "=r"(q[55]), "=r"(q[56]), "=r"(q[57]), "=r"(q[58]), "=r"(q[59]), "=r"(q[60]), "=r"(q[61]), "=r"(q[62]), "=r"(q[63])
      : "r"(taddr0), "r"(taddr1)
      : "memory");
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
  int flags;                     // bit 0: no L2 eviction hints on the TMA loads (tuning)
  int x_lo_rows;                 // row offset of the lo plane inside the activation tensor map (0: single plane)
  int* status;
  int* diag;                     // optional int[8]: where the first bounded wait gave up (site, cta, unit, units, grid, m, n, kb)
  long long* trace;              // optional [grid][8] nanosecond timestamps of each CTA's phases (tuning aid), or null
};

__device__ __forceinline__ long long global_ns() { long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
// Records the first wait that ran out (site: 1 producer/empty, 2 mma/acc-empty, 3 mma/full-w, 4 mma/full-x, 5 epilogue/acc-full).
#define GIVE_UP(site, unit) do { atomicOr(a.status, ST_TIMEOUT); \
    if (a.diag && atomicCAS(a.diag, 0, (site)) == 0) { a.diag[1] = blockIdx.x; a.diag[2] = (unit); a.diag[3] = n_units; \
      a.diag[4] = gridDim.x; a.diag[5] = a.m; a.diag[6] = a.n; a.diag[7] = a.kb; } } while (0)
#define TRACE(slot) do { if (a.trace) a.trace[blockIdx.x * 8 + (slot)] = global_ns(); } while (0)

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
    TRACE(0);
    s_abort = 0;
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(fullw_bar(s), 1); mbar_init(fullx_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(accfull_bar(i), 1); mbar_init(accempty_bar(i), 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmX) : "memory");
    // weights do not depend on the preceding kernel: request the first ring of weight tiles right away, before the
    // CTA-wide set-up (TMEM allocation, barrier hand-over) and before griddepcontrol.wait
    const uint64_t pol_w0 = policy_evict_first();
    const int pre0 = n_units < C::STAGES ? n_units : C::STAGES;
    for (int i = 0; i < pre0; ++i) {
      const int u = u_begin + i, tile = u / a.kb;
      mbar_arrive_expect_tx(fullw_bar(i), C::W_BYTES);
      tma_load_2d(tiles + i * C::STAGE_BYTES, &tmW, (u - tile * a.kb) * BLOCK_K, (tile % a.n_tiles) * BN, fullw_bar(i), pol_w0);
    }
  }
  if (warp == 1) tmem_alloc(tmem_slot, C::TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (threadIdx.x == 0) TRACE(1);
  grid_dep_launch();                       // all CTAs of this grid are resident: let the next kernel get ready
  uint32_t tmem_base;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

  if (warp == 0) {
    if (lane == 0) {
      uint64_t pol_w = policy_evict_first(), pol_x = policy_evict_last();
      if (a.flags & 1) { asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol_w)); pol_x = pol_w; }
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
      TRACE(2);
      grid_dep_wait();                     // activations are the preceding kernel's output
      for (int i = 0; i < n_units; ++i) {
        const uint32_t a_dst = tiles + s * C::STAGE_BYTES;
        if (i >= pre) {
          if (!mbar_wait(empty_bar(s), eph)) { GIVE_UP(1, i); s_abort = 1; break; }
          mbar_arrive_expect_tx(fullw_bar(s), C::W_BYTES);
          tma_load_2d(a_dst, &tmW, kcol, nrow, fullw_bar(s), pol_w);
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
        if (!mbar_wait(accempty_bar(acc), acc_ph ^ 1u)) { GIVE_UP(2, i); ok = false; break; }      // epilogue has drained this buffer
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * NH * C::ACC_COLS);
        for (int j = 0; j < seg_len; ++j, ++i) {
          if (!mbar_wait(fullw_bar(s), ph)) { GIVE_UP(3, i); ok = false; break; }
          if (!mbar_wait(fullx_bar(s), ph)) { GIVE_UP(4, i); ok = false; break; }
          if (i == 0) TRACE(3);
          tc_fence_after();
          const uint32_t a_addr = tiles + s * C::STAGE_BYTES;
          const uint64_t bdesc = smem_desc_sw128(a_addr + C::W_BYTES);
#pragma unroll
          for (int hh = 0; hh < NH; ++hh) {              // the unit's weight tiles, one accumulator each, same activation tile
            const uint64_t adesc = smem_desc_sw128(a_addr + hh * A_BYTES);
            const uint32_t d_h = tmem_d + (uint32_t)(hh * C::ACC_COLS);
#pragma unroll
            for (int k = 0; k < BLOCK_K / 16; ++k)       // 16 bf16 = 32 bytes per MMA: +2 in 16-byte units
              umma_bf16(d_h, adesc + 2u * k, bdesc + 2u * k, idesc, (uint32_t)((j | k) != 0));
            if (two_pass) {                              // the low-order plane of the activations, same weights
              const uint64_t ldesc = smem_desc_sw128(a_addr + C::W_BYTES + C::B_PLANE);
#pragma unroll
              for (int k = 0; k < BLOCK_K / 16; ++k) umma_bf16(d_h, adesc + 2u * k, ldesc + 2u * k, idesc, 1u);
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
      TRACE(4);
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
      if (!mbar_wait(accfull_bar(acc), acc_ph)) { if (lane == 0) GIVE_UP(5, i); break; }
      if (epi_tid == 0 && i + seg_len >= n_units) TRACE(5);
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
    if (epi_tid == 0) TRACE(6);
  }
  tc_fence_before();
  __syncthreads();
  if (s_abort) {                                         // let copies in flight land before the CTA retires
    for (int i = 0; i < 2000; ++i) __nanosleep(100);
  }
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, C::TMEM_COLS); }
  if (threadIdx.x == 32) TRACE(7);
}

// ---- GEMM chain ----------------------------------------------------------------------------------
// Several GEMMs over the same rows run as ONE persistent kernel: job j's activations are produced from job j-1's
// partial sums by a row-wise step (residual + RMSNorm, or SiLU(gate) * up) that the epilogue warps of all CTAs share
// out among themselves between two grid-wide counters.  The producer warp keeps requesting the next job's weight
// tiles (which depend on nothing) while that step runs, so HBM does not idle across the boundary, and the ramp and
// tail of a separate launch per GEMM and per row-wise kernel disappear.
//   done[j]  (sync[j])      counts CTAs whose partial sums of job j are in memory
//   ready[j] (sync[8 + j])  counts CTAs that finished their share of the step that makes job j's activations
//   sync[16]                counts CTAs at the exit; the last one clears all counters for the next launch
// The grid is launched cooperatively with one CTA per SM, so every CTA is resident and the counters fill;
// every spin is bounded all the same (ST_TIMEOUT + the usual unwinding through the bounded barrier waits).
constexpr int MAX_JOBS = 4;
constexpr uint32_t SPIN_LIMIT = 1u << 22;
struct ChainJob {
  int n, kb, n_tiles, total_units, q, x_lo_rows;
  int op, cols;                  // row-wise step after this job (CHAIN_NONE / CHAIN_RESID_NORM / CHAIN_SILU_MUL), its output width
  size_t slot_stride;
  float* resid; const bf16* gain; bf16* out; size_t out_ps; float* hn; float eps;
};
struct ChainArgs {
  CUtensorMap tmW[MAX_JOBS];
  CUtensorMap tmX[MAX_JOBS];
  ChainJob job[MAX_JOBS];
  float* part; int m, n_jobs; int* status; int* diag; int* sync;
};

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ bool spin_until(const int* p, int target) {
  for (uint32_t it = 0; it < SPIN_LIMIT; ++it) {
    if (ld_acquire(p) >= target) return true;
    __nanosleep(40);
  }
  return false;
}
__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async;" ::: "memory"); }

__device__ __forceinline__ void store_hl4(bf16* dst, size_t lo_off, const float4& v) {
  const __nv_bfloat162 h0 = __floats2bfloat162_rn(v.x, v.y), h1 = __floats2bfloat162_rn(v.z, v.w);
  *reinterpret_cast<uint2*>(dst) = make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
  if (lo_off) {
    const __nv_bfloat162 l0 = __floats2bfloat162_rn(v.x - __low2float(h0), v.y - __high2float(h0));
    const __nv_bfloat162 l1 = __floats2bfloat162_rn(v.z - __low2float(h1), v.w - __high2float(h1));
    *reinterpret_cast<uint2*>(dst + lo_off) = make_uint2(*reinterpret_cast<const uint32_t*>(&l0), *reinterpret_cast<const uint32_t*>(&l1));
  }
}

// act[r][c] = SiLU(gate[r][c]) * up[r][c] from the gate/up partial sums ([r][2 f] per slot): this CTA's share, 128 threads
__device__ void chain_silu_mul(const ChainArgs& a, const ChainJob& J, const SplitDesc& sd, int et) {
  const int f = J.cols;
  const long long items = (long long)a.m * f / 4, step = (long long)gridDim.x * 128;
  for (long long it0 = (long long)blockIdx.x * 128 + et; it0 < items; it0 += 2 * step) {
    size_t off[4]; int ns[4]; float4 acc[4];
    long long e[2] = {it0 * 4, (it0 + step) * 4};
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const bool valid = e[k] < (long long)a.m * f;
      const int r = valid ? (int)(e[k] / f) : 0, c = valid ? (int)(e[k] % f) : 0;
      off[2 * k] = (size_t)r * 2 * f + c; off[2 * k + 1] = off[2 * k] + f;
      ns[2 * k] = valid ? split_count(sd, r, c) : 0; ns[2 * k + 1] = valid ? split_count(sd, r, f + c) : 0;
    }
    sum_slots_multi<4>(a.part, sd.stride, off, ns, acc);
#pragma unroll
    for (int k = 0; k < 2; ++k)
      if (e[k] < (long long)a.m * f) {
        const float4 g = acc[2 * k], u = acc[2 * k + 1];
        store_hl4(J.out + e[k], J.out_ps, make_float4(silu_f(g.x) * u.x, silu_f(g.y) * u.y, silu_f(g.z) * u.z, silu_f(g.w) * u.w));
      }
  }
}

// resid[r] += sum of the partial slots; then (with a gain) out[r] = resid[r] * rsqrt(mean(resid[r]^2) + eps) * gain as hi/lo
// planes (and as float in hn): rows r = cta, cta + grid, ...; 128 threads per row
__device__ void chain_resid_norm(const ChainArgs& a, const ChainJob& J, const SplitDesc& sd, int et, float* red /* smem [4] */) {
  const int d = J.cols;
  for (int r = blockIdx.x; r < a.m; r += gridDim.x) {
    float* xr = J.resid + (size_t)r * d;
    float ss = 0.f;
    for (int c0 = et * 4; c0 < d; c0 += 4 * 512) {
      size_t off[4]; int ns[4]; float4 acc[4], v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int c = c0 + u * 512;
        const bool valid = c < d;
        off[u] = (size_t)r * d + (valid ? c : 0); ns[u] = valid ? split_count(sd, r, c) : 0;
        v[u] = valid ? *reinterpret_cast<const float4*>(xr + c) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
      sum_slots_multi<4>(a.part, sd.stride, off, ns, acc);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int c = c0 + u * 512;
        if (c < d) {
          v[u].x += acc[u].x; v[u].y += acc[u].y; v[u].z += acc[u].z; v[u].w += acc[u].w;
          *reinterpret_cast<float4*>(xr + c) = v[u];
          ss += v[u].x * v[u].x + v[u].y * v[u].y + v[u].z * v[u].z + v[u].w * v[u].w;
        }
      }
    }
    if (!J.gain) continue;
    ss = warp_sum(ss);
    epi_bar();                                           // red[] free again (previous row's readers are done)
    if ((et & 31) == 0) red[et >> 5] = ss;
    epi_bar();
    const float inv = rsqrtf((red[0] + red[1] + red[2] + red[3]) / (float)d + J.eps);
    for (int c = et * 4; c < d; c += 512) {
      float4 v = *reinterpret_cast<const float4*>(xr + c);           // this thread's own stores above
      const uint2 gr = *reinterpret_cast<const uint2*>(J.gain + c);
      const __nv_bfloat162 g0 = *reinterpret_cast<const __nv_bfloat162*>(&gr.x), g1 = *reinterpret_cast<const __nv_bfloat162*>(&gr.y);
      v.x *= inv * __low2float(g0); v.y *= inv * __high2float(g0); v.z *= inv * __low2float(g1); v.w *= inv * __high2float(g1);
      if (J.out) store_hl4(J.out + (size_t)r * d + c, J.out_ps, v);
      if (J.hn) *reinterpret_cast<float4*>(J.hn + (size_t)r * d + c) = v;
    }
  }
}

#define CHAIN_GIVE_UP(site, jj, ii) do { atomicOr(a.status, ST_TIMEOUT); \
    if (a.diag && atomicCAS(a.diag, 0, (site)) == 0) { a.diag[1] = blockIdx.x; a.diag[2] = (ii); a.diag[3] = (jj); \
      a.diag[4] = gridDim.x; a.diag[5] = a.m; a.diag[6] = a.job[jj].n; a.diag[7] = a.job[jj].kb; } } while (0)

template <int MT>
__global__ void __launch_bounds__(192, 1) gemm_chain_kernel(const __grid_constant__ ChainArgs a) {
  using C = TileCfg<MT, 200>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bars = tiles + C::STAGES * C::STAGE_BYTES;
  auto fullw_bar = [&](int s) { return bars + 8u * s; };
  auto fullx_bar = [&](int s) { return bars + 8u * (C::STAGES + s); };
  auto empty_bar = [&](int s) { return bars + 8u * (2 * C::STAGES + s); };
  auto accfull_bar = [&](int i) { return bars + 8u * (3 * C::STAGES + i); };
  auto accempty_bar = [&](int i) { return bars + 8u * (3 * C::STAGES + 2 + i); };
  const uint32_t tmem_slot = bars + 8u * (3 * C::STAGES + 4);
  __shared__ int s_abort, s_flag;
  __shared__ float s_red[4];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = gridDim.x;
  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(fullw_bar(s), 1); mbar_init(fullx_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(accfull_bar(i), 1); mbar_init(accempty_bar(i), 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    for (int j = 0; j < a.n_jobs; ++j) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&a.tmW[j]) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&a.tmX[j]) : "memory");
    }
  }
  if (warp == 1) tmem_alloc(tmem_slot, C::TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  grid_dep_launch();
  uint32_t tmem_base;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
  const bool cat = C::CAT && a.job[0].x_lo_rows != 0;

  if (warp == 0) {
    if (lane == 0) {
      const uint64_t pol_w = policy_evict_first(), pol_x = policy_evict_last();
      int ws = 0; uint32_t wph = 1;                      // ring stage and empty-barrier parity of the next weight tile (all jobs)
      bool ok = true;
      for (int j = 0; j < a.n_jobs && ok; ++j) {
        const ChainJob& J = a.job[j];
        const CUtensorMap* tw = &a.tmW[j];
        const CUtensorMap* tx = &a.tmX[j];
        const int kb = J.kb, n_tiles = J.n_tiles, lo_rows = J.x_lo_rows;
        const int ub = blockIdx.x * J.q, nu = max(min(ub + J.q, J.total_units) - ub, 0);
        const int pre = nu < C::STAGES ? nu : C::STAGES;
        // (k-block, weight-tile row, activation-tile row) of the next weight / activation load, advanced without divisions
        int wk = 0, wn = 0, xk = 0, xn = 0, xm = 0, xs = ws;
        if (nu > 0) {
          const int tile = ub / kb;
          wk = xk = (ub - tile * kb) * BLOCK_K;
          wn = xn = (tile % n_tiles) * BLOCK_N;
          xm = (tile / n_tiles) * MT;
        }
        const int kend = kb * BLOCK_K, nend = n_tiles * BLOCK_N;
        auto issue_w = [&](int i) {
          if (!mbar_wait(empty_bar(ws), wph)) { CHAIN_GIVE_UP(1, j, i); return false; }
          mbar_arrive_expect_tx(fullw_bar(ws), A_BYTES);
          tma_load_2d(tiles + ws * C::STAGE_BYTES, tw, wk, wn, fullw_bar(ws), pol_w);
          if (++ws == C::STAGES) { ws = 0; wph ^= 1u; }
          if ((wk += BLOCK_K) == kend) { wk = 0; if ((wn += BLOCK_N) == nend) wn = 0; }
          return true;
        };
        for (int i = 0; i < pre && ok; ++i) ok = issue_w(i);       // weights first: they wait for nothing but ring space
        if (!ok) break;
        if (j == 0) grid_dep_wait();                     // the first job's activations are the preceding kernel's output
        else {
          if (!spin_until(a.sync + 8 + j, G)) { CHAIN_GIVE_UP(6, j, 0); ok = false; break; }
          fence_async_proxy();                           // the rows were written with ordinary stores, TMA reads them
        }
        const uint32_t x_bytes = lo_rows ? C::B_BYTES : C::B_PLANE;
        for (int i = 0; i < nu; ++i) {
          if (i >= pre && !(ok = issue_w(i))) break;
          const uint32_t b_dst = tiles + xs * C::STAGE_BYTES + A_BYTES;
          mbar_arrive_expect_tx(fullx_bar(xs), x_bytes);
          tma_load_2d(b_dst, tx, xk, xm, fullx_bar(xs), pol_x);
          if (lo_rows) tma_load_2d(b_dst + C::B_PLANE, tx, xk, lo_rows + xm, fullx_bar(xs), pol_x);
          if (++xs == C::STAGES) xs = 0;
          if ((xk += BLOCK_K) == kend) { xk = 0; if ((xn += BLOCK_N) == nend) { xn = 0; xm += MT; } }
        }
      }
      if (!ok) s_abort = 1;
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = cat ? instr_desc(2 * MT) : instr_desc(MT);
      int seg = 0, st_ = 0;
      uint32_t ph = 0;                                   // ring stage and full-barrier parity of the next unit (all jobs)
      bool ok = true;
      for (int j = 0; j < a.n_jobs && ok; ++j) {
        const ChainJob& J = a.job[j];
        const int kb = J.kb;
        const bool two_pass = J.x_lo_rows && !cat;
        const int ub = blockIdx.x * J.q, ue = min(ub + J.q, J.total_units), nu = max(ue - ub, 0);
        int seg_len = nu > 0 ? min((ub / kb + 1) * kb, ue) - ub : 0;       // the first segment: the tail of a tile
        for (int i = 0; i < nu && ok;) {
          const int acc = seg & 1;
          if (!mbar_wait(accempty_bar(acc), ((seg >> 1) & 1) ^ 1u)) { CHAIN_GIVE_UP(2, j, i); ok = false; break; }
          tc_fence_after();
          const uint32_t tmem_d = tmem_base + (uint32_t)(acc * C::ACC_COLS);
          for (int k2 = 0; k2 < seg_len; ++k2, ++i) {
            if (!mbar_wait(fullw_bar(st_), ph)) { CHAIN_GIVE_UP(3, j, i); ok = false; break; }
            if (!mbar_wait(fullx_bar(st_), ph)) { CHAIN_GIVE_UP(4, j, i); ok = false; break; }
            tc_fence_after();
            const uint32_t a_addr = tiles + st_ * C::STAGE_BYTES;
            const uint64_t adesc = smem_desc_sw128(a_addr), bdesc = smem_desc_sw128(a_addr + A_BYTES);
#pragma unroll
            for (int k = 0; k < BLOCK_K / 16; ++k) umma_bf16(tmem_d, adesc + 2u * k, bdesc + 2u * k, idesc, (uint32_t)((k2 | k) != 0));
            if (two_pass) {
              const uint64_t ldesc = smem_desc_sw128(a_addr + A_BYTES + C::B_PLANE);
#pragma unroll
              for (int k = 0; k < BLOCK_K / 16; ++k) umma_bf16(tmem_d, adesc + 2u * k, ldesc + 2u * k, idesc, 1u);
            }
            umma_commit(empty_bar(st_));
            if (++st_ == C::STAGES) { st_ = 0; ph ^= 1u; }
          }
          if (!ok) break;
          umma_commit(accfull_bar(acc));
          ++seg;
          seg_len = min(kb, nu - i);                     // every later segment starts a tile
        }
      }
      if (!ok) { atomicOr(a.status, ST_TIMEOUT); s_abort = 1; }
    }
  } else {
    const int quarter = warp & 3;
    const int et = quarter * 32 + lane;
    grid_dep_wait();
    int seg = 0;
    bool ok = true;
    for (int j = 0; j < a.n_jobs && ok; ++j) {
      const ChainJob& J = a.job[j];
      const int ub = blockIdx.x * J.q, ue = min(ub + J.q, J.total_units), nu = max(ue - ub, 0);
      for (int i = 0; i < nu;) {
        const int u = ub + i, tile = u / J.kb;
        const int seg_len = min((tile + 1) * J.kb, ue) - u;
        const int acc = seg & 1;
        if (!mbar_wait(accfull_bar(acc), (seg >> 1) & 1)) { if (lane == 0) CHAIN_GIVE_UP(5, j, i); ok = false; break; }
        tc_fence_after();
        const int slot = blockIdx.x - (int)(((long long)tile * J.kb) / J.q);
        const int n0 = (tile % J.n_tiles) * BLOCK_N, m0 = (tile / J.n_tiles) * MT;
        float* dst = a.part + (size_t)slot * J.slot_stride + n0 + et;
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * C::ACC_COLS);
        store_accumulator<MT>(taddr, cat, dst, m0, a.m, J.n);
        tc_fence_before();
        if (lane == 0) mbar_arrive(accempty_bar(acc));
        i += seg_len;
        ++seg;
      }
      if (!ok || J.op == CHAIN_NONE) continue;
      // every CTA's partial sums of this job in memory -> this CTA's share of the row-wise step -> next job's rows ready
      __threadfence();
      epi_bar();
      if (et == 0) {
        atomicAdd(a.sync + j, 1);
        s_flag = spin_until(a.sync + j, G) ? 1 : 0;
        if (!s_flag) CHAIN_GIVE_UP(7, j, 0);
      }
      epi_bar();
      if (!s_flag) { ok = false; break; }
      const SplitDesc sd{J.q, J.kb, J.n_tiles, MT, 7, J.slot_stride};
      if (J.op == CHAIN_SILU_MUL) chain_silu_mul(a, J, sd, et);
      else chain_resid_norm(a, J, sd, et, s_red);
      __threadfence();
      fence_async_proxy();
      epi_bar();
      if (et == 0) atomicAdd(a.sync + 8 + j + 1, 1);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (s_abort) {
    for (int i = 0; i < 2000; ++i) __nanosleep(100);
  }
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, C::TMEM_COLS); }
  if (threadIdx.x == 0) {                                // the last CTA out clears the counters for the next launch
    __threadfence();
    if (atomicAdd(a.sync + 16, 1) == G - 1) {
      for (int k = 0; k <= 16; ++k) a.sync[k] = 0;
      __threadfence();
    }
  }
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

int sm_count() {
  static int n = []() {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v < 1)
      return 148;
    return v;
  }();
  return n;
}

template <int MT, int BUDGET_KB, int NH>
hydra_status launch_b(const CUtensorMap& tw, const CUtensorMap& tx, const GemmArgs& a, int grid, cudaStream_t st) {
  using C = TileCfg<MT, BUDGET_KB, NH>;
  static bool attr_done = false;
  if (!attr_done) {
    HYDRA_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<MT, BUDGET_KB, NH>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
    attr_done = true;
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

// Shared memory per CTA: a deep ring (one CTA per SM) by default; HYDRA_GEMM_SMEM_KB=100 selects a ring that lets
// the CTAs of two consecutive (programmatically overlapped) GEMMs share an SM (measured: no faster).
template <int MT, int NH>
hydra_status launch(const CUtensorMap& tw, const CUtensorMap& tx, const GemmArgs& a, int grid, cudaStream_t st) {
  static const int kb = []() { const char* e = getenv("HYDRA_GEMM_SMEM_KB"); return e ? atoi(e) : 200; }();
  if (kb >= 200 || NH > 1) return launch_b<MT, 200, NH>(tw, tx, a, grid, st);
  return launch_b<MT, 100, NH>(tw, tx, a, grid, st);
}

template <int MT>
hydra_status launch_chain(const ChainArgs& a, int grid, cudaStream_t st) {
  using C = TileCfg<MT, 200>;
  static bool attr_done = false;
  if (!attr_done) {
    HYDRA_CUDA(cudaFuncSetAttribute(gemm_chain_kernel<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
    attr_done = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(192); cfg.dynamicSmemBytes = C::SMEM_BYTES; cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeCooperative;           // all CTAs resident at once: the grid-wide counters need it
  attr[0].val.cooperative = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 2;
  HYDRA_CUDA(cudaLaunchKernelEx(&cfg, gemm_chain_kernel<MT>, a));
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

}  // namespace

bool gemm_tc_available() { return encode_fn() != nullptr; }

int gemm_tile_rows(int m) { return m <= 16 ? 16 : m <= 32 ? 32 : m <= 64 ? 64 : m <= 128 ? 128 : 256; }

// Stream-K plan: equal contiguous unit ranges, one per CTA, at most one CTA per SM and at least 4 k-blocks each.
// 128-row weight tiles per unit: outputs of 4096 columns and more take two (half the activation-tile traffic and half
// the issue work per weight byte, a third more weight bytes in flight: -5 % step time at the 7B shape).  Above 64
// activation rows tensor memory holds one set of two accumulators only (the epilogue no longer overlaps the next
// segment), still a small gain.  HYDRA_GEMM_NH=1 forces single tiles.
int gemm_tile_halves(int m, int n) {
  static const int force = []() { const char* e = getenv("HYDRA_GEMM_NH"); return e ? atoi(e) : 0; }();
  if (force == 1) return 1;
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
                     SplitDesc* sd_out, int* status, int* diag, long long* trace, cudaStream_t st) {
  if (m <= 0 || n <= 0 || k <= 0 || n % BLOCK_N || k % BLOCK_K || (x_planes != 1 && x_planes != 2)) return HYDRA_ERR_UNSUPPORTED;
  if (((uintptr_t)x | (uintptr_t)w) & 15) return HYDRA_ERR_INVALID;
  int grid = 1;
  SplitDesc sd = gemm_tc_plan(m, n, k, &grid, nullptr, 0);
  if (x_rows_alloc < m) x_rows_alloc = m;
  CUtensorMap tw, tx;
  const int nh = sd.bn_shift == 8 ? 2 : 1;
  if (!get_tensor_map(w, (uint64_t)n, (uint64_t)k, (uint32_t)(nh * BLOCK_N), &tw) ||
      !get_tensor_map(x, (uint64_t)x_rows_alloc * x_planes, (uint64_t)k, (uint32_t)sd.mt, &tx)) {
    set_last_error("cuTensorMapEncodeTiled", cudaErrorUnknown);
    return HYDRA_ERR_CUDA;
  }
  GemmArgs a{};
  a.part = part; a.slot_stride = sd.stride; a.m = m; a.n = n; a.kb = sd.kb; a.n_tiles = sd.n_tiles;
  a.total_units = sd.n_tiles * ((m + sd.mt - 1) / sd.mt) * sd.kb; a.q = sd.q; a.status = status;
  a.x_lo_rows = x_planes == 2 ? x_rows_alloc : 0; a.diag = diag; a.trace = trace;
  { static const int f = []() { const char* e = getenv("HYDRA_GEMM_NOHINT"); return e && e[0] == '1' ? 1 : 0; }(); a.flags = f; }
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

hydra_status gemm_chain(const ChainStep* steps, int n_steps, int m, int x_planes, float* part, size_t part_floats, SplitDesc* last_sd,
                        int* status, int* diag, int* sync, cudaStream_t st) {
  if (n_steps < 1 || n_steps > MAX_JOBS || m <= 0 || (x_planes != 1 && x_planes != 2)) return HYDRA_ERR_UNSUPPORTED;
  ChainArgs a{};
  a.part = part; a.m = m; a.n_jobs = n_steps; a.status = status; a.diag = diag; a.sync = sync;
  const int mt = gemm_tile_rows(m);
  for (int j = 0; j < n_steps; ++j) {
    const ChainStep& s = steps[j];
    if (s.n <= 0 || s.k <= 0 || s.n % BLOCK_N || s.k % BLOCK_K) return HYDRA_ERR_UNSUPPORTED;
    if (((uintptr_t)s.x | (uintptr_t)s.w) & 15) return HYDRA_ERR_INVALID;
    if (s.op != CHAIN_NONE && (s.cols & 3)) return HYDRA_ERR_UNSUPPORTED;
    if (s.op == CHAIN_NONE && j + 1 < n_steps) return HYDRA_ERR_INVALID;       // only the last job may leave raw partial sums
    int slots = 1;
    const SplitDesc sd = gemm_tc_plan(m, s.n, s.k, nullptr, &slots, 1);       // the chain kernel works on single weight tiles
    if ((size_t)slots * m * s.n > part_floats) return HYDRA_ERR_CAPACITY;
    const int rows_alloc = s.x_rows_alloc < m ? m : s.x_rows_alloc;
    if (!get_tensor_map(s.w, (uint64_t)s.n, (uint64_t)s.k, BLOCK_N, &a.tmW[j]) ||
        !get_tensor_map(s.x, (uint64_t)rows_alloc * x_planes, (uint64_t)s.k, (uint32_t)mt, &a.tmX[j])) {
      set_last_error("cuTensorMapEncodeTiled", cudaErrorUnknown);
      return HYDRA_ERR_CUDA;
    }
    ChainJob& J = a.job[j];
    J.n = s.n; J.kb = sd.kb; J.n_tiles = sd.n_tiles; J.total_units = sd.n_tiles * ((m + mt - 1) / mt) * sd.kb; J.q = sd.q;
    J.x_lo_rows = x_planes == 2 ? rows_alloc : 0; J.op = s.op; J.cols = s.cols; J.slot_stride = sd.stride;
    J.resid = s.resid; J.gain = s.gain; J.out = s.out; J.out_ps = s.out_ps; J.hn = s.hn; J.eps = s.eps;
    if (j + 1 == n_steps && last_sd) *last_sd = sd;
  }
  const int grid = sm_count();
  switch (mt) {
    case 16: return launch_chain<16>(a, grid, st);
    case 32: return launch_chain<32>(a, grid, st);
    case 64: return launch_chain<64>(a, grid, st);
    case 128: return launch_chain<128>(a, grid, st);
    default: return launch_chain<256>(a, grid, st);
  }
}

}  // namespace hydra

// Tree attention for the bfloat16 model path on the sm_100a tensor cores: TMA tile loads, tcgen05.mma with the
// score and output accumulators in tensor memory, softmax out of tensor memory.
//
// Operand format: q, the K cache (post-RoPE), the V cache and the softmax weights are float16 (the values are O(1),
// far inside the float16 range) in NP planes.  NP = 2: hi = f16(v), lo = f16(v - hi), about 22 significant bits;
// a product x y is taken as x_hi y_hi + x_hi y_lo + x_lo y_hi.  Stacking the planes of the B operand along its N
// dimension gives the first two terms in ONE instruction sequence (accumulator columns [0, n) and [n, 2n), added
// when the accumulator is read); the third is a second sequence into columns [0, n).  NP = 1: hi only, 11 bits
// (half the cache bytes; hidden states then drift to a few 1e-3 of a float reference over 32 layers).
// Scores, running maxima, sums and the output accumulate in float.  The result leaves as two bfloat16 planes
// (hi = bf16(v), lo = bf16(v - hi)), the operand format of the GEMM that consumes it.
//
// One CTA per (head, sequence, KV chunk).  A sequence's KV rows are cut into 64-row tiles and the tiles are dealt
// to the launch's chunks in equal contiguous runs, computed on the device from the real length (a captured graph
// keeps balanced chunks as the sequence grows).  256 threads:
//   warp 2 (one lane)  TMA producer: Q once, then K tiles and V tiles through rings of their own (a K stage is free
//                      as soon as the scores of its tile are done, a V stage after the tile's P V product), each stage
//                      with its own "full" barrier, so the scores of a tile start before its V has landed;
//   warp 3 (one lane)  MMA issue: S_i = Q K_i^T (M = 128 query lanes, N = 64 keys) into one of two score buffers in
//                      tensor memory, issued one tile ahead; O += P_i V_i (N = head_dim, V read as an MN-major operand
//                      straight from its [key][dim] tile) into one accumulator that lives across the chunk;
//   four softmax warps thread = query row (a tensor-memory lane).  With 64 query rows two warps share a quadrant of
//                      tensor memory (warps 0 and 4: rows 0..31, warps 1 and 5: rows 32..63) and each takes half of a
//                      tile's keys; the two swap their row maxima through shared memory, keep the same reference
//                      maximum and each its own part of the row sum.  With 128 rows warps 4..7 take a quadrant each
//                      and all keys.  A thread reads its scores from tensor memory, applies the scale and
//                      the mask (committed slots are visible to every row; tree slot j to row i iff bit j of the
//                      row's ancestor bitmask, or j <= i for a causal chunk), keeps the row's running reference
//                      maximum and sum in the exp2 domain, writes P_i as float16 into a swizzled shared-memory
//                      tile for the MMA.  The reference maximum only moves when a tile's maximum exceeds it by
//                      more than 8 (a factor 256, harmless in float16 and float); only then is the row's output
//                      accumulator rescaled in tensor memory (load, scale, store), so the common tile needs no
//                      round trip through registers for O.
// Query rows beyond the row count of the call ride along as unused lanes of the M = 128 tile.
// The chunks of a (head, sequence) pair (at most 8) form a thread-block cluster: every CTA leaves its partial rows
// (un-normalised output, reference maximum, sum) in its own shared memory, and each CTA merges a share of the rows
// out of its peers' shared memory, in chunk order (deterministic; no scratch traffic, no atomics).
// Every barrier wait is bounded; when one runs out the CTA raises the time-out bit of the status word, skips its
// stores, still takes part in the cluster barriers, frees its tensor memory and returns.
#include "tc.cuh"
#include <cuda_fp16.h>
#include <math.h>

namespace hydra {

namespace {

using namespace tc;

constexpr int TILE = 64;           // KV rows per tile
constexpr int MAX_CHUNKS = 8;      // chunks of a (head, sequence) pair = cluster size
constexpr float RESCALE_STEP = 8.f;

__device__ __forceinline__ int chunk_first_tile(int c, int nt, int nch) { return (int)(((unsigned)c * (unsigned)nt) / (unsigned)nch); }

__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t peer_smem(uint32_t saddr, uint32_t rank) {     // the same offset in CTA `rank`'s shared memory
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ float4 ld_peer4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

struct AttArgs {
  RowSet rs;
  int q_plane_rows, kv_plane_rows;     // rows between the hi and lo planes in the q and cache tensor maps
  bf16* out; size_t out_ps;
  int H, max_seq, nchunks;
  int* status;
  uint32_t wait_limit;
  int row_off;                         // first row (of each sequence's rs.tc row slots) this launch computes: a wide causal chunk
                                       // runs as several launches of QROWS rows, each seeing the earlier ones as cache rows
  int early;                           // the lengths (rs.pos0, rs.n_rows) and the committed cache rows were written by kernels that
                                       // completed before the preceding kernel started (see tree_attention_tc)
};

template <int HD, int QROWS, int NP> struct AttCfg {
  static constexpr int NHALF = HD / 64;                       // 64-column (128-byte) halves of a head row
  static constexpr int QP_BYTES = NHALF * QROWS * 128;        // one plane of Q: [half][query row][128 bytes]
  static constexpr int Q_BYTES = NP * QP_BYTES;
  static constexpr int PP_BYTES = QROWS * 128;                // one plane of a P tile: [query row][64 keys] float16
  static constexpr int P_BYTES = NP * PP_BYTES;
  static constexpr int KH_BYTES = NP * TILE * 128;            // one half of a K tile: [plane][key][128 bytes] (the planes stacked along N)
  static constexpr int K_BYTES = NHALF * KH_BYTES;
  static constexpr int V_BYTES = NP * NHALF * TILE * 128;     // a V tile: [plane][half][key][128 bytes] (N blocks of 64 output columns)
  // K and V tiles travel through rings of their own: a K stage is free again as soon as the scores of its tile are done,
  // long before the tile's P V product frees the V stage, so K runs further ahead inside the same shared memory.
  static constexpr int NSK = K_BYTES >= 32768 ? 3 : 4;            // K ring stages
  static constexpr int NSV = V_BYTES >= 32768 ? 2 : 4;            // V ring stages
  // MMA M is 128 whatever QROWS is: with 64 query rows the upper 64 accumulator lanes are unused (M = 64 instructions
  // measured slower per instruction), and the operand reads of a 64-row Q or P tile run 8 KB past the tile, into the next
  // piece of Q, of P or of the ring (never read back), so the order Q, P0, P1, ring keeps them inside the allocation.
  static constexpr int MROWS = 128;
  static constexpr int RPW = MROWS / 4;                       // accumulator rows (tensor-memory lanes) per softmax warp
  static constexpr int KRING_BYTES = NSK * K_BYTES;
  static constexpr int RING_BYTES = KRING_BYTES + NSV * V_BYTES;
  static constexpr int MERGE_BYTES = QROWS * HD * 4 + QROWS * 16;    // a chunk's partial rows + (max, sum, max, sum of the other key half); aliases the ring
  // 64 query rows: two softmax warps per tensor-memory quadrant, each with half of a tile's keys (SPLIT); they exchange
  // their row maxima through XM_BYTES of shared memory.  128 rows: one warp per quadrant, thread = row, all keys.
  static constexpr bool SPLIT = QROWS == 64;
  static constexpr int KPT = SPLIT ? TILE / 2 : TILE;                // keys per softmax thread and tile
  static constexpr int XM_BYTES = 2 * 2 * 64 * 4;                    // [tile parity][key half][row]
  static constexpr int NBAR = 1 + 2 * NSK + 2 * NSV + 8 + 4;
  static constexpr int SMEM_BYTES = 1024 + Q_BYTES + 2 * P_BYTES + (RING_BYTES > MERGE_BYTES ? RING_BYTES : MERGE_BYTES) + XM_BYTES + NBAR * 8 + 16;
  static constexpr int NTHREADS = 256;
  static constexpr int S_COLS = NP * TILE;                    // one score buffer: [Q_hi K_hi + Q_lo K_hi | Q_hi K_lo]
  static constexpr int O_COLS = NP * HD;                      // the output accumulator: [P_hi V_hi + P_lo V_hi | P_hi V_lo]
  static constexpr int O_COL0 = 2 * S_COLS;
  static constexpr int TMEM_COLS = O_COL0 + O_COLS <= 256 ? 256 : 512;
  static_assert(RING_BYTES >= MERGE_BYTES + 128 * MAX_CHUNKS * 4, "merge area and chunk weights must fit in the ring");
  static_assert(MERGE_BYTES % 16 == 0, "alignment of the chunk weights");
  static_assert(O_COL0 + O_COLS <= 512, "tensor memory");
  static_assert(SMEM_BYTES <= 232448, "shared memory of one SM");
};

template <int HD, int QROWS, int NP>
__global__ void __launch_bounds__(256, 1)
tree_attn_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const AttArgs a) {
  using C = AttCfg<HD, QROWS, NP>;
  constexpr int NSK = C::NSK, NSV = C::NSV;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t q_s = base, p_s = q_s + C::Q_BYTES, ring_s = p_s + 2 * C::P_BYTES, vring_s = ring_s + C::KRING_BYTES;
  const uint32_t xm_s = ring_s + (C::RING_BYTES > C::MERGE_BYTES ? C::RING_BYTES : C::MERGE_BYTES);
  const uint32_t bars = xm_s + C::XM_BYTES;
  const uint32_t q_full = bars;
  auto k_full = [&](int s) { return bars + 8u * (1 + s); };
  auto k_empty = [&](int s) { return bars + 8u * (1 + NSK + s); };
  auto v_full = [&](int s) { return bars + 8u * (1 + 2 * NSK + s); };
  auto v_empty = [&](int s) { return bars + 8u * (1 + 2 * NSK + NSV + s); };
  constexpr int B0 = 1 + 2 * NSK + 2 * NSV;
  auto s_full = [&](int i) { return bars + 8u * (B0 + i); };
  auto s_empty = [&](int i) { return bars + 8u * (B0 + 2 + i); };
  auto p_full = [&](int i) { return bars + 8u * (B0 + 4 + i); };
  auto pv_done = [&](int i) { return bars + 8u * (B0 + 6 + i); };
  auto xm_bar = [&](int par, int quad) { return bars + 8u * (B0 + 8 + 2 * par + quad); };   // both key halves of a quadrant have left their maxima
  const uint32_t tmem_slot = bars + 8u * C::NBAR;
  __shared__ int s_abort;
  // normalised chunk weights of the rows this CTA merges: in the idle ring, behind the merge area its peers read
  float* const s_w = reinterpret_cast<float*>(smem_raw + (ring_s - smem_u32(smem_raw)) + C::MERGE_BYTES);

  const RowSet& rs = a.rs;
  const int h = blockIdx.x, b = blockIdx.y, c = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nchunks = a.nchunks, H = a.H;

  if (tid == 0) {
    s_abort = 0;
    mbar_init(q_full, 1);
    for (int s = 0; s < NSK; ++s) { mbar_init(k_full(s), 1); mbar_init(k_empty(s), 1); }
    for (int s = 0; s < NSV; ++s) { mbar_init(v_full(s), 1); mbar_init(v_empty(s), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(s_full(i), 1); mbar_init(s_empty(i), 4); mbar_init(p_full(i), 4); mbar_init(pv_done(i), 1); }
    for (int i = 0; i < 4; ++i) mbar_init(xm_bar(i >> 1, i & 1), 2);
    mbar_init_fence();
    prefetch_tensormap(&tmQ); prefetch_tensormap(&tmK); prefetch_tensormap(&tmV);
  }
  if (warp == 3) tmem_alloc(tmem_slot, C::TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_trigger();
  // q and the new cache rows are the preceding kernel's output.  With a.early the lengths and the committed cache rows
  // are known to be older than anything still in flight, so the producer requests committed tiles before it waits.
  if (!a.early) pdl_wait();
  uint32_t tmem_base;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

  const int nr = min(max((rs.n_rows ? rs.n_rows[b] : rs.tc) - a.row_off, 0), QROWS);
  const int p_call = rs.pos0[b];                         // first cache slot written by this forward call
  const int p0 = p_call + a.row_off;                     // first slot of this launch's rows
  const int total = p0 + nr;
  const int nt = (total + TILE - 1) / TILE;
  const int tile0 = chunk_first_tile(c, nt, nchunks), tile1 = chunk_first_tile(c + 1, nt, nchunks);
  const bool has_work = tile0 < tile1 && nr > 0 && p0 >= 0 && total <= a.max_seq;
  const int ntiles = has_work ? tile1 - tile0 : 0;
  const uint32_t limit = a.wait_limit;

  // warp 2: TMA producer (one lane); warp 3: MMA issue (one lane); softmax: warps 0, 1, 4, 5 (quadrants 0, 1, 0, 1; key halves
  // 0, 0, 1, 1) for 64 query rows, warps 4..7 (quadrants 0..3) for 128
  const bool softmax_warp = C::SPLIT ? (warp & 2) == 0 : warp >= 4;
  if (warp == 2) {
    if (lane == 0 && has_work) {
      const uint64_t pol = policy_evict_first(), pol_q = policy_evict_last();
      const int row0 = (b * H + h) * a.max_seq;
      auto request_k = [&](int i) {
        const int s = i % NSK;
        const uint32_t k_dst = ring_s + s * C::K_BYTES;
        const int r = row0 + (tile0 + i) * TILE;
        mbar_arrive_expect_tx(k_full(s), C::K_BYTES);
#pragma unroll
        for (int pl = 0; pl < NP; ++pl)
#pragma unroll
          for (int hf = 0; hf < C::NHALF; ++hf)
            tma_load_2d(k_dst + hf * C::KH_BYTES + pl * TILE * 128, &tmK, hf * 64, pl * a.kv_plane_rows + r, k_full(s), pol);
      };
      auto request_v = [&](int i) {
        const int s = i % NSV;
        const uint32_t v_dst = vring_s + s * C::V_BYTES;
        const int r = row0 + (tile0 + i) * TILE;
        mbar_arrive_expect_tx(v_full(s), C::V_BYTES);
#pragma unroll
        for (int pl = 0; pl < NP; ++pl)
#pragma unroll
          for (int hf = 0; hf < C::NHALF; ++hf)
            tma_load_2d(v_dst + (pl * C::NHALF + hf) * TILE * 128, &tmV, hf * 64, pl * a.kv_plane_rows + r, v_full(s), pol);
      };
      int nk = 0, nv = 0;                                  // next K and V tile to request
      if (a.early) {                                       // committed rows only
        for (; nk < ntiles && nk < NSK && (tile0 + nk + 1) * TILE <= p_call; ++nk) {
          request_k(nk);
          if (nv == nk && nv < NSV) request_v(nv++);
        }
        pdl_wait();
      }
      mbar_arrive_expect_tx(q_full, C::Q_BYTES);
#pragma unroll
      for (int pl = 0; pl < NP; ++pl)
#pragma unroll
        for (int hf = 0; hf < C::NHALF; ++hf)
          tma_load_2d(q_s + pl * C::QP_BYTES + hf * QROWS * 128, &tmQ, h * HD + hf * 64, pl * a.q_plane_rows + b * rs.tc + a.row_off, q_full, pol_q);
      // K stage i % NSK was last read by the scores of tile i - NSK (completion i / NSK - 1 of its empty barrier), V stage
      // i % NSV by the P V product of tile i - NSV; whichever ring has room is served first, K ahead of V
      uint32_t idle = 0;
      while (nk < ntiles || nv < ntiles) {
        bool did = false;
        if (nk < ntiles && (nk < NSK || mbar_test(k_empty(nk % NSK), (uint32_t)((nk / NSK - 1) & 1)))) { request_k(nk++); did = true; }
        if (nv < nk && (nv < NSV || mbar_test(v_empty(nv % NSV), (uint32_t)((nv / NSV - 1) & 1)))) { request_v(nv++); did = true; }
        if (did) idle = 0;
        else if (++idle > limit) { atomicOr(a.status, ST_TIMEOUT); s_abort = 1; break; }
      }
    }
  } else if (warp == 3) {
    if (lane == 0 && has_work) {
      constexpr uint32_t idesc_s = instr_desc_f16(0, C::MROWS, NP * TILE, 0);      // Q_hi x [K_hi ; K_lo]
      constexpr uint32_t idesc_s2 = instr_desc_f16(0, C::MROWS, TILE, 0);          // Q_lo x K_hi
      constexpr uint32_t idesc_pv = instr_desc_f16(0, C::MROWS, NP * HD, 1);       // P_hi x [V_hi | V_lo]
      constexpr uint32_t idesc_pv2 = instr_desc_f16(0, C::MROWS, HD, 1);           // P_lo x V_hi
      // operand descriptors: built once; a byte offset inside shared memory adds offset / 16 to the start-address field
      const uint64_t q_desc = smem_desc_sw128(q_s), p_desc = smem_desc_sw128(p_s), k_desc = smem_desc_sw128(ring_s),
                     v_desc = smem_desc_sw128_mn(vring_s, TILE * 128);
      bool ok = mbar_wait(q_full, 0, limit);
      auto issue_s = [&](int i) {                        // S_i = Q K_i^T into score buffer i & 1
        const int s = i % NSK;
        if (!mbar_wait(k_full(s), (uint32_t)((i / NSK) & 1), limit)) return false;
        if (i >= 2 && !mbar_wait(s_empty(i & 1), (uint32_t)(((i >> 1) - 1) & 1), limit)) return false;
        tc_fence_after();
        const uint64_t kd = k_desc + (uint64_t)((s * C::K_BYTES) >> 4);
        const uint32_t d_s = tmem_base + (uint32_t)((i & 1) * C::S_COLS);
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk)
          umma_f16(d_s, q_desc + (uint64_t)(((kk >> 2) * QROWS * 128 + (kk & 3) * 32) >> 4),
                   kd + (uint64_t)(((kk >> 2) * C::KH_BYTES + (kk & 3) * 32) >> 4), idesc_s, (uint32_t)(kk != 0));
        if (NP == 2) {
#pragma unroll
          for (int kk = 0; kk < HD / 16; ++kk)
            umma_f16(d_s, q_desc + (uint64_t)((C::QP_BYTES + (kk >> 2) * QROWS * 128 + (kk & 3) * 32) >> 4),
                     kd + (uint64_t)(((kk >> 2) * C::KH_BYTES + (kk & 3) * 32) >> 4), idesc_s2, 1u);
        }
        umma_commit(k_empty(s));                        // frees the K stage once these MMAs have read it
        umma_commit(s_full(i & 1));
        return true;
      };
      if (ok) ok = issue_s(0);
      for (int i = 0; i < ntiles && ok; ++i) {
        if (i + 1 < ntiles) ok = issue_s(i + 1);
        if (!ok) break;
        const int s = i % NSV;
        if (!mbar_wait(p_full(i & 1), (uint32_t)((i >> 1) & 1), limit)) { ok = false; break; }
        if (!mbar_wait(v_full(s), (uint32_t)((i / NSV) & 1), limit)) { ok = false; break; }
        tc_fence_after();
        const uint64_t vd = v_desc + (uint64_t)((s * C::V_BYTES) >> 4), pd = p_desc + (uint64_t)(((i & 1) * C::P_BYTES) >> 4);
        const uint32_t d_o = tmem_base + (uint32_t)C::O_COL0;
#pragma unroll
        for (int kk = 0; kk < TILE / 16; ++kk)
          umma_f16(d_o, pd + (uint64_t)((kk * 32) >> 4), vd + (uint64_t)((kk * 2048) >> 4), idesc_pv, (uint32_t)((i | kk) != 0));
        if (NP == 2) {
#pragma unroll
          for (int kk = 0; kk < TILE / 16; ++kk)
            umma_f16(d_o, pd + (uint64_t)((C::PP_BYTES + kk * 32) >> 4), vd + (uint64_t)((kk * 2048) >> 4), idesc_pv2, 1u);
        }
        umma_commit(v_empty(s));
        umma_commit(pv_done(i & 1));
      }
      if (!ok) { atomicOr(a.status, ST_TIMEOUT); s_abort = 1; }
    }
  } else if (softmax_warp) {
    // ---- softmax warps: thread = accumulator row = a tensor-memory lane of the warp's quadrant; KPT of the tile's keys
    constexpr int KPT = C::KPT;
    const int quad = warp & 3, half = C::SPLIT ? warp >> 2 : 0, row = quad * C::RPW + lane;
    const int kb0 = half * KPT;                           // first key of the tile this thread looks at
    const bool row_valid = row < QROWS;
    const bool warp_rows = quad * C::RPW < nr;            // any row of this warp in use
    const bool row_live = row_valid && row < nr;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const uint64_t mask = (row_live && rs.mask) ? rs.mask[row] : 0ull;
    const bool causal = rs.mask == nullptr;
    const float sc = rsqrtf((float)HD) * 1.4426950408889634f;   // 1/sqrt(hd) * log2(e)
    float m_ref = -INFINITY, l = 0.f;                     // l: the sum over this thread's keys only
    bool ok = true;
    const int st = (C::SPLIT ? half * 2 + quad : warp - 4) * 32 + lane;      // 0..127 among the softmax threads
    for (int i = 0; i < ntiles; ++i) {
      if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }     // a wait that ran out in one lane ends the walk for the whole warp
      const int t0 = (tile0 + i) * TILE;
      if (!mbar_wait(s_full(i & 1), (uint32_t)((i >> 1) & 1), limit)) { ok = false; break; }
      tc_fence_after();
      uint32_t r[KPT];
      if (warp_rows) {
        const uint32_t s_addr = lane_addr + (uint32_t)((i & 1) * C::S_COLS + kb0);
        if constexpr (NP == 1) {
          if constexpr (KPT == 64) tmem_ld64(s_addr, r); else tmem_ld32(s_addr, r);
        } else {                                           // the two column halves of the score buffer in one round trip, added
          uint32_t y[KPT];
          if constexpr (KPT == 64) tmem_ld64x2(s_addr, s_addr + (uint32_t)TILE, r, y); else tmem_ld32x2(s_addr, s_addr + (uint32_t)TILE, r, y);
#pragma unroll
          for (int j = 0; j < KPT; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(y[j]));
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(s_empty(i & 1));
      float alpha = 1.f;
      if (warp_rows) {
        // visibility word of this row for the tile's 64 keys (bit j: key t0 + j), built once per tile
        uint64_t vis = row_live ? ~0ull : 0ull;
        if (t0 + TILE > p0 && row_live) {                  // the tile reaches into the new rows (or past the end)
          const int shift = t0 - p0;                       // new-slot index of the tile's first key; negative: it is a committed row
          if (causal) {                                    // new slots 0..row: keys j <= row - shift
            const int n = row - shift + 1;
            vis = n >= 64 ? ~0ull : (n <= 0 ? 0ull : ((1ull << n) - 1ull));
          } else if (shift >= 0) {
            vis = shift < 64 ? mask >> shift : 0ull;
          } else {
            vis = (mask << (-shift)) | ((1ull << (-shift)) - 1ull);
          }
          const int nv = total - t0;                       // keys of the tile that exist
          if (nv < 64) vis &= (1ull << nv) - 1ull;
        }
        if constexpr (C::SPLIT) vis >>= kb0;
        float mx = -INFINITY;
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
          const float v = ((vis >> j) & 1ull) ? __uint_as_float(r[j]) * sc : -INFINITY;
          r[j] = __float_as_uint(v);
          mx = fmaxf(mx, v);
        }
        if constexpr (C::SPLIT) {
          // the row's maximum over all 64 keys: the two warps of the quadrant swap theirs (buffer and barrier of the tile's
          // parity; a buffer is rewritten two tiles later, after the P V product that followed this read has been issued)
          const uint32_t xm = xm_s + (uint32_t)(((i & 1) * 2) * 64 * 4);
          asm volatile("st.shared.f32 [%0], %1;" ::"r"(xm + (uint32_t)((half * 64 + row) * 4)), "f"(mx) : "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive(xm_bar(i & 1, quad));
          if (!mbar_wait(xm_bar(i & 1, quad), (uint32_t)((i >> 1) & 1), limit)) { ok = false; break; }
          float other;
          asm volatile("ld.shared.f32 %0, [%1];" : "=f"(other) : "r"(xm + (uint32_t)(((half ^ 1) * 64 + row) * 4)) : "memory");
          mx = fmaxf(mx, other);
        }
        float m_new = m_ref;
        if (mx > m_ref + RESCALE_STEP) m_new = mx;          // also the first finite maximum (m_ref = -inf)
        const bool rescale = m_ref != -INFINITY && m_new != m_ref;
        if (rescale) alpha = ex2(m_ref - m_new);
        m_ref = m_new;
        const float bse = m_new == -INFINITY ? 0.f : m_new;
        float sum = 0.f;
        uint32_t pk[KPT / 2];
#pragma unroll
        for (int j = 0; j < KPT / 2; ++j) {
          const float p0v = ex2(__uint_as_float(r[2 * j]) - bse), p1v = ex2(__uint_as_float(r[2 * j + 1]) - bse);
          pk[j] = pack_half2(p0v, p1v);
          if (NP == 1) {
            const __half2 hv = *reinterpret_cast<const __half2*>(&pk[j]);
            sum += __low2float(hv) + __high2float(hv);     // the sum of what the MMA will really weigh V with
          } else {
            sum += p0v + p1v;
            r[2 * j] = __float_as_uint(p0v); r[2 * j + 1] = __float_as_uint(p1v);     // kept for the lo plane
          }
        }
        l = l * alpha + sum;
        // P buffer i & 1 was last read by P V of tile i - 2; the row's accumulator by P V of tile i - 1
        if (i >= 2 && !mbar_wait(pv_done(i & 1), (uint32_t)(((i >> 1) - 1) & 1), limit)) { ok = false; break; }
        if (__any_sync(0xffffffffu, rescale)) {            // both warps of a quadrant decide alike; each scales its half of the columns
          if (i >= 1 && !mbar_wait(pv_done((i - 1) & 1), (uint32_t)(((i - 1) >> 1) & 1), limit)) { ok = false; break; }
          tc_fence_after();
          constexpr int OC = C::SPLIT ? C::O_COLS / 2 : C::O_COLS;
#pragma unroll 1
          for (int c0 = half * OC; c0 < (half + 1) * OC; c0 += 32) {
            uint32_t o[32];
            tmem_ld32(lane_addr + (uint32_t)(C::O_COL0 + c0), o);
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
            tmem_st32(lane_addr + (uint32_t)(C::O_COL0 + c0), o);
          }
        }
        const uint32_t prow = p_s + (i & 1) * C::P_BYTES + (uint32_t)row * 128u;
        if (row_valid) {
#pragma unroll
          for (int ch = 0; ch < KPT / 8; ++ch) {
            const uint32_t dst = prow + (uint32_t)(((kb0 / 8 + ch) ^ (row & 7)) * 16);
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(pk[4 * ch]), "r"(pk[4 * ch + 1]), "r"(pk[4 * ch + 2]), "r"(pk[4 * ch + 3]) : "memory");
          }
          if (NP == 2) {
#pragma unroll
            for (int j = 0; j < KPT / 2; ++j) {            // lo = f16(p - f16(p))
              const __half2 hv = *reinterpret_cast<const __half2*>(&pk[j]);
              pk[j] = pack_half2(__uint_as_float(r[2 * j]) - __low2float(hv), __uint_as_float(r[2 * j + 1]) - __high2float(hv));
            }
#pragma unroll
            for (int ch = 0; ch < KPT / 8; ++ch) {
              const uint32_t dst = prow + (uint32_t)(C::PP_BYTES + ((kb0 / 8 + ch) ^ (row & 7)) * 16);
              asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(pk[4 * ch]), "r"(pk[4 * ch + 1]), "r"(pk[4 * ch + 2]), "r"(pk[4 * ch + 3]) : "memory");
            }
          }
        }
      } else {
        if (i >= 2 && !mbar_wait(pv_done(i & 1), (uint32_t)(((i >> 1) - 1) & 1), limit)) { ok = false; break; }
      }
      if (t0 + TILE > total) {
        // rows of the V tile past the end of the sequence hold whatever the cache holds: zero them, so that a
        // zero weight times a non-finite stale value cannot reach the accumulator
        const int s = i % NSV;
        if (!mbar_wait(v_full(s), (uint32_t)((i / NSV) & 1), limit)) { ok = false; break; }
        const uint32_t v_src = vring_s + s * C::V_BYTES;
        const int first = total - t0;                       // first row to clear (>= 1)
        constexpr int BLK = NP * C::NHALF;                  // 64-column blocks of a V tile
        for (int e = st; e < (TILE - first) * BLK * 8; e += 128) {
          const int rr = first + e / (BLK * 8), rem = e % (BLK * 8);
          const uint32_t dst = v_src + (uint32_t)((rem >> 3) * TILE * 128 + rr * 128 + (rem & 7) * 16);
          asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(dst), "r"(0u) : "memory");
        }
      }
      fence_proxy_async();                                 // P (and the cleared V rows) become visible to the tensor core
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(p_full(i & 1));
    }
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) { atomicOr(a.status, ST_TIMEOUT); s_abort = 1; }
    // ---- this chunk's partial rows -> shared memory (the ring is idle once the last P V has completed)
    if (ok && ntiles > 0 && !mbar_wait(pv_done((ntiles - 1) & 1), (uint32_t)(((ntiles - 1) >> 1) & 1), limit)) {
      ok = false; atomicOr(a.status, ST_TIMEOUT); s_abort = 1;
    }
    ok = __all_sync(0xffffffffu, ok);
    tc_fence_after();
    {
      const uint32_t xo = ring_s + (uint32_t)row * (HD * 4), xml = ring_s + QROWS * HD * 4 + (uint32_t)row * 16 + (uint32_t)half * 8;
      const bool have = ok && ntiles > 0 && row_live && m_ref != -INFINITY;
      if (ok && ntiles > 0 && warp_rows) {
        // 64 output columns (both planes' halves) per tensor-memory round trip; with two warps per quadrant each takes
        // every other block of 64
#pragma unroll 1
        for (int c0 = half * 64; c0 < HD; c0 += C::SPLIT ? 128 : 64) {
          uint32_t o[64];
          if (NP == 2) {
            uint32_t o2[64];
            tmem_ld64x2(lane_addr + (uint32_t)(C::O_COL0 + c0), lane_addr + (uint32_t)(C::O_COL0 + HD + c0), o, o2);
#pragma unroll
            for (int j = 0; j < 64; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) + __uint_as_float(o2[j]));
          } else {
            tmem_ld64(lane_addr + (uint32_t)(C::O_COL0 + c0), o);
          }
          if (row_valid) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {                 // float4 piece k4 of row i sits at position k4 ^ (i & (HD/4 - 1))
              const int k4 = c0 / 4 + j;
              const uint32_t dst = xo + (uint32_t)((k4 ^ (row & (HD / 4 - 1))) * 16);
              asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(o[4 * j]), "r"(o[4 * j + 1]), "r"(o[4 * j + 2]), "r"(o[4 * j + 3]) : "memory");
            }
          }
        }
      }
      if (row_valid) {                                     // (max, this thread's part of the sum); without a second key half its slot reads (max, 0)
        const float2 ml = have ? make_float2(m_ref, l) : make_float2(-INFINITY, 0.f);
        asm volatile("st.shared.v2.f32 [%0], {%1,%2};" ::"r"(xml), "f"(ml.x), "f"(ml.y) : "memory");
        if constexpr (!C::SPLIT) asm volatile("st.shared.v2.f32 [%0], {%1,%2};" ::"r"(xml + 8u), "f"(ml.x), "f"(0.f) : "memory");
      }
    }
  }
  __syncwarp();                                           // the one-lane roles rejoin their warps before the block-wide barrier
  tc_fence_before();
  __syncthreads();
  // ---- merge the chunks of this (head, sequence): out[r][h][:] = sum_c o_c 2^(m_c - M) / sum_c l_c 2^(m_c - M),
  // chunks in order; this CTA takes rows c, c + nchunks, ...
  cluster_sync_all();                                     // every chunk's rows are in its shared memory
  if (a.early) pdl_wait();                                // (the producer lane has waited already) before the first global store
  {
    constexpr int V4 = HD / 4;
    const uint32_t xo_s = ring_s, xml_s = ring_s + QROWS * HD * 4;
    const int d = H * HD;
    const int rows_cap = min(rs.tc - a.row_off, QROWS);
    const int my_rows = rows_cap > c ? (rows_cap - c + nchunks - 1) / nchunks : 0;
    // chunk weights of my rows, normalised: w_c = 2^(m_c - M) / sum_c l_c 2^(m_c - M)  (one thread per row, all (m, l) loads in flight together)
    for (int t = tid; t < my_rows; t += C::NTHREADS) {
      const int i = c + t * nchunks;
      float mc[MAX_CHUNKS], lc[MAX_CHUNKS];
      float M = -INFINITY, L = 0.f;
#pragma unroll
      for (int cc = 0; cc < MAX_CHUNKS; ++cc) {
        mc[cc] = -INFINITY; lc[cc] = 0.f;
        if (cc < nchunks && i < nr) { const float4 ml = ld_peer4(peer_smem(xml_s + (uint32_t)i * 16u, (uint32_t)cc)); mc[cc] = ml.x; lc[cc] = ml.y + ml.w; }
      }
#pragma unroll
      for (int cc = 0; cc < MAX_CHUNKS; ++cc) M = fmaxf(M, mc[cc]);
#pragma unroll
      for (int cc = 0; cc < MAX_CHUNKS; ++cc) { mc[cc] = mc[cc] == -INFINITY ? 0.f : exp2f(mc[cc] - M); L += lc[cc] * mc[cc]; }
      const float inv = L > 0.f ? 1.f / L : 0.f;
#pragma unroll
      for (int cc = 0; cc < MAX_CHUNKS; ++cc) s_w[t * MAX_CHUNKS + cc] = mc[cc] * inv;
    }
    __syncthreads();
    // two output pieces per thread and round, all their peer loads in flight together (a load that waits for the
    // previous one's use costs a shared-memory round trip across the cluster each)
    for (int e0 = tid; e0 < my_rows * V4; e0 += 2 * C::NTHREADS) {
      float4 v[2][MAX_CHUNKS];
      float w[2][MAX_CHUNKS];
#pragma unroll
      for (int ib = 0; ib < 2; ++ib) {
        const int e = e0 + ib * C::NTHREADS, t = e / V4, i = c + t * nchunks, k4 = e % V4;
        const bool live = e < my_rows * V4;
#pragma unroll
        for (int cc = 0; cc < MAX_CHUNKS; ++cc) {
          w[ib][cc] = live && cc < nchunks ? s_w[t * MAX_CHUNKS + cc] : 0.f;
          v[ib][cc] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (w[ib][cc] != 0.f)                              // a chunk of weight zero may hold nothing at all
            v[ib][cc] = ld_peer4(peer_smem(xo_s + (uint32_t)(i * HD * 4 + ((k4 ^ (i & (V4 - 1))) * 16)), (uint32_t)cc));
        }
      }
#pragma unroll
      for (int ib = 0; ib < 2; ++ib) {
        const int e = e0 + ib * C::NTHREADS, t = e / V4, i = c + t * nchunks, k4 = e % V4;
        if (e >= my_rows * V4 || s_abort) continue;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int cc = 0; cc < MAX_CHUNKS; ++cc) {
          acc.x += v[ib][cc].x * w[ib][cc]; acc.y += v[ib][cc].y * w[ib][cc]; acc.z += v[ib][cc].z * w[ib][cc]; acc.w += v[ib][cc].w * w[ib][cc];
        }
        bf16* dst = a.out + ((size_t)b * rs.tc + a.row_off + i) * d + h * HD + k4 * 4;      // rows past nr get zeros
        const __nv_bfloat162 h0 = __floats2bfloat162_rn(acc.x, acc.y), h1 = __floats2bfloat162_rn(acc.z, acc.w);
        *reinterpret_cast<uint2*>(dst) = make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
        if (a.out_ps) {
          const __nv_bfloat162 l0 = __floats2bfloat162_rn(acc.x - __low2float(h0), acc.y - __high2float(h0));
          const __nv_bfloat162 l1 = __floats2bfloat162_rn(acc.z - __low2float(h1), acc.w - __high2float(h1));
          *reinterpret_cast<uint2*>(dst + a.out_ps) = make_uint2(*reinterpret_cast<const uint32_t*>(&l0), *reinterpret_cast<const uint32_t*>(&l1));
        }
      }
    }
  }
  cluster_sync_all();                                     // peers may still be reading this CTA's rows
  if (s_abort) {                                          // let copies in flight land before the CTA retires
    for (int i = 0; i < 2000; ++i) __nanosleep(100);
  }
  if (warp == 3) { tc_fence_after(); tmem_dealloc(tmem_base, C::TMEM_COLS); }
}

// Number of KV chunks per (head, sequence) for lengths up to len_upper: the count (at most 8) that minimises the
// largest number of tiles any SM walks, with about three tiles' worth of set-up and merging per CTA; ties go to
// fewer chunks.  One CTA per SM (the rings take nearly all of its shared memory).
int pick_chunks(int pairs, int len_upper, int sms) {
  const int nt = (len_upper + TILE - 1) / TILE;
  int hi = nt < MAX_CHUNKS ? nt : MAX_CHUNKS;
  if (hi < 1) hi = 1;
  auto cost = [&](int n) {
    const long per_sm = ((long)pairs * n + sms - 1) / sms, tiles = (nt + n - 1) / n;
    return per_sm * (tiles + 3);
  };
  int best = 1; long best_cost = cost(1);
  for (int n = 2; n <= hi; ++n)
    if (cost(n) < best_cost) { best = n; best_cost = cost(n); }
  return best;
}

template <int HD, int QROWS, int NP>
hydra_status run(const __half* q, int q_rows, const __half* kc, const __half* vc, int cache_batch, RowSet rs, bf16* out, size_t out_ps,
                 int H, int max_seq, int len_upper, int* status, bool stable_lengths, int row_off, cudaStream_t st) {
  using C = AttCfg<HD, QROWS, NP>;
  CUtensorMap tq, tk, tv;
  const uint64_t cache_rows = (uint64_t)cache_batch * H * max_seq;
  if (cache_rows * NP > 0x7fffffffull) return HYDRA_ERR_UNSUPPORTED;          // tensor-map row coordinates are 32-bit
  if (!get_tensor_map(q, (uint64_t)NP * q_rows, (uint64_t)H * HD, QROWS, true, &tq) ||
      !get_tensor_map(kc, NP * cache_rows, HD, TILE, true, &tk) || !get_tensor_map(vc, NP * cache_rows, HD, TILE, true, &tv)) {
    set_last_error("cuTensorMapEncodeTiled", cudaErrorUnknown);
    return HYDRA_ERR_CUDA;
  }
  static PerDeviceFlag attr_done;
  if (!attr_done.get()) {
    HYDRA_CUDA(cudaFuncSetAttribute(tree_attn_tc_kernel<HD, QROWS, NP>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
    attr_done.set();
  }
  AttArgs a{};
  a.rs = rs; a.out = out; a.out_ps = out_ps; a.H = H; a.max_seq = max_seq; a.status = status; a.wait_limit = WAIT_LIMIT;
  a.q_plane_rows = q_rows; a.kv_plane_rows = (int)cache_rows; a.early = stable_lengths ? 1 : 0; a.row_off = row_off;
  a.nchunks = pick_chunks(H * rs.batch, len_upper, sm_count());
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(H, rs.batch, a.nchunks); cfg.blockDim = dim3(C::NTHREADS); cfg.dynamicSmemBytes = C::SMEM_BYTES; cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = (unsigned)a.nchunks;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 2;
  HYDRA_CUDA(cudaLaunchKernelEx(&cfg, tree_attn_tc_kernel<HD, QROWS, NP>, tq, tk, tv, a));
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

template <int NP>
hydra_status dispatch(const __half* q, int q_rows, const __half* kc, const __half* vc, int cache_batch, RowSet rs, bf16* out, size_t out_ps,
                      int H, int hd, int max_seq, int len_upper, int* status, bool stable_lengths, cudaStream_t st) {
  const bool wide = rs.tc > 64;
  if (hd == 128 && wide && NP == 2) {
    // Q, P and the rings of two planes for 128 query rows exceed the shared memory of an SM: 64 rows per launch; the rows of
    // an earlier launch are cache rows to a later one (the preceding kernel has appended the K and V rows of the whole chunk)
    for (int off = 0; off < rs.tc; off += 64) {
      hydra_status r = run<128, 64, 2>(q, q_rows, kc, vc, cache_batch, rs, out, out_ps, H, max_seq, len_upper, status, stable_lengths, off, st);
      if (r != HYDRA_OK) return r;
    }
    return HYDRA_OK;
  }
  if (hd == 128) return wide ? run<128, 128, 1>(q, q_rows, kc, vc, cache_batch, rs, out, out_ps, H, max_seq, len_upper, status, stable_lengths, 0, st)
                             : run<128, 64, NP>(q, q_rows, kc, vc, cache_batch, rs, out, out_ps, H, max_seq, len_upper, status, stable_lengths, 0, st);
  if (hd == 64) return wide ? run<64, 128, NP>(q, q_rows, kc, vc, cache_batch, rs, out, out_ps, H, max_seq, len_upper, status, stable_lengths, 0, st)
                            : run<64, 64, NP>(q, q_rows, kc, vc, cache_batch, rs, out, out_ps, H, max_seq, len_upper, status, stable_lengths, 0, st);
  return HYDRA_ERR_UNSUPPORTED;
}

}  // namespace

hydra_status tree_attention_tc(const __half* q, int q_rows, const __half* kc, const __half* vc, int cache_batch, int planes, RowSet rs,
                               bf16* out, size_t out_ps, int H, int hd, int max_seq, int len_upper, int* status, bool stable_lengths,
                               cudaStream_t st) {
  if (rs.tc > 128 || (rs.mask && rs.tc > 64) || (planes != 1 && planes != 2)) return HYDRA_ERR_UNSUPPORTED;
  if (!tensor_map_encoder_available()) { set_last_error("cuTensorMapEncodeTiled entry point", cudaErrorUnknown); return HYDRA_ERR_CUDA; }
  if (((uintptr_t)q | (uintptr_t)kc | (uintptr_t)vc) & 15) return HYDRA_ERR_INVALID;
  return planes == 2 ? dispatch<2>(q, q_rows, kc, vc, cache_batch, rs, out, out_ps, H, hd, max_seq, len_upper, status, stable_lengths, st)
                     : dispatch<1>(q, q_rows, kc, vc, cache_batch, rs, out, out_ps, H, hd, max_seq, len_upper, status, stable_lengths, st);
}

}  // namespace hydra

// Tree attention for bfloat16 caches on the tensor cores (mma.sync m16n8k16, float accumulate).
//
// One CTA per (head, sequence, KV chunk).  A sequence's KV rows are cut into TILE-row tiles and the tiles are dealt
// to the grid's chunks in equal contiguous runs (computed on the device from the real length, so every chunk of
// the launch has work whatever the length); Q and the chunk's K and V tiles are streamed once through a five-stage
// cp.async ring (four tiles in flight per CTA: the walk is bound by HBM latency otherwise).  Eight warps: warp w
// owns query rows 16 (w & 3) .. +15 (as MMA fragments) and the keys of half (w >> 2) of every tile.  Scores of
// committed slots are unmasked; a tree slot j is visible to row i iff bit j of the row's ancestor bitmask is set.
// Each warp keeps a running (max, sum, weighted V) per query row in the exp2 domain (online softmax, reductions by
// warp shuffles over the 4 lanes that share a row); the two key halves are merged through shared memory at the end.
// Merging the chunks of a (head, sequence) pair, in chunk order either way: with up to 8 chunks the pair's CTAs
// form a thread-block cluster, leave their partial rows in their own shared memory and each merges a share of the
// rows out of its peers' shared memory; with more chunks the partial rows go to a scratch buffer and the CTA that
// reports in last (an arrival counter that it resets) merges them.
// Precision: q, K, V and the attention output are stored as two bfloat16 planes (hi = bf16(v), lo = bf16(v - hi),
// about 16 mantissa bits together).  Products use the three significant cross terms (hi*hi + lo*hi + hi*lo); the
// softmax weights are split the same way before the P V product.  A plane distance of 0 selects hi-only operands.
#include "launch.h"
#include <math.h>
#include <cstdlib>

namespace hydra {

namespace {

constexpr int NWARP = 8;           // warp w: query rows 16 (w & 3) .. +15, key half w >> 2 of every tile

// First tile of chunk c when nt tiles are dealt to nch chunks in equal contiguous runs.
__device__ __forceinline__ int chunk_first_tile(int c, int nt, int nch) { return (int)(((unsigned)c * (unsigned)nt) / (unsigned)nch); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// thread-block cluster helpers (the chunks of one (head, sequence) pair form a cluster along z)
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
  asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ float2 ld_peer2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
  return v;
}

// CLUSTER: the nchunks (<= 8) CTAs of a (head, sequence) pair are one thread-block cluster; they leave their partial
// rows in their own shared memory and every CTA merges its share of the rows out of its peers' shared memory
// (no scratch, no counters).  Otherwise: partial rows in scratch, merged by the CTA that reports in last.
template <int HD, bool HL, int TILE, int NS, bool CLUSTER>
__global__ void __launch_bounds__(NWARP * 32) tree_attn_tc_kernel(const bf16* __restrict__ q, size_t q_ps, const bf16* __restrict__ kc,
                                                                  const bf16* __restrict__ vc, size_t kv_ps, RowSet rs,
                                                                  float* __restrict__ part_o, float* __restrict__ part_ml,
                                                                  int* __restrict__ arrived, bf16* __restrict__ out, size_t out_ps,
                                                                  int H, int max_seq, int nchunks) {
  pdl_trigger();
  pdl_wait();
  constexpr int LDS = HD + 8;                         // padded row (bf16 elements): conflict-free ldmatrix
  constexpr int KSTEPS = HD / 16;
  constexpr int NB = HD / 8;                          // output n-blocks
  constexpr int NP = HL ? 2 : 1;                      // planes
  constexpr int TSZ = TILE * LDS;                     // elements of one staged tile
  extern __shared__ __align__(16) unsigned char smem_raw[];
  bf16* Qs = reinterpret_cast<bf16*>(smem_raw);       // [NP][64][LDS]
  bf16* KVs = Qs + NP * 64 * LDS;                     // [NS stages][K planes, V planes][TILE][LDS]
  __shared__ int s_last;

  const int h = blockIdx.x, b = blockIdx.y, c = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int nr = rs.n_rows ? rs.n_rows[b] : rs.tc;
  const int p0 = rs.pos0[b];
  const int total = p0 + nr;
  const int nt = (total + TILE - 1) / TILE;
  const int s0 = chunk_first_tile(c, nt, nchunks) * TILE;
  const int s1 = min(chunk_first_tile(c + 1, nt, nchunks) * TILE, total);
  const int d = H * HD;
  const bool has_work = s0 < s1 && nr > 0;            // a chunk that got no tile only reports in (see the end)
  const size_t head_off = ((size_t)b * H + h) * max_seq * HD;
  constexpr int PIECES = HD / 8;                       // 16-byte pieces per row

  auto tile_ptr = [&](int buf, int kv, int plane) { return KVs + ((buf * 2 + kv) * NP + plane) * TSZ; };
  auto load_tile = [&](int buf, int t0) {
    for (int e = tid; e < TILE * PIECES; e += NWARP * 32) {
      const int r = e / PIECES, pc = e % PIECES;
      const int slot = t0 + r;
#pragma unroll
      for (int kv = 0; kv < 2; ++kv)
#pragma unroll
        for (int pl = 0; pl < NP; ++pl) {
          bf16* dst = tile_ptr(buf, kv, pl) + r * LDS + pc * 8;
          if (slot < s1) cp_async16((uint32_t)__cvta_generic_to_shared(dst), (kv ? vc : kc) + pl * kv_ps + head_off + (size_t)slot * HD + pc * 8);
          else *reinterpret_cast<uint4*>(dst) = make_uint4(0, 0, 0, 0);     // rows past the end (their scores are masked)
        }
    }
  };

  const int ntiles = has_work ? (s1 - s0 + TILE - 1) / TILE : 0;
  // request Q (rows past nr are zero) and the first NS-1 KV tiles: one cp.async group per tile, Q rides with the first
  for (int e = tid; has_work && e < 64 * PIECES; e += NWARP * 32) {
    const int r = e / PIECES, pc = e % PIECES;
#pragma unroll
    for (int pl = 0; pl < NP; ++pl) {
      bf16* dst = Qs + (pl * 64 + r) * LDS + pc * 8;
      if (r < nr) cp_async16((uint32_t)__cvta_generic_to_shared(dst), q + pl * q_ps + (size_t)(b * rs.tc + r) * d + h * HD + pc * 8);
      else *reinterpret_cast<uint4*>(dst) = make_uint4(0, 0, 0, 0);
    }
  }
#pragma unroll
  for (int i = 0; i < NS - 1; ++i) {
    if (i < ntiles) load_tile(i, s0 + i * TILE);
    cp_async_commit();
  }
  const int row0 = (warp & 3) * 16, khalf = warp >> 2;
  constexpr int HT = TILE / 2;                           // keys of a tile per warp
  const bool warp_active = has_work && row0 < nr;
  const int ra = row0 + g, rb = row0 + g + 8;            // the two query rows this thread owns
  const uint64_t mask_a = ra < nr ? rs.mask[ra] : 0ull, mask_b = rb < nr ? rs.mask[rb] : 0ull;
  float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;
  float o[NB][4];
#pragma unroll
  for (int n = 0; n < NB; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
  const float sc = rsqrtf((float)HD) * 1.4426950408889634f;   // 1/sqrt(hd) * log2(e)
  const uint32_t q_addr = (uint32_t)__cvta_generic_to_shared(Qs + (row0 + (lane & 15)) * LDS + (lane >> 4) * 8);

  for (int it = 0; it < ntiles; ++it) {
    const int t0 = s0 + it * TILE;
    const int buf = it % NS;
    if (it + NS - 1 < ntiles) load_tile((it + NS - 1) % NS, t0 + (NS - 1) * TILE);      // the buffer read in iteration it - 1
    cp_async_commit();
    cp_async_wait<NS - 1>();                             // tile `it` (and Q, stored before the first barrier) has landed
    __syncthreads();
    if (warp_active) {
      float s[HT / 8][4];
#pragma unroll
      for (int n = 0; n < HT / 8; ++n) { s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f; }
      const uint32_t k_off = (uint32_t)(((khalf * HT + (lane & 7) + (lane >> 4) * 8) * LDS + ((lane >> 3) & 1) * 8) * 2);
      const uint32_t kh_addr = (uint32_t)__cvta_generic_to_shared(tile_ptr(buf, 0, 0)) + k_off;
#pragma unroll
      for (int kk = 0; kk < KSTEPS; ++kk) {
        uint32_t qh[4], ql[4];
        ldsm_x4(q_addr + kk * 32, qh[0], qh[1], qh[2], qh[3]);
        if (HL) ldsm_x4(q_addr + 64 * LDS * 2 + kk * 32, ql[0], ql[1], ql[2], ql[3]);
#pragma unroll
        for (int np = 0; np < HT / 16; ++np) {         // 16 keys per ldmatrix.x4
          uint32_t b0, b1, b2, b3;
          const uint32_t addr = kh_addr + (uint32_t)((np * 16 * LDS + kk * 16) * 2);
          ldsm_x4(addr, b0, b1, b2, b3);
          mma_bf16(s[2 * np], qh[0], qh[1], qh[2], qh[3], b0, b1);
          mma_bf16(s[2 * np + 1], qh[0], qh[1], qh[2], qh[3], b2, b3);
          if (HL) {
            mma_bf16(s[2 * np], ql[0], ql[1], ql[2], ql[3], b0, b1);
            mma_bf16(s[2 * np + 1], ql[0], ql[1], ql[2], ql[3], b2, b3);
            ldsm_x4(addr + TSZ * 2, b0, b1, b2, b3);   // K lo plane
            mma_bf16(s[2 * np], qh[0], qh[1], qh[2], qh[3], b0, b1);
            mma_bf16(s[2 * np + 1], qh[0], qh[1], qh[2], qh[3], b2, b3);
          }
        }
      }
      // scale, mask, running max
      const int k0 = t0 + khalf * HT;                    // first key of this warp's half
      const bool need_mask = k0 + HT > p0 || k0 + HT > s1;
      float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
      for (int n = 0; n < HT / 8; ++n) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float v = s[n][e] * sc;
          if (need_mask) {
            int key = k0 + n * 8 + 2 * t + (e & 1);
            uint64_t mk = (e < 2) ? mask_a : mask_b;
            bool ok = key < s1 && (key < p0 || ((mk >> (key - p0)) & 1ull));
            v = ok ? v : -INFINITY;
          }
          s[n][e] = v;
          if (e < 2) mx_a = fmaxf(mx_a, v); else mx_b = fmaxf(mx_b, v);
        }
      }
      mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 1)); mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 2));
      mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 1)); mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 2));
      const float mn_a = fmaxf(m_a, mx_a), mn_b = fmaxf(m_b, mx_b);
      const float base_a = mn_a == -INFINITY ? 0.f : mn_a, base_b = mn_b == -INFINITY ? 0.f : mn_b;
      const float al_a = exp2f(m_a - base_a), al_b = exp2f(m_b - base_b);     // exp2(-inf) = 0 for the first tile
      m_a = mn_a; m_b = mn_b;
      float sum_a = 0.f, sum_b = 0.f;
#pragma unroll
      for (int n = 0; n < HT / 8; ++n) {
        s[n][0] = exp2f(s[n][0] - base_a); s[n][1] = exp2f(s[n][1] - base_a);
        s[n][2] = exp2f(s[n][2] - base_b); s[n][3] = exp2f(s[n][3] - base_b);
        sum_a += s[n][0] + s[n][1]; sum_b += s[n][2] + s[n][3];
      }
      l_a = l_a * al_a + sum_a; l_b = l_b * al_b + sum_b;      // per-thread partial sums; reduced over the quad at the end
#pragma unroll
      for (int n = 0; n < NB; ++n) { o[n][0] *= al_a; o[n][1] *= al_a; o[n][2] *= al_b; o[n][3] *= al_b; }
      // O += P V
      const uint32_t v_off = (uint32_t)(((khalf * HT + (lane & 7) + ((lane >> 3) & 1) * 8) * LDS + (lane >> 4) * 8) * 2);
      const uint32_t vh_addr = (uint32_t)__cvta_generic_to_shared(tile_ptr(buf, 1, 0)) + v_off;
#pragma unroll
      for (int kp = 0; kp < HT / 16; ++kp) {           // 16 keys per k-step
        uint32_t ah[4], al[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float x0 = s[2 * kp + (e >> 1)][(e & 1) * 2], x1 = s[2 * kp + (e >> 1)][(e & 1) * 2 + 1];
          ah[e] = pack_bf16(x0, x1);
          if (HL) {
            const __nv_bfloat162 hv = *reinterpret_cast<const __nv_bfloat162*>(&ah[e]);
            al[e] = pack_bf16(x0 - __low2float(hv), x1 - __high2float(hv));
          }
        }
#pragma unroll
        for (int np = 0; np < NB / 2; ++np) {          // 16 output columns per ldmatrix.x4.trans
          uint32_t b0, b1, b2, b3;
          const uint32_t addr = vh_addr + (uint32_t)((kp * 16 * LDS + np * 16) * 2);
          ldsm_x4_trans(addr, b0, b1, b2, b3);
          mma_bf16(o[2 * np], ah[0], ah[1], ah[2], ah[3], b0, b1);
          mma_bf16(o[2 * np + 1], ah[0], ah[1], ah[2], ah[3], b2, b3);
          if (HL) {
            mma_bf16(o[2 * np], al[0], al[1], al[2], al[3], b0, b1);
            mma_bf16(o[2 * np + 1], al[0], al[1], al[2], al[3], b2, b3);
            ldsm_x4_trans(addr + TSZ * 2, b0, b1, b2, b3);   // V lo plane
            mma_bf16(o[2 * np], ah[0], ah[1], ah[2], ah[3], b0, b1);
            mma_bf16(o[2 * np + 1], ah[0], ah[1], ah[2], ah[3], b2, b3);
          }
        }
      }
    }
    __syncthreads();
  }
  l_a += __shfl_xor_sync(0xffffffffu, l_a, 1); l_a += __shfl_xor_sync(0xffffffffu, l_a, 2);
  l_b += __shfl_xor_sync(0xffffffffu, l_b, 1); l_b += __shfl_xor_sync(0xffffffffu, l_b, 2);
  // merge the two key halves: the upper warps hand (m, l, o) to their partner through the (now idle) tile ring
  float* xch = reinterpret_cast<float*>(KVs) + ((warp & 3) * 32 + lane) * (NB * 4 + 4);
  if (khalf == 1 && warp_active) {
#pragma unroll
    for (int n = 0; n < NB; ++n) *reinterpret_cast<float4*>(xch + n * 4) = make_float4(o[n][0], o[n][1], o[n][2], o[n][3]);
    *reinterpret_cast<float4*>(xch + NB * 4) = make_float4(m_a, m_b, l_a, l_b);
  }
  __syncthreads();
  constexpr int XCH_FLOATS = 4 * 32 * (NB * 4 + 4);     // the hand-over area above
  float* xo = reinterpret_cast<float*>(KVs) + XCH_FLOATS;    // CLUSTER: this chunk's partial rows [64][HD], then (m, l) [64][2]
  float* xml = xo + 64 * HD;
  if (CLUSTER && !warp_active && khalf == 0) {           // rows this CTA has nothing for: weight zero
    if (t == 0) { *reinterpret_cast<float2*>(xml + ra * 2) = make_float2(-INFINITY, 0.f); *reinterpret_cast<float2*>(xml + rb * 2) = make_float2(-INFINITY, 0.f); }
  }
  if (khalf == 0 && warp_active) {
    const float4 ml = *reinterpret_cast<const float4*>(xch + NB * 4);
    const float mn_a = fmaxf(m_a, ml.x), mn_b = fmaxf(m_b, ml.y);
    const float base_a = mn_a == -INFINITY ? 0.f : mn_a, base_b = mn_b == -INFINITY ? 0.f : mn_b;
    const float w0a = exp2f(m_a - base_a), w1a = exp2f(ml.x - base_a), w0b = exp2f(m_b - base_b), w1b = exp2f(ml.y - base_b);
    m_a = mn_a; m_b = mn_b;
    l_a = l_a * w0a + ml.z * w1a; l_b = l_b * w0b + ml.w * w1b;
    // partials: o (un-normalised), m (log2 domain), l
    if (CLUSTER) {
#pragma unroll
      for (int n = 0; n < NB; ++n) {
        const float4 v = *reinterpret_cast<const float4*>(xch + n * 4);
        *reinterpret_cast<float2*>(xo + ra * HD + n * 8 + 2 * t) = make_float2(o[n][0] * w0a + v.x * w1a, o[n][1] * w0a + v.y * w1a);
        *reinterpret_cast<float2*>(xo + rb * HD + n * 8 + 2 * t) = make_float2(o[n][2] * w0b + v.z * w1b, o[n][3] * w0b + v.w * w1b);
      }
      if (t == 0) {
        *reinterpret_cast<float2*>(xml + ra * 2) = ra < nr ? make_float2(m_a, l_a) : make_float2(-INFINITY, 0.f);
        *reinterpret_cast<float2*>(xml + rb * 2) = rb < nr ? make_float2(m_b, l_b) : make_float2(-INFINITY, 0.f);
      }
    } else {
      const size_t idx_a = ((size_t)(b * rs.tc + ra) * H + h) * nchunks + c, idx_b = ((size_t)(b * rs.tc + rb) * H + h) * nchunks + c;
#pragma unroll
      for (int n = 0; n < NB; ++n) {
        const float4 v = *reinterpret_cast<const float4*>(xch + n * 4);
        if (ra < nr) __stcg(reinterpret_cast<float2*>(part_o + idx_a * HD + n * 8 + 2 * t), make_float2(o[n][0] * w0a + v.x * w1a, o[n][1] * w0a + v.y * w1a));
        if (rb < nr) __stcg(reinterpret_cast<float2*>(part_o + idx_b * HD + n * 8 + 2 * t), make_float2(o[n][2] * w0b + v.z * w1b, o[n][3] * w0b + v.w * w1b));
      }
      if (t == 0 && ra < nr) __stcg(reinterpret_cast<float2*>(part_ml + idx_a * 2), make_float2(m_a, l_a));
      if (t == 0 && rb < nr) __stcg(reinterpret_cast<float2*>(part_ml + idx_b * 2), make_float2(m_b, l_b));
    }
  }
  if (CLUSTER) {
    // out[r][h][:] = sum_c o_c 2^(m_c - M) / sum_c l_c 2^(m_c - M), chunks in order; this CTA takes rows c, c + nchunks, ...
    cluster_sync_all();                                  // every chunk's rows are in its shared memory
    constexpr int V4 = HD / 4;
    const uint32_t xo_s = (uint32_t)__cvta_generic_to_shared(xo), xml_s = (uint32_t)__cvta_generic_to_shared(xml);
    const int my_rows = (rs.tc - c + nchunks - 1) / nchunks;
    for (int e = tid; e < my_rows * V4; e += NWARP * 32) {
      const int i = c + (e / V4) * nchunks, k4 = e % V4;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      if (i < nr) {
        float mc[8], lc[8];
        float M = -INFINITY;
#pragma unroll
        for (int cc = 0; cc < 8; ++cc) {
          mc[cc] = -INFINITY; lc[cc] = 0.f;
          if (cc < nchunks) { const float2 ml = ld_peer2(peer_smem(xml_s + (uint32_t)i * 8u, (uint32_t)cc)); mc[cc] = ml.x; lc[cc] = ml.y; }
          M = fmaxf(M, mc[cc]);
        }
        float L = 0.f;
#pragma unroll
        for (int cc = 0; cc < 8; ++cc) {
          if (cc < nchunks && mc[cc] != -INFINITY) {
            const float w = exp2f(mc[cc] - M);
            const float4 v = ld_peer4(peer_smem(xo_s + (uint32_t)(i * HD + k4 * 4) * 4u, (uint32_t)cc));
            L += lc[cc] * w;
            acc.x += v.x * w; acc.y += v.y * w; acc.z += v.z * w; acc.w += v.w * w;
          }
        }
        const float inv = L > 0.f ? 1.f / L : 0.f;
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
      }
      bf16* dst = out + ((size_t)b * rs.tc + i) * d + h * HD + k4 * 4;      // rows past nr get zeros
      const __nv_bfloat162 h0 = __floats2bfloat162_rn(acc.x, acc.y), h1 = __floats2bfloat162_rn(acc.z, acc.w);
      *reinterpret_cast<uint2*>(dst) = make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
      if (out_ps) {
        const __nv_bfloat162 l0 = __floats2bfloat162_rn(acc.x - __low2float(h0), acc.y - __high2float(h0));
        const __nv_bfloat162 l1 = __floats2bfloat162_rn(acc.z - __low2float(h1), acc.w - __high2float(h1));
        *reinterpret_cast<uint2*>(dst + out_ps) = make_uint2(*reinterpret_cast<const uint32_t*>(&l0), *reinterpret_cast<const uint32_t*>(&l1));
      }
    }
    cluster_sync_all();                                  // peers may still be reading this CTA's rows
    return;
  }
  // The last of the (head, sequence)'s chunks to report in merges them:
  // out[r][h][:] = sum_c o_c 2^(m_c - M) / sum_c l_c 2^(m_c - M) over the chunks that were dealt tiles, in chunk order.
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int prev = atomicAdd(arrived + b * H + h, 1);
    s_last = prev == nchunks - 1;
    if (s_last) arrived[b * H + h] = 0;                  // ready for the next launch
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // Every thread owns up to PER float4 pieces of the output rows.  The partial rows of the first four chunks are
  // requested before anything else, so that they travel while the chunk weights are worked out (one (row, chunk)
  // pair per thread, through shared memory); further chunks follow four at a time.
  constexpr int V4 = HD / 4, PER = (64 * V4 + NWARP * 32 - 1) / (NWARP * 32), CB = 4;
  float4 v[CB][PER];
  auto dealt = [&](int cc) { return chunk_first_tile(cc, nt, nchunks) != chunk_first_tile(cc + 1, nt, nchunks); };   // else it wrote nothing
  auto load_batch = [&](int c0) {
#pragma unroll
    for (int cb = 0; cb < CB; ++cb) {
      const int cc = c0 + cb;
      const bool live = cc < nchunks && dealt(cc);
#pragma unroll
      for (int j = 0; j < PER; ++j) {
        const int e = tid + j * NWARP * 32, i = e / V4, k4 = e % V4;
        v[cb][j] = live && i < nr ? __ldcg(reinterpret_cast<const float4*>(part_o + ((((size_t)b * rs.tc + i) * H + h) * nchunks + cc) * HD + k4 * 4))
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
  };
  load_batch(0);
  float* sm_m = reinterpret_cast<float*>(KVs);         // [tc][nchunks] chunk maxima, then the normalised chunk weights
  float* sm_l = sm_m + rs.tc * nchunks;
  for (int e = tid; e < rs.tc * nchunks; e += NWARP * 32) {
    const int i = e / nchunks, cc = e % nchunks;
    float2 ml = make_float2(-INFINITY, 0.f);
    if (i < nr && dealt(cc)) ml = __ldcg(reinterpret_cast<const float2*>(part_ml + (((size_t)b * rs.tc + i) * H + h) * nchunks * 2 + cc * 2));
    sm_m[e] = ml.x; sm_l[e] = ml.y;
  }
  __syncthreads();
  for (int i = tid; i < rs.tc; i += NWARP * 32) {
    float M = -INFINITY, L = 0.f;
    for (int cc = 0; cc < nchunks; ++cc) M = fmaxf(M, sm_m[i * nchunks + cc]);
    for (int cc = 0; cc < nchunks; ++cc) {
      const float mc = sm_m[i * nchunks + cc];
      const float w = mc == -INFINITY ? 0.f : exp2f(mc - M);
      L += sm_l[i * nchunks + cc] * w;
      sm_m[i * nchunks + cc] = w;
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
    for (int cc = 0; cc < nchunks; ++cc) sm_m[i * nchunks + cc] *= inv;
  }
  __syncthreads();
  float4 acc[PER];
#pragma unroll
  for (int j = 0; j < PER; ++j) acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int c0 = 0; c0 < nchunks; c0 += CB) {
    if (c0 > 0) load_batch(c0);
#pragma unroll
    for (int cb = 0; cb < CB; ++cb) {
      const int cc = c0 + cb;
#pragma unroll
      for (int j = 0; j < PER; ++j) {
        const int i = (tid + j * NWARP * 32) / V4;
        const float w = cc < nchunks && i < rs.tc ? sm_m[i * nchunks + cc] : 0.f;
        acc[j].x += v[cb][j].x * w; acc[j].y += v[cb][j].y * w; acc[j].z += v[cb][j].z * w; acc[j].w += v[cb][j].w * w;
      }
    }
  }
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    const int e = tid + j * NWARP * 32, i = e / V4, k4 = e % V4;
    if (i >= rs.tc) continue;
    bf16* dst = out + ((size_t)b * rs.tc + i) * d + h * HD + k4 * 4;      // rows past nr get zeros
    const __nv_bfloat162 h0 = __floats2bfloat162_rn(acc[j].x, acc[j].y), h1 = __floats2bfloat162_rn(acc[j].z, acc[j].w);
    *reinterpret_cast<uint2*>(dst) = make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
    if (out_ps) {
      const __nv_bfloat162 l0 = __floats2bfloat162_rn(acc[j].x - __low2float(h0), acc[j].y - __high2float(h0));
      const __nv_bfloat162 l1 = __floats2bfloat162_rn(acc[j].z - __low2float(h1), acc[j].w - __high2float(h1));
      *reinterpret_cast<uint2*>(dst + out_ps) = make_uint2(*reinterpret_cast<const uint32_t*>(&l0), *reinterpret_cast<const uint32_t*>(&l1));
    }
  }
}

// Number of KV chunks per (head, sequence) for lengths up to len_upper.  Few (head, sequence) pairs: one CTA per SM
// at most and chunks as long as that allows (the kernel is bound by the MMA rate of an SM, so what counts is the
// largest number of tiles any SM walks, plus about four tiles' worth of set-up and merging per CTA: measured on the
// 13B shape at 2048 rows, 3 chunks in one wave beat 7 chunks in two); many pairs: chunks of about 128 rows at most.
int pick_chunks(int pairs, int len_upper, int tile, int nchunks_max, int sms, bool* cluster) {
  const int nt = (len_upper + tile - 1) / tile;
  int hi = (len_upper + ATT_CHUNK_ROWS - 1) / ATT_CHUNK_ROWS;
  hi = hi < 1 ? 1 : (hi > nchunks_max ? nchunks_max : hi);
  auto cost = [&](int n) {
    const long per_sm = ((long)pairs * n + sms - 1) / sms, tiles = (nt + n - 1) / n;
    return per_sm * (tiles + 4) + 1;
  };
  int best = hi; long best_cost = -1;
  for (int n = 1; n <= hi; ++n)
    if (best_cost < 0 || cost(n) < best_cost) { best = n; best_cost = cost(n); }     // ties: fewer chunks
  *cluster = best <= 8;        // up to 8 chunks: the pair's CTAs form a cluster and merge through shared memory
  return best;
}

template <int HD, bool HL, int NS>
hydra_status run_ns(const bf16* q, size_t q_ps, const bf16* kc, const bf16* vc, size_t kv_ps, RowSet rs, bf16* out, size_t out_ps,
                 float* scratch, int H, int max_seq, int len_upper, cudaStream_t st) {
  constexpr int TILE = 32;                    // 32-row tiles, four of them in flight: hides the HBM latency of a chunk's walk
  const int nchunks_max = (max_seq + ATT_CHUNK_ROWS - 1) / ATT_CHUNK_ROWS;     // what the scratch is sized for
  const int sms = sm_count();
  if ((size_t)H * rs.batch * sizeof(int) > ATT_SCRATCH_HEADER) return HYDRA_ERR_UNSUPPORTED;
  bool cluster = false;
  const int nchunks = pick_chunks(H * rs.batch, len_upper, TILE, nchunks_max, sms, &cluster);
  const size_t rows = (size_t)rs.batch * rs.tc;
  int* arrived = reinterpret_cast<int*>(scratch);     // one counter per (sequence, head): zero between launches
  float* part_o = scratch + ATT_SCRATCH_HEADER / sizeof(float);
  float* part_ml = part_o + rows * H * nchunks_max * HD;
  constexpr int LDS = HD + 8;
  constexpr int NP = HL ? 2 : 1;
  const size_t ring = (size_t)NP * 2 * NS * TILE * LDS * sizeof(bf16);
  const size_t xchg = (size_t)(4 * 32 * (HD / 2 + 4) + 64 * HD + 128) * sizeof(float);      // hand-over area + a chunk's partial rows + (m, l)
  const size_t smem = (size_t)NP * 64 * LDS * sizeof(bf16) + (ring > xchg ? ring : xchg);
  static PerDeviceFlag attr_done;
  if (!attr_done.get()) {
    HYDRA_CUDA(cudaFuncSetAttribute(tree_attn_tc_kernel<HD, HL, TILE, NS, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    HYDRA_CUDA(cudaFuncSetAttribute(tree_attn_tc_kernel<HD, HL, TILE, NS, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    attr_done.set();
  }
  if (!cluster) {
    launch_pdl(tree_attn_tc_kernel<HD, HL, TILE, NS, false>, dim3(H, rs.batch, nchunks), dim3(NWARP * 32), smem, st, q, q_ps, kc, vc, kv_ps, rs, part_o,
               part_ml, arrived, out, out_ps, H, max_seq, nchunks);
    HYDRA_LAUNCH_CHECK();
    return HYDRA_OK;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(H, rs.batch, nchunks); cfg.blockDim = dim3(NWARP * 32); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = (unsigned)nchunks;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 2;
  HYDRA_CUDA(cudaLaunchKernelEx(&cfg, tree_attn_tc_kernel<HD, HL, TILE, NS, true>, q, q_ps, kc, vc, kv_ps, rs, part_o, part_ml, arrived, out, out_ps, H,
                                max_seq, nchunks));
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

template <int HD, bool HL>
hydra_status run(const bf16* q, size_t q_ps, const bf16* kc, const bf16* vc, size_t kv_ps, RowSet rs, bf16* out, size_t out_ps,
                 float* scratch, int H, int max_seq, int len_upper, cudaStream_t st) {
  return run_ns<HD, HL, 5>(q, q_ps, kc, vc, kv_ps, rs, out, out_ps, scratch, H, max_seq, len_upper, st);
}

}  // namespace

hydra_status tree_attention_tc(const bf16* q, size_t q_ps, const bf16* kc, const bf16* vc, size_t kv_ps, RowSet rs, bf16* out,
                               size_t out_ps, void* scratch, int H, int hd, int max_seq, int len_upper, cudaStream_t st) {
  if (rs.tc > 64) return HYDRA_ERR_UNSUPPORTED;
  if ((q_ps == 0) != (kv_ps == 0)) return HYDRA_ERR_UNSUPPORTED;           // q and the caches split the same way
  const bool hl = q_ps != 0;
  if (hd == 128 && hl) return run<128, true>(q, q_ps, kc, vc, kv_ps, rs, out, out_ps, (float*)scratch, H, max_seq, len_upper, st);
  if (hd == 128) return run<128, false>(q, q_ps, kc, vc, kv_ps, rs, out, out_ps, (float*)scratch, H, max_seq, len_upper, st);
  if (hd == 64 && hl) return run<64, true>(q, q_ps, kc, vc, kv_ps, rs, out, out_ps, (float*)scratch, H, max_seq, len_upper, st);
  if (hd == 64) return run<64, false>(q, q_ps, kc, vc, kv_ps, rs, out, out_ps, (float*)scratch, H, max_seq, len_upper, st);
  return HYDRA_ERR_UNSUPPORTED;
}

}  // namespace hydra

// Tree attention for bfloat16 caches on the tensor cores (mma.sync m16n8k16, float accumulate).
//
// One CTA per (head, sequence, KV chunk): the chunk's K and V rows are streamed once from HBM through a
// double-buffered cp.async ring of 64-row tiles; the (at most 64) query rows of the call stay in registers
// as MMA fragments, 16 rows per warp.  Scores of committed slots are unmasked; a tree slot j is visible to
// row i iff bit j of the row's ancestor bitmask is set.  Each warp keeps a running (max, sum, weighted V)
// per query row in the exp2 domain (online softmax, reductions by warp shuffles over the 4 lanes that share
// a row); per-chunk partial results are merged by the combine kernel in fixed order.
// Precision: q, K, V and the attention output are stored as two bfloat16 planes (hi = bf16(v), lo = bf16(v - hi),
// about 16 mantissa bits together).  Products use the three significant cross terms (hi*hi + lo*hi + hi*lo); the
// softmax weights are split the same way before the P V product.  A plane distance of 0 selects hi-only operands.
#include "launch.h"
#include <math.h>
#include <cstdlib>

namespace hydra {

namespace {

constexpr int NWARP = 4;           // 16 query rows each

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

template <int HD, bool HL, int TILE>
__global__ void __launch_bounds__(NWARP * 32) tree_attn_tc_kernel(const bf16* __restrict__ q, size_t q_ps, const bf16* __restrict__ kc,
                                                                  const bf16* __restrict__ vc, size_t kv_ps, RowSet rs,
                                                                  float* __restrict__ part_o, float* __restrict__ part_ml,
                                                                  int H, int max_seq, int nchunks, int chunk) {
  pdl_trigger();
  pdl_wait();
  constexpr int LDS = HD + 8;                         // padded row (bf16 elements): conflict-free ldmatrix
  constexpr int KSTEPS = HD / 16;
  constexpr int NB = HD / 8;                          // output n-blocks
  constexpr int NP = HL ? 2 : 1;                      // planes
  constexpr int TSZ = TILE * LDS;                     // elements of one staged tile
  extern __shared__ __align__(16) unsigned char smem_raw[];
  bf16* Qs = reinterpret_cast<bf16*>(smem_raw);       // [NP][64][LDS]
  bf16* KVs = Qs + NP * 64 * LDS;                     // [2 stages][K planes, V planes][TILE][LDS]

  const int h = blockIdx.x, b = blockIdx.y, c = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int nr = rs.n_rows ? rs.n_rows[b] : rs.tc;
  const int p0 = rs.pos0[b];
  const int total = p0 + nr;
  const int s0 = c * chunk;
  const int s1 = min(s0 + chunk, total);
  const int d = H * HD;
  if (s0 >= s1 || nr <= 0) return;                    // nothing in this chunk: the combine kernel skips it
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

  // stage Q (rows past nr are zero) and the first KV tile
  for (int e = tid; e < 64 * PIECES; e += NWARP * 32) {
    const int r = e / PIECES, pc = e % PIECES;
#pragma unroll
    for (int pl = 0; pl < NP; ++pl) {
      uint4 v = make_uint4(0, 0, 0, 0);
      if (r < nr) v = *reinterpret_cast<const uint4*>(q + pl * q_ps + (size_t)(b * rs.tc + r) * d + h * HD + pc * 8);
      *reinterpret_cast<uint4*>(Qs + (pl * 64 + r) * LDS + pc * 8) = v;
    }
  }
  load_tile(0, s0);
  cp_async_commit();
  __syncthreads();

  const int row0 = warp * 16;
  const bool warp_active = row0 < nr;
  const int ra = row0 + g, rb = row0 + g + 8;            // the two query rows this thread owns
  const uint64_t mask_a = ra < nr ? rs.mask[ra] : 0ull, mask_b = rb < nr ? rs.mask[rb] : 0ull;
  float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;
  float o[NB][4];
#pragma unroll
  for (int n = 0; n < NB; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
  const float sc = rsqrtf((float)HD) * 1.4426950408889634f;   // 1/sqrt(hd) * log2(e)
  const uint32_t q_addr = (uint32_t)__cvta_generic_to_shared(Qs + (row0 + (lane & 15)) * LDS + (lane >> 4) * 8);

  const int ntiles = (s1 - s0 + TILE - 1) / TILE;
  for (int it = 0; it < ntiles; ++it) {
    const int t0 = s0 + it * TILE;
    const int buf = it & 1;
    if (it + 1 < ntiles) load_tile(buf ^ 1, t0 + TILE);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    if (warp_active) {
      float s[TILE / 8][4];
#pragma unroll
      for (int n = 0; n < TILE / 8; ++n) { s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f; }
      const uint32_t k_off = (uint32_t)((((lane & 7) + (lane >> 4) * 8) * LDS + ((lane >> 3) & 1) * 8) * 2);
      const uint32_t kh_addr = (uint32_t)__cvta_generic_to_shared(tile_ptr(buf, 0, 0)) + k_off;
#pragma unroll
      for (int kk = 0; kk < KSTEPS; ++kk) {
        uint32_t qh[4], ql[4];
        ldsm_x4(q_addr + kk * 32, qh[0], qh[1], qh[2], qh[3]);
        if (HL) ldsm_x4(q_addr + 64 * LDS * 2 + kk * 32, ql[0], ql[1], ql[2], ql[3]);
#pragma unroll
        for (int np = 0; np < TILE / 16; ++np) {       // 16 keys per ldmatrix.x4
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
      const bool need_mask = t0 + TILE > p0 || t0 + TILE > s1;
      float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
      for (int n = 0; n < TILE / 8; ++n) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float v = s[n][e] * sc;
          if (need_mask) {
            int key = t0 + n * 8 + 2 * t + (e & 1);
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
      for (int n = 0; n < TILE / 8; ++n) {
        s[n][0] = exp2f(s[n][0] - base_a); s[n][1] = exp2f(s[n][1] - base_a);
        s[n][2] = exp2f(s[n][2] - base_b); s[n][3] = exp2f(s[n][3] - base_b);
        sum_a += s[n][0] + s[n][1]; sum_b += s[n][2] + s[n][3];
      }
      l_a = l_a * al_a + sum_a; l_b = l_b * al_b + sum_b;      // per-thread partial sums; reduced over the quad at the end
#pragma unroll
      for (int n = 0; n < NB; ++n) { o[n][0] *= al_a; o[n][1] *= al_a; o[n][2] *= al_b; o[n][3] *= al_b; }
      // O += P V
      const uint32_t v_off = (uint32_t)((((lane & 7) + ((lane >> 3) & 1) * 8) * LDS + (lane >> 4) * 8) * 2);
      const uint32_t vh_addr = (uint32_t)__cvta_generic_to_shared(tile_ptr(buf, 1, 0)) + v_off;
#pragma unroll
      for (int kp = 0; kp < TILE / 16; ++kp) {         // 16 keys per k-step
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
  if (!warp_active) return;
  l_a += __shfl_xor_sync(0xffffffffu, l_a, 1); l_a += __shfl_xor_sync(0xffffffffu, l_a, 2);
  l_b += __shfl_xor_sync(0xffffffffu, l_b, 1); l_b += __shfl_xor_sync(0xffffffffu, l_b, 2);
  // partials: o (un-normalised), m (log2 domain), l
  if (ra < nr) {
    size_t idx = ((size_t)(b * rs.tc + ra) * H + h) * nchunks + c;
#pragma unroll
    for (int n = 0; n < NB; ++n) *reinterpret_cast<float2*>(part_o + idx * HD + n * 8 + 2 * t) = make_float2(o[n][0], o[n][1]);
    if (t == 0) { part_ml[idx * 2] = m_a; part_ml[idx * 2 + 1] = l_a; }
  }
  if (rb < nr) {
    size_t idx = ((size_t)(b * rs.tc + rb) * H + h) * nchunks + c;
#pragma unroll
    for (int n = 0; n < NB; ++n) *reinterpret_cast<float2*>(part_o + idx * HD + n * 8 + 2 * t) = make_float2(o[n][2], o[n][3]);
    if (t == 0) { part_ml[idx * 2] = m_b; part_ml[idx * 2 + 1] = l_b; }
  }
}

// out[r][h][:] = sum_c o_c 2^(m_c - M) / sum_c l_c 2^(m_c - M) over the chunks that hold slots of sequence b.
template <int HD>
__global__ void __launch_bounds__(HD) tree_attn_tc_combine_kernel(const float* __restrict__ part_o, const float* __restrict__ part_ml,
                                                                  RowSet rs, bf16* __restrict__ out, size_t out_ps, int H, int nchunks, int chunk) {
  pdl_trigger();
  pdl_wait();
  const int r = blockIdx.x, h = blockIdx.y, b = r / rs.tc, i = r % rs.tc;
  const int nr = rs.n_rows ? rs.n_rows[b] : rs.tc;
  const int k = threadIdx.x;
  bf16* dst = out + (size_t)r * H * HD + h * HD;
  if (i >= nr) { dst[k] = __float2bfloat16_rn(0.f); if (out_ps) dst[out_ps + k] = __float2bfloat16_rn(0.f); return; }
  const int used = min(nchunks, (rs.pos0[b] + nr + chunk - 1) / chunk);
  const size_t idx = ((size_t)r * H + h) * nchunks;
  float M = -INFINITY;
  for (int c = 0; c < used; ++c) M = fmaxf(M, part_ml[(idx + c) * 2]);
  float L = 0.f, acc = 0.f;
  for (int c = 0; c < used; ++c) {
    float mc = part_ml[(idx + c) * 2];
    if (mc == -INFINITY) continue;
    float w = exp2f(mc - M);
    L += part_ml[(idx + c) * 2 + 1] * w;
    acc += part_o[(idx + c) * HD + k] * w;
  }
  const float v = acc / L;
  const bf16 hi = __float2bfloat16_rn(v);
  dst[k] = hi;
  if (out_ps) dst[out_ps + k] = __float2bfloat16_rn(v - __bfloat162float(hi));
}

template <int HD, bool HL, int TILE>
hydra_status run_t(const bf16* q, size_t q_ps, const bf16* kc, const bf16* vc, size_t kv_ps, RowSet rs, bf16* out, size_t out_ps,
                 float* scratch, int H, int max_seq, int len_upper, int chunk, cudaStream_t st) {
  const int nchunks_max = (max_seq + chunk - 1) / chunk;
  int nchunks = (len_upper + chunk - 1) / chunk;
  nchunks = nchunks < 1 ? 1 : (nchunks > nchunks_max ? nchunks_max : nchunks);
  const size_t rows = (size_t)rs.batch * rs.tc;
  float* part_o = scratch;
  float* part_ml = scratch + rows * H * nchunks_max * HD;
  constexpr int LDS = HD + 8;
  constexpr int NP = HL ? 2 : 1;
  const size_t smem = (size_t)NP * (64 + 4 * TILE) * LDS * sizeof(bf16);
  static bool attr_done = false;
  if (!attr_done) {
    HYDRA_CUDA(cudaFuncSetAttribute(tree_attn_tc_kernel<HD, HL, TILE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    attr_done = true;
  }
  launch_pdl(tree_attn_tc_kernel<HD, HL, TILE>, dim3(H, rs.batch, nchunks), dim3(NWARP * 32), smem, st, q, q_ps, kc, vc, kv_ps, rs, part_o, part_ml, H,
             max_seq, nchunks, chunk);
  HYDRA_LAUNCH_CHECK();
  launch_pdl(tree_attn_tc_combine_kernel<HD>, dim3((unsigned)rows, H), dim3(HD), 0, st, (const float*)part_o, (const float*)part_ml, rs, out, out_ps, H,
             nchunks, chunk);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

// KV rows per pipeline stage: 32 lets two CTAs share an SM with two-plane operands (HYDRA_ATT_TILE=64: one CTA, fewer syncs).
template <int HD, bool HL>
hydra_status run(const bf16* q, size_t q_ps, const bf16* kc, const bf16* vc, size_t kv_ps, RowSet rs, bf16* out, size_t out_ps,
                 float* scratch, int H, int max_seq, int len_upper, int chunk, cudaStream_t st) {
  static const int tile = []() { const char* e = getenv("HYDRA_ATT_TILE"); return e ? atoi(e) : 32; }();
  if (tile == 64) return run_t<HD, HL, 64>(q, q_ps, kc, vc, kv_ps, rs, out, out_ps, scratch, H, max_seq, len_upper, chunk, st);
  return run_t<HD, HL, 32>(q, q_ps, kc, vc, kv_ps, rs, out, out_ps, scratch, H, max_seq, len_upper, chunk, st);
}

}  // namespace

hydra_status tree_attention_tc(const bf16* q, size_t q_ps, const bf16* kc, const bf16* vc, size_t kv_ps, RowSet rs, bf16* out,
                               size_t out_ps, void* scratch, int H, int hd, int max_seq, int len_upper, cudaStream_t st) {
  if (rs.tc > 64) return HYDRA_ERR_UNSUPPORTED;
  if ((q_ps == 0) != (kv_ps == 0)) return HYDRA_ERR_UNSUPPORTED;           // q and the caches split the same way
  const int chunk = ATT_CHUNK_ROWS;
  const bool hl = q_ps != 0;
  if (hd == 128 && hl) return run<128, true>(q, q_ps, kc, vc, kv_ps, rs, out, out_ps, (float*)scratch, H, max_seq, len_upper, chunk, st);
  if (hd == 128) return run<128, false>(q, q_ps, kc, vc, kv_ps, rs, out, out_ps, (float*)scratch, H, max_seq, len_upper, chunk, st);
  if (hd == 64 && hl) return run<64, true>(q, q_ps, kc, vc, kv_ps, rs, out, out_ps, (float*)scratch, H, max_seq, len_upper, chunk, st);
  if (hd == 64) return run<64, false>(q, q_ps, kc, vc, kv_ps, rs, out, out_ps, (float*)scratch, H, max_seq, len_upper, chunk, st);
  return HYDRA_ERR_UNSUPPORTED;
}

}  // namespace hydra

// Row-wise, element-wise, attention, draft-head and acceptance kernels of libhydra (everything that is
// not the tensor-core GEMM).  float or bfloat16 storage, float arithmetic.
#include "launch.h"
#include <math.h>

namespace hydra {

// ------------------------------------------------------------------------------------------------
// SIMT GEMM: out[m][n] = sum_k x[m][k] w[n][k].  One warp per output feature, MR rows per pass.
// ------------------------------------------------------------------------------------------------
template <typename T> struct Vec4 { };
template <> struct Vec4<float> {
  static __device__ __forceinline__ void load(const float* p, float (&v)[4]) {
    float4 t = *reinterpret_cast<const float4*>(p); v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
};
template <> struct Vec4<bf16> {
  static __device__ __forceinline__ void load(const bf16* p, float (&v)[4]) {
    uint2 t = *reinterpret_cast<const uint2*>(p);
    __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&t.x), b = *reinterpret_cast<__nv_bfloat162*>(&t.y);
    v[0] = __low2float(a); v[1] = __high2float(a); v[2] = __low2float(b); v[3] = __high2float(b); }
};

template <typename T, int MR>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const T* __restrict__ x, const T* __restrict__ w,
                                                        float* __restrict__ out, int m, int n, int k) {
  pdl_trigger();
  pdl_wait();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int col = blockIdx.x * 8 + warp;
  const int m0 = blockIdx.y * MR;
  if (col >= n) return;
  float acc[MR];
#pragma unroll
  for (int r = 0; r < MR; ++r) acc[r] = 0.f;
  const T* wr = w + (size_t)col * k;
  for (int kk = lane * 4; kk < k; kk += 128) {
    float wv[4];
    Vec4<T>::load(wr + kk, wv);
#pragma unroll
    for (int r = 0; r < MR; ++r) {
      int row = m0 + r < m ? m0 + r : m - 1;
      float xv[4];
      Vec4<T>::load(x + (size_t)row * k + kk, xv);
      acc[r] += wv[0] * xv[0] + wv[1] * xv[1] + wv[2] * xv[2] + wv[3] * xv[3];
    }
  }
#pragma unroll
  for (int r = 0; r < MR; ++r) {
    float s = warp_sum(acc[r]);
    if (lane == 0 && m0 + r < m) out[(size_t)(m0 + r) * n + col] = s;
  }
}

hydra_status gemm_simt(const void* x, const void* w, float* out, int m, int n, int k, int dtype, cudaStream_t st) {
  if (m <= 0 || n <= 0 || k <= 0 || (k & 3)) return HYDRA_ERR_UNSUPPORTED;
  constexpr int MR = 16;
  dim3 grid((n + 7) / 8, (m + MR - 1) / MR);
  if (dtype == 0) launch_pdl(gemm_simt_kernel<float, MR>, dim3(grid), dim3(256), 0, st, (const float*)x, (const float*)w, out, m, n, k);
  else launch_pdl(gemm_simt_kernel<bf16, MR>, dim3(grid), dim3(256), 0, st, (const bf16*)x, (const bf16*)w, out, m, n, k);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

__global__ void reduce_splits_kernel(const float* __restrict__ part, SplitDesc sd, float* __restrict__ out, int m, int n) {
  pdl_trigger();
  pdl_wait();
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (size_t)m * n) return;
  const int ns = split_count(sd, (int)(i / n), (int)(i % n));
  float s = 0.f;
  for (int p = 0; p < ns; ++p) s += part[p * sd.stride + i];
  out[i] = s;
}
hydra_status reduce_splits(const float* part, SplitDesc sd, float* out, int m, int n, cudaStream_t st) {
  launch_pdl(reduce_splits_kernel, dim3((unsigned)(((size_t)m * n + 255) / 256)), dim3(256), 0, st, part, sd, out, m, n);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

// ------------------------------------------------------------------------------------------------
// Embedding gather
// ------------------------------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float4 load4(const T* p);
template <> __device__ __forceinline__ float4 load4<float>(const float* p) { return *reinterpret_cast<const float4*>(p); }
template <> __device__ __forceinline__ float4 load4<bf16>(const bf16* p) {
  float v[4]; Vec4<bf16>::load(p, v); return make_float4(v[0], v[1], v[2], v[3]);
}

template <typename T>
__global__ void embed_rows_kernel(const T* __restrict__ embed, const int* __restrict__ tok, float* __restrict__ x, int d,
                                  int vocab, int* status) {
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x;
  int t = tok[r];
  if (t < 0 || t >= vocab) { if (threadIdx.x == 0) atomicOr(status, ST_BOUNDS); t = 0; }
  const T* e = embed + (size_t)t * d;
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) *reinterpret_cast<float4*>(x + (size_t)r * d + i) = load4<T>(e + i);   // d % 4 == 0
}
hydra_status embed_rows(const void* embed, const int* tok, float* x, int rows, int d, int vocab, int dtype, int* status,
                        cudaStream_t st) {
  if (dtype == 0) launch_pdl(embed_rows_kernel<float>, dim3(rows), dim3(256), 0, st, (const float*)embed, tok, x, d, vocab, status);
  else launch_pdl(embed_rows_kernel<bf16>, dim3(rows), dim3(256), 0, st, (const bf16*)embed, tok, x, d, vocab, status);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

// ------------------------------------------------------------------------------------------------
// Residual add of split-K partial sums + RMSNorm (Llama: x * gain / sqrt(mean(x^2) + eps))
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float block_sum(float v, float* sh) {
  v = warp_sum(v);
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) sh[warp] = v;
  __syncthreads();
  float t = (threadIdx.x < (blockDim.x >> 5)) ? sh[threadIdx.x] : 0.f;
  if (warp == 0) { t = warp_sum(t); if (lane == 0) sh[0] = t; }
  __syncthreads();
  t = sh[0];
  __syncthreads();
  return t;
}

template <typename T> __device__ __forceinline__ void store4(T* p, float4 v);
template <> __device__ __forceinline__ void store4<float>(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
template <> __device__ __forceinline__ void store4<bf16>(bf16* p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  uint2 u; u.x = *reinterpret_cast<uint32_t*>(&a); u.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}
template <> __device__ __forceinline__ void store4<__half>(__half* p, float4 v) {
  __half2 a = __floats2half2_rn(v.x, v.y), b = __floats2half2_rn(v.z, v.w);
  uint2 u; u.x = *reinterpret_cast<uint32_t*>(&a); u.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}
// float: one plane.  float16: hi = f16(v) and, ps elements further on, lo = f16(v - hi) (ps = 0: hi only).
template <typename T> __device__ __forceinline__ void put4h(T* p, size_t ps, float4 v);
template <> __device__ __forceinline__ void put4h<float>(float* p, size_t, float4 v) { *reinterpret_cast<float4*>(p) = v; }
template <> __device__ __forceinline__ void put4h<__half>(__half* p, size_t ps, float4 v) {
  const float4 h = make_float4(__half2float(__float2half_rn(v.x)), __half2float(__float2half_rn(v.y)),
                               __half2float(__float2half_rn(v.z)), __half2float(__float2half_rn(v.w)));
  store4<__half>(p, h);
  if (ps) store4<__half>(p + ps, make_float4(v.x - h.x, v.y - h.y, v.z - h.z, v.w - h.w));
}

// Operand storage.  float buffers hold one plane.  bfloat16 operand buffers hold two planes `ps` elements apart:
// hi = bf16(v) and lo = bf16(v - hi), together about 16 mantissa bits (ps = 0 stores hi only).
template <typename T> __device__ __forceinline__ void put(T* p, size_t ps, float v);
template <> __device__ __forceinline__ void put<float>(float* p, size_t, float v) { *p = v; }
template <> __device__ __forceinline__ void put<bf16>(bf16* p, size_t ps, float v) {
  const bf16 h = __float2bfloat16_rn(v);
  *p = h;
  if (ps) p[ps] = __float2bfloat16_rn(v - __bfloat162float(h));
}
template <typename T> __device__ __forceinline__ void put4(T* p, size_t ps, float4 v);
template <> __device__ __forceinline__ void put4<float>(float* p, size_t, float4 v) { *reinterpret_cast<float4*>(p) = v; }
template <> __device__ __forceinline__ void put4<bf16>(bf16* p, size_t ps, float4 v) {
  const float4 h = make_float4(__bfloat162float(__float2bfloat16_rn(v.x)), __bfloat162float(__float2bfloat16_rn(v.y)),
                               __bfloat162float(__float2bfloat16_rn(v.z)), __bfloat162float(__float2bfloat16_rn(v.w)));
  store4<bf16>(p, h);
  if (ps) store4<bf16>(p + ps, make_float4(v.x - h.x, v.y - h.y, v.z - h.z, v.w - h.w));
}

constexpr int NORM_THREADS = 1024;
// x_out = res + sum of the partial-sum slots; with `gain`, also xn = rmsnorm(x_out) * gain (operand planes) and hn (float).
// A row is shared by the CS CTAs of a thread-block cluster (CTA `part` owns d / CS consecutive columns), so that few rows
// still pull their partial sums through many SMs; the CTAs push their sums of squares into each other's shared memory and
// add them in rank order after one cluster barrier.
template <typename T, int CS>
__global__ void __launch_bounds__(NORM_THREADS) residual_rmsnorm_kernel(const float* res, const float* __restrict__ part,
                                                                        SplitDesc sd, float* x_out,
                                                                        const T* __restrict__ gain, T* __restrict__ xn, size_t xn_ps,
                                                                        float* __restrict__ hn, int d, float eps) {
  pdl_trigger();
  pdl_wait();
  __shared__ float sh[32];
  __shared__ float s_ss[CS];
  const int row = blockIdx.x / CS, rank = blockIdx.x % CS;
  const int dc = d / CS, c0 = rank * dc;
  const size_t base = (size_t)row * d;
  float ss = 0.f;
  float4 v0 = make_float4(0.f, 0.f, 0.f, 0.f);                          // this thread's first piece stays in registers
  for (int i = c0 + threadIdx.x * 4, it = 0; i < c0 + dc; i += blockDim.x * 4, ++it) {   // one 16-byte piece per thread and round, all its slot loads in flight together
    size_t off[1] = {base + i};
    int ns[1] = {part ? split_count(sd, row, i) : 0};
    float4 acc[1];
    float4 v = res ? *reinterpret_cast<const float4*>(res + base + i) : make_float4(0.f, 0.f, 0.f, 0.f);
    sum_slots_multi<1, 12>(part, sd.stride, off, ns, acc);             // narrow outputs are cut into up to ~11 slots per tile
    v.x += acc[0].x; v.y += acc[0].y; v.z += acc[0].z; v.w += acc[0].w;
    *reinterpret_cast<float4*>(x_out + base + i) = v;
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    if (it == 0) v0 = v;
  }
  if (!gain) return;
  float tot = block_sum(ss, sh);
  if constexpr (CS > 1) {
    if (threadIdx.x < CS) {                                              // thread r leaves this CTA's sum in CTA r's slot `rank`
      uint32_t local = (uint32_t)__cvta_generic_to_shared(&s_ss[rank]), remote;
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"((uint32_t)threadIdx.x));
      asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(tot) : "memory");
    }
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    tot = 0.f;
#pragma unroll
    for (int r = 0; r < CS; ++r) tot += s_ss[r];
  }
  const float inv = rsqrtf(tot / (float)d + eps);
  for (int i = c0 + threadIdx.x * 4, it = 0; i < c0 + dc; i += blockDim.x * 4, ++it) {
    float4 v = it == 0 ? v0 : *reinterpret_cast<const float4*>(x_out + base + i);
    float4 gn = load4<T>(gain + i);
    v.x *= inv * gn.x; v.y *= inv * gn.y; v.z *= inv * gn.z; v.w *= inv * gn.w;
    if (xn) put4<T>(xn + base + i, xn_ps, v);
    if (hn) *reinterpret_cast<float4*>(hn + base + i) = v;
  }
}
template <typename T, int CS>
static cudaError_t launch_norm(int rows, int d, cudaStream_t st, const float* res, const float* part, SplitDesc sd, float* x_out,
                               const void* gain, void* xn, size_t xn_ps, float* hn, float eps) {
  int threads = (d / CS / 4 + 31) / 32 * 32;
  if (threads > NORM_THREADS) threads = NORM_THREADS;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(rows * CS); cfg.blockDim = dim3(threads); cfg.dynamicSmemBytes = 0; cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = CS; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = CS > 1 ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, residual_rmsnorm_kernel<T, CS>, res, part, sd, x_out, (const T*)gain, (T*)xn, xn_ps, hn, d, eps);
}
hydra_status residual_rmsnorm(const float* res, const float* part, SplitDesc sd, float* x_out,
                              const void* gain, void* xn, size_t xn_ps, float* hn, int rows, int d, float eps, int dtype,
                              cudaStream_t st) {
  if (d & 3) return HYDRA_ERR_UNSUPPORTED;
  // few rows: 4 or 2 CTAs per row (the columns must split into whole 16-byte pieces)
  const int cs = (rows <= 40 && d % 16 == 0) ? 4 : (rows <= 96 && d % 8 == 0) ? 2 : 1;
  if (dtype == 0) {
    if (cs == 4) launch_norm<float, 4>(rows, d, st, res, part, sd, x_out, gain, xn, xn_ps, hn, eps);
    else if (cs == 2) launch_norm<float, 2>(rows, d, st, res, part, sd, x_out, gain, xn, xn_ps, hn, eps);
    else launch_norm<float, 1>(rows, d, st, res, part, sd, x_out, gain, xn, xn_ps, hn, eps);
  } else {
    if (cs == 4) launch_norm<bf16, 4>(rows, d, st, res, part, sd, x_out, gain, xn, xn_ps, hn, eps);
    else if (cs == 2) launch_norm<bf16, 2>(rows, d, st, res, part, sd, x_out, gain, xn, xn_ps, hn, eps);
    else launch_norm<bf16, 1>(rows, d, st, res, part, sd, x_out, gain, xn, xn_ps, hn, eps);
  }
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

// ------------------------------------------------------------------------------------------------
// Rotary table + QKV post-processing (sum partials, rotate q and k, append K,V to the cache)
// ------------------------------------------------------------------------------------------------
// The first kernel of every forward call.  It lets its successors start only AFTER it has waited for everything before
// it (trigger after wait): no kernel of this call can be resident, however early the following launches are, while a
// kernel of an earlier call (the acceptance kernel that wrote the lengths, the kernels that filled the committed cache
// rows) is still running.  The early cache fetches of the attention kernel rely on that.
__global__ void rope_table_kernel(RowSet rs, float2* __restrict__ table, int half, float theta) {
  pdl_wait();
  pdl_trigger();
  int r = blockIdx.x, b = r / rs.tc, i = r % rs.tc;
  int pos = rs.pos0[b] + rs.depth[i];
  for (int j = threadIdx.x; j < half; j += blockDim.x) {
    double inv = exp2(-((double)j / (double)half) * log2((double)theta));
    double s, c;
    sincos((double)pos * inv, &s, &c);
    table[(size_t)r * half + j] = make_float2((float)c, (float)s);
  }
}
hydra_status rope_table(RowSet rs, float2* table, int head_dim, float theta, cudaStream_t st) {
  launch_pdl(rope_table_kernel, dim3(rs.batch * rs.tc), dim3(64), 0, st, rs, table, head_dim / 2, theta);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

// One thread rotates four consecutive pairs (j..j+3, j+half..j+half+3) of one head of q and k and copies the
// matching v elements; all loads and stores are 16 bytes wide.
// T: float (float model path) or float16 (bfloat16 model path: q and the caches are float16 in one or two planes).
template <typename T>
__global__ void __launch_bounds__(256) qkv_rope_store_kernel(const float* __restrict__ part, SplitDesc sd,
                                                             const float2* __restrict__ table, T* __restrict__ q, size_t q_ps,
                                                             T* __restrict__ kc, T* __restrict__ vc, size_t kv_ps,
                                                             RowSet rs, int H, int hd, int max_seq,
                                                             int* status) {
  pdl_trigger();
  pdl_wait();
  const int r = blockIdx.x, b = r / rs.tc, i = r % rs.tc;
  const int nr = rs.n_rows ? rs.n_rows[b] : rs.tc;
  if (i >= nr) return;
  const int d = H * hd, half = hd >> 1;
  const int slot = rs.pos0[b] + i;
  if (slot < 0 || slot >= max_seq) { if (threadIdx.x == 0 && blockIdx.y == 0) atomicOr(status, ST_BOUNDS); return; }
  const int tph = half >> 2;                                       // threads per head
  const int h = blockIdx.y * (blockDim.x / tph) + threadIdx.x / tph;
  if (h >= H) return;
  const int j = (threadIdx.x % tph) * 4;
  const int c0 = h * hd + j, c1 = c0 + half;
  const int cols[6] = {c0, c1, d + c0, d + c1, 2 * d + c0, 2 * d + c1};
  float4 v6[6];
  {
    size_t off[6]; int ns[6];
#pragma unroll
    for (int e = 0; e < 6; ++e) { off[e] = (size_t)r * 3 * d + cols[e]; ns[e] = split_count(sd, r, cols[e]); }
    sum_slots_multi<6>(part, sd.stride, off, ns, v6);
  }
  const float4 t01 = *reinterpret_cast<const float4*>(table + (size_t)r * half + j);        // (cos, sin) of j, j+1
  const float4 t23 = *reinterpret_cast<const float4*>(table + (size_t)r * half + j + 2);    // (cos, sin) of j+2, j+3
  const float cs[4] = {t01.x, t01.z, t23.x, t23.z}, sn[4] = {t01.y, t01.w, t23.y, t23.w};
  auto rot = [&](const float4& a, const float4& bq, float4& lo, float4& hi) {
    const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {bq.x, bq.y, bq.z, bq.w};
    float l[4], hh[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) { l[e] = av[e] * cs[e] - bv[e] * sn[e]; hh[e] = bv[e] * cs[e] + av[e] * sn[e]; }
    lo = make_float4(l[0], l[1], l[2], l[3]); hi = make_float4(hh[0], hh[1], hh[2], hh[3]);
  };
  float4 qlo, qhi, klo, khi;
  rot(v6[0], v6[1], qlo, qhi);
  rot(v6[2], v6[3], klo, khi);
  put4h<T>(q + (size_t)r * d + c0, q_ps, qlo);
  put4h<T>(q + (size_t)r * d + c1, q_ps, qhi);
  const size_t o = (((size_t)b * H + h) * max_seq + slot) * hd;
  put4h<T>(kc + o + j, kv_ps, klo);
  put4h<T>(kc + o + j + half, kv_ps, khi);
  put4h<T>(vc + o + j, kv_ps, v6[4]);
  put4h<T>(vc + o + j + half, kv_ps, v6[5]);
}
hydra_status qkv_rope_store(const float* part, SplitDesc sd, const float2* table, void* q, size_t q_ps, void* kcache, void* vcache,
                            size_t kv_ps, RowSet rs, int H, int hd, int max_seq, int dtype, int* status, cudaStream_t st) {
  if (hd % 8) return HYDRA_ERR_UNSUPPORTED;
  // 128 threads per CTA: with 64 rows twice as many SMs pull the partial sums as with 256
  const int threads = 128 % (hd / 8) == 0 ? 128 : 256;
  const int heads_per_block = threads / (hd / 8);
  dim3 grid(rs.batch * rs.tc, (H + heads_per_block - 1) / heads_per_block);
  if (dtype == 0)
    launch_pdl(qkv_rope_store_kernel<float>, grid, dim3(threads), 0, st, part, sd, table, (float*)q, q_ps, (float*)kcache, (float*)vcache,
               kv_ps, rs, H, hd, max_seq, status);
  else
    launch_pdl(qkv_rope_store_kernel<__half>, grid, dim3(threads), 0, st, part, sd, table, (__half*)q, q_ps, (__half*)kcache, (__half*)vcache,
               kv_ps, rs, H, hd, max_seq, status);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

// ------------------------------------------------------------------------------------------------
// Tree attention, split over the KV length.  One CTA per (head, sequence, KV chunk); the chunk's K,V
// rows are read once; every query row keeps an online softmax (running max, sum, weighted V) per warp.
// ------------------------------------------------------------------------------------------------
constexpr int ATT_CHUNK = ATT_CHUNK_ROWS;
constexpr int ATT_TILE = 32;      // KV rows staged per iteration
constexpr int ATT_WARPS = 8;

template <typename T, int HD>
__global__ void __launch_bounds__(ATT_WARPS * 32) tree_attn_kernel(const T* __restrict__ q, const T* __restrict__ kc,
                                                                   const T* __restrict__ vc, RowSet rs,
                                                                   float* __restrict__ part_o, float* __restrict__ part_ml,
                                                                   int H, int max_seq, int nchunks) {
  pdl_trigger();
  pdl_wait();
  extern __shared__ float smem[];
  constexpr int RPW = 8;                                  // query rows per warp (tc <= 64)
  constexpr int KPL = HD / 32;                            // output dims per lane
  float* qs = smem;                                       // [64][HD]
  float* ks = qs + 64 * HD;                               // [ATT_TILE][HD+1]
  float* vs = ks + ATT_TILE * (HD + 1);                   // [ATT_TILE][HD]
  const int h = blockIdx.x, b = blockIdx.y, c = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nr = rs.n_rows ? rs.n_rows[b] : rs.tc;
  const int p0 = rs.pos0[b];
  const int total = p0 + nr;
  const int s0 = c * ATT_CHUNK;
  const int s1 = min(s0 + ATT_CHUNK, total);
  const int d = H * HD;
  const float scale = rsqrtf((float)HD);

  for (int e = threadIdx.x; e < nr * HD; e += blockDim.x) {
    int i = e / HD, k = e % HD;
    qs[i * HD + k] = to_f<T>(q[((size_t)(b * rs.tc + i)) * d + h * HD + k]) * scale;
  }
  float m[RPW], l[RPW], o[RPW][KPL];
  uint64_t msk[RPW];
#pragma unroll
  for (int j = 0; j < RPW; ++j) {
    m[j] = -INFINITY; l[j] = 0.f;
    int r = warp * RPW + j;
    msk[j] = r < nr ? rs.mask[r] : 0ull;
#pragma unroll
    for (int kk = 0; kk < KPL; ++kk) o[j][kk] = 0.f;
  }
  const T* kbase = kc + ((size_t)b * H + h) * max_seq * HD;
  const T* vbase = vc + ((size_t)b * H + h) * max_seq * HD;

  for (int t0 = s0; t0 < s1; t0 += ATT_TILE) {
    __syncthreads();
    for (int e = threadIdx.x; e < ATT_TILE * HD; e += blockDim.x) {
      int j = e / HD, k = e % HD;
      int slot = t0 + j;
      float kv = 0.f, vv = 0.f;
      if (slot < s1) { kv = to_f<T>(kbase[(size_t)slot * HD + k]); vv = to_f<T>(vbase[(size_t)slot * HD + k]); }
      ks[j * (HD + 1) + k] = kv;
      vs[j * HD + k] = vv;
    }
    __syncthreads();
    const int slot = t0 + lane;
#pragma unroll
    for (int j = 0; j < RPW; ++j) {
      const int r = warp * RPW + j;
      if (r >= nr) continue;
      bool valid = slot < s1 && (slot < p0 || ((msk[j] >> (slot - p0)) & 1ull));
      float sc = 0.f;
      const float* qr = qs + r * HD;
      const float* kr = ks + lane * (HD + 1);
#pragma unroll 8
      for (int k = 0; k < HD; ++k) sc += qr[k] * kr[k];
      sc = valid ? sc : -INFINITY;
      float mn = fmaxf(m[j], warp_max(sc));
      if (mn == -INFINITY) continue;
      float alpha = expf(m[j] - mn);
      float p = valid ? expf(sc - mn) : 0.f;
      l[j] = l[j] * alpha + warp_sum(p);
      float acc[KPL];
#pragma unroll
      for (int kk = 0; kk < KPL; ++kk) acc[kk] = o[j][kk] * alpha;
      for (int jj = 0; jj < ATT_TILE; ++jj) {
        float pj = __shfl_sync(0xffffffffu, p, jj);
#pragma unroll
        for (int kk = 0; kk < KPL; ++kk) acc[kk] += pj * vs[jj * HD + lane + 32 * kk];
      }
#pragma unroll
      for (int kk = 0; kk < KPL; ++kk) o[j][kk] = acc[kk];
      m[j] = mn;
    }
  }
#pragma unroll
  for (int j = 0; j < RPW; ++j) {
    const int r = warp * RPW + j;
    if (r >= nr) continue;
    size_t idx = ((size_t)(b * rs.tc + r) * H + h) * nchunks + c;
#pragma unroll
    for (int kk = 0; kk < KPL; ++kk) part_o[idx * HD + lane + 32 * kk] = o[j][kk];
    if (lane == 0) { part_ml[idx * 2] = m[j]; part_ml[idx * 2 + 1] = l[j]; }
  }
}

template <typename T, int HD>
__global__ void tree_attn_combine_kernel(const float* __restrict__ part_o, const float* __restrict__ part_ml, RowSet rs,
                                         T* __restrict__ out, int H, int nchunks) {
  pdl_trigger();
  pdl_wait();
  const int r = blockIdx.x, h = blockIdx.y, b = r / rs.tc, i = r % rs.tc;
  const int nr = rs.n_rows ? rs.n_rows[b] : rs.tc;
  const int k = threadIdx.x;
  T* dst = out + (size_t)r * H * HD + h * HD;
  if (i >= nr) { dst[k] = from_f<T>(0.f); return; }
  const int used = min(nchunks, (rs.pos0[b] + nr + ATT_CHUNK - 1) / ATT_CHUNK);
  size_t idx = ((size_t)r * H + h) * nchunks;
  float M = -INFINITY;
  for (int c = 0; c < used; ++c) M = fmaxf(M, part_ml[(idx + c) * 2]);
  float L = 0.f, acc = 0.f;
  for (int c = 0; c < used; ++c) {
    float mc = part_ml[(idx + c) * 2];
    if (mc == -INFINITY) continue;
    float w = expf(mc - M);
    L += part_ml[(idx + c) * 2 + 1] * w;
    acc += part_o[(idx + c) * HD + k] * w;
  }
  dst[k] = from_f<T>(acc / L);
}

size_t attention_scratch_bytes(int batch, int tc, int n_heads, int head_dim, int max_seq) {
  size_t nchunks = (size_t)(max_seq + ATT_CHUNK - 1) / ATT_CHUNK;
  return (size_t)batch * tc * n_heads * nchunks * (head_dim + 2) * sizeof(float);
}

template <typename T, int HD>
static hydra_status tree_attention_t(const T* q, const T* kc, const T* vc, RowSet rs, T* out, float* scratch, int H,
                                     int max_seq, int len_upper, cudaStream_t st) {
  int nchunks_max = (max_seq + ATT_CHUNK - 1) / ATT_CHUNK;
  int nchunks = (len_upper + ATT_CHUNK - 1) / ATT_CHUNK;
  if (nchunks < 1) nchunks = 1;
  if (nchunks > nchunks_max) nchunks = nchunks_max;
  size_t rows = (size_t)rs.batch * rs.tc;
  float* part_o = scratch;
  float* part_ml = scratch + rows * H * nchunks_max * HD;
  size_t smem = (size_t)(64 * HD + ATT_TILE * (HD + 1) + ATT_TILE * HD) * sizeof(float);
  static PerDeviceFlag attr_done;
  if (!attr_done.get()) {
    HYDRA_CUDA(cudaFuncSetAttribute(tree_attn_kernel<T, HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    attr_done.set();
  }
  launch_pdl(tree_attn_kernel<T, HD>, dim3(dim3(H, rs.batch, nchunks)), dim3(ATT_WARPS * 32), smem, st, q, kc, vc, rs, part_o, part_ml, H,
                                                                                   max_seq, nchunks);
  HYDRA_LAUNCH_CHECK();
  launch_pdl(tree_attn_combine_kernel<T, HD>, dim3(dim3((unsigned)rows, H)), dim3(HD), 0, st, part_o, part_ml, rs, out, H, nchunks);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

hydra_status tree_attention_f32(const float* q, const float* kc, const float* vc, RowSet rs, float* out, void* scratch, int H, int hd,
                                int max_seq, int len_upper, cudaStream_t st) {
  if (rs.tc > 64 || !rs.mask) return HYDRA_ERR_UNSUPPORTED;
  if (hd == 64) return tree_attention_t<float, 64>(q, kc, vc, rs, out, (float*)scratch, H, max_seq, len_upper, st);
  if (hd == 128) return tree_attention_t<float, 128>(q, kc, vc, rs, out, (float*)scratch, H, max_seq, len_upper, st);
  return HYDRA_ERR_UNSUPPORTED;
}

// ------------------------------------------------------------------------------------------------
// SiLU(gate) * up from the gate/up partial sums
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void silu_mul_kernel(const float* __restrict__ part, SplitDesc sd, T* __restrict__ act, size_t act_ps, int rows, int f) {
  pdl_trigger();
  pdl_wait();
  size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i >= (size_t)rows * f) return;
  const int r = (int)(i / f), c = (int)(i % f);
  size_t off[2] = {(size_t)r * 2 * f + c, (size_t)r * 2 * f + f + c};
  int ns[2] = {split_count(sd, r, c), split_count(sd, r, f + c)};
  float4 gu[2];
  sum_slots_multi<2>(part, sd.stride, off, ns, gu);
  const float4 g = gu[0], u = gu[1];
  put4<T>(act + i, act_ps, make_float4(silu_f(g.x) * u.x, silu_f(g.y) * u.y, silu_f(g.z) * u.z, silu_f(g.w) * u.w));
}
hydra_status silu_mul(const float* part, SplitDesc sd, void* act, size_t act_ps, int rows, int f, int dtype, cudaStream_t st) {
  if (f & 3) return HYDRA_ERR_UNSUPPORTED;
  size_t n = (size_t)rows * f / 4;
  unsigned grid = (unsigned)((n + 255) / 256);
  if (dtype == 0) launch_pdl(silu_mul_kernel<float>, dim3(grid), dim3(256), 0, st, part, sd, (float*)act, act_ps, rows, f);
  else launch_pdl(silu_mul_kernel<bf16>, dim3(grid), dim3(256), 0, st, part, sd, (bf16*)act, act_ps, rows, f);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

// ------------------------------------------------------------------------------------------------
// argmax / top-k with total order (value descending, token id ascending)
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ bool better(float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); }

// The best (value, index) of a warp, in every lane.
__device__ __forceinline__ void warp_best(float& v, int& i) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    float ov = __shfl_xor_sync(0xffffffffu, v, o);
    int oi = __shfl_xor_sync(0xffffffffu, i, o);
    if (better(ov, oi, v, i)) { v = ov; i = oi; }
  }
}

__device__ __forceinline__ float summed(const float* part, const SplitDesc& sd, int row, int col, int n) {
  return sum_slots_scalar<4>(part, sd.stride, (size_t)row * n + col, split_count(sd, row, col));
}

// Top-c of every logits row in two stages.  Stage 1: grid (rows, blocks of TOPK_SPAN columns); each block sums the
// partial slots of its columns (optionally storing the sums as the row's logits); every warp then picks the c best of
// its register-resident values in c rounds of a warp-wide reduction (no block barrier inside the rounds), and one warp
// merges the eight sorted lists.  Stage 2: one warp per winner list merges the sorted candidate lists of all column
// blocks out of shared memory and writes the winners (children of a tree node, or the argmax).
constexpr int TOPK_SPAN = 2048;           // columns per stage-1 block (8 per thread)
constexpr int TOPK_MAX = 64;              // a tree node has at most 63 children
constexpr int TOPK_LISTS_PER_LANE = 4;    // stage 2: at most 128 column blocks (262144 tokens)

__global__ void __launch_bounds__(256) topk_stage1_kernel(const float* __restrict__ part, SplitDesc sd,
                                                          float* __restrict__ logits_out, float* __restrict__ cand_v,
                                                          int* __restrict__ cand_i, int vocab, int c) {
  pdl_trigger();
  pdl_wait();
  __shared__ float wv[8][TOPK_MAX];
  __shared__ int wi[8][TOPK_MAX];
  const int row = blockIdx.x, blk = blockIdx.y, nblk = gridDim.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float v[8]; int idx[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int col = blk * TOPK_SPAN + j * 256 + threadIdx.x;
    idx[j] = col;
    v[j] = -INFINITY;
    if (col < vocab) {
      v[j] = summed(part, sd, row, col, vocab);
      if (logits_out) logits_out[(size_t)row * vocab + col] = v[j];
    } else {
      idx[j] = 0x7fffffff;
    }
  }
  for (int t = 0; t < c; ++t) {                            // this warp's c best, in order
    float bv = -INFINITY; int bi = 0x7fffffff;
#pragma unroll
    for (int j = 0; j < 8; ++j) if (better(v[j], idx[j], bv, bi)) { bv = v[j]; bi = idx[j]; }
    warp_best(bv, bi);
    if (lane == 0) { wv[warp][t] = bv; wi[warp][t] = bi; }
#pragma unroll
    for (int j = 0; j < 8; ++j) if (idx[j] == bi) { v[j] = -INFINITY; idx[j] = 0x7fffffff; }    // taken
  }
  __syncthreads();
  if (warp == 0) {                                         // merge: lane w < 8 walks warp w's list
    int ptr = 0;
    for (int t = 0; t < c; ++t) {
      float hv = -INFINITY; int hi = 0x7fffffff;
      if (lane < 8 && ptr < c) { hv = wv[lane][ptr]; hi = wi[lane][ptr]; }
      float bv = hv; int bi = hi;
      warp_best(bv, bi);
      if (lane == 0) {
        cand_v[((size_t)row * nblk + blk) * TOPK_MAX + t] = bv;
        cand_i[((size_t)row * nblk + blk) * TOPK_MAX + t] = bi;
      }
      if (hi == bi && bi != 0x7fffffff) ++ptr;
    }
  }
}

// out_of(row) and count_of(row): where the winners go.  lv.parents == null: argmax (one winner per row to amax[row]).
// One warp per winner list; dynamic shared memory: nblk * c (value, index) pairs.
__global__ void __launch_bounds__(32) topk_stage2_kernel(const float* __restrict__ cand_v, const int* __restrict__ cand_i,
                                                         int nblk, int c, LevelDesc lv, const int* __restrict__ first_child,
                                                         const int* __restrict__ n_child, int* __restrict__ out, int T, int cand_div) {
  pdl_trigger();
  pdl_wait();
  extern __shared__ float s_cand[];
  float* sv = s_cand;
  int* si = reinterpret_cast<int*>(s_cand + nblk * c);
  const int row = blockIdx.x, lane = threadIdx.x;
  const int crow = row / cand_div;                         // row of the candidate lists (one per sequence when the parents share them)
  int* dst = out + row;
  int count = 1;
  if (lv.parents) {
    const int b = row / lv.n_parents, p = lv.parents[row % lv.n_parents];
    dst = out + b * T + first_child[p];
    count = n_child[p];
  }
  for (int e = lane; e < nblk * c; e += 32) {
    const size_t at = ((size_t)crow * nblk + e / c) * TOPK_MAX + e % c;
    sv[e] = cand_v[at]; si[e] = cand_i[at];
  }
  __syncwarp();
  int ptr[TOPK_LISTS_PER_LANE];                            // lane l walks the sorted lists l, l + 32, ...
#pragma unroll
  for (int q = 0; q < TOPK_LISTS_PER_LANE; ++q) ptr[q] = 0;
  for (int t = 0; t < count; ++t) {
    float bv = -INFINITY; int bi = 0x7fffffff;
#pragma unroll
    for (int q = 0; q < TOPK_LISTS_PER_LANE; ++q) {
      const int l = lane + 32 * q;
      if (l < nblk && ptr[q] < c && better(sv[l * c + ptr[q]], si[l * c + ptr[q]], bv, bi)) { bv = sv[l * c + ptr[q]]; bi = si[l * c + ptr[q]]; }
    }
    warp_best(bv, bi);
    if (lane == 0) dst[t] = bi;
#pragma unroll
    for (int q = 0; q < TOPK_LISTS_PER_LANE; ++q) {
      const int l = lane + 32 * q;
      if (l < nblk && ptr[q] < c && si[l * c + ptr[q]] == bi && bi != 0x7fffffff) ++ptr[q];
    }
  }
}

size_t topk_scratch_bytes(int rows, int vocab) {
  const size_t nblk = (size_t)(vocab + TOPK_SPAN - 1) / TOPK_SPAN;
  return (size_t)rows * nblk * TOPK_MAX * (sizeof(float) + sizeof(int));
}

// rows: logits rows (stage 1); out_rows: winner lists (stage 2), out_rows / rows of them per logits row
static hydra_status topk_rows(const float* part, SplitDesc sd, float* logits_out, void* scratch, int rows_cap, int rows, int out_rows, int vocab,
                              int c, LevelDesc lv, const int* first_child, const int* n_child, int* out, int T, cudaStream_t st) {
  if (c < 1 || c > TOPK_MAX || rows > rows_cap || rows < 1 || out_rows % rows) return HYDRA_ERR_UNSUPPORTED;
  const int nblk = (vocab + TOPK_SPAN - 1) / TOPK_SPAN;
  const size_t merge_bytes = (size_t)nblk * c * 8;         // stage 2 keeps every candidate of a row in shared memory
  if (nblk > 32 * TOPK_LISTS_PER_LANE || merge_bytes > 48 * 1024) return HYDRA_ERR_UNSUPPORTED;
  float* cand_v = (float*)scratch;
  int* cand_i = (int*)(cand_v + (size_t)rows_cap * nblk * TOPK_MAX);
  launch_pdl(topk_stage1_kernel, dim3(rows, nblk), dim3(256), 0, st, part, sd, logits_out, cand_v, cand_i, vocab, c);
  HYDRA_LAUNCH_CHECK();
  launch_pdl(topk_stage2_kernel, dim3(out_rows), dim3(32), merge_bytes, st, (const float*)cand_v, (const int*)cand_i, nblk, c, lv, first_child, n_child, out, T,
             out_rows / rows);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

hydra_status argmax_rows(const float* part, SplitDesc sd, float* logits_out, int* amax, void* scratch, int rows_cap, int rows,
                         int vocab, cudaStream_t st) {
  return topk_rows(part, sd, logits_out, scratch, rows_cap, rows, rows, vocab, 1, LevelDesc{0, 0, nullptr}, nullptr, nullptr, amax, 0, st);
}

hydra_status topk_children(const float* part, SplitDesc sd, float* logits, LevelDesc lv, int max_children, const int* first_child,
                           const int* n_child, int* tree_tok, void* scratch, int rows_cap, int batch, int T, int vocab, int shared_rows,
                           cudaStream_t st) {
  return topk_rows(part, sd, logits, scratch, rows_cap, shared_rows ? batch : batch * lv.n_parents, batch * lv.n_parents, vocab, max_children, lv,
                   first_child, n_child, tree_tok, T, st);
}

// ------------------------------------------------------------------------------------------------
// Hydra heads: input gather and the residual SiLU layer epilogue
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) head_gather_kernel(const float* __restrict__ hprime, const T* __restrict__ embed,
                                                          const int* __restrict__ root_tok, int* tree_tok,
                                                          const int* __restrict__ path_tab, LevelDesc lv, int write_root, T* __restrict__ z,
                                                          size_t z_ps, int T_rows, int kp1, int d_model, int vocab, int* status) {
  pdl_trigger();
  pdl_wait();
  const int row = blockIdx.x, b = row / lv.n_parents, j = row % lv.n_parents;
  const int blk = blockIdx.y;                               // 0: hidden, 1..d: path tokens root..parent
  const int p = lv.parents[j];
  T* dst = z + ((size_t)row * (lv.d + 1) + blk) * d_model;
  if (blk == 0) {                                          // 16-byte pieces (d_model is a multiple of 4)
    for (int i = threadIdx.x * 4; i < d_model; i += blockDim.x * 4)
      put4<T>(dst + i, z_ps, *reinterpret_cast<const float4*>(hprime + (size_t)b * d_model + i));
    if (write_root && j == 0 && threadIdx.x == 0) tree_tok[b * T_rows] = root_tok[b];
    return;
  }
  int node = path_tab[p * kp1 + (blk - 1)];
  int t = node == 0 ? root_tok[b] : tree_tok[b * T_rows + node];
  if (t < 0 || t >= vocab) { if (threadIdx.x == 0) atomicOr(status, ST_BOUNDS); t = 0; }
  const T* e = embed + (size_t)t * d_model;
  for (int i = threadIdx.x * 4; i < d_model; i += blockDim.x * 4) put4<T>(dst + i, z_ps, load4<T>(e + i));      // embeddings are exact: lo = 0
}
hydra_status head_gather(const float* hprime, const void* embed, const int* root_tok, int* tree_tok, const int* path_tab,
                         LevelDesc lv, int write_root, void* z, size_t z_ps, int batch, int T, int kp1, int d_model, int vocab, int dtype,
                         int* status, cudaStream_t st) {
  dim3 grid(batch * lv.n_parents, lv.d + 1);
  if (dtype == 0)
    launch_pdl(head_gather_kernel<float>, dim3(grid), dim3(256), 0, st, hprime, (const float*)embed, root_tok, tree_tok, path_tab, lv, write_root,
               (float*)z, z_ps, T, kp1, d_model, vocab, status);
  else
    launch_pdl(head_gather_kernel<bf16>, dim3(grid), dim3(256), 0, st, hprime, (const bf16*)embed, root_tok, tree_tok, path_tab, lv, write_root,
               (bf16*)z, z_ps, T, kp1, d_model, vocab, status);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

template <typename T>
__global__ void head_act_kernel(const float* res, int res_is_hprime, int rows_per_b, const float* __restrict__ part,
                                SplitDesc sd, const T* __restrict__ bias, float* y_out, T* __restrict__ yb, size_t yb_ps,
                                int rows, int d) {
  pdl_trigger();
  pdl_wait();
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (size_t)rows * d) return;
  int r = (int)(i / d), c = (int)(i % d);
  float v = bias ? to_f<T>(bias[c]) : 0.f;
  v += sum_slots_scalar<12>(part, sd.stride, i, split_count(sd, r, c));
  float base = res_is_hprime ? res[(size_t)(r / rows_per_b) * d + c] : res[i];
  float y = base + silu_f(v);
  y_out[i] = y;
  put<T>(yb + i, yb_ps, y);
}
hydra_status head_act(const float* res, int res_is_hprime, int rows_per_b, const float* part, SplitDesc sd,
                      const void* bias, float* y_out, void* yb, size_t yb_ps, int rows, int d, int dtype, cudaStream_t st) {
  size_t n = (size_t)rows * d;
  unsigned grid = (unsigned)((n + 255) / 256);
  if (dtype == 0)
    launch_pdl(head_act_kernel<float>, dim3(grid), dim3(256), 0, st, res, res_is_hprime, rows_per_b, part, sd, (const float*)bias,
                                                 y_out, (float*)yb, yb_ps, rows, d);
  else
    launch_pdl(head_act_kernel<bf16>, dim3(grid), dim3(256), 0, st, res, res_is_hprime, rows_per_b, part, sd, (const bf16*)bias,
                                                y_out, (bf16*)yb, yb_ps, rows, d);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

// ------------------------------------------------------------------------------------------------
// Greedy acceptance + in-place KV compaction + state update, one kernel.
// grid (G, batch).  Every CTA recomputes the accepted path of its sequence (cheap), then moves its
// share of 16-byte KV pieces.  A thread moves its piece for k = 1..n in batches of 8 positions, reading a
// batch before writing it: the destination slot k can only be the source of a path position j <= k (a row
// at depth j has index >= j), which the same thread reads in the same or an earlier batch, before the
// write, so the in-place move is hazard-free.  The last CTA of a sequence to
// finish publishes the new length / root token; all CTAs read the old length before they signal.
// ------------------------------------------------------------------------------------------------
// Typical criterion for candidate row i of sequence b (Section "Typical acceptance sampling"): with p = softmax(l / tau) at
// the parent row and H its entropy, accept when p[token] > min(eps, alpha exp(-H)).  From the row statistics (max m,
// Z = sum exp((l - m)/tau), S = sum exp((l - m)/tau) (l - m)/tau): p[x] = exp((l_x - m)/tau) / Z, H = log Z - S / Z.
__device__ __forceinline__ bool typical_pass(const AcceptArgs& a, int b, int i) {
  const int prow = b * a.T + a.parent[i];
  const int tok = a.tree_tok[b * a.T + i];
  if (tok < 0 || tok >= a.vocab) return false;
  const float4 st = a.row_stats[prow];
  const float z = (a.logits[(size_t)prow * a.vocab + tok] - st.x) / a.tau;
  const float p = __expf(z) / st.y;
  const float H = __logf(st.y) - st.z / st.y;
  return p > fminf(a.eps, a.alpha * __expf(-H));
}

__global__ void __launch_bounds__(256) accept_compact_kernel(AcceptArgs a) {
  pdl_trigger();
  pdl_wait();
  __shared__ int s_path[72];
  __shared__ int s_n, s_best, s_bonus;
  __shared__ float s_scan[256];
  const int b = blockIdx.y;
  const int T = a.T;
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    uint64_t bits = 0;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      int i = lane + 32 * half;
      bool mt = false;
      if (i >= 1 && i < T) mt = a.mode == 1 ? typical_pass(a, b, i) : a.tree_tok[b * T + i] == a.amax[b * T + a.parent[i]];
      bits |= (uint64_t)__ballot_sync(0xffffffffu, mt) << (32 * half);
    }
    if (lane == 0 && blockIdx.x == 0 && a.pass_bits) a.pass_bits[b] = bits;
    int key = -1;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      int i = lane + 32 * half;
      if (i < T) {
        bool acc = ((a.anc[i] & ~1ull) & ~bits) == 0ull;
        if (acc) key = max(key, a.depth[i] * 64 + (63 - i));
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) key = max(key, __shfl_xor_sync(0xffffffffu, key, o));
    // walk from the best row to the root through the parents held in registers (lane i: rows i and i + 32)
    const int p_lo = lane < T ? a.parent[lane] : 0, p_hi = lane + 32 < T ? a.parent[lane + 32] : 0;
    const int best = 63 - (key & 63), n = key >> 6;
    int node = best;
    for (int k = n; k >= 0; --k) {
      if (lane == 0) s_path[k] = node;
      const int up_lo = __shfl_sync(0xffffffffu, p_lo, node & 31), up_hi = __shfl_sync(0xffffffffu, p_hi, node & 31);
      node = node < 32 ? up_lo : up_hi;
    }
    if (lane == 0) { s_n = n; s_best = best; }
  }
  __syncthreads();
  const int n = s_n, best = s_best;
  // the token after the accepted path: the best row's argmax, or (typical mode with uniform numbers) a draw from its
  // temperature distribution by inverse CDF in token-id order; only CTA 0 of the sequence works it out
  const bool sampled = a.mode == 1 && a.u != nullptr;
  if (blockIdx.x == 0) {
    if (!sampled) {
      if (threadIdx.x == 0) s_bonus = a.amax[b * T + best];
    } else {
      const float* lg = a.logits + (size_t)(b * T + best) * a.vocab;
      const float mx = a.row_stats[b * T + best].x, inv_tau = 1.f / a.tau;
      const int per = (a.vocab + 255) / 256, v0 = threadIdx.x * per, v1 = min(v0 + per, a.vocab);
      float part = 0.f;
      for (int v = v0; v < v1; ++v) part += __expf((lg[v] - mx) * inv_tau);
      s_scan[threadIdx.x] = part;
      __syncthreads();
      if (threadIdx.x == 0) {                                          // sequential scan of 256 partial sums: fixed order
        float run = 0.f;
        for (int t = 0; t < 256; ++t) { const float p = s_scan[t]; s_scan[t] = run; run += p; }
        const float target = a.u[b] * run;
        int owner = 255;
        for (int t = 0; t < 256; ++t) if (s_scan[t] <= target) owner = t;      // last thread whose range starts at or below the target
        float acc = s_scan[owner];
        int pick = -1;
        const int w0 = owner * per, w1 = min(w0 + per, a.vocab);
        for (int v = w0; v < w1 && pick < 0; ++v) { acc += __expf((lg[v] - mx) * inv_tau); if (acc > target) pick = v; }
        if (pick < 0) {                                                   // rounding at a range boundary: the next token of non-zero weight
          for (int v = w1; v < a.vocab && pick < 0; ++v) if (__expf((lg[v] - mx) * inv_tau) > 0.f) pick = v;
          if (pick < 0) pick = a.vocab - 1;
        }
        s_bonus = pick;
      }
    }
    __syncthreads();
    if (threadIdx.x == 0 && a.bonus_tmp) a.bonus_tmp[b] = s_bonus;       // published with the fence before this CTA signs off below
  }
  const int L = a.len[b];
  const bool in_range = L >= 0 && L + T <= a.max_seq;
  if (!in_range) {
    if (threadIdx.x == 0) atomicOr(a.status, ST_BOUNDS);
  } else {
    const int row_bytes = a.head_dim * a.esize;
    const int ppr = row_bytes / 16;                                    // 16-byte pieces per row
    const long long units = (long long)a.n_layers * 2 * a.kv_planes * a.n_heads * ppr;
    for (long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x; u < units; u += (long long)gridDim.x * blockDim.x) {
      int piece = (int)(u % ppr);
      long long t = u / ppr;
      int head = (int)(t % a.n_heads);
      long long lk = t / a.n_heads;                                    // (layer*2 + kv)*planes + plane
      char* base = (char*)a.kv_base + ((((size_t)lk * a.max_batch + b) * a.n_heads + head) * a.max_seq) * row_bytes;
      for (int k0 = 1; k0 <= n; k0 += 8) {                             // all reads of a batch in flight before its writes
        uint4 v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (k0 + j <= n) v[j] = *reinterpret_cast<const uint4*>(base + (size_t)(L + s_path[k0 + j]) * row_bytes + piece * 16);
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (k0 + j <= n && s_path[k0 + j] != k0 + j) *reinterpret_cast<uint4*>(base + (size_t)(L + k0 + j) * row_bytes + piece * 16) = v[j];
      }
    }
    // hidden rows of the accepted path feed the next draft
    const int d4 = a.d_model / 4;
    for (int u = blockIdx.x * blockDim.x + threadIdx.x; u < (n + 1) * d4; u += gridDim.x * blockDim.x) {
      int k = u / d4, c = u % d4;
      reinterpret_cast<float4*>(a.h_new + ((size_t)b * (a.K + 1) + k) * a.d_model)[c] =
          reinterpret_cast<const float4*>(a.h_tree + ((size_t)b * a.h_tree_stride + s_path[k]) * a.d_model)[c];
    }
  }
  if (blockIdx.x == 0 && threadIdx.x <= a.K) {
    int k = threadIdx.x;
    if (a.path) a.path[b * (a.K + 1) + k] = k <= n ? s_path[k] : -1;
    if (a.out_tok) {
      int v = -1;
      if (k < n) v = a.tree_tok[b * T + s_path[k + 1]];
      else if (k == n) v = s_bonus;
      a.out_tok[b * (a.K + 1) + k] = v;
    }
    if (k == 0 && a.n_acc) a.n_acc[b] = n;
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned prev = atomicAdd(&a.done_counter[b], 1u);
    if (prev == gridDim.x - 1) {
      a.done_counter[b] = 0;
      if (in_range) {
        a.len[b] = L + n + 1;
        __threadfence();
        a.root_tok[b] = a.bonus_tmp ? *((volatile int*)a.bonus_tmp + b) : a.amax[b * T + best];
        a.n_new[b] = n + 1;
      }
    }
  }
}
// (max, sum exp((l - max)/tau), sum exp((l - max)/tau) (l - max)/tau) of every logits row; one CTA per row, fixed reduction order
__global__ void __launch_bounds__(1024) softmax_row_stats_kernel(const float* __restrict__ logits, float4* __restrict__ stats, int vocab, float tau) {
  pdl_trigger();
  pdl_wait();
  __shared__ float sh[32];
  const float* lg = logits + (size_t)blockIdx.x * vocab;
  float mx = -INFINITY;
  for (int v = threadIdx.x; v < vocab; v += 1024) mx = fmaxf(mx, lg[v]);
  mx = warp_max(mx);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = mx;
  __syncthreads();
  mx = sh[0];
  for (int w = 1; w < 32; ++w) mx = fmaxf(mx, sh[w]);
  __syncthreads();
  float z_sum = 0.f, s_sum = 0.f;
  const float inv_tau = 1.f / tau;
  for (int v = threadIdx.x; v < vocab; v += 1024) {
    const float z = (lg[v] - mx) * inv_tau, e = __expf(z);
    z_sum += e; s_sum += e * z;
  }
  const float Z = block_sum(z_sum, sh), S = block_sum(s_sum, sh);
  if (threadIdx.x == 0) stats[blockIdx.x] = make_float4(mx, Z, S, 0.f);
}
hydra_status softmax_row_stats(const float* logits, float4* row_stats, int rows, int vocab, float tau, cudaStream_t st) {
  launch_pdl(softmax_row_stats_kernel, dim3(rows), dim3(1024), 0, st, logits, row_stats, vocab, tau);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

hydra_status accept_compact(const AcceptArgs& a, cudaStream_t st) {
  long long units = (long long)a.n_layers * 2 * a.kv_planes * a.n_heads * (a.head_dim * a.esize / 16);
  int G = (int)((units + 255) / 256);
  int cap = (sm_count() * 4 + a.batch - 1) / a.batch;
  if (G > cap) G = cap;
  if (G < 1) G = 1;
  launch_pdl(accept_compact_kernel, dim3(dim3(G, a.batch)), dim3(256), 0, st, a);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

// ------------------------------------------------------------------------------------------------
// Small state kernels
// ------------------------------------------------------------------------------------------------
__global__ void set_chunk_kernel(const int* prompt_len, int chunk, int tc, int* pos0, int* n_rows, int batch) {
  pdl_trigger();
  pdl_wait();
  int b = threadIdx.x;
  if (b >= batch) return;
  int rem = prompt_len[b] - chunk * tc;
  pos0[b] = rem > 0 ? chunk * tc : prompt_len[b];
  n_rows[b] = rem < 0 ? 0 : (rem > tc ? tc : rem);
}
hydra_status set_chunk(const int* prompt_len, int chunk, int tc, int* pos0, int* n_rows, int batch, cudaStream_t st) {
  launch_pdl(set_chunk_kernel, dim3(1), dim3(64), 0, st, prompt_len, chunk, tc, pos0, n_rows, batch);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

__global__ void gather_chunk_tokens_kernel(const int* tokens, const int* offsets, int chunk, int tc, int* tok_out) {
  pdl_trigger();
  pdl_wait();
  int b = blockIdx.x, i = threadIdx.x;
  if (i >= tc) return;
  int n = offsets[b + 1] - offsets[b];
  int idx = chunk * tc + i;
  tok_out[b * tc + i] = idx < n ? tokens[offsets[b] + idx] : 0;
}
hydra_status gather_chunk_tokens(const int* tokens, const int* offsets, int chunk, int tc, int* tok_out, int batch,
                                 cudaStream_t st) {
  launch_pdl(gather_chunk_tokens_kernel, dim3(batch), dim3((tc + 31) / 32 * 32), 0, st, tokens, offsets, chunk, tc, tok_out);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

__global__ void capture_last_kernel(const float* h, const int* prompt_len, int chunk, int tc, float* h_new, int kp1,
                                    int* n_new, int* len, int d) {
  pdl_trigger();
  pdl_wait();
  int b = blockIdx.x;
  int last = prompt_len[b] - 1;
  if (last < chunk * tc || last >= (chunk + 1) * tc) return;
  int i = last - chunk * tc;
  for (int c = threadIdx.x; c < d; c += blockDim.x) h_new[(size_t)b * kp1 * d + c] = h[((size_t)b * tc + i) * d + c];
  if (threadIdx.x == 0) { n_new[b] = 1; len[b] = prompt_len[b]; }
}
hydra_status capture_last(const float* h, const int* prompt_len, int chunk, int tc, float* h_new, int kp1, int* n_new,
                          int* len, int batch, int d, cudaStream_t st) {
  launch_pdl(capture_last_kernel, dim3(batch), dim3(256), 0, st, h, prompt_len, chunk, tc, h_new, kp1, n_new, len, d);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

__global__ void prefix_rowset_kernel(const int* len, const int* n_new, int* pos0, int* n_rows, int batch) {
  pdl_trigger();
  pdl_wait();
  int b = threadIdx.x;
  if (b >= batch) return;
  pos0[b] = len[b] - n_new[b];
  n_rows[b] = n_new[b];
}
hydra_status prefix_rowset(const int* len, const int* n_new, int* pos0, int* n_rows, int batch, cudaStream_t st) {
  launch_pdl(prefix_rowset_kernel, dim3(1), dim3(64), 0, st, len, n_new, pos0, n_rows, batch);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

__global__ void pick_last_row_kernel(const float* x, const int* n_rows, int tc, float* hprime, int d) {
  pdl_trigger();
  pdl_wait();
  int b = blockIdx.x;
  int i = n_rows[b] - 1;
  if (i < 0) i = 0;
  for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4)                                  // d % 4 == 0
    *reinterpret_cast<float4*>(hprime + (size_t)b * d + c) = *reinterpret_cast<const float4*>(x + ((size_t)b * tc + i) * d + c);
}
hydra_status pick_last_row(const float* x, const int* n_rows, int tc, float* hprime, int batch, int d, cudaStream_t st) {
  launch_pdl(pick_last_row_kernel, dim3(batch), dim3(256), 0, st, x, n_rows, tc, hprime, d);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

__global__ void apply_plant_kernel(int* tree_tok, const int* plant, int count) {
  pdl_trigger();
  pdl_wait();
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count && plant[i] >= 0) tree_tok[i] = plant[i];
}
hydra_status apply_plant(int* tree_tok, const int* plant, int count, cudaStream_t st) {
  launch_pdl(apply_plant_kernel, dim3((count + 255) / 256), dim3(256), 0, st, tree_tok, plant, count);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

template <typename T>
__global__ void cast_rows_kernel(const float* __restrict__ src, T* __restrict__ dst, size_t dst_ps, size_t count) {
  pdl_trigger();
  pdl_wait();
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) put<T>(dst + i, dst_ps, src[i]);
}
hydra_status cast_rows(const float* src, void* dst, size_t dst_ps, size_t count, int dtype, cudaStream_t st) {
  unsigned grid = (unsigned)((count + 255) / 256);
  if (dtype == 0) launch_pdl(cast_rows_kernel<float>, dim3(grid), dim3(256), 0, st, src, (float*)dst, dst_ps, count);
  else launch_pdl(cast_rows_kernel<bf16>, dim3(grid), dim3(256), 0, st, src, (bf16*)dst, dst_ps, count);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

__global__ void copy_i32_kernel(int* dst, const int* src, int count) {
  pdl_trigger();
  pdl_wait();
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) dst[i] = src[i];
}
hydra_status copy_i32(int* dst, const int* src, int count, cudaStream_t st) {
  launch_pdl(copy_i32_kernel, dim3((count + 255) / 256), dim3(256), 0, st, dst, src, count);
  HYDRA_LAUNCH_CHECK();
  return HYDRA_OK;
}

}  // namespace hydra

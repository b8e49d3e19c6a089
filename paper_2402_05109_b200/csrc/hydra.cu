// libhydra: context, workspace carving, host orchestration of the decode step and the C ABI.
#include "launch.h"
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <tuple>
#include <new>
#include <string>
#include <vector>

namespace hydra {

thread_local long long* g_launch_counter = nullptr;
static thread_local char g_err[512] = "";
void set_last_error(const char* what, cudaError_t e) {
  snprintf(g_err, sizeof(g_err), "%s: %s", what, cudaGetErrorString(e));
}

namespace {

constexpr int CHUNK = 64;          // rows per sequence that a masked forward call can hold (64-bit ancestor masks)
// Rows per sequence of one prefill pass: 128 causal rows on the bfloat16 path (half as many passes over the weights; the
// attention kernel takes them as a causal chunk), 64 chain-masked rows on the float path.
inline int prefill_chunk(const hydra_model_cfg& m) { return m.dtype == 1 ? 2 * CHUNK : CHUNK; }

struct LayerW { const void *attn_norm, *wqkv, *wo, *ffn_norm, *w_gate_up, *w_down; };

struct Bump {                      // 256-byte aligned bump allocator; base == nullptr only measures
  char* base; size_t off;
  template <typename T> T* take(size_t count) {
    off = (off + 255) & ~(size_t)255;
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * sizeof(T);
    return p;
  }
};

int pad_rows(int m) { int t = gemm_tile_rows(m); return (m + t - 1) / t * t; }

enum State { ST_CREATED = 0, ST_READY = 1, ST_DRAFTED = 2, ST_VERIFIED = 3 };

}  // namespace
}  // namespace hydra

using namespace hydra;

struct hydra_ctx {
  hydra_model_cfg m; hydra_head_cfg h;
  int T, Ktree;                                  // tree rows, tree depth
  std::vector<int> parent, depth, first_child, n_child, path_tab;
  std::vector<uint64_t> anc;
  std::vector<std::vector<int>> level_parents;   // [Ktree]
  std::vector<LayerW> layers; LayerW pfx;
  std::vector<const void*> head_w1, head_b1, head_wr, head_br;
  const void *embed, *lm_head, *final_norm;
  int esize;                                     // bytes per weight element
  int planes;                                    // planes of every GEMM operand buffer: 2 (hi, lo) for bfloat16, 1 for float
  int kv_esize;                                  // bytes per element of q and the KV caches: 4 (float) or 2 (float16)
  int kv_planes;                                 // planes of q and the KV caches: 1, or 2 (float16 hi + lo)
  int R;                                         // row capacity of a forward call (padded)
  int RH;                                        // row capacity of the head buffers (padded)
  int maxP;
  // device buffers
  int *d_parent, *d_depth, *d_first_child, *d_n_child, *d_path_tab, *d_chain_depth;
  uint64_t *d_anc, *d_chain_mask;
  std::vector<int*> d_level_parents;
  int *d_len, *d_n_new, *d_root_tok, *d_status, *d_pos0, *d_nrows, *d_prompt_len, *d_offsets, *d_tok, *d_tree_tok, *d_amax;
  unsigned int* d_done;
  unsigned long long* d_pass_bits; int* d_bonus; float4* d_row_stats;
  const float* last_logits;                      // logits of the last verification (the caller's buffer or c->logits)
  int acc_mode; float acc_tau, acc_eps, acc_alpha; const float* acc_u;
  char *kv_base, *kv_pfx;
  float *x, *part, *h_tree, *logits, *h_new, *hprime, *y, *head_logits;
  float2* rope;
  void *topk_scratch; int topk_rows_cap;
  void *q, *xn, *attn_out, *act, *z, *yb, *att_scratch;
  size_t part_floats;
  // host state
  int batch, state, gemm_mode;
  std::vector<int> len_ub;
  const int* plant;
  long long launches;
  // optional per-kernel-class timing (benchmarks): event pairs recorded around launches of a class
  struct Timed { cudaEvent_t a, b; int cls; double bytes; };
  // whole-step CUDA graphs, keyed by everything a captured step freezes (attention grid sizes, buffer pointers)
  struct GraphKey {
    int len_verify, len_prefix; const void *plant, *n_acc, *out_tok;
    bool operator<(const GraphKey& o) const {
      return std::tie(len_verify, len_prefix, plant, n_acc, out_tok) < std::tie(o.len_verify, o.len_prefix, o.plant, o.n_acc, o.out_tok);
    }
  };
  struct StepGraph { cudaGraphExec_t exec; long long launches; };
  std::map<GraphKey, StepGraph> graphs;
  int use_graph; long long steps_done;
  int timing;
  std::vector<Timed> timed;
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> event_pool;
};

namespace {

size_t kv_layer_elems(const hydra_model_cfg& m) { return (size_t)m.max_batch * m.n_heads * m.max_seq * m.head_dim; }

struct TreeHost {
  int T = 0, K = 0, maxP = 1;
  std::vector<int> parent, depth, first_child, n_child, path_tab;
  std::vector<uint64_t> anc;
  std::vector<std::vector<int>> level_parents;
};

// Tables of the static tree: depth, ancestor-or-self bitmask, children ranges, root paths, per-level parents.
bool build_tree(const hydra_tree_cfg* t, int max_depth, TreeHost& o) {
  if (!t || !t->parent || t->n_rows < 1 || t->n_rows > 64 || t->parent[0] != -1) return false;
  int T = t->n_rows;
  o.T = T; o.parent.assign(t->parent, t->parent + T);
  o.depth.assign(T, 0); o.anc.assign(T, 0); o.first_child.assign(T, 0); o.n_child.assign(T, 0);
  o.anc[0] = 1ull;
  for (int i = 1; i < T; ++i) {
    int p = o.parent[i];
    if (p < 0 || p >= i) return false;
    o.depth[i] = o.depth[p] + 1;
    o.anc[i] = o.anc[p] | (1ull << i);
    if (o.n_child[p] == 0) o.first_child[p] = i;
    else if (o.first_child[p] + o.n_child[p] != i) return false;     // children of a parent must be adjacent rows
    o.n_child[p]++;
    if (o.depth[i] < o.depth[i - 1]) return false;                   // rows ordered by depth
    if (o.depth[i] == o.depth[i - 1] && i > 1 && p < o.parent[i - 1]) return false;   // ... then by rank path
  }
  o.K = *std::max_element(o.depth.begin(), o.depth.end());
  if (o.K > max_depth) return false;
  int kp1 = max_depth + 1;
  o.path_tab.assign((size_t)T * kp1, -1);
  for (int i = 0; i < T; ++i) { int node = i; for (int k = o.depth[i]; k >= 0; --k) { o.path_tab[i * kp1 + k] = node; node = o.parent[node]; } }
  o.level_parents.assign(o.K, {});
  for (int d = 1; d <= o.K; ++d)
    for (int i = 0; i < T; ++i) if (o.depth[i] == d - 1 && o.n_child[i] > 0) o.level_parents[d - 1].push_back(i);
  o.maxP = 1;
  for (auto& lv : o.level_parents) o.maxP = std::max(o.maxP, (int)lv.size());
  return true;
}

bool valid_cfg(const hydra_model_cfg* m, const hydra_head_cfg* h) {
  if (!m || !h) return false;
  if (m->n_layers < 1 || m->d_model < 1 || m->n_heads < 1 || m->d_ffn < 1 || m->vocab < 1 || m->max_batch < 1 || m->max_seq < 1)
    return false;
  if (m->n_heads * m->head_dim != m->d_model) return false;
  if (m->dtype != 0 && m->dtype != 1) return false;
  if (m->kv_planes < 0 || m->kv_planes > 2) return false;
  if (h->n_heads < 0 || h->n_mlp_layers < 1) return false;
  return true;
}
hydra_status supported_cfg(const hydra_model_cfg* m) {
  if (m->head_dim != 64 && m->head_dim != 128) return HYDRA_ERR_UNSUPPORTED;
  if (m->d_model % 4 || m->d_ffn % 4) return HYDRA_ERR_UNSUPPORTED;
  if (m->max_batch > 64) return HYDRA_ERR_UNSUPPORTED;
  if (m->dtype == 1 && (m->d_model % 128 || m->d_ffn % 64 || m->vocab % 128)) return HYDRA_ERR_UNSUPPORTED;
  return HYDRA_OK;
}

// Lays every library buffer out in the workspace (or just measures it when ws == nullptr).
size_t carve(hydra_ctx* c, const hydra_model_cfg& m, const hydra_head_cfg& h, const TreeHost& t, char* ws) {
  Bump b{ws, 0};
  const int es = m.dtype == 0 ? 4 : 2;
  const int np = m.dtype == 0 ? 1 : 2;          // bfloat16 GEMM operands are stored as hi + lo planes
  const int ces = m.dtype == 0 ? 4 : 2;         // q and the KV caches: float, or float16 in kvp planes
  const int kvp = m.dtype == 0 ? 1 : (m.kv_planes == 1 ? 1 : 2);
  const int d = m.d_model, f = m.d_ffn, V = m.vocab, K = h.n_heads, T = t.T;
  const int PC = prefill_chunk(m);
  const int R = pad_rows(m.max_batch * PC);
  const int RH = pad_rows(m.max_batch * t.maxP);
  // largest partial-sum buffer over every GEMM shape and row count the library issues
  size_t part_floats = 0;
  {
    auto need = [&](int mm, int n, int k) {
      int slots = 1;
      if (m.dtype == 1) gemm_tc_plan(mm, n, k, nullptr, &slots);
      part_floats = std::max(part_floats, (size_t)slots * mm * n);
    };
    const int shapes[][2] = {{3 * d, d}, {d, d}, {2 * f, d}, {d, f}, {V, d}};
    const int per_seq[] = {PC, T, K + 1, 1};
    for (auto& sh : shapes)
      for (int rows : per_seq)
        for (int bb = 1; bb <= m.max_batch; ++bb) need(rows * bb, sh[0], sh[1]);
    for (int mm = 1; mm <= m.max_batch * t.maxP; ++mm) {
      for (int i = 1; i <= K; ++i) need(mm, d, (i + 1) * d);
      need(mm, d, d);
      need(mm, V, d);
    }
  }
  auto* parent = b.take<int>(T); auto* depth = b.take<int>(T); auto* fc = b.take<int>(T); auto* nc = b.take<int>(T);
  auto* path_tab = b.take<int>((size_t)T * (K + 1)); auto* chain_depth = b.take<int>(PC);
  auto* anc = b.take<uint64_t>(T); auto* chain_mask = b.take<uint64_t>(CHUNK);
  std::vector<int*> lvl;
  for (auto& lv : t.level_parents) lvl.push_back(b.take<int>(lv.size()));
  auto* len = b.take<int>(m.max_batch); auto* n_new = b.take<int>(m.max_batch); auto* root = b.take<int>(m.max_batch);
  auto* status = b.take<int>(64);          // [0] status word, [8..15] where a bounded wait gave up
  auto* pos0 = b.take<int>(m.max_batch); auto* nrows = b.take<int>(m.max_batch);
  auto* plen = b.take<int>(m.max_batch); auto* offs = b.take<int>(m.max_batch + 1);
  auto* tok = b.take<int>(R); auto* tree_tok = b.take<int>((size_t)m.max_batch * T); auto* amax = b.take<int>(R);
  auto* done = b.take<unsigned int>(m.max_batch);
  auto* pass_bits = b.take<unsigned long long>(m.max_batch); auto* bonus = b.take<int>(m.max_batch);
  auto* row_stats = b.take<float4>(R);
  auto* kvb = b.take<char>((size_t)m.n_layers * 2 * kvp * kv_layer_elems(m) * ces);
  auto* kvpfx = b.take<char>(h.prefix_attn ? (size_t)2 * kvp * kv_layer_elems(m) * ces : 0);
  auto* x = b.take<float>((size_t)R * d); auto* q = b.take<char>((size_t)kvp * R * d * ces);
  auto* part = b.take<float>(part_floats);
  auto* h_tree = b.take<float>((size_t)R * d);
  auto* logits = b.take<float>((size_t)pad_rows(m.max_batch * T) * V);
  auto* h_new = b.take<float>((size_t)pad_rows(m.max_batch * (K + 1)) * d);
  auto* hprime = b.take<float>((size_t)m.max_batch * d);
  auto* y = b.take<float>((size_t)RH * d); auto* head_logits = b.take<float>((size_t)RH * V);
  auto* rope = b.take<float2>((size_t)R * (m.head_dim / 2));
  auto* xn = b.take<char>((size_t)np * R * d * es); auto* attn_out = b.take<char>((size_t)np * R * d * es);
  auto* act = b.take<char>((size_t)np * R * f * es);
  auto* z = b.take<char>((size_t)np * RH * (K + 1) * d * es); auto* yb = b.take<char>((size_t)np * RH * d * es);
  const int topk_cap = std::max(R, RH);
  auto* topk_s = b.take<char>(topk_scratch_bytes(topk_cap, V));
  auto* att = b.take<char>(m.dtype == 0 ? attention_scratch_bytes(m.max_batch, CHUNK, m.n_heads, m.head_dim, m.max_seq) : 0);
  if (c) {
    c->R = R; c->RH = RH; c->part_floats = part_floats; c->esize = es; c->planes = np; c->kv_esize = ces; c->kv_planes = kvp;
    c->d_parent = parent; c->d_depth = depth; c->d_first_child = fc; c->d_n_child = nc; c->d_path_tab = path_tab;
    c->d_chain_depth = chain_depth; c->d_anc = anc; c->d_chain_mask = chain_mask; c->d_level_parents = lvl;
    c->d_len = len; c->d_n_new = n_new; c->d_root_tok = root; c->d_status = status; c->d_pos0 = pos0; c->d_nrows = nrows;
    c->d_prompt_len = plen; c->d_offsets = offs; c->d_tok = tok; c->d_tree_tok = tree_tok; c->d_amax = amax; c->d_done = done;
    c->d_pass_bits = pass_bits; c->d_bonus = bonus; c->d_row_stats = row_stats;
    c->kv_base = kvb; c->kv_pfx = kvpfx; c->x = x; c->q = q; c->part = part; c->h_tree = h_tree; c->logits = logits;
    c->h_new = h_new; c->hprime = hprime; c->y = y; c->head_logits = head_logits; c->rope = rope; c->xn = xn;
    c->attn_out = attn_out; c->act = act; c->z = z; c->yb = yb; c->att_scratch = att; c->topk_scratch = topk_s; c->topk_rows_cap = topk_cap;
  }
  return (b.off + 255) & ~(size_t)255;
}

struct TimeScope {                // brackets the launches issued during its lifetime with an event pair
  hydra_ctx* c; cudaStream_t st; cudaEvent_t a = nullptr, b = nullptr; int cls; double bytes;
  TimeScope(hydra_ctx* c_, int cls_, double bytes_, cudaStream_t st_) : c(c_), st(st_), cls(cls_), bytes(bytes_) {
    if (!c->timing) return;
    if (!c->event_pool.empty()) { a = c->event_pool.back().first; b = c->event_pool.back().second; c->event_pool.pop_back(); }
    else if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { a = b = nullptr; return; }
    cudaEventRecord(a, st);
  }
  ~TimeScope() { if (a) { cudaEventRecord(b, st); c->timed.push_back({a, b, cls, bytes}); } }
};

// Partial sums of x @ w^T into c->part; *sd says where the slots of each output tile are.
hydra_status run_gemm(hydra_ctx* c, const void* x, int x_rows_alloc, const void* w, int m, int n, int k, SplitDesc* sd,
                      cudaStream_t st) {
  // algorithmic bytes of the launch: the weight matrix and the activation slab read once, the output written once
  TimeScope ts(c, HYDRA_TIME_GEMM, (double)c->esize * ((double)n * k + (double)c->planes * m * k) + 4.0 * m * n, st);
  if (c->m.dtype == 1 && c->gemm_mode != 1) {
    int slots = 1;
    gemm_tc_plan(m, n, k, nullptr, &slots);
    if ((size_t)slots * m * n > c->part_floats) return HYDRA_ERR_CAPACITY;
    return gemm_tc((const bf16*)x, x_rows_alloc, c->planes, (const bf16*)w, c->part, m, n, k, sd, c->d_status, c->d_status + 8, nullptr, st);
  }
  *sd = single_slot((size_t)m * n);
  return gemm_simt(x, w, c->part, m, n, k, c->m.dtype, st);      // bfloat16: the hi plane only (debug mode)
}

// element distance between the hi and lo planes of an operand buffer of `rows_alloc` rows of `cols` (0 for float)
size_t ps(const hydra_ctx* c, int rows_alloc, size_t cols) { return c->planes == 2 ? (size_t)rows_alloc * cols : 0; }

// RoPE + KV append + tree attention of one layer from the QKV partial sums (*sd) in c->part; result in c->attn_out.
// stable_lengths: every forward call of the library starts with rope_table, which lets nothing of the call start before all
// earlier kernels have completed; the row set's lengths and the committed cache rows are written before that kernel, so
// the attention kernels of the call may fetch committed tiles ahead of their predecessor.
hydra_status attention_block(hydra_ctx* c, char* kc, char* vc, const RowSet& rs, int len_upper, const SplitDesc& sd, bool stable_lengths,
                             cudaStream_t st) {
  const hydra_model_cfg& m = c->m;
  const int d = m.d_model, dt = m.dtype;
  const size_t q_ps = c->kv_planes == 2 ? (size_t)c->R * d : 0, kv_ps = c->kv_planes == 2 ? kv_layer_elems(m) : 0;
  HYDRA_TRY(qkv_rope_store(c->part, sd, c->rope, c->q, q_ps, kc, vc, kv_ps, rs, m.n_heads, m.head_dim, m.max_seq, dt, c->d_status, st));
  TimeScope ts(c, HYDRA_TIME_ATTENTION, 0.0, st);
  if (dt == 0)
    return tree_attention_f32((const float*)c->q, (const float*)kc, (const float*)vc, rs, (float*)c->attn_out, c->att_scratch, m.n_heads,
                              m.head_dim, m.max_seq, len_upper, st);
  return tree_attention_tc((const __half*)c->q, c->R, (const __half*)kc, (const __half*)vc, m.max_batch, c->kv_planes, rs, (bf16*)c->attn_out,
                           ps(c, c->R, d), m.n_heads, m.head_dim, m.max_seq, len_upper, c->d_status, stable_lengths, st);
}

double gemm_bytes(const hydra_ctx* c, int m, int n, int k) {        // weights + activation slab read once, output written once
  return (double)c->esize * ((double)n * k + (double)c->planes * m * k) + 4.0 * m * n;
}

// The rest of a layer after its attention: O projection, + residual, RMSNorm, gate/up, SiLU * up, down, + residual and,
// when next_gain is given, xn = rmsnorm(x) * next_gain (hn: the same in float); when next_w is given, also the
// GEMM xn @ next_w^T (the next layer's QKV projection, or the LM head), whose partial sums stay in c->part (*sd).
hydra_status mlp_block(hydra_ctx* c, const LayerW& w, int rows, const void* next_gain, float* hn, const void* next_w, int next_n,
                       SplitDesc* sd, cudaStream_t st) {
  const hydra_model_cfg& m = c->m;
  const int d = m.d_model, f = m.d_ffn, dt = m.dtype;
  SplitDesc s1;
  HYDRA_TRY(run_gemm(c, c->attn_out, c->R, w.wo, rows, d, d, &s1, st));
  HYDRA_TRY(residual_rmsnorm(c->x, c->part, s1, c->x, w.ffn_norm, c->xn, ps(c, c->R, d), nullptr, rows, d, m.rms_eps, dt, st));
  HYDRA_TRY(run_gemm(c, c->xn, c->R, w.w_gate_up, rows, 2 * f, d, &s1, st));
  HYDRA_TRY(silu_mul(c->part, s1, c->act, ps(c, c->R, f), rows, f, dt, st));
  HYDRA_TRY(run_gemm(c, c->act, c->R, w.w_down, rows, d, f, &s1, st));
  HYDRA_TRY(residual_rmsnorm(c->x, c->part, s1, c->x, next_gain, next_gain ? c->xn : nullptr, ps(c, c->R, d), hn, rows, d, m.rms_eps, dt, st));
  if (next_w) HYDRA_TRY(run_gemm(c, c->xn, c->R, next_w, rows, next_n, d, sd, st));
  return HYDRA_OK;
}

// Base model over the rows of `rs` whose tokens are tok[rows]: leaves post-final-norm hidden rows in c->h_tree
// (float) and c->xn (operand type); with tail_w also the partial sums of xn @ tail_w^T (the LM head) in c->part (*tail_sd).
hydra_status run_base(hydra_ctx* c, const int* tok, const RowSet& rs, int len_upper, const void* tail_w, int tail_n, SplitDesc* tail_sd,
                      bool stable_lengths, cudaStream_t st) {
  const hydra_model_cfg& m = c->m;
  const int rows = rs.batch * rs.tc, d = m.d_model;
  const size_t kvl = kv_layer_elems(m) * c->kv_esize * c->kv_planes;      // bytes of one layer's K (or V) cache, all planes
  HYDRA_TRY(rope_table(rs, c->rope, m.head_dim, m.rope_theta, st));
  HYDRA_TRY(embed_rows(c->embed, tok, c->x, rows, d, m.vocab, m.dtype, c->d_status, st));
  HYDRA_TRY(residual_rmsnorm(c->x, nullptr, single_slot(0), c->x, c->layers[0].attn_norm, c->xn, ps(c, c->R, d), nullptr, rows, d, m.rms_eps, m.dtype, st));
  SplitDesc sd;
  HYDRA_TRY(run_gemm(c, c->xn, c->R, c->layers[0].wqkv, rows, 3 * d, d, &sd, st));
  for (int l = 0; l < m.n_layers; ++l) {
    const bool last = l + 1 == m.n_layers;
    HYDRA_TRY(attention_block(c, c->kv_base + (size_t)(2 * l) * kvl, c->kv_base + (size_t)(2 * l + 1) * kvl, rs, len_upper, sd, stable_lengths, st));
    HYDRA_TRY(mlp_block(c, c->layers[l], rows, last ? c->final_norm : c->layers[l + 1].attn_norm, last ? c->h_tree : nullptr,
                        last ? tail_w : c->layers[l + 1].wqkv, last ? tail_n : 3 * d, last ? tail_sd : &sd, st));
  }
  return HYDRA_OK;
}

// Prefix-attention layer over rows whose input (post-final-norm hidden) is `src` laid out like rs.
hydra_status run_prefix(hydra_ctx* c, const float* src, const RowSet& rs, int len_upper, cudaStream_t st) {
  const hydra_model_cfg& m = c->m;
  const int rows = rs.batch * rs.tc, d = m.d_model;
  const size_t kvl = kv_layer_elems(m) * c->kv_esize * c->kv_planes;      // bytes of one layer's K (or V) cache, all planes
  HYDRA_TRY(rope_table(rs, c->rope, m.head_dim, m.rope_theta, st));
  HYDRA_TRY(residual_rmsnorm(src, nullptr, single_slot(0), c->x, c->pfx.attn_norm, c->xn, ps(c, c->R, d), nullptr, rows, d, m.rms_eps, m.dtype, st));
  SplitDesc sd;
  HYDRA_TRY(run_gemm(c, c->xn, c->R, c->pfx.wqkv, rows, 3 * d, d, &sd, st));
  HYDRA_TRY(attention_block(c, c->kv_pfx, c->kv_pfx + kvl, rs, len_upper, sd, true, st));
  return mlp_block(c, c->pfx, rows, nullptr, nullptr, nullptr, 0, nullptr, st);
}

int max_len_ub(const hydra_ctx* c) { int v = 0; for (int b = 0; b < c->batch; ++b) v = std::max(v, c->len_ub[b]); return v; }
// Upper bound of the KV length used to size attention grids, rounded up so that it (and a captured step graph)
// stays valid for many steps; CTAs beyond the real length exit at once.
int len_bucket(const hydra_ctx* c, int v) { v = (v + 511) / 512 * 512; return std::min(v, c->m.max_seq); }

hydra_status do_draft(hydra_ctx* c, int* tree_tok, cudaStream_t st) {
  const hydra_model_cfg& m = c->m;
  const int B = c->batch, K = c->h.n_heads, d = m.d_model, dt = m.dtype;
  if (c->h.prefix_attn) {
    HYDRA_TRY(prefix_rowset(c->d_len, c->d_n_new, c->d_pos0, c->d_nrows, B, st));
    RowSet rs{B, K + 1, c->d_nrows, c->d_pos0, c->d_chain_depth, c->d_chain_mask};
    HYDRA_TRY(run_prefix(c, c->h_new, rs, len_bucket(c, max_len_ub(c)), st));
    HYDRA_TRY(pick_last_row(c->x, c->d_nrows, K + 1, c->hprime, B, d, st));
  } else {
    HYDRA_TRY(pick_last_row(c->h_new, c->d_n_new, K + 1, c->hprime, B, d, st));
  }
  if (c->Ktree == 0) return copy_i32(tree_tok, c->d_root_tok, B, st);      // root-only tree (T == 1)
  const bool medusa = c->h.medusa != 0;
  for (int lvl = 1; lvl <= c->Ktree; ++lvl) {
    const int P = (int)c->level_parents[lvl - 1].size();
    // Hydra heads: one row per (sequence, parent), input [h' ; E of the path tokens].  Sequentially independent heads: one row
    // per sequence, input h' alone (level 1's parent list, the root, stands in as a one-parent level for the gather)
    const int rows = medusa ? B : B * P;
    const int rows_per_b = medusa ? 1 : P;
    const int in_blocks = medusa ? 1 : lvl + 1;
    LevelDesc lv{lvl, P, c->d_level_parents[lvl - 1]};
    LevelDesc lv_in = medusa ? LevelDesc{0, 1, c->d_level_parents[0]} : lv;
    HYDRA_TRY(head_gather(c->hprime, c->embed, c->d_root_tok, tree_tok, c->d_path_tab, lv_in, lvl == 1, c->z, ps(c, c->RH, (size_t)in_blocks * d), B, c->T,
                          K + 1, d, m.vocab, dt, c->d_status, st));
    SplitDesc sd;
    HYDRA_TRY(run_gemm(c, c->z, c->RH, c->head_w1[lvl - 1], rows, d, in_blocks * d, &sd, st));
    HYDRA_TRY(head_act(c->hprime, 1, rows_per_b, c->part, sd, c->h.has_bias ? c->head_b1[lvl - 1] : nullptr, c->y, c->yb, ps(c, c->RH, d), rows, d, dt, st));
    for (int l = 0; l + 1 < c->h.n_mlp_layers; ++l) {
      const char* wr = (const char*)c->head_wr[lvl - 1] + (size_t)l * d * d * c->esize;
      const char* br = c->h.has_bias ? (const char*)c->head_br[lvl - 1] + (size_t)l * d * c->esize : nullptr;
      HYDRA_TRY(run_gemm(c, c->yb, c->RH, wr, rows, d, d, &sd, st));
      HYDRA_TRY(head_act(c->y, 0, rows_per_b, c->part, sd, br, c->y, c->yb, ps(c, c->RH, d), rows, d, dt, st));
    }
    HYDRA_TRY(run_gemm(c, c->yb, c->RH, c->lm_head, rows, m.vocab, d, &sd, st));
    int max_children = 1;
    for (int p : c->level_parents[lvl - 1]) max_children = std::max(max_children, c->n_child[p]);
    HYDRA_TRY(topk_children(c->part, sd, c->head_logits, lv, max_children, c->d_first_child, c->d_n_child, tree_tok, c->topk_scratch,
                            c->topk_rows_cap, B, c->T, m.vocab, medusa ? 1 : 0, st));
  }
  return HYDRA_OK;
}

hydra_status do_verify(hydra_ctx* c, const int* tree_tok, int* amax, float* logits, cudaStream_t st) {
  const hydra_model_cfg& m = c->m;
  const int rows = c->batch * c->T;
  RowSet rs{c->batch, c->T, nullptr, c->d_len, c->d_depth, c->d_anc};
  SplitDesc sd;
  HYDRA_TRY(run_base(c, tree_tok, rs, len_bucket(c, max_len_ub(c) + c->T), c->lm_head, m.vocab, &sd, true, st));
  if (c->acc_mode == 1 && !logits) logits = c->logits;              // the typical criterion reads whole rows of logits
  c->last_logits = logits;
  HYDRA_TRY(argmax_rows(c->part, sd, logits, amax, c->topk_scratch, c->topk_rows_cap, rows, m.vocab, st));
  if (c->acc_mode == 1) HYDRA_TRY(softmax_row_stats(logits, c->d_row_stats, rows, m.vocab, c->acc_tau, st));
  return HYDRA_OK;
}

hydra_status do_accept(hydra_ctx* c, const int* tree_tok, const int* amax, int* n_acc, int* path, int* out_tok, cudaStream_t st) {
  const hydra_model_cfg& m = c->m;
  AcceptArgs a{};
  a.tree_tok = tree_tok; a.amax = amax; a.parent = c->d_parent; a.depth = c->d_depth; a.anc = c->d_anc;
  a.T = c->T; a.K = c->h.n_heads; a.batch = c->batch; a.n_layers = m.n_layers; a.n_heads = m.n_heads; a.head_dim = m.head_dim;
  a.max_seq = m.max_seq; a.max_batch = m.max_batch; a.d_model = m.d_model; a.esize = c->kv_esize; a.kv_planes = c->kv_planes;
  a.kv_base = c->kv_base; a.h_tree = c->h_tree; a.h_tree_stride = c->T;
  a.h_new = c->h_new; a.n_new = c->d_n_new; a.len = c->d_len; a.root_tok = c->d_root_tok;
  a.n_acc = n_acc; a.path = path; a.out_tok = out_tok; a.done_counter = c->d_done; a.status = c->d_status;
  a.mode = c->acc_mode; a.tau = c->acc_tau; a.eps = c->acc_eps; a.alpha = c->acc_alpha; a.logits = c->last_logits;
  a.row_stats = c->d_row_stats; a.vocab = m.vocab; a.u = c->acc_mode == 1 ? c->acc_u : nullptr; a.pass_bits = c->d_pass_bits;
  a.bonus_tmp = c->d_bonus;
  if (a.mode == 1 && !a.logits) return HYDRA_ERR_STATE;
  {
    TimeScope ts(c, HYDRA_TIME_ACCEPT, 0.0, st);
    HYDRA_TRY(accept_compact(a, st));
  }
  return HYDRA_OK;
}

void bump_len_ub(hydra_ctx* c) { for (int b = 0; b < c->batch; ++b) c->len_ub[b] += c->Ktree + 1; }

hydra_status enqueue_step(hydra_ctx* c, int* n_acc, int* out_tok, cudaStream_t st) {
  HYDRA_TRY(do_draft(c, c->d_tree_tok, st));
  if (c->plant) HYDRA_TRY(apply_plant(c->d_tree_tok, c->plant, c->batch * c->T, st));
  HYDRA_TRY(do_verify(c, c->d_tree_tok, c->d_amax, nullptr, st));
  return do_accept(c, c->d_tree_tok, c->d_amax, n_acc, nullptr, out_tok, st);
}

void drop_graphs(hydra_ctx* c) {
  for (auto& g : c->graphs) cudaGraphExecDestroy(g.second.exec);
  c->graphs.clear();
}

bool capacity_ok(const hydra_ctx* c) {
  for (int b = 0; b < c->batch; ++b) if (c->len_ub[b] + c->T > c->m.max_seq) return false;
  return true;
}

struct CounterScope {
  explicit CounterScope(hydra_ctx* c) { g_launch_counter = c ? &c->launches : nullptr; }
  ~CounterScope() { g_launch_counter = nullptr; }
};

}  // namespace

extern "C" {

size_t hydra_workspace_bytes(const hydra_model_cfg* m, const hydra_head_cfg* h, const hydra_tree_cfg* t) {
  TreeHost th;
  if (!valid_cfg(m, h) || !build_tree(t, h->n_heads, th)) return 0;
  return carve(nullptr, *m, *h, th, nullptr);
}

hydra_status hydra_create(hydra_ctx** out, const hydra_model_cfg* m, const hydra_head_cfg* h, const hydra_tree_cfg* t,
                          const hydra_weights* w, void* ws, size_t ws_bytes) {
  if (!out || !w || !ws) return HYDRA_ERR_INVALID;
  *out = nullptr;
  TreeHost th;
  if (!valid_cfg(m, h) || !build_tree(t, h->n_heads, th)) return HYDRA_ERR_INVALID;
  hydra_status sup = supported_cfg(m);
  if (sup != HYDRA_OK) return sup;
  if ((uintptr_t)ws & 255) return HYDRA_ERR_INVALID;
  if (!w->embed || !w->lm_head || !w->final_norm || !w->attn_norm || !w->wqkv || !w->wo || !w->ffn_norm || !w->w_gate_up || !w->w_down)
    return HYDRA_ERR_INVALID;
  if (th.K > 0 && (!w->head_w1 || (h->has_bias && !w->head_b1))) return HYDRA_ERR_INVALID;
  if (th.K > 0 && h->n_mlp_layers > 1 && (!w->head_wr || (h->has_bias && !w->head_br))) return HYDRA_ERR_INVALID;
  if (h->prefix_attn && (!w->pfx_attn_norm || !w->pfx_wqkv || !w->pfx_wo || !w->pfx_ffn_norm || !w->pfx_w_gate_up || !w->pfx_w_down))
    return HYDRA_ERR_INVALID;
  size_t need = carve(nullptr, *m, *h, th, nullptr);
  if (ws_bytes < need) return HYDRA_ERR_CAPACITY;
  if (m->dtype == 1 && !gemm_tc_available()) { set_last_error("cuTensorMapEncodeTiled entry point", cudaErrorUnknown); return HYDRA_ERR_CUDA; }
  hydra_ctx* c = new (std::nothrow) hydra_ctx();
  if (!c) return HYDRA_ERR_INVALID;
  c->m = *m; c->h = *h; c->T = th.T; c->Ktree = th.K; c->maxP = th.maxP;
  c->parent = th.parent; c->depth = th.depth; c->first_child = th.first_child; c->n_child = th.n_child;
  c->path_tab = th.path_tab; c->anc = th.anc; c->level_parents = th.level_parents;
  for (int l = 0; l < m->n_layers; ++l) {
    LayerW lw{w->attn_norm[l], w->wqkv[l], w->wo[l], w->ffn_norm[l], w->w_gate_up[l], w->w_down[l]};
    if (!lw.attn_norm || !lw.wqkv || !lw.wo || !lw.ffn_norm || !lw.w_gate_up || !lw.w_down) { delete c; return HYDRA_ERR_INVALID; }
    c->layers.push_back(lw);
  }
  c->pfx = LayerW{w->pfx_attn_norm, w->pfx_wqkv, w->pfx_wo, w->pfx_ffn_norm, w->pfx_w_gate_up, w->pfx_w_down};
  for (int i = 0; i < th.K; ++i) {
    c->head_w1.push_back(w->head_w1[i]);
    c->head_b1.push_back(h->has_bias ? w->head_b1[i] : nullptr);
    c->head_wr.push_back(h->n_mlp_layers > 1 ? w->head_wr[i] : nullptr);
    c->head_br.push_back(h->n_mlp_layers > 1 && h->has_bias ? w->head_br[i] : nullptr);
    if (!c->head_w1[i] || (h->n_mlp_layers > 1 && !c->head_wr[i])) { delete c; return HYDRA_ERR_INVALID; }
  }
  c->embed = w->embed; c->lm_head = w->lm_head; c->final_norm = w->final_norm;
  carve(c, *m, *h, th, (char*)ws);
  c->batch = 0; c->state = ST_CREATED; c->gemm_mode = 0; c->plant = nullptr; c->launches = 0; c->timing = 0; c->steps_done = 0;
  c->use_graph = 1;
  c->acc_mode = 0; c->acc_tau = 1.f; c->acc_eps = 0.f; c->acc_alpha = 0.f; c->acc_u = nullptr; c->last_logits = nullptr;
  c->len_ub.assign(m->max_batch, 0);
  // clear the workspace, upload the static tables
  auto fail = [&](cudaError_t e, const char* what) { set_last_error(what, e); delete c; return HYDRA_ERR_CUDA; };
  cudaError_t e;
  // the workspace may be memory that work still queued on some (non-blocking) stream is using: drain the device first
  if ((e = cudaDeviceSynchronize()) != cudaSuccess) return fail(e, "cudaDeviceSynchronize");
  if ((e = cudaMemset(ws, 0, need)) != cudaSuccess) return fail(e, "cudaMemset(workspace)");
  const int T = th.T, K = h->n_heads;
  const int PC = prefill_chunk(c->m);
  std::vector<int> chain_depth(PC); std::vector<uint64_t> chain_mask(CHUNK);
  for (int i = 0; i < PC; ++i) chain_depth[i] = i;
  for (int i = 0; i < CHUNK; ++i) chain_mask[i] = i == 63 ? ~0ull : ((1ull << (i + 1)) - 1);
#define UP(dst, src, bytes) if ((bytes) && (e = cudaMemcpy(dst, src, bytes, cudaMemcpyHostToDevice)) != cudaSuccess) return fail(e, "cudaMemcpy(tables)")
  UP(c->d_parent, th.parent.data(), T * sizeof(int)); UP(c->d_depth, th.depth.data(), T * sizeof(int));
  UP(c->d_first_child, th.first_child.data(), T * sizeof(int)); UP(c->d_n_child, th.n_child.data(), T * sizeof(int));
  UP(c->d_path_tab, th.path_tab.data(), (size_t)T * (K + 1) * sizeof(int));
  UP(c->d_chain_depth, chain_depth.data(), PC * sizeof(int)); UP(c->d_chain_mask, chain_mask.data(), CHUNK * sizeof(uint64_t));
  UP(c->d_anc, th.anc.data(), T * sizeof(uint64_t));
  for (size_t i = 0; i < th.level_parents.size(); ++i) UP(c->d_level_parents[i], th.level_parents[i].data(), th.level_parents[i].size() * sizeof(int));
#undef UP
  if ((e = cudaDeviceSynchronize()) != cudaSuccess) return fail(e, "cudaDeviceSynchronize");
  *out = c;
  return HYDRA_OK;
}

hydra_status hydra_destroy(hydra_ctx* c) {
  if (!c) return HYDRA_ERR_INVALID;
  cudaError_t e = cudaDeviceSynchronize();
  drop_graphs(c);
  for (auto& t : c->timed) { cudaEventDestroy(t.a); cudaEventDestroy(t.b); }
  for (auto& p : c->event_pool) { cudaEventDestroy(p.first); cudaEventDestroy(p.second); }
  delete c;
  if (e != cudaSuccess) { set_last_error("cudaDeviceSynchronize", e); return HYDRA_ERR_CUDA; }
  return HYDRA_OK;
}

hydra_status hydra_prefill(hydra_ctx* c, int batch, const int32_t* tokens, const int32_t* offs, void* stream) {
  if (!c || !tokens || !offs || batch < 1 || batch > c->m.max_batch) return HYDRA_ERR_INVALID;
  CounterScope cs(c);
  cudaStream_t st = (cudaStream_t)stream;
  const hydra_model_cfg& m = c->m;
  std::vector<int> plen(batch);
  int maxlen = 0;
  for (int b = 0; b < batch; ++b) {
    plen[b] = offs[b + 1] - offs[b];
    if (plen[b] < 1) return HYDRA_ERR_INVALID;
    if (plen[b] + c->T > m.max_seq) return HYDRA_ERR_CAPACITY;
    maxlen = std::max(maxlen, plen[b]);
  }
  c->batch = batch;
  HYDRA_CUDA(cudaMemcpyAsync(c->d_prompt_len, plen.data(), batch * sizeof(int), cudaMemcpyHostToDevice, st));
  HYDRA_CUDA(cudaMemcpyAsync(c->d_offsets, offs, (batch + 1) * sizeof(int), cudaMemcpyHostToDevice, st));
  HYDRA_CUDA(cudaStreamSynchronize(st));           // the host vectors above go out of scope
  const int PC = prefill_chunk(m);
  const int nchunks = (maxlen + PC - 1) / PC;
  // a chunk is a chain: row i sees the rows before it (an explicit mask for 64 rows, the causal rule of the attention kernel for 128)
  RowSet rs{batch, PC, c->d_nrows, c->d_pos0, c->d_chain_depth, PC > CHUNK ? nullptr : c->d_chain_mask};
  for (int ch = 0; ch < nchunks; ++ch) {
    HYDRA_TRY(set_chunk(c->d_prompt_len, ch, PC, c->d_pos0, c->d_nrows, batch, st));
    HYDRA_TRY(gather_chunk_tokens(tokens, c->d_offsets, ch, PC, c->d_tok, batch, st));
    HYDRA_TRY(run_base(c, c->d_tok, rs, (ch + 1) * PC, nullptr, 0, nullptr, true, st));
    HYDRA_TRY(capture_last(c->h_tree, c->d_prompt_len, ch, PC, c->h_new, c->h.n_heads + 1, c->d_n_new, c->d_len, batch, m.d_model, st));
    if (c->h.prefix_attn) HYDRA_TRY(run_prefix(c, c->h_tree, rs, (ch + 1) * PC, st));
  }
  // root token = argmax of the logits of the last prompt row
  HYDRA_TRY(pick_last_row(c->h_new, c->d_n_new, c->h.n_heads + 1, c->hprime, batch, m.d_model, st));
  HYDRA_TRY(cast_rows(c->hprime, c->yb, ps(c, c->RH, m.d_model), (size_t)batch * m.d_model, m.dtype, st));
  SplitDesc sd;
  HYDRA_TRY(run_gemm(c, c->yb, c->RH, c->lm_head, batch, m.vocab, m.d_model, &sd, st));
  HYDRA_TRY(argmax_rows(c->part, sd, nullptr, c->d_root_tok, c->topk_scratch, c->topk_rows_cap, batch, m.vocab, st));
  for (int b = 0; b < batch; ++b) c->len_ub[b] = plen[b];
  drop_graphs(c);
  c->state = ST_READY;
  return HYDRA_OK;
}

hydra_status hydra_draft(hydra_ctx* c, int32_t* tree_tok, void* stream) {
  if (!c || !tree_tok) return HYDRA_ERR_INVALID;
  if (c->state != ST_READY && c->state != ST_DRAFTED) return HYDRA_ERR_STATE;
  if (!capacity_ok(c)) return HYDRA_ERR_CAPACITY;
  CounterScope cs(c);
  HYDRA_TRY(do_draft(c, tree_tok, (cudaStream_t)stream));
  c->state = ST_DRAFTED;
  return HYDRA_OK;
}

hydra_status hydra_verify(hydra_ctx* c, const int32_t* tree_tok, int32_t* amax, float* logits, void* stream) {
  if (!c || !tree_tok || !amax) return HYDRA_ERR_INVALID;
  if (c->state != ST_READY && c->state != ST_DRAFTED && c->state != ST_VERIFIED) return HYDRA_ERR_STATE;
  if (!capacity_ok(c)) return HYDRA_ERR_CAPACITY;
  CounterScope cs(c);
  HYDRA_TRY(do_verify(c, tree_tok, amax, logits, (cudaStream_t)stream));
  c->state = ST_VERIFIED;
  return HYDRA_OK;
}

hydra_status hydra_accept_compact(hydra_ctx* c, const int32_t* tree_tok, const int32_t* amax, int32_t* n_acc, int32_t* path,
                                  int32_t* out_tok, void* stream) {
  if (!c || !tree_tok || !amax) return HYDRA_ERR_INVALID;
  if (c->state != ST_VERIFIED) return HYDRA_ERR_STATE;
  CounterScope cs(c);
  HYDRA_TRY(do_accept(c, tree_tok, amax, n_acc, path, out_tok, (cudaStream_t)stream));
  bump_len_ub(c);
  c->state = ST_READY;
  return HYDRA_OK;
}

hydra_status hydra_step(hydra_ctx* c, int32_t* n_acc, int32_t* out_tok, void* stream) {
  if (!c) return HYDRA_ERR_INVALID;
  if (c->state != ST_READY) return HYDRA_ERR_STATE;
  if (!capacity_ok(c)) return HYDRA_ERR_CAPACITY;
  CounterScope cs(c);
  cudaStream_t st = (cudaStream_t)stream;
  const bool capturable = st != nullptr && st != cudaStreamLegacy && st != cudaStreamPerThread;   // default streams cannot be captured
  if (!c->use_graph || !capturable || c->timing || c->steps_done == 0) {      // the first step runs uncaptured (one-time lazy set-up)
    HYDRA_TRY(enqueue_step(c, n_acc, out_tok, st));
  } else {
    const int lu = max_len_ub(c);
    hydra_ctx::GraphKey key{len_bucket(c, lu + c->T), len_bucket(c, lu), c->plant, n_acc, out_tok};
    auto it = c->graphs.find(key);
    if (it == c->graphs.end()) {
      if (c->graphs.size() >= 8) drop_graphs(c);
      const long long before = c->launches;
      HYDRA_CUDA(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
      hydra_status es = enqueue_step(c, n_acc, out_tok, st);
      cudaGraph_t graph = nullptr;
      cudaError_t ce = cudaStreamEndCapture(st, &graph);
      const long long captured = c->launches - before;
      c->launches = before;
      if (es != HYDRA_OK) { if (graph) cudaGraphDestroy(graph); return es; }
      if (ce != cudaSuccess) { set_last_error("cudaStreamEndCapture", ce); return HYDRA_ERR_CUDA; }
      cudaGraphExec_t exec = nullptr;
      ce = cudaGraphInstantiate(&exec, graph, 0);
      cudaGraphDestroy(graph);
      if (ce != cudaSuccess) { set_last_error("cudaGraphInstantiate", ce); return HYDRA_ERR_CUDA; }
      it = c->graphs.emplace(key, hydra_ctx::StepGraph{exec, captured}).first;
    }
    HYDRA_CUDA(cudaGraphLaunch(it->second.exec, st));
    c->launches += it->second.launches;
  }
  bump_len_ub(c);
  ++c->steps_done;
  return HYDRA_OK;
}

hydra_status hydra_set_plant(hydra_ctx* c, const int32_t* plant) {
  if (!c) return HYDRA_ERR_INVALID;
  c->plant = plant;
  return HYDRA_OK;
}

hydra_status hydra_set_acceptance(hydra_ctx* c, int mode, float tau, float eps, float alpha, const float* u_dev) {
  if (!c || (mode != 0 && mode != 1)) return HYDRA_ERR_INVALID;
  if (mode == 1 && !(tau > 0.f && eps >= 0.f && alpha >= 0.f)) return HYDRA_ERR_INVALID;
  if (c->state == ST_VERIFIED && mode != c->acc_mode) return HYDRA_ERR_STATE;      // the last verification prepared for the other criterion
  c->acc_mode = mode; c->acc_tau = tau; c->acc_eps = eps; c->acc_alpha = alpha; c->acc_u = mode == 1 ? u_dev : nullptr;
  drop_graphs(c);
  return HYDRA_OK;
}

hydra_status hydra_get_buffer(hydra_ctx* c, int which, void** ptr, size_t* bytes) {
  if (!c || !ptr) return HYDRA_ERR_INVALID;
  const hydra_model_cfg& m = c->m;
  const size_t kvl = kv_layer_elems(m) * c->kv_esize * c->kv_planes;      // bytes of one layer's K (or V) cache, all planes
  const int K = c->h.n_heads;
  void* p = nullptr; size_t n = 0;
  switch (which) {
    case HYDRA_BUF_LEN: p = c->d_len; n = m.max_batch * sizeof(int); break;
    case HYDRA_BUF_ROOT_TOK: p = c->d_root_tok; n = m.max_batch * sizeof(int); break;
    case HYDRA_BUF_H_TREE: p = c->h_tree; n = (size_t)c->R * m.d_model * sizeof(float); break;
    case HYDRA_BUF_H_NEW: p = c->h_new; n = (size_t)m.max_batch * (K + 1) * m.d_model * sizeof(float); break;
    case HYDRA_BUF_KV_BASE: p = c->kv_base; n = (size_t)m.n_layers * 2 * kvl; break;
    case HYDRA_BUF_KV_PREFIX: p = c->h.prefix_attn ? c->kv_pfx : nullptr; n = c->h.prefix_attn ? 2 * kvl : 0; break;
    case HYDRA_BUF_TREE_MASK: p = c->d_anc; n = c->T * sizeof(uint64_t); break;
    case HYDRA_BUF_TREE_TOK: p = c->d_tree_tok; n = (size_t)m.max_batch * c->T * sizeof(int); break;
    case HYDRA_BUF_AMAX: p = c->d_amax; n = (size_t)m.max_batch * c->T * sizeof(int); break;
    case HYDRA_BUF_HEAD_LOGITS: p = c->head_logits; n = (size_t)c->RH * m.vocab * sizeof(float); break;
    case HYDRA_BUF_N_NEW: p = c->d_n_new; n = m.max_batch * sizeof(int); break;
    case HYDRA_BUF_H_PRIME: p = c->hprime; n = (size_t)m.max_batch * m.d_model * sizeof(float); break;
    case HYDRA_BUF_STATUS: p = c->d_status; n = 64 * sizeof(int); break;
    case HYDRA_BUF_PASS_BITS: p = c->d_pass_bits; n = m.max_batch * sizeof(unsigned long long); break;
    default: return HYDRA_ERR_INVALID;
  }
  *ptr = p;
  if (bytes) *bytes = n;
  return HYDRA_OK;
}

hydra_status hydra_poll_status(hydra_ctx* c, void* stream) {
  if (!c) return HYDRA_ERR_INVALID;
  cudaStream_t st = (cudaStream_t)stream;
  int word = 0;
  HYDRA_CUDA(cudaStreamSynchronize(st));
  HYDRA_CUDA(cudaMemcpy(&word, c->d_status, sizeof(int), cudaMemcpyDeviceToHost));
  if (c->batch > 0 && (c->state == ST_READY || c->state == ST_DRAFTED)) {
    // the stream is drained: replace the host's upper bounds of the lengths (which assume every step accepted a
    // full path) by the real ones, so that the capacity check and the attention grids follow the real cache use
    std::vector<int> len(c->batch);
    HYDRA_CUDA(cudaMemcpy(len.data(), c->d_len, c->batch * sizeof(int), cudaMemcpyDeviceToHost));
    for (int b = 0; b < c->batch; ++b) if (len[b] >= 0 && len[b] < c->len_ub[b]) c->len_ub[b] = len[b];
  }
  if (word & ST_TIMEOUT) {
    int d[8] = {0};
    cudaMemcpy(d, c->d_status + 8, sizeof(d), cudaMemcpyDeviceToHost);
    snprintf(g_err, sizeof(g_err), "GEMM wait gave up: site %d cta %d unit %d/%d grid %d m %d n %d kb %d", d[0], d[1], d[2], d[3], d[4], d[5], d[6], d[7]);
  }
  if (word) HYDRA_CUDA(cudaMemset(c->d_status, 0, 64 * sizeof(int)));
  if (word & ST_TIMEOUT) return HYDRA_ERR_TIMEOUT;
  if (word & ST_BOUNDS) return HYDRA_ERR_BOUNDS;
  return HYDRA_OK;
}

long long hydra_launch_count(hydra_ctx* c) { return c ? c->launches : 0; }

hydra_status hydra_set_timing(hydra_ctx* c, int on) {
  if (!c) return HYDRA_ERR_INVALID;
  c->timing = on ? 1 : 0;
  return HYDRA_OK;
}

hydra_status hydra_get_timing(hydra_ctx* c, int kclass, double* ms_total, long long* launches, double* bytes_total) {
  if (!c || kclass < 0 || kclass > HYDRA_TIME_ACCEPT) return HYDRA_ERR_INVALID;
  HYDRA_CUDA(cudaDeviceSynchronize());
  double ms = 0, bytes = 0; long long n = 0;
  std::vector<hydra_ctx::Timed> keep;
  for (auto& t : c->timed) {
    if (t.cls != kclass) { keep.push_back(t); continue; }
    float dt = 0.f;
    HYDRA_CUDA(cudaEventElapsedTime(&dt, t.a, t.b));
    ms += dt; bytes += t.bytes; ++n;
    c->event_pool.push_back({t.a, t.b});
  }
  c->timed.swap(keep);
  if (ms_total) *ms_total = ms;
  if (launches) *launches = n;
  if (bytes_total) *bytes_total = bytes;
  return HYDRA_OK;
}

hydra_status hydra_set_step_graph(hydra_ctx* c, int on) {
  if (!c) return HYDRA_ERR_INVALID;
  c->use_graph = on ? 1 : 0;
  return HYDRA_OK;
}

hydra_status hydra_set_gemm_mode(hydra_ctx* c, int mode) {
  if (!c || mode < 0 || mode > 1) return HYDRA_ERR_INVALID;
  c->gemm_mode = mode;
  drop_graphs(c);
  return HYDRA_OK;
}

const char* hydra_status_str(hydra_status s) {
  switch (s) {
    case HYDRA_OK: return "ok";
    case HYDRA_ERR_INVALID: return "invalid argument";
    case HYDRA_ERR_CAPACITY: return "capacity exceeded";
    case HYDRA_ERR_STATE: return "call out of order";
    case HYDRA_ERR_UNSUPPORTED: return "unsupported shape";
    case HYDRA_ERR_CUDA: return "CUDA error";
    case HYDRA_ERR_TIMEOUT: return "device-side wait timed out";
    case HYDRA_ERR_BOUNDS: return "device-side index out of range";
  }
  return "unknown";
}

const char* hydra_last_error(void) { return g_err; }

size_t hydra_gemm_partial_floats(int m, int n, int k, int dtype, int mode) {
  if (m < 1 || n < 1 || k < 1) return 0;
  if (dtype != 1 || mode != 0 || n % 128 || k % 64) return (size_t)m * n;
  int slots = 1;
  gemm_tc_plan(m, n, k, nullptr, &slots);
  return (size_t)slots * m * n;
}

hydra_status hydra_gemm(const void* x, const void* w, float* out, float* partial, int m, int n, int k, int dtype, int mode,
                        int x_planes, int32_t* status, void* stream) {
  if (!x || !w || !out || !partial || m < 1 || n < 1 || k < 1 || (dtype != 0 && dtype != 1)) return HYDRA_ERR_INVALID;
  if (x_planes != 1 && !(x_planes == 2 && dtype == 1 && mode == 0)) return HYDRA_ERR_INVALID;
  cudaStream_t st = (cudaStream_t)stream;
  CounterScope cs(nullptr);
  if (dtype == 1 && mode == 0) {
    if (!status) return HYDRA_ERR_INVALID;
    if (!gemm_tc_available()) { set_last_error("cuTensorMapEncodeTiled entry point", cudaErrorUnknown); return HYDRA_ERR_CUDA; }
    SplitDesc sd;
    HYDRA_TRY(gemm_tc((const bf16*)x, m, x_planes, (const bf16*)w, partial, m, n, k, &sd, status, nullptr, nullptr, st));
    return reduce_splits(partial, sd, out, m, n, st);
  }
  return gemm_simt(x, w, out, m, n, k, dtype, st);
}

hydra_status hydra_gemm_bounded_wait_probe(const void* x, const void* w, float* partial, int m, int n, int k, int skip_unit,
                                           unsigned wait_limit, int32_t* status, int32_t* diag, void* stream) {
  if (!x || !w || !partial || !status || !diag || m < 1 || n < 1 || k < 1 || wait_limit < 1 || wait_limit > (1u << 16)) return HYDRA_ERR_INVALID;
  int grid = 0;
  gemm_tc_plan(m, n, k, &grid, nullptr);
  if (n % 128 || k % 64 || grid != 1) return HYDRA_ERR_UNSUPPORTED;     // one CTA: nothing else waits on the missing tile
  if (!gemm_tc_available()) { set_last_error("cuTensorMapEncodeTiled entry point", cudaErrorUnknown); return HYDRA_ERR_CUDA; }
  CounterScope cs(nullptr);
  GemmDebug dbg{wait_limit, skip_unit};
  SplitDesc sd;
  return gemm_tc((const bf16*)x, m, 1, (const bf16*)w, partial, m, n, k, &sd, status, diag, &dbg, (cudaStream_t)stream);
}

size_t hydra_attention_scratch_bytes(int batch, int tc, int n_heads, int head_dim, int max_seq) {
  if (batch < 1 || tc < 1 || n_heads < 1 || head_dim < 1 || max_seq < 1) return 0;
  return attention_scratch_bytes(batch, tc, n_heads, head_dim, max_seq);
}

hydra_status hydra_tree_attention(const void* q, const void* kc, const void* vc, const int32_t* pos0, const int32_t* n_rows,
                                  const uint64_t* mask, void* out, void* scratch, int batch, int tc, int n_heads, int head_dim,
                                  int max_seq, int dtype, int planes, int out_planes, int32_t* status, void* stream) {
  if (!q || !kc || !vc || !pos0 || !out || batch < 1 || tc < 1 || n_heads < 1 || max_seq < 1 || (dtype != 0 && dtype != 1)) return HYDRA_ERR_INVALID;
  CounterScope cs(nullptr);
  RowSet rs{batch, tc, n_rows, pos0, nullptr, mask};
  if (dtype == 0) {
    if (!mask || !scratch || out_planes != 1 || planes != 1) return HYDRA_ERR_INVALID;
    return tree_attention_f32((const float*)q, (const float*)kc, (const float*)vc, rs, (float*)out, scratch, n_heads, head_dim, max_seq, max_seq,
                              (cudaStream_t)stream);
  }
  if (!status || (out_planes != 1 && out_planes != 2) || (planes != 1 && planes != 2)) return HYDRA_ERR_INVALID;
  const size_t d = (size_t)n_heads * head_dim;
  return tree_attention_tc((const __half*)q, batch * tc, (const __half*)kc, (const __half*)vc, batch, planes, rs, (bf16*)out,
                           out_planes == 2 ? (size_t)batch * tc * d : 0, n_heads, head_dim, max_seq, max_seq, status, false,
                           (cudaStream_t)stream);
}

}  // extern "C"

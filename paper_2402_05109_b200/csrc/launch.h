// Host-side launchers of every kernel (internal).  Each enqueues on `st` and returns a hydra_status.
#pragma once
#include "common.cuh"

namespace hydra {

// ---- GEMM: partial sums of x[m][k] * w[n][k] (see SplitDesc for where they land)
// tcgen05 path (bfloat16 operands).  x_rows_alloc = rows the x buffer really holds (>= m); rows of the last
// tile beyond m are computed and dropped.  part needs gemm_tc_plan(...)'s max_slots * m * n floats.
// x holds x_planes (1 or 2) planes of x_rows_alloc rows each: plane 0 = bf16(v), plane 1 = bf16(v - plane 0).
// dbg (tests of the bounded waits only): a shorter poll limit and one weight-tile request that CTA 0 leaves out.
struct GemmDebug { uint32_t wait_limit; int skip_unit; };
hydra_status gemm_tc(const bf16* x, int x_rows_alloc, int x_planes, const bf16* w, float* part, int m, int n, int k,
                     SplitDesc* sd_out, int* status, int* diag /*int[8] or null*/, const GemmDebug* dbg /*null: defaults*/, cudaStream_t st);
SplitDesc gemm_tc_plan(int m, int n, int k, int* grid, int* max_slots, int force_nh = 0);   // force_nh: 128-row weight tiles per unit (0: the kernel's own choice)
int gemm_tile_rows(int m);                // activation rows per MMA tile for an m-row GEMM: 16, 32, 64, 128 or 256
bool gemm_tc_available();                 // driver entry point for tensor-map encoding found
// SIMT path (float or bfloat16 operands), single slot.
hydra_status gemm_simt(const void* x, const void* w, float* out, int m, int n, int k, int dtype, cudaStream_t st);
// out[m][n] = sum of the slots of part
hydra_status reduce_splits(const float* part, SplitDesc sd, float* out, int m, int n, cudaStream_t st);

// ---- element-wise / row-wise stages of a decoder layer (dtype: 0 float, 1 bfloat16 for the "act" outputs)
hydra_status embed_rows(const void* embed, const int* tok, float* x, int rows, int d, int vocab, int dtype, int* status,
                        cudaStream_t st);
// x_out = (res ? res : 0) + sum_s part[s]; if gain: xn = rmsnorm(x_out)*gain (act dtype, optional) and hn = the same in
// float (optional).  part may be null.  x_out may alias res.
hydra_status residual_rmsnorm(const float* res, const float* part, SplitDesc sd, float* x_out,
                              const void* gain, void* xn, size_t xn_ps, float* hn, int rows, int d, float eps, int dtype,
                              cudaStream_t st);
// table[r][j] = (cos, sin) of (pos0[b]+depth[i]) * theta^(-2j/head_dim), evaluated in double
hydra_status rope_table(RowSet rs, float2* table, int head_dim, float theta, cudaStream_t st);
// q ([rows][H][hd], rotated) and the K/V cache rows (rotated K) from the QKV partial sums; float for dtype 0; for dtype 1
// float16 with a lo plane (f16(v - f16(v))) q_ps / kv_ps elements after the hi plane (0: hi only).
hydra_status qkv_rope_store(const float* part, SplitDesc sd, const float2* table, void* q, size_t q_ps, void* kcache, void* vcache,
                            size_t kv_ps, RowSet rs, int n_heads, int head_dim, int max_seq, int dtype, int* status, cudaStream_t st);
// Float model path: SIMT kernel + combine kernel, partial rows of ATT_CHUNK_ROWS-row chunks in `scratch`
// (attention_scratch_bytes).  q, caches and out are float.
constexpr int ATT_CHUNK_ROWS = 128;
size_t attention_scratch_bytes(int batch, int tc, int n_heads, int head_dim, int max_seq);
hydra_status tree_attention_f32(const float* q, const float* kcache, const float* vcache, RowSet rs, float* out, void* scratch,
                                int n_heads, int head_dim, int max_seq, int len_upper, cudaStream_t st);
// bfloat16 model path: tensor-core kernel (attention_tc.cu).  q [planes][q_rows][H*hd] and the caches
// [planes][cache_batch][H][max_seq][hd] are float16 in 1 or 2 planes (hi = f16(v), lo = f16(v - hi)); out is bfloat16
// [rows][H*hd] in two planes out_ps elements apart (0: hi only).  rs.mask == null selects a causal chunk (row i sees
// the committed slots and new slots 0..i) of up to 128 rows (one plane, or head_dim 64); with a mask, up to 64 rows.
// stable_lengths: rs.pos0 / rs.n_rows and every cache row below pos0 were written by kernels that had COMPLETED before the
// kernel preceding this one in the stream started (true inside a forward call of the library, whose first kernel holds
// its successors back until everything earlier has completed); the kernel then requests committed cache tiles before it
// waits for its predecessor.
hydra_status tree_attention_tc(const __half* q, int q_rows, const __half* kc, const __half* vc, int cache_batch, int planes, RowSet rs,
                               bf16* out, size_t out_ps, int n_heads, int head_dim, int max_seq, int len_upper, int* status,
                               bool stable_lengths, cudaStream_t st);
hydra_status silu_mul(const float* part, SplitDesc sd, void* act, size_t act_ps, int rows, int f, int dtype,
                      cudaStream_t st);
// amax[r] = argmax_v of the summed partial logits (lowest id among equal maxima); the sums go to logits_out if given
// scratch: topk_scratch_bytes(rows_cap, vocab) bytes of candidate storage
size_t topk_scratch_bytes(int rows, int vocab);
hydra_status argmax_rows(const float* part, SplitDesc sd, float* logits_out, int* amax, void* scratch, int rows_cap, int rows,
                         int vocab, cudaStream_t st);

// ---- Hydra heads
struct LevelDesc {           // one tree level d (1-based): the parents that have children
  int d, n_parents;
  const int* parents;        // device [n_parents] row ids
};
// z[b*P+j] = [hprime[b] ; E[tok[b][path(parent j)]]] in act dtype (lv.d path tokens; lv.d = 0: the hidden state alone);
// with write_root also tree_tok[b][0] = root_tok[b].
hydra_status head_gather(const float* hprime, const void* embed, const int* root_tok, int* tree_tok, const int* path_tab,
                         LevelDesc lv, int write_root, void* z, size_t z_ps, int batch, int T, int kp1, int d_model, int vocab, int dtype,
                         int* status, cudaStream_t st);
// y_out = res + silu(sum_s part[s] + bias); res row = hprime[b] when res_is_hprime else y row.  yb = act-dtype copy.
hydra_status head_act(const float* res, int res_is_hprime, int rows_per_b, const float* part, SplitDesc sd,
                      const void* bias, float* y_out, void* yb, size_t yb_ps, int rows, int d, int dtype, cudaStream_t st);
// children of parent j of sequence b = top n_child tokens of logits row b*P+j, descending (ties: lower id first);
// the logits are the summed partials, also written to `logits` [rows][vocab].  shared_rows: the logits have ONE row per
// sequence (sequentially independent heads) and every parent of the level takes its children from that row.
hydra_status topk_children(const float* part, SplitDesc sd, float* logits, LevelDesc lv, int max_children, const int* first_child,
                           const int* n_child, int* tree_tok, void* scratch, int rows_cap, int batch, int T, int vocab, int shared_rows,
                           cudaStream_t st);

// ---- acceptance + compaction (one kernel)
struct AcceptArgs {
  const int* tree_tok; const int* amax;
  const int* parent; const int* depth; const uint64_t* anc;
  int T, K, batch, n_layers, n_heads, head_dim, max_seq, max_batch, d_model, esize, kv_planes;
  void* kv_base; const float* h_tree; int h_tree_stride;   // h_tree row = b*h_tree_stride + i
  float* h_new; int* n_new; int* len; int* root_tok;
  int* n_acc; int* path; int* out_tok; unsigned int* done_counter; int* status;
  // acceptance criterion: 0 greedy (token == argmax at the parent); 1 typical (probability of the token under the
  // temperature-tau distribution at the parent > min(eps, alpha * exp(-entropy)))
  int mode; float tau, eps, alpha;
  const float* logits;       // [batch*T][vocab] of the last verification (typical mode)
  const float4* row_stats;   // [batch*T] (max logit, sum exp((l - max)/tau), sum exp(.) (l - max)/tau, 0) (typical mode)
  int vocab;
  const float* u;            // [batch] uniform numbers for the token after the accepted path, or null (= its argmax)
  unsigned long long* pass_bits;   // [batch] out: bit i = candidate row i passed the criterion at its parent
  int* bonus_tmp;            // [batch] scratch: the sampled token, handed from CTA 0 of a sequence to the CTA that publishes the state
};
// row_stats[r] for every logits row (typical acceptance)
hydra_status softmax_row_stats(const float* logits, float4* row_stats, int rows, int vocab, float tau, cudaStream_t st);
hydra_status accept_compact(const AcceptArgs& a, cudaStream_t st);

// ---- small state kernels
hydra_status set_chunk(const int* prompt_len, int chunk, int tc, int* pos0, int* n_rows, int batch, cudaStream_t st);
hydra_status gather_chunk_tokens(const int* tokens, const int* offsets, int chunk, int tc, int* tok_out, int batch,
                                 cudaStream_t st);
// for sequences whose last prompt row lies in this chunk: h_new[b][0] = h[b*tc + i], n_new = 1, len = prompt_len
hydra_status capture_last(const float* h, const int* prompt_len, int chunk, int tc, float* h_new, int kp1, int* n_new,
                          int* len, int batch, int d, cudaStream_t st);
// pos0[b] = len[b] - n_new[b]; n_rows[b] = n_new[b]
hydra_status prefix_rowset(const int* len, const int* n_new, int* pos0, int* n_rows, int batch, cudaStream_t st);
// hprime[b] = x[b*tc + n_rows[b]-1]
hydra_status pick_last_row(const float* x, const int* n_rows, int tc, float* hprime, int batch, int d, cudaStream_t st);
hydra_status apply_plant(int* tree_tok, const int* plant, int count, cudaStream_t st);
// dst = src converted to the operand type
hydra_status cast_rows(const float* src, void* dst, size_t dst_ps, size_t count, int dtype, cudaStream_t st);
hydra_status copy_i32(int* dst, const int* src, int count, cudaStream_t st);

}  // namespace hydra

/* hydra.h -- C ABI of libhydra: one Hydra speculative-decode step on one sm_100a GPU.
 *
 * The calls follow the paper's statement of the problem (Hydra: Sequentially-Dependent Draft Heads
 * for Medusa Decoding): a static candidate tree is populated by the draft heads (Background, "Tree
 * decoding"; Section "Hydra Heads", second displayed equation; Section "Hydra++"), verified by one
 * base-model forward in which a token attends only to its ancestors (Background, "Tree decoding"),
 * a prefix is accepted by the greedy criterion (Background, verification criteria) and the rest is
 * discarded (Background, "Speculative decoding").
 *
 * Conventions
 *  - Every call returns a hydra_status; nothing throws, aborts or exits.
 *  - "dev" pointers are device pointers, "host" pointers are host pointers.  All matrices are
 *    row-major [out][in].  dtype 0: weights, KV cache and GEMM operands are float; dtype 1: weights are
 *    bfloat16; activations that feed a GEMM are stored as TWO bfloat16 planes (hi = bf16(v), lo = bf16(v - hi),
 *    about 16 mantissa bits together); the attention operands (q, the post-rotation K cache, the V cache and the
 *    softmax weights) are float16 in two planes (hi = f16(v), lo = f16(v - hi); hydra_model_cfg.kv_planes = 1 keeps
 *    hi only); accumulation, residual stream, norms and softmax stay float.
 *  - The caller owns the weights, the workspace and every in/out buffer and keeps them alive until
 *    hydra_destroy.  The library owns only the opaque context; KV caches, tables and scratch are
 *    carved out of the caller's workspace (hydra_workspace_bytes, 256-byte aligned base).
 *  - Calls enqueue work on `stream` (a cudaStream_t passed as void*) and do not synchronise, except
 *    hydra_create (uploads tables; synchronises the device), hydra_prefill (synchronises the stream once,
 *    after uploading the prompt offsets, before its first kernel), hydra_poll_status, hydra_get_timing and
 *    hydra_destroy.
 *  - Order: create -> prefill -> (draft -> verify -> accept_compact | step)*.  A call out of order
 *    returns HYDRA_ERR_STATE.  The host keeps an upper bound of every sequence length (it grows by
 *    K+1 per step, as if every step accepted a full path); a step whose bound could exceed max_seq returns
 *    HYDRA_ERR_CAPACITY before any launch.  hydra_poll_status replaces the bounds by the real lengths, so a
 *    caller that polls now and then can use the whole cache.
 *  - Device-side problems (token id / slot out of range, a bounded wait that ran out) set a status
 *    word that hydra_poll_status returns; kernels skip the offending access and never trap.
 */
#ifndef HYDRA_H_
#define HYDRA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hydra_ctx hydra_ctx;

typedef enum {
  HYDRA_OK = 0,
  HYDRA_ERR_INVALID = 1,     /* null pointer, non-positive size, malformed tree */
  HYDRA_ERR_CAPACITY = 2,    /* workspace too small, or a sequence could outgrow max_seq */
  HYDRA_ERR_STATE = 3,       /* call out of order */
  HYDRA_ERR_UNSUPPORTED = 4, /* shape outside what the kernels cover */
  HYDRA_ERR_CUDA = 5,        /* a CUDA runtime/driver call failed (see hydra_last_error) */
  HYDRA_ERR_TIMEOUT = 6,     /* a bounded device-side wait ran out */
  HYDRA_ERR_BOUNDS = 7       /* a device-side index check failed */
} hydra_status;

/* Base model: Llama-style decoder (RMSNorm, rotary embedding with half-split pairing, SiLU-gated FFN). */
typedef struct {
  int n_layers, d_model, n_heads, head_dim, d_ffn, vocab;
  float rms_eps, rope_theta;
  int dtype;               /* 0 = float, 1 = bfloat16 */
  int max_batch, max_seq;  /* capacity of the KV caches */
  int kv_planes;           /* dtype 1 only: float16 planes of q and the KV caches.  0 or 2: hi + lo (about 22 bits: hidden states
                              stay within ~1e-4 of a float reference over 60 layers); 1: hi only (half the cache bytes; a few
                              1e-3 over 32 layers, not enough for the deepest shapes) */
} hydra_model_cfg;

/* Draft model: K heads, head i an m-layer residual SiLU MLP over [h ; E[x_t] ; E of the i-1 tokens
 * speculated before it] (Section "Hydra Heads"); prefix_attn adds the extra decoder layer that is
 * queried once per step (Section "Hydra++", "Prefix Attention"). */
typedef struct {
  int n_heads;       /* K */
  int n_mlp_layers;  /* m >= 1 */
  int prefix_attn;   /* 0 | 1 */
  int has_bias;      /* 0 | 1 */
  int medusa;        /* 0: Hydra heads (sequentially dependent).  1: sequentially independent heads, the Medusa baseline
                        (Background, "Lightweight heads as a draft model" / "Medusa decoding"): head i sees the hidden state
                        only, head_w1[i-1] is [d][d], and every parent of a tree level gets the same children */
} hydra_head_cfg;

/* Static candidate tree (Background, "Tree decoding").  parent is a HOST array of n_rows entries:
 * parent[0] = -1 (root = the committed token not yet run through the base model), 0 <= parent[i] < i,
 * rows ordered by (depth, rank path), depth <= K, n_rows <= 64. */
typedef struct {
  int n_rows;
  const int32_t* parent;
} hydra_tree_cfg;

/* Device weight pointers.  Arrays of pointers (attn_norm[l], ...) are HOST arrays of n_layers (or K)
 * DEVICE pointers.  wqkv rows are q, k, v in that order; w_gate_up rows are gate then up. */
typedef struct {
  const void *embed /*[V][d]*/, *lm_head /*[V][d]*/, *final_norm /*[d]*/;
  const void *const *attn_norm /*[d]*/, *const *wqkv /*[3d][d]*/, *const *wo /*[d][d]*/;
  const void *const *ffn_norm /*[d]*/, *const *w_gate_up /*[2f][d]*/, *const *w_down /*[d][f]*/;
  const void *const *head_w1 /*[K] -> [d][(i+1)d], i = 1..K*/, *const *head_b1 /*[K] -> [d]*/;
  const void *const *head_wr /*[K] -> [m-1][d][d]*/, *const *head_br /*[K] -> [m-1][d]*/;
  const void *pfx_attn_norm, *pfx_wqkv, *pfx_wo, *pfx_ffn_norm, *pfx_w_gate_up, *pfx_w_down; /* prefix layer or NULL */
} hydra_weights;

/* Bytes of device workspace hydra_create needs for these configs (0 if they are invalid). */
size_t hydra_workspace_bytes(const hydra_model_cfg*, const hydra_head_cfg*, const hydra_tree_cfg*);

/* Validate the configs, build and upload the tree tables (depth, ancestor bitmask, paths, levels),
 * carve the workspace (256-byte aligned; it is cleared by this call).  Synchronises the whole device before
 * and after, so the workspace may be memory that earlier work on any stream was still using. */
hydra_status hydra_create(hydra_ctx** out, const hydra_model_cfg*, const hydra_head_cfg*, const hydra_tree_cfg*,
                          const hydra_weights*, void* workspace_dev, size_t workspace_bytes);
hydra_status hydra_destroy(hydra_ctx*);

/* Set-up of speculative decoding (Background, "Speculative decoding": the base model has processed the
 * sequence so far and proposes the next token).  Base-model forward over the prompts (ordinary causal
 * attention) filling the KV caches, and, with prefix_attn, the extra layer's cache (Section "Hydra++",
 * "Prefix Attention"); leaves, per sequence, the committed length, the root token (argmax after the last
 * prompt token) and the last hidden state.  tokens_dev holds the prompts back to back; seq_offsets_host
 * has batch+1 entries (read before the call returns).  The prompts are processed in passes of 128 rows per sequence
 * (dtype 1) or 64 (dtype 0), every pass streaming the weights once.  Synchronises the stream once (see Conventions).
 * Errors: INVALID (null pointer, batch outside 1..max_batch, empty prompt), CAPACITY (prompt + tree rows
 * exceed max_seq). */
hydra_status hydra_prefill(hydra_ctx*, int batch, const int32_t* tokens_dev, const int32_t* seq_offsets_host,
                           void* stream);

/* Drafting (Section "Hydra Heads", second displayed equation: head i sees the last hidden state and the
 * tokens speculated before it; Section "Hydra++": deeper MLPs and the extra decoder layer queried once per
 * step; Background, "Tree decoding": children of a node = the top tokens of its head in descending order).
 * Populates the candidate tree level by level; ties: lower token id first.  tree_tok_dev [batch][n_rows]
 * int32 out, row 0 = root.  Errors: STATE, CAPACITY. */
hydra_status hydra_draft(hydra_ctx*, int32_t* tree_tok_dev, void* stream);

/* Verification (Background, "Tree decoding": all candidates packed into one input, a token attends only
 * to its ancestors).  One base forward over all tree rows of all sequences with the ancestor mask; K,V of
 * row i land in cache slot len+i, its rotary position is len+depth(i).  amax_dev [batch][n_rows] int32 out:
 * argmax of each row's logits (ties: lowest id).  logits_dev [batch][n_rows][vocab] float out, or NULL.
 * tree_tok_dev [batch][n_rows] int32 in; the caller may have edited it since hydra_draft.  A token id outside
 * [0, vocab) raises the BOUNDS bit of the status word (the row is computed for token 0).  Errors: STATE, CAPACITY. */
hydra_status hydra_verify(hydra_ctx*, const int32_t* tree_tok_dev, int32_t* amax_dev, float* logits_dev, void* stream);

/* Acceptance and compaction (Background, verification criteria: the greedy criterion keeps a candidate
 * that equals the base model's most likely token; Background, "Speculative decoding": the accepted tokens
 * are appended to the sequence, the rest is discarded).  One kernel.  A candidate is accepted when it
 * equals amax of its parent and its parent is accepted; the deepest accepted row wins (lowest row
 * among equals); the accepted rows' K,V move to cache slots len+1..len+n in place.  n_acc_dev [batch]: accepted candidates (0..K); path_dev [batch][K+1]: accepted rows
 * root..best, -1 padded; out_tok_dev [batch][K+1]: accepted tokens then the bonus token, -1 padded.
 * Any of the three outputs may be NULL.  Updates the committed lengths, root tokens and hidden rows. */
hydra_status hydra_accept_compact(hydra_ctx*, const int32_t* tree_tok_dev, const int32_t* amax_dev,
                                  int32_t* n_acc_dev, int32_t* path_dev, int32_t* out_tok_dev, void* stream);

/* One whole decoding step (the three passages above): draft + (optional planting) + verify + accept_compact
 * on the library's own buffers.  n_acc_dev [batch], out_tok_dev [batch][K+1] as in hydra_accept_compact (either
 * may be NULL).  From the second step after a prefill on, the step is captured into a CUDA graph (re-captured
 * when an attention grid must grow or a pointer argument changes) and replayed with one launch, unless the stream
 * is a default stream (not capturable) or hydra_set_step_graph switched graphs off.  Errors: STATE, CAPACITY. */
hydra_status hydra_step(hydra_ctx*, int32_t* n_acc_dev, int32_t* out_tok_dev, void* stream);
/* on = 0: hydra_step launches kernel by kernel (for profilers that list kernels); on = 1 (default): graph replay. */
hydra_status hydra_set_step_graph(hydra_ctx*, int on);

/* Acceptance criterion.  mode 0 (default): greedy, as described at hydra_accept_compact.  mode 1: typical acceptance
 * (Section "Typical acceptance sampling", paragraph "Typical acceptance criterion"): with p = softmax(logits / tau) of the
 * base model at a candidate's parent row and H the entropy of p, the candidate passes when
 * p[token] > min(eps, alpha * exp(-H)) (eps: posterior threshold, alpha: posterior alpha; the paper uses tau = 0.7,
 * eps in 0.05..0.25, alpha = sqrt(eps)); it is accepted when it passes and its parent is accepted; the deepest accepted
 * row wins, lowest row among equals, and the cache is compacted as in the greedy case.  The token after the accepted
 * path is drawn from p at the best row by inverse CDF in token-id order with the uniform number u_dev[b] in [0, 1)
 * (u_dev: DEVICE float [max_batch], read by every acceptance until replaced; the caller draws the numbers), or is that
 * row's most likely token when u_dev is NULL.  In mode 1 hydra_verify also writes every row's logits (to logits_dev,
 * or to a library buffer when that is NULL) and their softmax statistics, which hydra_accept_compact then reads; amax_dev
 * is still needed (the most likely token).  Errors: INVALID (mode, tau <= 0, negative eps / alpha); STATE (changing the
 * mode between a verification and its acceptance). */
hydra_status hydra_set_acceptance(hydra_ctx*, int mode, float tau, float eps, float alpha, const float* u_dev);

/* Accept-exercise mode: plant_dev [batch][n_rows], -1 keeps the drafted token; applied between draft
 * and verify inside hydra_step.  NULL disables.  The buffer is read at every step. */
hydra_status hydra_set_plant(hydra_ctx*, const int32_t* plant_dev);

/* Introspection for parity tests: device pointers into library buffers, valid until destroy. */
enum {
  HYDRA_BUF_LEN = 0,        /* int32 [max_batch] committed lengths */
  HYDRA_BUF_ROOT_TOK = 1,   /* int32 [max_batch] */
  HYDRA_BUF_H_TREE = 2,     /* float [batch*n_rows][d] post-final-norm hidden of the last verify */
  HYDRA_BUF_H_NEW = 3,      /* float [max_batch][K+1][d] hidden rows committed by the last step */
  HYDRA_BUF_KV_BASE = 4,    /* [n_layers][k,v][planes][max_batch][n_heads][max_seq][head_dim]; float, planes = 1 for dtype 0;
                               float16, planes = kv_planes (hi, lo) for dtype 1 */
  HYDRA_BUF_KV_PREFIX = 5,  /* [k,v][planes][max_batch][n_heads][max_seq][head_dim], same element type */
  HYDRA_BUF_TREE_MASK = 6,  /* uint64 [n_rows] ancestor-or-self bitmask */
  HYDRA_BUF_TREE_TOK = 7,   /* int32 [batch][n_rows] tokens of the last hydra_step */
  HYDRA_BUF_AMAX = 8,       /* int32 [batch][n_rows] */
  HYDRA_BUF_HEAD_LOGITS = 9,/* float [rows][vocab] logits of the last drafted level, row = b*parents+j */
  HYDRA_BUF_N_NEW = 10,     /* int32 [max_batch] rows in H_NEW */
  HYDRA_BUF_H_PRIME = 11,   /* float [max_batch][d] hidden state the heads consumed */
  HYDRA_BUF_STATUS = 12,    /* int32 [64]: [0] the device status word (bit 1 bounds, bit 2 timeout) that hydra_poll_status
                               reads and clears, [8..15] where a bounded wait gave up (site, cta, unit, units, grid, m, n, k-blocks) */
  HYDRA_BUF_PASS_BITS = 13  /* uint64 [max_batch]: bit i = candidate row i passed the acceptance criterion at its parent in the
                               last hydra_accept_compact (greedy: equals the parent's argmax; typical: the inequality) */
};
hydra_status hydra_get_buffer(hydra_ctx*, int which, void** dev_ptr, size_t* bytes);

/* Synchronises the stream and returns (and clears) the device status word as a hydra_status. */
hydra_status hydra_poll_status(hydra_ctx*, void* stream);

/* Number of kernels the library has launched for this context since create. */
long long hydra_launch_count(hydra_ctx*);

/* Per-kernel-class device timing for benchmarks.  While on, every launch of a class is bracketed by a pair
 * of CUDA events on the call's stream (this separates back-to-back kernels, so whole-step times taken
 * with timing on are slightly longer).  hydra_get_timing synchronises the device, returns the summed
 * event time (ms), the number of bracketed launches and, for GEMMs, their summed algorithmic bytes
 * (weight matrix + activation slab read once, output written once), then forgets those records. */
enum { HYDRA_TIME_GEMM = 0, HYDRA_TIME_ATTENTION = 1, HYDRA_TIME_ACCEPT = 2 };
hydra_status hydra_set_timing(hydra_ctx*, int on);
hydra_status hydra_get_timing(hydra_ctx*, int kclass, double* ms_total, long long* launches, double* bytes_total);

/* Which GEMM the bfloat16 path uses: 0 = tcgen05/TMA (default); 1 = the plain SIMT kernel (debugging; it reads
 * only the hi plane of the activations). */
hydra_status hydra_set_gemm_mode(hydra_ctx*, int mode);

const char* hydra_status_str(hydra_status);
const char* hydra_last_error(void); /* text of the last CUDA error seen by this thread, "" if none */

/* Single-kernel entry points for kernel-level parity tests.  No context; the library makes its own
 * tensor maps.  All pointers are device pointers.
 * hydra_gemm: out[m][n] = sum_k x[m][k] * w[n][k] (float accumulate, float out), dtype as above;
 *   n % 128 == 0 and k % 64 == 0 for mode 0.  x_planes = 1: x is [m][k]; x_planes = 2 (dtype 1, mode 0 only): x is
 *   [2][m][k], the hi and lo bfloat16 planes of the activations, and the product uses both.  partial_dev needs
 *   hydra_gemm_partial_floats(m, n, k, dtype, mode) floats: the tensor-core GEMM leaves per-CTA partial sums
 *   there, which a second kernel adds in fixed order.  mode as in hydra_set_gemm_mode; status_dev is an int32
 *   status word (bit 1 bounds, bit 2 timeout).
 * hydra_tree_attention (Background, "Tree decoding": a token attends only to its ancestors): q [planes][rows][n_heads][head_dim]
 *   (rows = batch*tc), caches [planes][batch][n_heads][max_seq][head_dim], pos0 [batch] committed lengths, n_rows [batch] or
 *   NULL (= tc), mask [tc] ancestor bitmasks.  Row i of sequence b sees slots < pos0[b] and slot pos0[b]+j when bit j
 *   of mask[i] is set; mask NULL (dtype 1 only) means a causal chunk: slot pos0[b]+j is visible when j <= i.
 *   dtype 0: q, caches and out [rows][n_heads*head_dim] are float, tc <= 64, scratch_dev needs
 *   hydra_attention_scratch_bytes(...) bytes, planes = out_planes = 1, status_dev unused.  dtype 1: q and the caches are
 *   float16 in `planes` planes (2: hi = f16(v), lo = f16(v - hi)), out is bfloat16 [out_planes][rows][n_heads*head_dim]
 *   (2: hi = bf16(v) and lo = bf16(v - hi)); tc <= 64 with a mask, <= 128 causal (two planes at head_dim 128: computed as launches of 64 rows each, the rows of
 *   an earlier launch being cache rows to a later one, so the K and V rows of the whole chunk must be in the caches); scratch_dev unused (may be NULL); status_dev is an int32 status word (bit 2: a bounded wait ran out). */
size_t hydra_gemm_partial_floats(int m, int n, int k, int dtype, int mode);
hydra_status hydra_gemm(const void* x_dev, const void* w_dev, float* out_dev, float* partial_dev, int m, int n, int k,
                        int dtype, int mode, int x_planes, int32_t* status_dev, void* stream);
/* hydra_gemm_noalloc: the bfloat16 tensor-core GEMM of hydra_gemm (dtype 1, mode 0, x_planes 1) for callers that
 * may not allocate device memory.  (The paper has no counterpart; this is a convenience of the library.)
 * Serving loops that must stay clear of the allocator's locks and implicit synchronisation, plugins living
 * inside a host's fixed memory budget, and processes whose free memory already belongs to a pool cannot
 * supply hydra_gemm's partial_dev buffer; here the partial sums live in an 8 MiB array that is part of the
 * library image (every GPU that loads the library holds it until the process exits).
 *   - x [m][k], w [n][k] bfloat16, out [m][n] float, status_dev as in hydra_gemm: all caller-owned device
 *     memory; n % 128 == 0, k % 64 == 0.
 *   - hydra_gemm_partial_floats(m, n, k, 1, 0) * 4 bytes must fit in the 8 MiB array, otherwise HYDRA_ERR_CAPACITY (text in
 *     hydra_last_error) and nothing is launched.
 *   - The call allocates nothing on the device.  The first call on each device looks up the array's device
 *     address (cudaGetSymbolAddress, with that device current); make that first call outside any stream
 *     capture.
 *   - All calls on a GPU share the one array and it keeps the previous call's partial sums; the GEMM
 *     overwrites every element it later reads, so no clearing is needed, but two calls whose kernels overlap
 *     on the GPU (different streams, different threads) race on it: serialise them. */
hydra_status hydra_gemm_noalloc(const void* x_dev, const void* w_dev, float* out_dev, int m, int n, int k,
                                int32_t* status_dev, void* stream);
/* hydra_gemm_bounded_wait_probe: exercises the give-up path of the tensor-core GEMM's bounded waits.  Runs the
 * GEMM of hydra_gemm (dtype 1, mode 0, x_planes 1) on a problem small enough for ONE CTA (else UNSUPPORTED), with
 * barrier waits limited to wait_limit polls (1..65536) and with the weight-tile request of k-block `skip_unit` left
 * out, so the tensor-core lane's wait for that tile runs out: the kernel raises the TIMEOUT bit (2) in status_dev[0],
 * records where it gave up in diag_dev (int32[8]: site, cta, unit, units, grid, m, n, k-blocks; site 3 = weight tile),
 * lets its copies land, frees its tensor memory and returns; nothing faults and the context stays usable.
 * partial_dev as in hydra_gemm; its contents are unspecified afterwards. */
hydra_status hydra_gemm_bounded_wait_probe(const void* x_dev, const void* w_dev, float* partial_dev, int m, int n, int k,
                                           int skip_unit, unsigned wait_limit, int32_t* status_dev, int32_t* diag_dev,
                                           void* stream);
size_t hydra_attention_scratch_bytes(int batch, int tc, int n_heads, int head_dim, int max_seq);
hydra_status hydra_tree_attention(const void* q_dev, const void* k_cache_dev, const void* v_cache_dev,
                                  const int32_t* pos0_dev, const int32_t* n_rows_dev, const uint64_t* mask_dev,
                                  void* out_dev, void* scratch_dev, int batch, int tc, int n_heads, int head_dim,
                                  int max_seq, int dtype, int planes, int out_planes, int32_t* status_dev, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HYDRA_H_ */

/*
 * specvlm.h -- C ABI of the B200 (sm_100a) hot path of SpecVLM's pruned-draft speculative
 * decoding step (arXiv 2508.16201).
 *
 * One speculative step of the paper runs, in this order:
 *   specvlm_stage1_scores   token rating A from the verifier's language-to-video attention
 *   specvlm_select          Stage I retention (top-k of A) + Stage II spatially uniform reduction
 *   specvlm_gather_kv       compaction of the surviving video tokens' K/V into the draft cache
 *   specvlm_draft_decode_attn   (gamma times) draft decode attention over the pruned cache
 *   specvlm_verify_attn     (gamma+1)-query causal verification attention over the full cache
 *   specvlm_accept          greedy acceptance length and next token
 *
 * Conventions (all entry points)
 *   - Return value: SPECVLM_OK (0) or a negative specvlm_status code.  Argument errors are
 *     detected on the host and nothing is launched.
 *   - Pointers marked "device" are device memory owned by the caller; pointers marked "host"
 *     are ordinary host memory read during the call.  Unless an entry point says otherwise the
 *     library allocates nothing and keeps no state between calls.
 *   - Work is enqueued on the CUDA stream passed as `stream` (a cudaStream_t cast to void*;
 *     NULL = the legacy default stream).  No call synchronises the host with the device.
 *   - `d_status` (device int32_t*, optional): a kernel that gives up a bounded wait stores
 *     SPECVLM_ERR_TIMEOUT there and returns.  A kernel that finds device-side data it would have
 *     to turn into an address out of range (a kept index, a block-table entry, a tree-path node,
 *     a sequence length) skips that access and stores SPECVLM_ERR_INVALID_ARG.  It is never
 *     written otherwise; the caller zeroes it and reads it when convenient.
 *   - Scratch memory comes from the caller: `ws` (device, 256-byte aligned) of at least the
 *     size the matching *_workspace_bytes query returns.  Its contents need not be initialised
 *     and are unspecified afterwards.  Calls that share a workspace must not overlap on the GPU.
 *   - bf16 = 2-byte bfloat16.  "Token row" = head_dim consecutive bf16 values.
 */
#ifndef SPECVLM_H_
#define SPECVLM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum specvlm_status {
  SPECVLM_OK = 0,
  SPECVLM_ERR_INVALID_ARG = -1,       /* null pointer, negative size, inconsistent arguments   */
  SPECVLM_ERR_UNSUPPORTED_SHAPE = -2, /* a shape outside the documented supported set          */
  SPECVLM_ERR_WORKSPACE_TOO_SMALL = -3,
  SPECVLM_ERR_CUDA = -4,              /* a CUDA runtime / driver call failed                   */
  SPECVLM_ERR_TIMEOUT = -5,           /* device-side bounded wait expired (via d_status only)  */
  SPECVLM_ERR_TOO_LARGE = -6          /* problem exceeds the fixed capacity of a no-allocation call */
} specvlm_status;

/*
 * A K/V cache, contiguous or paged (the caches of Section 3.1 of the paper: the draft's pruned
 * cache and the target's full cache).  Token p of sequence b lives in logical block
 * p / block_tokens at offset p % block_tokens; the physical block is block_table[b][logical]
 * when block_table is non-NULL, else block b itself (then block_tokens >= max_seq_len, i.e. one
 * block per sequence = a contiguous cache).  The element (layer l, physical block n, KV head g,
 * offset t, channel c) is at
 *     k[l*stride_layer + n*stride_block + g*stride_head + t*stride_token + c]      (bf16 units).
 * Requirements: head_dim in {64, 128}; every stride a multiple of 8 elements (16 bytes);
 * k and v 16-byte aligned; with a block table, block_tokens a multiple of 64.
 * The struct itself is host memory; k, v, block_table, seq_lens are device pointers.
 */
typedef struct specvlm_kv {
  void* k;
  void* v;
  int64_t stride_layer, stride_block, stride_head, stride_token;
  int32_t n_layers, n_kv_heads, head_dim;
  int32_t block_tokens;         /* tokens per block                                          */
  int32_t n_blocks;             /* blocks in the pool (paged) / sequences (contiguous)       */
  int32_t max_blocks;           /* row length of block_table                                 */
  const int32_t* block_table;   /* device [batch][max_blocks] or NULL                        */
  const int32_t* seq_lens;      /* device [batch]: valid tokens per sequence                 */
  int32_t max_seq_len;          /* host-side upper bound on seq_lens (sizes the launch)      */
} specvlm_kv_t;

const char* specvlm_version(void);
const char* specvlm_status_string(int32_t status);

/* ---------------------------------------------------------------------------------------------
 * Step 1a -- token rating (Section 4.1, Eq. 4-5).
 * For every verifier layer l, query head h and language query i, the full causal softmax row
 * over the keys 0..p_i (p_i = absolute position of query i) is formed with logits
 * sm_scale * <q, K>; G_{i,j} is its value at video token j (Eq. 4); the score of video token j is
 * the mean of G_{i,j} over the language queries (Eq. 5) and over all layers and query heads.
 *
 *   target_kv   host struct; K of the verifier (V is not read).  All layers are used.
 *   q_text      device bf16 [n_layers][sum_text][n_q_heads][head_dim], language queries of all
 *               sequences concatenated (sequence b owns rows text_cu[b] .. text_cu[b+1]-1)
 *   text_cu     host int32 [batch+1]
 *   text_start  host int32 [batch]: absolute position of sequence b's first language query; its
 *               i-th query is at text_start[b]+i and sees keys 0 .. text_start[b]+i
 *   video_start, video_len   host int32 [batch]; video_start+video_len <= text_start
 *   video_cu    host int32 [batch+1]: offsets of each sequence's scores in `scores`
 *   scores      device fp32 [video_cu[batch]] out
 *   row_lse_or_null  device fp32 [n_layers][sum_text][n_q_heads] or NULL: the natural-log
 *               sum-exp of each language query's scaled causal logits.  An attention kernel that ran
 *               the prefill usually has it; when NULL it is computed first (one more pass over QK^T),
 *               exactly as specvlm_stage1_row_lse would.
 *   ws          device scratch, specvlm_stage1_scores_workspace_bytes(...)
 * Deterministic: the reduction order over rows, heads and layers is fixed.
 * Supported: head_dim 128 or 64, n_q_heads / n_kv_heads in 1..16, batch <= 64.
 *
 * specvlm_stage1_row_lse is the first half on its own: it writes row_lse (same layout) and
 * needs no scratch.
 */
size_t specvlm_stage1_scores_workspace_bytes(const specvlm_kv_t* target_kv, const int32_t* text_cu,
                                             const int32_t* video_len, int32_t batch,
                                             int32_t n_q_heads);
int32_t specvlm_stage1_row_lse(const specvlm_kv_t* target_kv, const void* q_text,
                               const int32_t* text_cu, const int32_t* text_start, int32_t batch,
                               int32_t n_q_heads, float sm_scale, float* row_lse, int32_t* d_status,
                               void* stream);
int32_t specvlm_stage1_scores(const specvlm_kv_t* target_kv, const void* q_text,
                              const int32_t* text_cu, const int32_t* text_start,
                              const int32_t* video_start, const int32_t* video_len,
                              const int32_t* video_cu, int32_t batch, int32_t n_q_heads,
                              float sm_scale, const float* row_lse_or_null, float* scores, void* ws,
                              size_t ws_bytes, int32_t* d_status, void* stream);
/*
 * The same rating, a range of layers at a time (Eq. 5 averages over the layers, so their
 * contributions can be gathered as the verifier's prefill produces them, or as their queries arrive
 * from the host).  All arguments describe the whole problem, exactly as for specvlm_stage1_scores
 * (target_kv and q_text cover all n_layers layers); this call rates layers layer_begin ..
 * layer_end-1 and leaves each layer's unnormalised column sums in `ws`.  With finish != 0 it then
 * adds up the sums of ALL layers, in layer order, and writes `scores`: the result is bit-identical to
 * one call of specvlm_stage1_scores, provided every layer has been rated by some earlier call (or
 * this one) with the same `ws`, whose contents must be left alone in between.  An empty range with
 * finish != 0 only reduces.  row_lse_or_null, when given, is the full [n_layers][sum_text][n_q_heads]
 * array; only the range's rows are read.
 */
int32_t specvlm_stage1_scores_layers(const specvlm_kv_t* target_kv, const void* q_text,
                                     const int32_t* text_cu, const int32_t* text_start,
                                     const int32_t* video_start, const int32_t* video_len,
                                     const int32_t* video_cu, int32_t batch, int32_t n_q_heads,
                                     float sm_scale, const float* row_lse_or_null, float* scores, void* ws,
                                     size_t ws_bytes, int32_t layer_begin, int32_t layer_end, int32_t finish,
                                     int32_t* d_status, void* stream);

/*
 * Where a rating call leaves its per-layer sums (Eq. 5 before the average over layers): after
 * specvlm_stage1_scores, or after the specvlm_stage1_scores_layers calls that rated a layer, the
 * workspace holds, at the byte offset this query returns, fp32 [n_layers][video_cu[batch]]:
 * entry (l, j) is the softmax probability that layer l puts on video token j, summed over all
 * query heads and over the language queries of j's sequence (a fixed summation order).
 * scores[j] = sum_l entry(l, j) / (n_layers * n_q_heads * n_text of the sequence).  Lets a caller
 * inspect or re-weight single layers.  Returns 0 for invalid arguments.
 */
size_t specvlm_stage1_scores_layer_sums_offset(const specvlm_kv_t* target_kv, const int32_t* text_cu,
                                               int32_t batch, int32_t n_q_heads);

/* ---------------------------------------------------------------------------------------------
 * Steps 1b + 2 -- two-stage selection (Section 4.2).
 * Stage I keeps the k_stage1[b] highest-scored video tokens V_R (ranking "sort A, add in order"
 * of the paragraph before Eq. 6; order key: score descending, index ascending, compared on the
 * fp32 bit patterns; scores must be finite and >= 0).  Stage II keeps, from V \ V_R, tokens at a
 * fixed interval (Eq. 7) with budget n_U = k_total[b] - k_stage1[b] so that the final set has
 * exactly k_total[b] tokens: frame f's remaining tokens (raster order, c_f of them, C_f before
 * it, m in total) get the quota floor(C_{f+1} n_U / m) - floor(C_f n_U / m) and the picks are
 * the remaining tokens of rank floor(t c_f / n_f), t = 0..n_f-1.
 *
 *   scores      device fp32, sequence b at video_cu[b] .. ; length n_frames[b]*tokens_per_frame
 *   video_cu, n_frames, k_stage1, k_total, kept_cu    host int32 arrays ([batch+1] for *_cu)
 *   kept_idx    device int32 out: sequence b's kept video indices (sequence-local, ascending) at
 *               kept_cu[b] .. kept_cu[b]+k_total[b]-1
 * Requires 0 <= k_stage1 <= k_total <= n_video <= 57344 per sequence, n_frames <= 1024.
 * Uses no scratch memory.  d_status is accepted for uniformity and never written: the kernel has
 * no bounded wait, and everything that becomes an address is host data checked before the launch.
 */
int32_t specvlm_select(const float* scores, const int32_t* video_cu, const int32_t* n_frames,
                       int32_t tokens_per_frame, const int32_t* k_stage1, const int32_t* k_total,
                       const int32_t* kept_cu, int32_t batch, int32_t* kept_idx, int32_t* d_status,
                       void* stream);

/*
 * The same selection with the Stage-I count chosen by the paper's Top-P rule (Section 4.2, Eq. 6):
 * V_R is the shortest prefix of the ranking (score descending, index ascending) whose cumulative
 * score reaches lambda_r times the sum of all scores; the paper uses lambda_r = 0.4 and 0.5.  The
 * count is bounded by k_total[b] (Stage II then adds nothing); otherwise Stage II fills the rest
 * of the budget exactly as in specvlm_select.
 *   lambda_permille   host int32 [batch]: lambda_r in thousandths, 0..1000
 *   k_stage1_out_or_null   device int32 [batch] out: the Stage-I count of each sequence
 * The cumulative comparison runs in integers so that the count is a function of the scores alone,
 * not of a summation order: each score is truncated to a multiple of 2^-36 (values above 1 count
 * as 1) and  1000 * sum_{i<c} q_(i) >= lambda_permille * sum q  is evaluated exactly.
 * Other arguments, requirements and errors as for specvlm_select.
 */
int32_t specvlm_select_top_p(const float* scores, const int32_t* video_cu, const int32_t* n_frames,
                             int32_t tokens_per_frame, const int32_t* lambda_permille,
                             const int32_t* k_total, const int32_t* kept_cu, int32_t batch,
                             int32_t* kept_idx, int32_t* k_stage1_out_or_null, int32_t* d_status,
                             void* stream);

/*
 * Attention-agnostic selectors the paper compares its method with (random token pruning in the
 * sensitivity study of Section 3.2; a window over the front, middle or end of the video tokens
 * and full-frame dropping at regular temporal intervals in the ablations).  Uniform-only and
 * attention-only pruning are specvlm_select with k_stage1 = 0 and k_stage1 = k_total.
 *   WINDOW_*  the k_total consecutive tokens at the front / centred ((n_video - k_total) / 2) / end
 *   FRAMES    floor(k_total / tokens_per_frame) whole frames, the i-th of n being frame floor(i F / n)
 *   RANDOM    the k_total tokens with the largest keys, the key of token j of sequence b being the top
 *             24 bits of the first word of Philox-4x32-10 at counter (j, b, 0, 0) under the 64-bit
 *             seed; equal keys go to the lower index
 *   kept_idx  device int32 out, ascending, sequence b at kept_cu[b]
 *   kept_n_out_or_null  device int32 [batch] out: indices written (k_total, less for FRAMES)
 * Arguments as in specvlm_select; n_video <= 57344 per sequence for RANDOM.
 */
typedef enum specvlm_selector {
  SPECVLM_SEL_WINDOW_FRONT = 0,
  SPECVLM_SEL_WINDOW_MIDDLE = 1,
  SPECVLM_SEL_WINDOW_END = 2,
  SPECVLM_SEL_FRAMES = 3,
  SPECVLM_SEL_RANDOM = 4
} specvlm_selector;
int32_t specvlm_select_baseline(int32_t mode, uint64_t seed, const int32_t* n_frames,
                                int32_t tokens_per_frame, const int32_t* k_total, const int32_t* kept_cu,
                                int32_t batch, int32_t* kept_idx, int32_t* kept_n_out_or_null, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Step 3 -- pruned draft context (end of Section 4.2: the draft sees V_R u V_U and the language
 * prompt, its cache reduced to 1-r of the original).
 * For every layer and KV head, copies the token rows
 *   [0, video_start)  ++  video_start + kept_idx[...]  ++  [video_start+video_len, src seq_len)
 * of sequence b from `src` to positions 0,1,2,... of sequence b in `dst`, K and V alike, bit for
 * bit.  The caller sets dst->seq_lens (= src length - video_len + kept count) itself.
 *   src, dst    host structs with the same n_layers, n_kv_heads, head_dim; either may be paged
 *   kept_idx    device int32 (as written by specvlm_select); kept_cu, video_start, video_len,
 *               src_len host int32 ([batch+1] / [batch]); src_len[b] = tokens of sequence b in src
 * Device-side range checks: a kept index outside [0, video_len[b]) or a block-table entry outside
 * [0, n_blocks) of its cache makes the kernel skip that row (nothing is read or written for it)
 * and store SPECVLM_ERR_INVALID_ARG to d_status.
 */
int32_t specvlm_gather_kv(const specvlm_kv_t* src, const int32_t* kept_idx, const int32_t* kept_cu,
                          const int32_t* video_start, const int32_t* video_len,
                          const int32_t* src_len, int32_t batch, const specvlm_kv_t* dst,
                          int32_t* d_status, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Steps 4a / 4b -- attention (Section 3.1: each draft step streams the draft's whole KV cache;
 * the target verifies the gamma drafted tokens in one memory-bound pass).
 *   o[l][b][t][h] = softmax_k( sm_scale * <q[l][b][t][h], K[l][b][g(h)][k]> ) V[l][b][g(h)][k]
 * with g(h) = h / (n_q_heads / n_kv_heads).  The cache already contains the K/V of the n_q new
 * tokens at its end (kv->seq_lens counts them); query t sees keys 0 .. seq_len - n_q + t.
 * specvlm_draft_decode_attn is the n_q = 1 case, specvlm_verify_attn has n_q = gamma + 1.
 *
 *   q, out      device bf16 [n_layers][batch][n_q][n_q_heads][head_dim]
 *   lse_or_null device fp32 [n_layers][batch][n_q][n_q_heads]: natural-log sum-exp of the logits
 *   ws          device scratch, specvlm_attn_workspace_bytes(kv, batch, n_q_heads, gamma)
 * fp32 softmax and accumulation; probabilities are rounded to bf16 before the PV product.
 * Stream order: the decode kernel (windows of at most 16 rows) is launched with programmatic stream
 * serialization; it may begin while the kernel before it on the stream is still running, and
 * touches no global memory until that kernel's writes are complete and visible.
 * Supported: head_dim 64/128; group = n_q_heads/n_kv_heads in 1..16; 0 <= gamma <= 8;
 * batch <= 127 when group * (gamma+1) > 16.  A window of more than 128 rows (group * (gamma+1))
 * is cut into parts of at most 128 rows that run side by side in one launch, so that the cache
 * still comes from HBM once (the later readers of a tile find it in the L2 cache).
 */
size_t specvlm_attn_workspace_bytes(const specvlm_kv_t* kv, int32_t batch, int32_t n_q_heads,
                                    int32_t gamma);
int32_t specvlm_draft_decode_attn(const specvlm_kv_t* kv, const void* q, int32_t batch,
                                  int32_t n_q_heads, float sm_scale, void* out, float* lse_or_null,
                                  void* ws, size_t ws_bytes, int32_t* d_status, void* stream);
int32_t specvlm_verify_attn(const specvlm_kv_t* kv, const void* q, int32_t batch,
                            int32_t n_q_heads, int32_t gamma, float sm_scale, void* out,
                            float* lse_or_null, void* ws, size_t ws_bytes, int32_t* d_status,
                            void* stream);

/* ---------------------------------------------------------------------------------------------
 * Step 4c -- greedy acceptance (Section 3.1 and the experimental set-up: the target decodes
 * greedily and speculative decoding is lossless).
 *   g[b][t] = argmax_v target_logits[b][t][v]   (lowest index among equal maxima)
 *   accept_len[b] = number of leading positions t < gamma with draft_tokens[b][t] == g[b][t]
 *   next_token[b] = g[b][accept_len[b]]
 *   target_logits  device fp32 [batch][gamma+1][vocab] (finite values)
 *   draft_tokens   device int32 [batch][gamma]
 *   accept_len, next_token   device int32 [batch] out
 *   target_argmax_or_null    device int32 [batch][gamma+1] out (optional)
 *   ws             device scratch, specvlm_accept_workspace_bytes(batch, gamma, vocab)
 */
size_t specvlm_accept_workspace_bytes(int32_t batch, int32_t gamma, int32_t vocab);
int32_t specvlm_accept(const float* target_logits, const int32_t* draft_tokens, int32_t batch,
                       int32_t gamma, int32_t vocab, int32_t* accept_len, int32_t* next_token,
                       int32_t* target_argmax_or_null, void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Cache maintenance around a step (Section 3.1: the gamma drafted tokens are generated by the
 * draft one at a time and verified by the target in one pass; rejected tokens are discarded).
 *
 * specvlm_append_kv writes the K/V rows of n_new new tokens of every sequence behind its current
 * end -- token t of sequence b goes to position seq_lens[b] + t of every layer and KV head -- and
 * then adds n_new to seq_lens[b].  The attention calls expect exactly that state (the cache
 * already holds the new tokens).
 *   kv           host struct of the cache to extend (kv->seq_lens is ignored, see seq_lens_inout)
 *   new_k, new_v device bf16 [n_layers][batch][n_new][n_kv_heads][head_dim]
 *   seq_lens_inout  device int32 [batch], read then updated on the stream
 * A sequence without room (seq_lens[b] + n_new > kv->max_seq_len) is left unchanged and
 * SPECVLM_ERR_INVALID_ARG is stored to d_status: none of its n_new rows is written and its length
 * stays.  With a block table the pages of the new positions must already be mapped; a row whose
 * table entry is outside [0, n_blocks) is skipped and reported the same way.
 *
 * specvlm_rollback_kv drops the rejected drafts after verification: a cache that held the
 * gamma + 1 tokens of the window keeps accept_len[b] + 1 of them,
 *   seq_lens[b] -= gamma - accept_len[b].
 * No row is moved: rows past a sequence's length are never read.
 *   accept_len   device int32 [batch], as written by specvlm_accept (0 .. gamma)
 */
int32_t specvlm_append_kv(const specvlm_kv_t* kv, const void* new_k, const void* new_v, int32_t batch,
                          int32_t n_new, int32_t* seq_lens_inout, int32_t* d_status, void* stream);
int32_t specvlm_rollback_kv(int32_t* seq_lens_inout, const int32_t* accept_len, int32_t batch,
                            int32_t gamma, int32_t* d_status, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Tree drafting (the paper's experimental set-up drafts a static token tree and reports chain
 * drafting as the ablation): the verification window holds the n_nodes nodes of a tree instead
 * of a chain.  Node 0 is the root (the last committed token); parents[b][t] < t is the parent of
 * node t, -1 marks a root.  A chain is the tree parents[t] = t - 1.
 *
 * specvlm_verify_tree_attn: as specvlm_verify_attn, but query node t sees the keys before the
 * window (positions 0 .. seq_len - n_nodes - 1) and, inside the window, the rows of its
 * ancestors and its own.
 *   parents   device int32 [batch][n_nodes]
 *   q, out    device bf16 [n_layers][batch][n_nodes][n_q_heads][head_dim]
 *   ws        device scratch, specvlm_verify_tree_workspace_bytes(kv, batch, n_q_heads, n_nodes)
 * Supported: n_nodes <= 64, n_q_heads / n_kv_heads in 1..16, batch <= 127.  A tree of more than 128
 * rows ((n_q_heads / n_kv_heads) * n_nodes) is cut into parts of at most 128 rows that run side by
 * side in one launch (see specvlm_verify_attn).  A parents array that is not in topological order stores
 * SPECVLM_ERR_INVALID_ARG to d_status.
 *
 * specvlm_accept_tree: greedy acceptance along the tree.  With g[t] = argmax of node t's target
 * logits (lowest index among equal maxima), start at the root and step to the child whose token is
 * g[current] (lowest node index among equal children) until no child matches.
 *   target_logits  device fp32 [batch][n_nodes][vocab]
 *   node_tokens    device int32 [batch][n_nodes]: the drafted token of each node (entry 0 unused)
 *   accept_len     device int32 [batch] out: accepted drafts
 *   next_token     device int32 [batch] out: g of the last accepted node
 *   path           device int32 [batch][n_nodes] out: the accepted nodes in order, then -1
 *   ws             device scratch, specvlm_accept_workspace_bytes(batch, n_nodes - 1, vocab)
 *
 * specvlm_compact_tree_kv: after acceptance the rows of the accepted nodes move up behind the
 * root (window position path[i] -> position 1 + i) and the sequence keeps 1 + accept_len of the
 * window's n_nodes rows, so that the cache is a plain sequence again.  A path node outside
 * [1, n_nodes), a block-table entry outside [0, n_blocks) or a sequence longer than max_seq_len
 * makes the kernel skip that row's move and store SPECVLM_ERR_INVALID_ARG to d_status.
 */
size_t specvlm_verify_tree_workspace_bytes(const specvlm_kv_t* kv, int32_t batch, int32_t n_q_heads,
                                           int32_t n_nodes);
int32_t specvlm_verify_tree_attn(const specvlm_kv_t* kv, const void* q, const int32_t* parents,
                                 int32_t batch, int32_t n_q_heads, int32_t n_nodes, float sm_scale,
                                 void* out, float* lse_or_null, void* ws, size_t ws_bytes,
                                 int32_t* d_status, void* stream);
int32_t specvlm_accept_tree(const float* target_logits, const int32_t* node_tokens, const int32_t* parents,
                            int32_t batch, int32_t n_nodes, int32_t vocab, int32_t* accept_len,
                            int32_t* next_token, int32_t* path, int32_t* target_argmax_or_null, void* ws,
                            size_t ws_bytes, void* stream);
int32_t specvlm_compact_tree_kv(const specvlm_kv_t* kv, const int32_t* path, const int32_t* accept_len,
                                int32_t batch, int32_t n_nodes, int32_t* seq_lens_inout, int32_t* d_status,
                                void* stream);

/* ---------------------------------------------------------------------------------------------
 * specvlm_accept without any caller-provided scratch.  (The paper has no counterpart: this is a
 * packaging variant of step 4c, same results.)
 *
 * For callers that cannot allocate device memory at the point of the call and have no workspace
 * to hand over: code running inside another framework's pre-planned memory arena, a latency-
 * critical serving loop that forbids cudaMalloc (it synchronises the device), or a plug-in that
 * only receives input and output buffers.  The per-(row, vocabulary-chunk) candidates live in a
 * fixed array inside the library (128 KB of device memory on every GPU that loads the library,
 * held until the process exits) instead of `ws`.
 *
 * Arguments and results are those of specvlm_accept, minus ws / ws_bytes.
 * Limit: batch * (gamma+1) * ceil(vocab / 8192) <= 16384 candidates (e.g. batch 16, gamma 8,
 * vocab 152064 needs 2736); larger problems return SPECVLM_ERR_TOO_LARGE and launch nothing.
 * The call allocates and frees nothing, on the host side or the device side.
 * The first call on each device looks up the device address of that device's copy of the array
 * (a cheap runtime query, cached afterwards); make that first call with the device current and
 * before starting any stream capture.
 * All calls on a device share the one array: two calls whose kernels may overlap on the GPU
 * (different streams without an ordering between them) race on it and give wrong results.
 * Calls ordered on one stream are safe; nothing needs clearing between calls, because each call
 * overwrites every slot it later reads.
 */
int32_t specvlm_accept_noalloc(const float* target_logits, const int32_t* draft_tokens, int32_t batch,
                               int32_t gamma, int32_t vocab, int32_t* accept_len,
                               int32_t* next_token, int32_t* target_argmax_or_null, void* stream);

/*
 * Diagnostic for tests; the paper has no counterpart.  Launches a kernel on `stream` that fills
 * the shared memory of the SMs with NaN bit patterns (0xffffffff words).  Shared memory keeps its
 * contents from one kernel to the next, so a kernel that reads a word it never wrote usually
 * sees something harmless and a test passes by luck; after this call it sees NaNs.  Computes
 * nothing, allocates nothing, touches no global memory.
 */
int32_t specvlm_debug_poison_shared_memory(void* stream);

/*
 * Diagnostic for tests; the paper has no counterpart.  Runs the library's bounded barrier wait on
 * a barrier that nothing ever arrives at, with a limit of limit_ms (1..1000) milliseconds instead
 * of the product kernels' 2 s: the wait gives up, the kernel stores SPECVLM_ERR_TIMEOUT to
 * d_status (device, required) and the CTA's abort flag to d_abort_flag_or_null (device int32),
 * and returns normally -- the way every kernel of the library reports an expired wait.
 */
int32_t specvlm_debug_wait_timeout(int32_t limit_ms, int32_t* d_status, int32_t* d_abort_flag_or_null,
                                   void* stream);

/*
 * Test hook; the paper has no counterpart.  n_splits > 0 makes every later attention call of up
 * to 16 rows per KV head cut each sequence into that many CTAs (capped by its tile count), so
 * that tests reach the split-merge path at any size; 0 restores the built-in choice.  Process-wide.
 */
void specvlm_debug_set_attn_splits(int32_t n_splits);

/*
 * Test hook, host only; the paper has no counterpart.  Reports how a verification window of n_q
 * query tokens at `group` = n_q_heads / n_kv_heads heads per KV head is cut into the parts that run
 * side by side in one launch: n_parts parts of q_per tokens (the last may be shorter), each of at
 * most 128 rows.  n_parts, q_per: host int32 out.  Launches nothing.
 */
int32_t specvlm_debug_window_parts(int32_t n_q, int32_t group, int32_t* n_parts, int32_t* q_per);

#ifdef __cplusplus
}
#endif
#endif /* SPECVLM_H_ */

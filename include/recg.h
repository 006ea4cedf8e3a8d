/*
 * recg.h -- C ABI of the fused draft+verify step for diffusion-AR self-speculation on one B200.
 *
 * One round of shared-backbone self-speculation (paper Sec. 3.1) runs ONE forward over a ragged,
 * padding-free batch (Sec. 5.3).  Request r contributes
 *     v_r pending verify tokens y_0..y_{v-1} at positions L_r .. L_r+v_r-1   (causal rows), and
 *     b_r mask tokens at positions L_r+v_r .. L_r+v_r+b_r-1                  (bidirectional rows),
 * over its L_r committed context tokens, whose K/V live in a paged pool.  Visibility is Eq. 1's
 * M^Diff with the prefix set = context + verify tokens and the draft set = the mask block; restricted
 * to the verify rows this is M^AR, so the same forward verifies the previous drafts and drafts the
 * next block (Sec. 5.1, continuation branch).  The round ends with greedy verification (accept the
 * drafted prefix up to the first mismatch, Sec. 3.1), the confidence statistics that guide the
 * runtime (P_1st, P_1st - P_2nd: Sec. 4.1; mean verifier entropy over valid rows: Sec. 5.2) and the
 * KV commit / rollback, which is index work only.
 *
 * General rules
 *   - every entry point returns a recg_status and never aborts; recg_last_error() gives the text;
 *   - all device work is enqueued on the CUDA stream given to recg_init(); nothing synchronises
 *     the stream unless stated;
 *   - "DEVICE" / "HOST" on a pointer says where the memory lives.  bf16 is the 16-bit brain float
 *     bit pattern; ids, lengths and slots are int32;
 *   - weights and the KV pool are BORROWED: the caller allocates them, keeps them alive while the
 *     context lives and frees them; the library allocates only its own workspace, in recg_init();
 *   - there is no CPU fallback: without a CUDA device every call fails with RECG_ERR_CUDA.
 */
#ifndef RECG_H_
#define RECG_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  RECG_OK = 0,
  RECG_ERR_INVALID_ARG = 1, /* null pointer, negative length, unknown enum                     */
  RECG_ERR_SHAPE = 2,       /* model dimensions the kernels do not support                     */
  RECG_ERR_CAPACITY = 3,    /* more requests / tokens / pages than the context was sized for   */
  RECG_ERR_CUDA = 4,        /* a CUDA runtime or driver call failed                            */
  RECG_ERR_TIMEOUT = 5,     /* a bounded device-side wait gave up (status word set by kernel)  */
  RECG_ERR_INTERNAL = 6
} recg_status;

typedef enum { RECG_DTYPE_BF16 = 0, RECG_DTYPE_F32 = 1 } recg_dtype;
typedef enum { RECG_MEM_DEVICE = 0, RECG_MEM_HOST = 1 } recg_mem;

enum {
  RECG_FLAG_LOGITS_BF16 = 1, /* recg_step() stores logits as bf16 instead of fp32               */
  RECG_FLAG_SIMT_GEMM = 2,   /* run the projections on the legacy mma.sync kernel (A/B checks)  */
  RECG_FLAG_SIMT_ATTENTION = 4, /* run attention on the legacy mma.sync kernel (A/B checks)     */
  RECG_FLAG_FOLD_NORM = 16,  /* fold every RMSNorm into the projections around it instead of running it as a kernel of
                                its own: the projection that updates the residual stream also writes x = bf16(h * gain)
                                and per-row partial sums of squares, the projection that reads x scales its rows by the
                                row's rstd.  Same results within bf16 rounding (x is rounded before the division instead
                                of after it); measured 3 % slower than the separate kernel, which hides behind the next
                                projection's weight prefetch, hence off by default                            */
  RECG_FLAG_CHAIN = 32,      /* steps of at most 128 rows (low concurrency): run the projections between two attention
                                calls (output projection, gate|up, down, the next layer's QKV projection or the LM head)
                                as ONE persistent kernel with grid-wide barriers, so that the weight stream does not stop
                                at kernel boundaries; implies the folded RMSNorm.  head_dim 128 only; larger steps and
                                captured streams take the ordinary path                                       */
  RECG_FLAG_DEBUG_CHECKS = 8 /* guard bands behind every workspace region, checked by recg_sync() (RECG_ERR_INTERNAL
                                if a kernel wrote past the end of one), and a host check that no page which receives
                                new rows is named by two requests (RECG_ERR_INVALID_ARG)          */
};

typedef struct recg_ctx recg_ctx;

/* Model and capacity description; immutable after recg_init(). */
typedef struct {
  int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab;
  float rope_base;        /* rotary base; pairing is (i, i + head_dim/2)                         */
  float rms_eps;
  int32_t mask_token_id;  /* id fed to the mask rows; < 0 means vocab - 1                        */
  int32_t page_size;      /* tokens per KV page; must be 16                                      */
  int32_t max_requests;   /* capacity: requests per step, at most 4096                            */
  int32_t max_tokens;     /* capacity: rows of a step, the sum of n_r (see recg_batch), at most 1048576 */
  int32_t max_pages_per_request;
  int32_t flags;          /* RECG_FLAG_*                                                         */
} recg_config;

/*
 * Weights, DEVICE, bf16, every matrix row-major [out_features, in_features]:
 *   embed [vocab, hidden]; final_norm [hidden]; lm_head [vocab, hidden];
 *   per layer l (the arrays of pointers themselves are HOST arrays of n_layers DEVICE pointers):
 *   attn_norm[l] [hidden]; wqkv[l] [(n_q + 2 n_kv) * head_dim, hidden] (q heads, k heads, v heads);
 *   wo[l] [hidden, n_q * head_dim]; ffn_norm[l] [hidden];
 *   w_gate_up[l] [2 * ffn, hidden] (gate rows then up rows); w_down[l] [hidden, ffn].
 * All base addresses must be 16-byte aligned.
 */
typedef struct {
  const void *embed, *final_norm, *lm_head;
  const void *const *attn_norm;
  const void *const *wqkv;
  const void *const *wo;
  const void *const *ffn_norm;
  const void *const *w_gate_up;
  const void *const *w_down;
} recg_weights;

/*
 * One round's batch descriptor.  The small arrays are HOST memory and are copied by the call.
 *   ctx_len[r]     L_r, committed context tokens whose K/V are already in the pool
 *   verify_len[r]  v_r >= 0, pending verify tokens (y_0 known-correct, y_1.. drafts)
 *   block_size[r]  b_r >= 0, mask tokens;  v_r + b_r >= 1
 *   verify_tokens  the y of all requests, concatenated in request order (sum of v_r ids)
 *   page_table     [n_req, page_table_stride] physical page ids; row r must cover
 *                  ceil((L_r + n_r) / page_size) pages (n_r = v_r + b_r without branches), else RECG_ERR_CAPACITY
 *   kv_pool        DEVICE, recg_kv_pool_bytes(cfg, kv_pool_pages) bytes, library-defined layout
 *                  (per layer, per page, per KV head: a K tile then a V tile of 16 tokens, stored in
 *                  the swizzled order the attention kernel loads; use recg_kv_write / recg_kv_read
 *                  to move logical K/V in and out).  May be NULL for a verify-only call.
 *
 * Prospective correction branches of the predictive draft-verify overlap (Sec. 5.1); n_corr == NULL
 * means no request has any, and block_size[r] is then the only draft block (the continuation branch):
 *   n_corr[r]        0..2 correction branches of request r
 *   corr_index[2r+k] i, 1 <= i <= v_r - 1, strictly increasing in k: the draft y_i the branch replaces
 *   corr_token[2r+k] the replacement token (the draft's second candidate)
 *   corr_block[r]    bc_r >= 0, mask tokens that follow the replacement token in each branch of r
 * Request r then has n_r = v_r + b_r + n_corr[r] * (1 + bc_r) rows in the ragged batch, in the order
 * [verify | continuation masks | branch 0: replacement, masks | branch 1: replacement, masks], and their
 * K/V occupy cache positions L_r .. L_r + n_r - 1 in that order (the page-table row must cover them).
 * A branch token is rotated as the position it hypothesises (replacement: L_r + i, masks: L_r + i + 1 ..).
 * It sees the committed context and y_0 .. y_{i-1}; besides those the replacement token sees itself and a
 * mask token sees its whole branch.  Branch rows are always rolled back by recg_verify.
 *   risk_delta       margin threshold of the risky-position outputs of recg_verify; <= 0 means 0.5
 */
typedef struct {
  int32_t n_req;
  const int32_t *ctx_len;
  const int32_t *verify_len;
  const int32_t *block_size;
  const int32_t *verify_tokens;
  const int32_t *page_table;
  int32_t page_table_stride;
  void *kv_pool;
  int64_t kv_pool_pages;
  const int32_t *n_corr;
  const int32_t *corr_index;
  const int32_t *corr_token;
  const int32_t *corr_block;
  float risk_delta;
} recg_batch;

/* Logits of the last recg_step(): DEVICE, library-owned, valid until the next recg_step(). */
typedef struct {
  const void *data;  /* [n_rows, vocab], row t = t-th token of the ragged batch */
  int32_t dtype;     /* recg_dtype */
  int32_t n_rows;
  int32_t vocab;
} recg_logits;

/*
 * Outputs of greedy verification.  All buffers are caller-provided and live where `mem` says
 * (every pointer in one struct in the same place); any pointer may be NULL to skip that output.
 * With RECG_MEM_HOST the call copies the results out and synchronises the stream before returning.
 * T = sum(n_r) rows of the batch, Tv = sum(v_r), Tb = T - Tv (all rows that are not verify rows).
 *   accept_len[n_req]    a_r: drafts y_1..y_a accepted (longest prefix equal to the verifier argmax)
 *   n_emitted[n_req]     a_r + 1 (0 if v_r = 0)
 *   emitted[Tv]          per request, at its verify offset: y_1..y_a then the verifier's token at row a
 *                        (correction if a < v-1, bonus if a = v-1); entries beyond n_emitted are -1
 *   new_ctx_len[n_req]   L_r + a_r + 1: K/V of y_0..y_a are now committed
 *   slot_state[T]        per token of the batch: +slot (page*page_size + offset) if its K/V is committed,
 *                        -(slot+1) if it is rolled back (rejected draft or mask row)
 *   freed_pages[n_req]   number of pages of request r that hold no committed token any more
 *                        (its page-table entries from ceil(new_ctx_len/page_size) on)
 *   next_draft[Tb]       argmax of every row that is not a verify row, in batch order: per request its
 *                        continuation masks, then per branch the replacement row and the branch's masks
 *   cont_hit[n_req]      1 if the block was fully accepted and the first drafted token equals the
 *                        bonus token (the continuation branch can be reused), else 0
 *   top1, top2 [T]       ids of the largest and second-largest logit per row (lowest index wins ties)
 *   p1, p2, entropy [T]  float32: softmax probability of top1 and top2, entropy in nats
 *   entropy_mean[n_req]  float32: mean verifier entropy over rows 0..a_r
 * Branch reuse and the next round's risky positions (Sec. 5.1):
 *   corr_hit[2 n_req]    entry 2r+k: 1 if the verifier rejected exactly the draft branch k replaced
 *                        (a_r == i - 1) and its own token there equals the replacement token, else 0
 *   risky_n[3 n_req]     entry 3r+j: how many drafts of block j of request r (j = 0 the continuation block,
 *                        j = 1 + k correction branch k) have margin p1 - p2 < risk_delta; 0 for absent blocks
 *   risky_index, risky_token [6 n_req]  entries 6r+2j+{0,1}: the earliest two of them, as the index the
 *                        draft would have in the next round's verify tokens (continuation: mask row m is
 *                        y'_m, m >= 1, since y'_0 is the bonus token; correction: mask row m is y'_{m+1})
 *                        and the row's second candidate; -1 where there is none
 */
typedef struct {
  int32_t mem; /* recg_mem */
  int32_t *accept_len, *n_emitted, *emitted, *new_ctx_len, *slot_state, *freed_pages;
  int32_t *next_draft, *cont_hit, *top1, *top2;
  float *p1, *p2, *entropy, *entropy_mean;
  int32_t *corr_hit, *risky_n, *risky_index, *risky_token;
  int32_t *freed_page_ids;
} recg_verify_out;

/* Bytes of KV pool needed for n_pages physical pages (all layers). */
size_t recg_kv_pool_bytes(const recg_config *cfg, int64_t n_pages);

/*
 * Create a context: validates cfg, allocates the workspace (activations for max_tokens rows, logits,
 * attention partials, descriptors) and records the weight pointers.  `weights` may be NULL for a
 * context that only runs the standalone operations (recg_verify with explicit logits,
 * recg_attention, recg_linear, recg_kv_*); recg_step() then fails with RECG_ERR_INVALID_ARG.
 * cuda_stream is a cudaStream_t (NULL = the default stream).  Uses the current CUDA device.
 */
recg_status recg_init(recg_ctx **out, const recg_config *cfg, const recg_weights *weights, void *cuda_stream);

/*
 * One fused draft+verify forward (ragged layout, embedding, n_layers x {RMSNorm, QKV projection with
 * rotary embedding and KV append, hybrid-mask paged attention (Eq. 1), output projection + residual,
 * RMSNorm, gate|up projection + SwiGLU, down projection + residual}, final norm, LM head).
 * K/V of all n_r new rows are written into the pool slots the page table names
 * (tentatively: recg_verify decides which stay).  `logits` (may be NULL) receives the view of the
 * logits.  Does not synchronise.
 */
recg_status recg_step(recg_ctx *ctx, const recg_batch *batch, recg_logits *logits);

/*
 * Greedy verification, statistics and KV commit / rollback (Sec. 3.1, 4.1, 5.1, 5.2) for `batch`.
 * logits == NULL: use the logits of the last recg_step() (same batch).  Otherwise `logits` is a
 * DEVICE array [T, vocab] of `logits_dtype`; batch->kv_pool may then be NULL and page_table may be
 * NULL (slot_state and freed_pages are then not produced).
 */
recg_status recg_verify(recg_ctx *ctx, const recg_batch *batch, const void *logits, int32_t logits_dtype,
                        recg_verify_out *out);

/*
 * The hybrid-mask paged attention of one layer as a standalone operation (Eq. 1 over a shared prefix).
 * q, o: DEVICE bf16 [T, n_q_heads, head_dim] (q already rotated).  K/V of ALL L_r + n_r
 * positions of every request must already be in layer `layer` of the pool.
 */
recg_status recg_attention(recg_ctx *ctx, const recg_batch *batch, int32_t layer, const void *q, void *o);

/*
 * Move logical K/V rows of one request into / out of the pool.  k, v: DEVICE bf16
 * [n_pos, n_kv_heads, head_dim] for positions pos0 .. pos0+n_pos-1; page_table_row: HOST, the
 * request's page ids covering those positions.
 */
recg_status recg_kv_write(recg_ctx *ctx, void *kv_pool, int64_t kv_pool_pages, int32_t layer,
                          const int32_t *page_table_row, int32_t n_table, int32_t pos0, int32_t n_pos,
                          const void *k, const void *v);
recg_status recg_kv_read(recg_ctx *ctx, const void *kv_pool, int64_t kv_pool_pages, int32_t layer,
                         const int32_t *page_table_row, int32_t n_table, int32_t pos0, int32_t n_pos,
                         void *k, void *v);

/*
 * y[M, N] = x[M, K] . w[N, K]^T, the projection kernel without an epilogue (for checking it alone).
 * x, w: DEVICE bf16, 16-byte aligned, K a multiple of 64 and N a multiple of 16; y: DEVICE, out_dtype.
 */
recg_status recg_linear(recg_ctx *ctx, const void *x, const void *w, void *y, int32_t M, int32_t N, int32_t K,
                        int32_t out_dtype);

/*
 * Read back an internal activation of the last recg_step() for parity checks.  which: 0 = residual
 * stream after the last layer, fp32 [T, hidden]; 1 = attention output of the last layer, bf16
 * [T, n_q*head_dim]; 2 = rotated queries of the last layer, bf16 [T, n_q*head_dim].
 * Returns DEVICE pointers into the workspace.
 */
recg_status recg_debug_buffer(recg_ctx *ctx, int32_t which, const void **ptr, int32_t *dtype, int32_t *rows,
                              int32_t *cols);

/*
 * Debugging aids (the paper has no counterpart).
 * recg_debug_gemm_config(): force the tile configuration of the projection launches that follow on this context,
 *   instead of the cost model's choice: tile = 64, 128 or 256 (single CTAs, 128-row tiles of that width), 384 (CTA
 *   pairs, 256 x 128 tiles), 512 (CTA pairs, 256 x 256 tiles), 0 = back to the cost model; stream_k = 1 cuts the
 *   K range of the tiles evenly over the SMs, stream_k = 2 does the same and also (with any tile value, 0 included)
 *   keeps problems of at most 128 rows from handing their partial tiles over inside thread-block clusters: they go
 *   through the partial-tile workspace like everything else; stream_k = 0: whole tiles.  A configuration that does not
 *   fit a shape is ignored for that launch.
 * recg_debug_wait_timeout(): enqueue a one-thread kernel that waits on a barrier nobody arrives on, bounded by
 *   max_polls polls (1 .. 1048576) exactly like the waits inside the kernels; it gives up, records the timeout in the
 *   device status word and returns.  The next recg_sync() then reports RECG_ERR_TIMEOUT and clears the word; the
 *   context stays usable.  Nothing traps or faults.
 * recg_debug_map_cache_selftest(): host only (no device needed): pushes n_keys distinct keys through the cache of
 *   encoded tensor maps, three per simulated launch, and returns how many maps came back wrong (0 = pass);
 *   *evictions receives how often the full cache was emptied on the way.
 */
recg_status recg_debug_gemm_config(recg_ctx *ctx, int32_t tile, int32_t stream_k);
recg_status recg_debug_wait_timeout(recg_ctx *ctx, int32_t max_polls);
int32_t recg_debug_map_cache_selftest(int32_t n_keys, int32_t *evictions);

/*
 * Per-kernel-class device timing of recg_step()/recg_verify() for roofline reports (measurement aid; the
 * forward-time profiling of Sec. 3.2 is the closest thing in the paper).  recg_timing_enable(ctx, 1) makes
 * the following calls record CUDA events at class boundaries on the context's stream;
 * recg_timing_read() synchronises the stream, adds the elapsed milliseconds per class since the last read
 * into ms[0..RECG_TIMING_CLASSES) and launches[...] (either may be NULL) and resets the accumulation.
 * Classes: 0 layout+embedding+rotary table, 1 RMSNorm, 2 QKV projection, 3 attention (+combine),
 * 4 output projection, 5 gate|up projection, 6 down projection, 7 LM head, 8 verify.
 */
#define RECG_TIMING_CLASSES 9
recg_status recg_timing_enable(recg_ctx *ctx, int32_t enable);
recg_status recg_timing_read(recg_ctx *ctx, float *ms, int32_t *launches);

/*
 * Verification-guided choice of the next block size (Sec. 5.2, Eq. 2-3), on the device.
 *
 * recg_policy_load() copies a lookup table into the context (HOST arrays, copied by the call):
 *   blocks[n_blocks]   candidate block sizes, ascending (the paper uses 8, 16, 32); n_blocks <= 8
 *   s_edges[n_bins-1]  ascending edges of the certainty bins; s falls into bin (number of edges <= s); n_bins <= 64
 *   value              float32 [n_blocks][n_bins][n_blocks][2]: the calibrated estimate V_B(s, z) of the
 *                      expected accepted progress, indexed [candidate B][bin of s][previous block][F]
 *   cost[n_blocks]     rho_C * T_C(B): the profiled execution cost of each candidate at the current load,
 *                      already weighted
 * recg_policy_step() runs after recg_verify() on the batch laid out last.  Per request r (state arrays are
 * DEVICE, caller-owned, [n_req], carried from round to round; the caller initialises them):
 *   if v_r > 0:  e2 <- e1;  e1 <- entropy_mean[r];  full <- (v_r > 1 and accept_len[r] == v_r - 1)
 *   s = -(e1 + e2) / 2                                                     (Eq. 2, float32)
 *   j* = argmax_j  value[j][bin(s)][block_index][full] - cost[j]           (Eq. 3; the first maximum wins)
 *   next_block[r] = blocks[j*];  block_index <- j*
 * entropy_mean / accept_len: DEVICE [n_req], or NULL for the library's own buffers, which hold the results
 * of the last recg_verify() unless that call was given DEVICE output pointers for these two fields.
 * next_block: DEVICE int32 [n_req].  Does not synchronise and copies nothing to the host.
 * Errors: RECG_ERR_INVALID_ARG (no table loaded, no batch laid out, null pointers, table out of limits or
 * not ascending).
 */
#define RECG_POLICY_MAX_BLOCKS 8
#define RECG_POLICY_MAX_BINS 64
typedef struct {
  int32_t n_blocks, n_bins;
  const int32_t *blocks;
  const float *s_edges;
  const float *value;
  const float *cost;
} recg_policy_table;
typedef struct {
  float *e1, *e2;       /* e_{t-1}, e_{t-2} */
  int32_t *block_index; /* index of B_{t-1} among the candidates */
  int32_t *full;        /* F_{t-1} */
} recg_policy_state;
recg_status recg_policy_load(recg_ctx *ctx, const recg_policy_table *table);
recg_status recg_policy_step(recg_ctx *ctx, const recg_policy_state *state, const float *entropy_mean,
                             const int32_t *accept_len, int32_t *next_block);

/*
 * Device-resident rounds (Sec. 5.2: the verification history of one round guides the next one; nothing has to come back
 * to the host in between).  The descriptor arrays live on the DEVICE and belong to the caller; the library reads them
 * when the step executes and recg_next_round() rewrites them in place, so N rounds are N x { recg_step_device,
 * recg_verify(ctx, NULL, NULL, 0, out with mem = RECG_MEM_DEVICE), optionally recg_policy_step, recg_next_round }
 * enqueued back to back with one synchronisation at the end.
 *
 * recg_device_batch (all pointers DEVICE):
 *   ctx_len, verify_len, block_size [n_req]   as in recg_batch; rewritten by recg_next_round()
 *   verify_tokens [n_req, max_verify]         request r's y_0.. at r * max_verify (a fixed stride, not ragged)
 *   page_table [n_req, page_table_stride]     fixed over the loop: row r must cover every position the request can
 *                                             reach (a request whose next round would not fit stops drafting: its
 *                                             block size becomes 0; if even one more token does not fit the status
 *                                             word is set)
 *   rows_hint                                 the expected number of rows per round, used to choose the projections'
 *                                             tile configurations (0: the context's max_tokens)
 * Correction branches are not available in this mode.  Because the row count of a round is only known on the device,
 * every launch is sized for the context's max_tokens and max_requests, projections use whole tiles only, and
 * recg_logits.n_rows reports max_tokens; the true counts are in the device arrays.  Lengths that break a capacity
 * (negative, a request without rows, verify_len > max_verify, rows beyond the page-table row, more than max_tokens rows
 * in total) set the device status word and turn the round into an empty one: recg_sync() then returns
 * RECG_ERR_INTERNAL.  Not available with RECG_FLAG_SIMT_GEMM or RECG_FLAG_FOLD_NORM.
 *
 * recg_next_round() turns the finished round (the library's own verification buffers: call recg_verify with NULL
 * output pointers or leave them out) into the next one, per request:
 *   a = accept_len; the tokens y_1..y_a and the verifier's token t at row a are appended to the log;
 *   ctx_len += a + 1;  if the continuation block is reusable (cont_hit): verify tokens = [t, d_1 .. d_{b-1}] (the drafted
 *   block, whose first token only confirmed t), else [t];  block_size = next_block[r] (DEVICE, e.g. the output of
 *   recg_policy_step; NULL keeps the block size).
 *   planted_emitted (DEVICE [n_req] or NULL): synthetic acceptance for random-weight runs -- the round is taken to have
 *   emitted min(planted_emitted[r], verify_len) tokens (at least 1), and its continuation block to be reusable exactly
 *   when every draft was accepted.
 * recg_round_log (DEVICE, caller-owned, any part may be NULL): tokens [n_req, max_tokens_per_request] with n_tokens
 * [n_req] (initialise to 0); accept_len / block_size / verify_len (int32) and entropy_mean (float32) [max_rounds, n_req]
 * receive row `round` (the caller's round counter): what the round accepted, the block size and verify length it ran
 * with and its mean verifier entropy; n_rounds [1] receives round + 1.
 */
typedef struct {
  int32_t n_req, max_verify, page_table_stride, rows_hint;
  int32_t *ctx_len, *verify_len, *block_size, *verify_tokens;
  const int32_t *page_table;
  void *kv_pool;
  int64_t kv_pool_pages;
} recg_device_batch;
typedef struct {
  int32_t *tokens, *n_tokens;
  int32_t max_tokens_per_request;
  int32_t max_rounds;
  int32_t *accept_len, *block_size, *verify_len, *n_rounds;
  float *entropy_mean;
} recg_round_log;
recg_status recg_step_device(recg_ctx *ctx, const recg_device_batch *batch, recg_logits *logits);
recg_status recg_next_round(recg_ctx *ctx, const recg_device_batch *batch, const int32_t *next_block,
                            const int32_t *planted_emitted, const recg_round_log *log, int32_t round);

/*
 * Per-row logit statistics with no allocation anywhere (the paper has no counterpart: this entry point
 * exists for callers that are not allowed to allocate device memory).
 *
 * Some hosts of this library cannot call cudaMalloc at the moment they need the statistics: code running
 * inside a stream capture, a serving loop that has handed all device memory to its own pool allocator
 * and forbids further driver allocations, or a plugin that runs under a sandbox whose allocation hooks
 * must not be re-entered.  recg_verify() needs a context, and creating a context allocates a workspace.
 * This variant needs neither: it runs the same vocabulary scan (top-1 / top-2 ids with lowest-index
 * ties, P_1st, P_2nd, entropy in nats per row), but keeps the per-chunk partial results in a fixed
 * array that is part of the library image, and it calls no cudaMalloc, cudaFree or any allocating routine.
 *
 *   logits   DEVICE [rows, vocab] of logits_dtype (recg_dtype), row-major
 *   top1, top2 DEVICE int32 [rows]; p1, p2, entropy DEVICE float32 [rows]; any output may be NULL
 *   cuda_stream  cudaStream_t the work is enqueued on (NULL = default stream); the call does not wait
 *
 * Limits and rules:
 *   - the static scratch holds 65536 chunk partials (1.5 MiB of device memory that every GPU which loads
 *     the library keeps until the process exits).  rows may not exceed 65536 and rows x chunks-per-row
 *     must fit; larger requests are refused with RECG_ERR_CAPACITY and nothing is launched;
 *   - the first call on each device looks up the device address of the scratch array (with that device
 *     current).  Make that first call outside any stream capture;
 *   - all calls on one device share the scratch, which keeps whatever the previous call left there.
 *     Every partial a call reads is written by that same call first, so stale contents are harmless, but
 *     two calls whose kernels overlap on the GPU (different streams, or different host threads) race on
 *     it: serialise them;
 *   - errors: RECG_ERR_INVALID_ARG, RECG_ERR_CAPACITY, RECG_ERR_CUDA; recg_last_error(NULL) does NOT carry
 *     this entry point's text, use recg_row_stats_static_error().
 */
recg_status recg_row_stats_static(const void *logits, int32_t logits_dtype, int32_t rows, int32_t vocab,
                                  int32_t *top1, int32_t *top2, float *p1, float *p2, float *entropy,
                                  void *cuda_stream);
const char *recg_row_stats_static_error(void);

/* Wait for the stream, then report (and clear) the device status word: RECG_OK or RECG_ERR_TIMEOUT /
 * RECG_ERR_INTERNAL if a kernel flagged a bounded wait that gave up or an out-of-range index. */
recg_status recg_sync(recg_ctx *ctx);

recg_status recg_free(recg_ctx *ctx);

/* Text of the last error on this context (or of the last failed recg_init if ctx is NULL). */
const char *recg_last_error(const recg_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* RECG_H_ */

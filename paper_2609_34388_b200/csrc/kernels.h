// Internal launcher interface between the C ABI (recg_api.cu) and the kernel files.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace recg {

struct Dims {
  int n_layers, hidden, n_q, n_kv, head_dim, ffn, vocab;
  float rope_base, rms_eps;
  int mask_id;
};

// One attention work item: rows of one (request, kv head, row tile) against a range of 64-token KV blocks.
struct AttnItem {
  int req, kv_head;
  int tok0, ntok;        // first token of the tile (index into the ragged batch) and tokens in it
  int blk_begin, blk_end;
  int part;              // index into the partial buffers, or -1 when the item covers the whole KV range
  int kv_len;            // L + n of the request
};
struct AttnTile {        // per (request, kv head, row tile): where its partials are, and which rows it covers
  int part_begin, n_parts;
  int tok0, ntok, kv_head;
};

// Device-resident ragged layout of one batch (all pointers DEVICE, int32 unless noted).
struct BatchLayout {
  int n_req, n_tok, n_ver, pt_stride;
  // Device-resident rounds: the row counts are only known on the device.  dyn (null otherwise) points to
  // {n_tok, n_ver}; n_tok / n_ver above are then the capacities the launches are sized for, and every kernel takes the
  // true counts from dyn.
  const int* dyn;
  float risk_delta;       // margin threshold of the risky-position outputs
  const int* ctx_len;     // [C]
  const int* verify_len;  // [C]
  const int* block_size;  // [C]
  const int* corr;        // [C][6] correction branches: count (0..2), mask tokens per branch, index 0, index 1, token 0, token 1
  const int* cu_tok;      // [C+1] exclusive prefix sum of the rows per request, v + b + count * (1 + mask tokens per branch)
  const int* cu_ver;      // [C+1] exclusive prefix sum of v
  const int* verify_tokens;  // [Tv]
  const int* page_table;  // [C, pt_stride] (may be null for verify-only batches)
  // per token, written by the layout kernel
  int* tok_id;
  int* tok_req;
  int* tok_pos;     // rotary position (a branch token: the position its branch hypothesises)
  int* tok_slot;    // page*16 + offset of cache position L + (row within the request), -1 without a page table
  int* tok_climit;  // sees every cache position <= climit ...
  int* tok_lo;      // ... and every cache position in [lo, hi)
  int* tok_hi;
  // attention work list
  AttnItem* items;
  AttnTile* tiles;
  int* tile_off;    // [C+1] first tile entry of each request
  int* cta_off;     // [4 n_ctas] per CTA of the persistent attention grid: the two item index ranges [b0, e0), [b1, e1) it walks
  int* item_cta;    // [max_items] owning CTA of each item (scratch of the layout kernel)
  int* counts;      // [0] number of items, [1] number of tiles, [2], [3] cost units per CTA / per CTA pair
  int max_items, max_parts;
};

// S1: per-token arrays and the attention work list.
void launch_layout(const BatchLayout& bl, const Dims& dm, int tok_per_tile, int n_ctas, int64_t n_pages,
                   int* status, cudaStream_t st);
// the layout kernel keeps eight ints per request in shared memory: requests per step are bounded by this
constexpr int kMaxLayoutRequests = 4096;
size_t layout_smem_bytes(int n_req, int n_ctas);
// debug checks
void launch_guard_fill(void* base, const size_t* offs_dev, int n, cudaStream_t st);
void launch_guard_check(const void* base, const size_t* offs_dev, int n, int* status, cudaStream_t st);
void launch_wait_timeout(uint32_t max_polls, int* status, cudaStream_t st);
// S2: h[t] = embed[tok_id[t]] (fp32 residual stream).  With gain != null also the input of the first normalised
// projection: x[t] = bf16(h[t] * gain) and ss[t] = sum h[t]^2 (one slot).
void launch_embed(const BatchLayout& bl, const Dims& dm, const void* embed, float* h, const void* gain, void* x, float* ss,
                  cudaStream_t st);
// x = rmsnorm(h) * g, bf16 out.  rows_dev (may be null): the true row count on the device (rows is then the capacity).
void launch_rmsnorm(const float* h, const void* gain, void* x, int rows, int hidden, float eps, cudaStream_t st,
                    const int* rows_dev = nullptr);

struct VerifyBuffers;
// Device-resident rounds (Sec. 5.2).  pack: builds the packed descriptor (the layout recg_api.cu uploads in the host
// mode: ctx_len | verify_len | block_size | corr | cu_tok | cu_ver | verify_tokens) in `desc` from the caller's device
// arrays and writes {n_tok, n_ver} to dyn; violations of the capacities set the status word and give an empty round.
struct DeviceRound {
  int n_req, max_verify, pt_stride, max_tokens;
  int *ctx_len, *verify_len, *block_size, *verify_tokens;    // caller's device arrays; verify tokens of request r at r * max_verify
};
void launch_pack_device(const DeviceRound& dr, int* desc, int* dyn, int* status, cudaStream_t st);
// next: turns the results of the finished round into the next round's arrays (in place) and appends to the logs.
struct RoundLog {
  int* tokens;       // [n_req][max_out] emitted tokens
  int max_out;
  int* n_tokens;     // [n_req]
  int* accept_len;   // [max_rounds][n_req] accepted drafts, block size used and verify length of every round
  int* block_size;
  int* verify_len;
  int max_rounds;
  int* n_rounds;     // [1]
  float* entropy_mean;   // [max_rounds][n_req]
};
void launch_next_round(const DeviceRound& dr, const BatchLayout& bl, const VerifyBuffers& vb, const int* next_block,
                       const int* planted_emitted, const RoundLog& log, int round, int* status, cudaStream_t st);

// (cos, sin) of pos * base^(-2i/d), angles evaluated in double: cs float2 [head_dim/2][T] (frequency-major).
void launch_rope_table(const int* tok_pos, int n_tok, int head_dim, float rope_base, void* cs, cudaStream_t st,
                       const int* n_tok_dev = nullptr);

// Projection epilogues.
enum Epilogue : int {
  EPI_PLAIN_BF16 = 0,  // C bf16 [M,N]
  EPI_PLAIN_F32 = 1,   // C fp32 [M,N]
  EPI_RESIDUAL = 2,    // h fp32 [M,N] += acc
  EPI_SWIGLU = 3,      // w is [2F,K]; out bf16 [M,F] = silu(x.wg) * (x.wu)
  EPI_QKV_ROPE = 4,    // rotate q and k heads, q -> bf16 [M, n_q*d], k/v -> paged pool at tok_slot
  EPI_RESIDUAL_NORM = 5  // h fp32 [M,N] += acc, and the input of the next RMSNorm-ed projection: x_out bf16 [M,N] =
                         // h * gain, ss_out[column tile][row] = sum over the tile's columns of h^2 (tcgen05 path only)
};
struct GemmArgs {
  const void* x;   // bf16 [M,K]
  const void* w;   // bf16 [N,K]  (EPI_SWIGLU: [2N,K], gate rows then up rows)
  void* out;       // see Epilogue
  int M, N, K;
  int epi;
  // EPI_QKV_ROPE only
  const int* tok_pos;
  const int* tok_slot;
  void* kv_pool;
  int64_t n_pages;
  int layer, n_q, n_kv, head_dim;
  const void* rope_cs;  // float2 [head_dim/2][M]: (cos, sin) of each token's rotary angles, frequency-major
  // device-resident rounds: the true row count (M is then the capacity the tensor maps cover), and the row count the
  // tile configuration is chosen for (0: M)
  const int* m_dev;
  int m_hint;
  bool m_dev_settled;   // a projection of this stream has already run since the count was written (no need to wait before reading it)
  // folded RMSNorm (see EpiParams in epilogue.cuh); all null / 0 when unused
  const float* ss_in;   // consumer: partial sums of squares of the rows of x's source, [ss_slots][ss_stride]
  int ss_slots, ss_stride;
  float norm_eps;       // the mean is over K (the width of x)
  void* x_out;          // EPI_RESIDUAL_NORM: bf16 [M,N]
  const void* gain;     // EPI_RESIDUAL_NORM: bf16 [N]
  float* ss_out;        // EPI_RESIDUAL_NORM: [column tiles][ss_stride]; *ss_slots_out receives the tile count
};
// legacy tensor path (mma.sync), any M; N multiple of 64 (EPI_SWIGLU: F multiple of 32), K multiple of 32
void launch_gemm_simt(const GemmArgs& a, int* status, cudaStream_t st);
// tcgen05 + TMA path; returns false if the shape is not supported by it
struct TcGemmPlan;  // opaque: cached tensor maps
// ss_slots_out (may be null): how many slots of ss_out an EPI_RESIDUAL_NORM launch fills
bool launch_gemm_tc(const GemmArgs& a, void* tc_state, int* status, cudaStream_t st, int* ss_slots_out = nullptr);
void* tc_state_create(int n_sm);
void tc_state_destroy(void* s);
// debugging aid: force the tile configuration of the following launches (bn 64 / 128 / 256 single CTAs, 384 = CTA pairs
// with 256 x 128 tiles, 512 = CTA pairs with 256 x 256 tiles; 0 = back to the cost model) and the decomposition
// (0 whole tiles, 1 tiles cut over K, 2 the same without the cluster hand-over of thin problems)
void tc_state_force(void* s, int bn, int stream_k);
// zero the arrival counters of cut tiles (after a launch that ended with an error status)
void tc_state_reset(void* s, cudaStream_t st);
// host-only self-test of the tensor-map cache; returns the number of wrong maps handed out
int tc_map_cache_selftest(int n_keys, int* evictions);

// A chain of projections in one persistent kernel (steps with at most 128 rows; see gemm_chain.cu).  Every op reads
// x [M, K] bf16 and w (layout as in GemmArgs); RMSNorm is folded as in EpiParams: EPI_RESIDUAL_NORM ops write x_out and
// the sum-of-squares slots (one per 128-column tile), ops with scale_in multiply their rows by the rstd of ss_slots_in slots.
constexpr int kChainMaxOps = 5;
struct ChainOp {
  const void* x;
  const void* w;
  void* out;
  int N, K, epi;
  int scale_in, ss_slots_in;
  void* x_out;          // EPI_RESIDUAL_NORM
  const void* gain;     // EPI_RESIDUAL_NORM
};
struct ChainCommon {
  float* ss;
  int ss_stride;
  float eps;
  // EPI_QKV_ROPE
  const int* tok_slot;
  const void* rope_cs;
  void* kv_pool;
  int64_t n_pages;
  int layer, n_q, n_kv, head_dim;
};
void* chain_state_create(int n_sm);
void chain_state_destroy(void* s);
void chain_state_reset(void* s, cudaStream_t st);    // after an error status: the grid barrier's counter starts from zero again
bool chain_state_reserve(void* s, int max_rows, long long max_total_kblocks, int min_kb);
// false: not launched (shape not supported, no workspace, or the stream is being captured)
bool launch_gemm_chain(void* s, const ChainOp* ops, int n_ops, int M, const ChainCommon& cm, int* status, cudaStream_t st);

// S5
// use_tc: run the tcgen05 kernel (head_dim 128 only); otherwise the mma.sync kernel
// layout_settled: the work list was written by a kernel that is known to have finished when this one starts (anything but
// the launch right before it): the tcgen05 kernel then reads its work range before it waits for its predecessor
void launch_attention(const BatchLayout& bl, const Dims& dm, int layer, const void* q, void* o, const void* kv_pool,
                      int64_t n_pages, float* part_o, float* part_ml, int tok_per_tile, int n_sm, int* status,
                      cudaStream_t st, bool use_tc, bool layout_settled = false);
void launch_attention_tc_main(const BatchLayout& bl, const Dims& dm, int layer, const void* q, void* o,
                              const void* kv_pool, int64_t n_pages, float* part_o, float* part_ml, int n_sm, int* status,
                              cudaStream_t st, bool layout_settled);
size_t attention_smem_bytes(int head_dim);

// S9b + S10
struct VerifyBuffers {   // DEVICE outputs (library workspace or caller buffers), any may be null
  int *accept_len, *n_emitted, *emitted, *new_ctx_len, *slot_state, *freed_pages, *next_draft, *cont_hit, *top1,
      *top2;
  float *p1, *p2, *entropy, *entropy_mean;
  int *corr_hit, *risky_n, *risky_index, *risky_token;
  int *freed_page_ids;
};
struct RowPartial {      // per (row, vocab chunk)
  float m1, m2;          // largest and second-largest logit of the chunk
  int i1, i2;
  float s, t;            // sum exp(x - m1), sum x exp(x - m1)
};
void launch_verify(const BatchLayout& bl, const void* logits, int logits_dtype, int vocab, RowPartial* partials,
                   int max_chunks_total, const VerifyBuffers& vb, int n_sm, cudaStream_t st);   // (bl.dyn: rows from the device)
int verify_chunks_per_row(int rows, int vocab, int n_sm);

// Block-size rule (Eq. 2-3): table = [blocks (int) x8 | cost x8 | edges x64 | value n_blocks*n_bins*n_blocks*2]
struct PolicyTable {
  int n_blocks, n_bins;
  const int* blocks;
  const float *cost, *edges, *value;
};
void launch_policy(const BatchLayout& bl, const PolicyTable& tb, float* e1, float* e2, int* block_index, int* full,
                   const float* entropy_mean, const int* accept_len, int* next_block, cudaStream_t st);

// KV import / export
void launch_kv_io(bool write, void* pool, int64_t n_pages, int layer, const Dims& dm, const int* page_row_dev, int pos0,
                  int n_pos, void* k, void* v, int* status, cudaStream_t st);

}  // namespace recg

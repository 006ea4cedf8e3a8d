// The C ABI: context, workspace, descriptor validation and the per-step launch sequence.
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#include "../../include/recg.h"
#include "common.cuh"
#include "kernels.h"

using namespace recg;

namespace {

thread_local std::string g_init_error;
constexpr size_t kVoutMirrorMax = 1 << 20;   // verify outputs up to this size come back to the host in one copy

// One cudaMalloc, carved with 256-byte alignment.  With guard = true (RECG_FLAG_DEBUG_CHECKS) every region is followed
// by a 256-byte guard band; the offsets of the bands are recorded so that they can be filled with a pattern at init
// and checked by recg_sync(): a kernel that writes past the end of a workspace region shows up there.
struct DeviceArena {
  uint8_t* base = nullptr;
  size_t size = 0, used = 0;
  bool guard = false;
  std::vector<size_t> guards;   // byte offsets of the guard bands
  template <typename T> T* take(size_t n) {
    used = (used + 255) & ~size_t(255);
    T* p = reinterpret_cast<T*>(base ? base + used : nullptr);
    used += n * sizeof(T);
    if (guard) {
      used = (used + 255) & ~size_t(255);
      guards.push_back(used);
      used += 256;
    }
    return p;
  }
};

}  // namespace

struct recg_ctx {
  recg_config cfg;
  Dims dm;
  bool has_weights = false;
  const void *embed = nullptr, *final_norm = nullptr, *lm_head = nullptr;
  std::vector<const void*> attn_norm, wqkv, wo, ffn_norm, w_gate_up, w_down;
  cudaStream_t stream = nullptr;
  int n_sm = 0, tok_per_tile = 0, target_items = 0;
  std::string err;

  DeviceArena arena;
  // descriptor staging (device)
  int* d_desc = nullptr;
  size_t desc_ints = 0;
  BatchLayout bl{};
  bool layout_valid = false;
  bool layout_has_pages = false;
  int64_t last_pool_pages = 0;
  void* last_pool = nullptr;
  // activations
  float* h = nullptr;
  __nv_bfloat16 *x = nullptr, *q = nullptr, *o = nullptr, *act = nullptr;
  void* logits = nullptr;
  bool logits_valid = false;
  float2* rope_cs = nullptr;
  float* ss = nullptr;           // folded RMSNorm: partial sums of squares of the residual rows, [slot][max_tokens]
  int ss_slots = 0;              // slots the last producer filled
  float *part_o = nullptr, *part_ml = nullptr;
  RowPartial* vpart = nullptr;
  int max_chunks_total = 0;
  VerifyBuffers vws{};
  size_t vout_off = 0, vout_bytes = 0;   // the verify outputs are one contiguous region of the arena ...
  uint8_t* h_vout = nullptr;             // ... mirrored by one pinned host buffer: a single copy brings all results back
  int* d_status = nullptr;
  int* d_dyn = nullptr;          // device-resident rounds: {n_tok, n_ver} of the round laid out last
  int* d_page_row = nullptr;
  size_t* d_guards = nullptr;    // RECG_FLAG_DEBUG_CHECKS: offsets of the guard bands, on the device
  int n_guards = 0;
  int* d_policy = nullptr;       // block-size rule: [blocks x8 | cost x8 | edges x64 | value]
  PolicyTable policy{};
  bool policy_loaded = false;
  std::vector<int> h_policy;
  void* tc_state = nullptr;
  void* chain_state = nullptr;   // RECG_FLAG_CHAIN
  std::vector<int> h_desc;
  std::vector<int> h_page_owner;   // debug checks: which request names a page
  // optional per-class timing
  bool timing = false;
  std::vector<cudaEvent_t> ev_pool;
  size_t ev_used = 0;
  std::vector<int> ev_class;  // class of the interval that ENDS at event i (-1 for an opening event)
  int ev_launches[RECG_TIMING_CLASSES] = {0};

  void mark(int cls, int launches = 0) {  // cls < 0 opens a sequence; otherwise closes an interval of that class
    if (!timing) return;
    if (ev_used == ev_pool.size()) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) return;
      ev_pool.push_back(e);
      ev_class.push_back(-1);
    }
    cudaEventRecord(ev_pool[ev_used], stream);
    ev_class[ev_used] = cls;
    if (cls >= 0) ev_launches[cls] += launches;
    ++ev_used;
  }
};

namespace {

recg_status fail(recg_ctx* c, recg_status s, const std::string& msg) {
  if (c) c->err = msg; else g_init_error = msg;
  return s;
}
#define CU(call)                                                                                    \
  do {                                                                                              \
    cudaError_t e__ = (call);                                                                       \
    if (e__ != cudaSuccess)                                                                         \
      return fail(ctx, RECG_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e__));         \
  } while (0)

size_t carve(recg_ctx* c, DeviceArena& A) {
  const recg_config& g = c->cfg;
  const size_t Cm = g.max_requests, Tm = g.max_tokens, Pm = g.max_pages_per_request;
  const Dims& d = c->dm;
  c->desc_ints = 9 * Cm + 2 * (Cm + 1) + Tm + Cm * Pm;
  c->d_desc = A.take<int>(c->desc_ints);
  BatchLayout& bl = c->bl;
  bl.tok_id = A.take<int>(Tm);
  bl.tok_req = A.take<int>(Tm);
  bl.tok_pos = A.take<int>(Tm);
  bl.tok_slot = A.take<int>(Tm);
  bl.tok_climit = A.take<int>(Tm);
  bl.tok_lo = A.take<int>(Tm);
  bl.tok_hi = A.take<int>(Tm);
  const size_t max_tiles = (size_t)d.n_kv * (Cm + Tm / c->tok_per_tile + 1);
  bl.max_parts = 4 * c->target_items;      // two lines of work, each cut at fewer than target_items places (see layout.cu)
  bl.max_items = (int)(4 * c->target_items + max_tiles);
  bl.items = A.take<AttnItem>(bl.max_items);
  bl.item_cta = A.take<int>(bl.max_items);
  bl.tiles = A.take<AttnTile>(max_tiles);
  bl.tile_off = A.take<int>(Cm + 1);
  bl.cta_off = A.take<int>(4 * (c->target_items + 1));
  bl.counts = A.take<int>(4);
  c->d_status = A.take<int>(1);
  c->d_dyn = A.take<int>(4);
  c->d_page_row = A.take<int>(Pm);
  c->d_policy = A.take<int>(8 + 8 + 64 + RECG_POLICY_MAX_BLOCKS * RECG_POLICY_MAX_BINS * RECG_POLICY_MAX_BLOCKS * 2);
  c->rope_cs = A.take<float2>(Tm * (d.head_dim / 2));
  c->part_o = A.take<float>((size_t)bl.max_parts * 128 * d.head_dim);
  c->part_ml = A.take<float>((size_t)bl.max_parts * 128 * 2);
  c->max_chunks_total = (int)(Tm + 4 * c->n_sm + 64);
  c->vpart = A.take<RowPartial>(c->max_chunks_total);
  VerifyBuffers& v = c->vws;
  c->vout_off = (A.used + 255) & ~size_t(255);
  v.accept_len = A.take<int>(Cm);
  v.n_emitted = A.take<int>(Cm);
  v.emitted = A.take<int>(Tm);
  v.new_ctx_len = A.take<int>(Cm);
  v.slot_state = A.take<int>(Tm);
  v.freed_pages = A.take<int>(Cm);
  v.next_draft = A.take<int>(Tm);
  v.cont_hit = A.take<int>(Cm);
  v.top1 = A.take<int>(Tm);
  v.top2 = A.take<int>(Tm);
  v.p1 = A.take<float>(Tm);
  v.p2 = A.take<float>(Tm);
  v.entropy = A.take<float>(Tm);
  v.entropy_mean = A.take<float>(Cm);
  v.corr_hit = A.take<int>(2 * Cm);
  v.risky_n = A.take<int>(3 * Cm);
  v.risky_index = A.take<int>(6 * Cm);
  v.risky_token = A.take<int>(6 * Cm);
  v.freed_page_ids = A.take<int>(Tm);
  c->vout_bytes = A.used - c->vout_off;
  c->q = A.take<__nv_bfloat16>(Tm * d.n_q * d.head_dim);
  c->o = A.take<__nv_bfloat16>(Tm * d.n_q * d.head_dim);
  if (c->has_weights) {
    c->h = A.take<float>(Tm * d.hidden);
    c->x = A.take<__nv_bfloat16>(Tm * d.hidden);
    c->ss = A.take<float>(Tm * (size_t)(d.hidden / 64 + 1));   // a column tile is at least 64 wide
    c->act = A.take<__nv_bfloat16>(Tm * d.ffn);
    const size_t esz = (g.flags & RECG_FLAG_LOGITS_BF16) ? 2 : 4;
    c->logits = A.take<uint8_t>(Tm * (size_t)d.vocab * esz);
  }
  if (A.guard) {
    c->n_guards = (int)A.guards.size();
    const bool was = A.guard;
    A.guard = false;
    c->d_guards = A.take<size_t>(A.guards.size() + 1);
    A.guard = was;
  }
  return A.used + 256;
}

// Rows of request r: verify tokens, continuation masks and the correction branches (replacement + masks each).
static inline int request_rows(const recg_batch* b, int r) {
  const int nc = b->n_corr ? b->n_corr[r] : 0;
  return b->verify_len[r] + b->block_size[r] + nc * (1 + (nc ? b->corr_block[r] : 0));
}

// Validate a batch and pack [ctx_len | verify_len | block_size | corr | cu_tok | cu_ver | verify_tokens | page_table].
recg_status pack_batch(recg_ctx* ctx, const recg_batch* b, bool need_pages, bool need_tokens, int* T_out, int* Tv_out) {
  if (!b || b->n_req <= 0 || !b->ctx_len || !b->verify_len || !b->block_size)
    return fail(ctx, RECG_ERR_INVALID_ARG, "batch: null descriptor array or n_req <= 0");
  const int C = b->n_req;
  if (C > ctx->cfg.max_requests) return fail(ctx, RECG_ERR_CAPACITY, "batch: n_req exceeds max_requests");
  const bool pages = b->page_table != nullptr;
  if (need_pages && (!pages || !b->kv_pool || b->kv_pool_pages <= 0))
    return fail(ctx, RECG_ERR_INVALID_ARG, "batch: page_table and kv_pool are required");
  if (pages && (b->page_table_stride <= 0 || b->page_table_stride > ctx->cfg.max_pages_per_request))
    return fail(ctx, RECG_ERR_CAPACITY, "batch: page_table_stride exceeds max_pages_per_request");
  if (b->n_corr && (!b->corr_index || !b->corr_token || !b->corr_block))
    return fail(ctx, RECG_ERR_INVALID_ARG, "batch: n_corr given without corr_index, corr_token and corr_block");
  long long T = 0, Tv = 0;
  for (int r = 0; r < C; ++r) {
    const int L = b->ctx_len[r], v = b->verify_len[r], k = b->block_size[r];
    if (L < 0 || v < 0 || k < 0 || v + k < 1)
      return fail(ctx, RECG_ERR_INVALID_ARG, "batch: negative length or a request without rows");
    if (b->n_corr && b->n_corr[r] != 0) {
      const int nc = b->n_corr[r];
      if (nc < 0 || nc > 2 || b->corr_block[r] < 0)
        return fail(ctx, RECG_ERR_INVALID_ARG, "batch: n_corr must be 0, 1 or 2 and corr_block >= 0");
      for (int q = 0; q < nc; ++q) {
        const int i = b->corr_index[2 * r + q], tok = b->corr_token[2 * r + q];
        if (i < 1 || i > v - 1 || (q > 0 && i <= b->corr_index[2 * r + q - 1]))
          return fail(ctx, RECG_ERR_INVALID_ARG, "batch: corr_index must name drafts y_1 .. y_{v-1} in increasing order");
        if (tok < 0 || tok >= ctx->cfg.vocab) return fail(ctx, RECG_ERR_INVALID_ARG, "batch: corr_token outside the vocabulary");
      }
    }
    const int n = request_rows(b, r);
    if (pages) {
      const long long need = ((long long)L + n + kPageSize - 1) / kPageSize;
      if (need > b->page_table_stride)
        return fail(ctx, RECG_ERR_CAPACITY, "batch: page table row does not cover ctx_len plus the rows of the request");
    }
    T += n;
    Tv += v;
  }
  if (T > ctx->cfg.max_tokens) return fail(ctx, RECG_ERR_CAPACITY, "batch: token count exceeds max_tokens");
  if (Tv > 0 && !b->verify_tokens && need_tokens) return fail(ctx, RECG_ERR_INVALID_ARG, "batch: verify_tokens is null");
  const int stride = pages ? b->page_table_stride : 0;
  std::vector<int>& hd = ctx->h_desc;
  hd.resize(9 * (size_t)C + 2 * ((size_t)C + 1) + (size_t)Tv + (size_t)C * stride);
  int* p = hd.data();
  memcpy(p, b->ctx_len, C * sizeof(int));
  memcpy(p + C, b->verify_len, C * sizeof(int));
  memcpy(p + 2 * C, b->block_size, C * sizeof(int));
  int* corr = p + 3 * C;   // per request: count, mask tokens per branch, index 0, index 1, token 0, token 1
  int* cu_tok = p + 9 * C;
  int* cu_ver = cu_tok + (C + 1);
  cu_tok[0] = cu_ver[0] = 0;
  for (int r = 0; r < C; ++r) {
    const int nc = b->n_corr ? b->n_corr[r] : 0;
    int* cr = corr + 6 * r;
    cr[0] = nc;
    cr[1] = nc ? b->corr_block[r] : 0;
    for (int q = 0; q < 2; ++q) {
      cr[2 + q] = q < nc ? b->corr_index[2 * r + q] : 0;
      cr[4 + q] = q < nc ? b->corr_token[2 * r + q] : 0;
    }
    cu_tok[r + 1] = cu_tok[r] + request_rows(b, r);
    cu_ver[r + 1] = cu_ver[r] + b->verify_len[r];
  }
  int* vt = cu_ver + (C + 1);
  if (Tv && b->verify_tokens) memcpy(vt, b->verify_tokens, Tv * sizeof(int));
  else if (Tv) memset(vt, 0, Tv * sizeof(int));
  int* pt = vt + Tv;
  if (pages) {
    for (int r = 0; r < C; ++r) {
      const long long need = ((long long)b->ctx_len[r] + request_rows(b, r) + kPageSize - 1) / kPageSize;
      for (int i = 0; i < stride; ++i) {
        const int pg = b->page_table[(size_t)r * stride + i];
        if (i < need && (pg < 0 || pg >= b->kv_pool_pages) && b->kv_pool)
          return fail(ctx, RECG_ERR_INVALID_ARG, "batch: page id outside the pool");
        pt[(size_t)r * stride + i] = pg;
      }
    }
  }
  if (pages && (ctx->cfg.flags & RECG_FLAG_DEBUG_CHECKS)) {
    // debug checks: a page that takes new rows of one request must not appear in another request's table (two
    // requests would overwrite each other's tentative K/V), nor twice in its own
    std::vector<int>& seen = ctx->h_page_owner;
    seen.assign((size_t)b->kv_pool_pages, -1);
    for (int r = 0; r < C; ++r) {
      const long long need = ((long long)b->ctx_len[r] + request_rows(b, r) + kPageSize - 1) / kPageSize;
      const int first_new = b->ctx_len[r] / kPageSize;
      for (int i = 0; i < need; ++i) {
        const int pg = pt[(size_t)r * stride + i];
        if (pg < 0 || pg >= b->kv_pool_pages) continue;    // reported above when a pool was given
        const int tag = i >= first_new ? 2 * r + 1 : 2 * r;  // odd: the page takes new rows
        const int old = seen[pg];
        if (old >= 0 && ((old >> 1) == r || (old & 1) || (tag & 1)))
          return fail(ctx, RECG_ERR_INVALID_ARG, "batch (debug checks): a page that receives new rows is named twice (requests " +
                                                     std::to_string(old >> 1) + " and " + std::to_string(r) + ")");
        if (old < 0 || (tag & 1)) seen[pg] = tag;
      }
    }
  }
  BatchLayout& bl = ctx->bl;
  int* d = ctx->d_desc;
  bl.dyn = nullptr;
  bl.n_req = C;
  bl.n_tok = (int)T;
  bl.n_ver = (int)Tv;
  bl.pt_stride = stride;
  bl.ctx_len = d;
  bl.verify_len = d + C;
  bl.block_size = d + 2 * C;
  bl.corr = d + 3 * C;
  bl.cu_tok = d + 9 * C;
  bl.risk_delta = b->risk_delta > 0.f ? b->risk_delta : 0.5f;
  bl.cu_ver = bl.cu_tok + (C + 1);
  bl.verify_tokens = bl.cu_ver + (C + 1);
  bl.page_table = pages ? bl.verify_tokens + Tv : nullptr;
  *T_out = (int)T;
  *Tv_out = (int)Tv;
  return RECG_OK;
}

recg_status upload_and_layout(recg_ctx* ctx, const recg_batch* b, bool need_pages, bool need_tokens = true) {
  int T = 0, Tv = 0;
  ctx->layout_valid = false;
  recg_status s = pack_batch(ctx, b, need_pages, need_tokens, &T, &Tv);
  if (s != RECG_OK) return s;
  CU(cudaMemcpyAsync(ctx->d_desc, ctx->h_desc.data(), ctx->h_desc.size() * sizeof(int), cudaMemcpyHostToDevice,
                     ctx->stream));
  const int64_t n_pages = b->page_table ? (b->kv_pool ? b->kv_pool_pages : (int64_t)1 << 40) : 0;
  launch_layout(ctx->bl, ctx->dm, ctx->tok_per_tile, ctx->target_items, n_pages, ctx->d_status, ctx->stream);
  CU(cudaGetLastError());
  ctx->layout_valid = true;
  ctx->layout_has_pages = b->page_table != nullptr;
  ctx->last_pool = b->kv_pool;
  ctx->last_pool_pages = b->kv_pool_pages;
  return RECG_OK;
}

recg_status run_gemm(recg_ctx* ctx, const GemmArgs& a, int* ss_slots_out = nullptr) {
  bool done = false;
  if (!(ctx->cfg.flags & RECG_FLAG_SIMT_GEMM)) done = launch_gemm_tc(a, ctx->tc_state, ctx->d_status, ctx->stream, ss_slots_out);
  if (!done) {
    // the folded RMSNorm and device-side row counts exist on the tcgen05 path only: such a projection must not fall back
    if (a.ss_in || a.epi == EPI_RESIDUAL_NORM || a.m_dev) {
      cudaGetLastError();
      return fail(ctx, RECG_ERR_INTERNAL, "projection: the tcgen05 kernel refused a shape of the step");
    }
    launch_gemm_simt(a, ctx->d_status, ctx->stream);
  }
  CU(cudaGetLastError());
  return RECG_OK;
}

}  // namespace

extern "C" {

size_t recg_kv_pool_bytes(const recg_config* cfg, int64_t n_pages) {
  if (!cfg || n_pages <= 0) return 0;
  return (size_t)cfg->n_layers * (size_t)n_pages * cfg->n_kv_heads * 2 * kPageSize * cfg->head_dim * 2;
}

const char* recg_last_error(const recg_ctx* ctx) { return ctx ? ctx->err.c_str() : g_init_error.c_str(); }

recg_status recg_init(recg_ctx** out, const recg_config* cfg, const recg_weights* w, void* cuda_stream) {
  recg_ctx* ctx = nullptr;  // errors before allocation go to the thread-local text
  if (!out || !cfg) return fail(ctx, RECG_ERR_INVALID_ARG, "recg_init: null argument");
  *out = nullptr;
  const recg_config& g = *cfg;
  if (g.n_layers < 0 || g.hidden <= 0 || g.n_q_heads <= 0 || g.n_kv_heads <= 0 || g.vocab <= 1 || g.ffn <= 0 ||
      g.max_requests <= 0 || g.max_tokens <= 0 || g.max_pages_per_request <= 0)
    return fail(ctx, RECG_ERR_INVALID_ARG, "recg_init: non-positive dimension or capacity");
  if (g.max_requests > kMaxLayoutRequests || g.max_tokens > (1 << 20))
    return fail(ctx, RECG_ERR_CAPACITY, "recg_init: at most 4096 requests and 1048576 rows per step");
  if (g.page_size != kPageSize) return fail(ctx, RECG_ERR_SHAPE, "recg_init: page_size must be 16");
  if (g.head_dim != 64 && g.head_dim != 128) return fail(ctx, RECG_ERR_SHAPE, "recg_init: head_dim must be 64 or 128");
  if (g.n_q_heads % g.n_kv_heads) return fail(ctx, RECG_ERR_SHAPE, "recg_init: n_q_heads must be a multiple of n_kv_heads");
  const int group = g.n_q_heads / g.n_kv_heads;
  if (group > 16) return fail(ctx, RECG_ERR_SHAPE, "recg_init: at most 16 query heads per kv head");
  if (g.hidden % 64 || g.ffn % 64 || g.vocab % 16 || ((g.n_q_heads + 2 * g.n_kv_heads) * g.head_dim) % 128)
    return fail(ctx, RECG_ERR_SHAPE, "recg_init: hidden and ffn must be multiples of 64, vocab of 16, qkv width of 128");
  if (g.mask_token_id >= g.vocab) return fail(ctx, RECG_ERR_INVALID_ARG, "recg_init: mask_token_id outside the vocabulary");
  if (w && g.n_layers > 0 &&
      (!w->embed || !w->final_norm || !w->lm_head || !w->attn_norm || !w->wqkv || !w->wo || !w->ffn_norm ||
       !w->w_gate_up || !w->w_down))
    return fail(ctx, RECG_ERR_INVALID_ARG, "recg_init: null weight pointer");
  int dev = 0, n_sm = 0, cc_major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return fail(ctx, RECG_ERR_CUDA, "recg_init: no usable CUDA device (there is no CPU fallback)");
  if (cc_major != 10) return fail(ctx, RECG_ERR_CUDA, "recg_init: the kernels are built for sm_100a only");

  ctx = new recg_ctx();
  ctx->cfg = g;
  ctx->dm = Dims{g.n_layers, g.hidden, g.n_q_heads, g.n_kv_heads, g.head_dim, g.ffn, g.vocab, g.rope_base, g.rms_eps,
                 g.mask_token_id < 0 ? g.vocab - 1 : g.mask_token_id};
  ctx->stream = static_cast<cudaStream_t>(cuda_stream);
  ctx->n_sm = n_sm;
  ctx->tok_per_tile = 128 / group;
  ctx->target_items = n_sm;
  ctx->has_weights = w != nullptr;
  if (w) {
    ctx->embed = w->embed;
    ctx->final_norm = w->final_norm;
    ctx->lm_head = w->lm_head;
    for (int l = 0; l < g.n_layers; ++l) {
      ctx->attn_norm.push_back(w->attn_norm[l]);
      ctx->wqkv.push_back(w->wqkv[l]);
      ctx->wo.push_back(w->wo[l]);
      ctx->ffn_norm.push_back(w->ffn_norm[l]);
      ctx->w_gate_up.push_back(w->w_gate_up[l]);
      ctx->w_down.push_back(w->w_down[l]);
      if (!w->attn_norm[l] || !w->wqkv[l] || !w->wo[l] || !w->ffn_norm[l] || !w->w_gate_up[l] || !w->w_down[l]) {
        delete ctx;
        ctx = nullptr;
        return fail(ctx, RECG_ERR_INVALID_ARG, "recg_init: null per-layer weight pointer");
      }
    }
  }
  DeviceArena probe;
  probe.guard = ctx->arena.guard = (g.flags & RECG_FLAG_DEBUG_CHECKS) != 0;
  const size_t bytes = carve(ctx, probe);
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&ctx->arena.base), bytes);
  if (e != cudaSuccess) {
    std::string msg = std::string("recg_init: workspace cudaMalloc of ") + std::to_string(bytes) + " bytes: " + cudaGetErrorString(e);
    delete ctx;
    ctx = nullptr;
    return fail(ctx, RECG_ERR_CUDA, msg);
  }
  ctx->arena.size = bytes;
  carve(ctx, ctx->arena);
  if (ctx->n_guards) {   // fill the guard bands behind every workspace region
    if (cudaMemcpyAsync(ctx->d_guards, ctx->arena.guards.data(), ctx->n_guards * sizeof(size_t), cudaMemcpyHostToDevice,
                        ctx->stream) != cudaSuccess || cudaStreamSynchronize(ctx->stream) != cudaSuccess) {
      cudaFree(ctx->arena.base);
      delete ctx;
      ctx = nullptr;
      return fail(ctx, RECG_ERR_CUDA, "recg_init: cannot upload the guard-band offsets");
    }
    launch_guard_fill(ctx->arena.base, ctx->d_guards, ctx->n_guards, ctx->stream);
  }
  if (ctx->vout_bytes <= kVoutMirrorMax && cudaMallocHost(reinterpret_cast<void**>(&ctx->h_vout), ctx->vout_bytes) != cudaSuccess) {
    cudaGetLastError();
    ctx->h_vout = nullptr;   // fall back to one copy per output array
  }
  cudaMemsetAsync(ctx->d_status, 0, sizeof(int), ctx->stream);
  ctx->tc_state = tc_state_create(n_sm);
  if ((g.flags & RECG_FLAG_CHAIN) && w && g.head_dim == 128 && !(g.flags & RECG_FLAG_SIMT_GEMM)) {
    ctx->chain_state = chain_state_create(n_sm);
    // the widest line of k-blocks in the model: the LM head (128-column tiles) or gate|up (64 output columns per tile)
    const long long kb_h = g.hidden / 64;
    long long most = (long long)((g.vocab + 127) / 128) * kb_h;
    const long long gu = (long long)((g.ffn + 63) / 64) * kb_h;
    if (gu > most) most = gu;
    if (ctx->chain_state && !chain_state_reserve(ctx->chain_state, g.max_tokens < 128 ? g.max_tokens : 128, most, (int)kb_h)) {
      chain_state_destroy(ctx->chain_state);
      ctx->chain_state = nullptr;
    }
  }
  *out = ctx;
  return RECG_OK;
}

recg_status recg_timing_enable(recg_ctx* ctx, int32_t enable) {
  if (!ctx) return RECG_ERR_INVALID_ARG;
  ctx->timing = enable != 0;
  return RECG_OK;
}

recg_status recg_timing_read(recg_ctx* ctx, float* ms, int32_t* launches) {
  if (!ctx) return RECG_ERR_INVALID_ARG;
  CU(cudaStreamSynchronize(ctx->stream));
  for (int c = 0; c < RECG_TIMING_CLASSES; ++c) {
    if (ms) ms[c] = 0.f;
    if (launches) launches[c] = ctx->ev_launches[c];
    ctx->ev_launches[c] = 0;
  }
  for (size_t i = 1; i < ctx->ev_used; ++i) {
    const int cls = ctx->ev_class[i];
    if (cls < 0) continue;
    float t = 0.f;
    if (cudaEventElapsedTime(&t, ctx->ev_pool[i - 1], ctx->ev_pool[i]) == cudaSuccess && ms) ms[cls] += t;
  }
  ctx->ev_used = 0;
  return RECG_OK;
}

recg_status recg_free(recg_ctx* ctx) {
  if (!ctx) return RECG_OK;
  cudaStreamSynchronize(ctx->stream);
  for (cudaEvent_t e : ctx->ev_pool) cudaEventDestroy(e);
  if (ctx->tc_state) tc_state_destroy(ctx->tc_state);
  if (ctx->chain_state) chain_state_destroy(ctx->chain_state);
  if (ctx->arena.base) cudaFree(ctx->arena.base);
  if (ctx->h_vout) cudaFreeHost(ctx->h_vout);
  delete ctx;
  return RECG_OK;
}

recg_status recg_sync(recg_ctx* ctx) {
  if (!ctx) return RECG_ERR_INVALID_ARG;
  int st = 0;
  if (ctx->n_guards) launch_guard_check(ctx->arena.base, ctx->d_guards, ctx->n_guards, ctx->d_status, ctx->stream);
  CU(cudaMemcpyAsync(&st, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  if (st != DEV_OK) {
    cudaMemsetAsync(ctx->d_status, 0, sizeof(int), ctx->stream);
    // a projection that gave up may have left arrival counters of cut tiles behind: the next launch starts clean
    tc_state_reset(ctx->tc_state, ctx->stream);
    chain_state_reset(ctx->chain_state, ctx->stream);
    if (st == DEV_GUARD) {
      launch_guard_fill(ctx->arena.base, ctx->d_guards, ctx->n_guards, ctx->stream);
      return fail(ctx, RECG_ERR_INTERNAL, "device: a guard band behind a workspace region was overwritten");
    }
    if (st == DEV_BAD_INDEX) return fail(ctx, RECG_ERR_INTERNAL, "device: a page id or slot was out of range");
    return fail(ctx, RECG_ERR_TIMEOUT, "device: a bounded wait gave up (code " + std::to_string(st) + ")");
  }
  return RECG_OK;
}

// The forward over the batch laid out last (ctx->bl): embedding, the layers, final norm and LM head.  m_hint: device-
// resident rounds only, the row count the projections' tile configurations are chosen for.
static recg_status run_forward(recg_ctx* ctx, void* kv_pool, int64_t kv_pool_pages, int m_hint, recg_logits* logits) {
  recg_status s = RECG_OK;
  const Dims& d = ctx->dm;
  const BatchLayout& bl = ctx->bl;
  const int T = bl.n_tok;
  cudaStream_t st = ctx->stream;
  launch_rope_table(bl.tok_pos, T, d.head_dim, d.rope_base, ctx->rope_cs, st, bl.dyn);
  // RMSNorm runs as a kernel of its own, or (RECG_FLAG_FOLD_NORM, tcgen05 path only) folded into the projections:
  // whoever writes the residual stream also writes x = bf16(h * gain of the next norm) and partial sums of squares per
  // row, and the projection that reads x scales its accumulator rows by the row's rstd.
  // (RECG_FLAG_CHAIN: steps of at most 128 rows run the projections between two attention calls as one persistent kernel)
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  const bool chain = ctx->chain_state && !bl.dyn && T <= 128 && d.n_layers > 0 && (d.n_q * d.head_dim) % 64 == 0 &&
                     d.hidden % 128 == 0 && d.ffn % 64 == 0 &&
                     cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone;
  const bool fold = ((ctx->cfg.flags & RECG_FLAG_FOLD_NORM) || chain) && !(ctx->cfg.flags & RECG_FLAG_SIMT_GEMM);
  const int Tm = ctx->cfg.max_tokens;
  const void* first_gain = d.n_layers > 0 ? ctx->attn_norm[0] : ctx->final_norm;
  launch_embed(bl, d, ctx->embed, ctx->h, fold ? first_gain : nullptr, ctx->x, ctx->ss, st);
  int slots = 1;
  CU(cudaGetLastError());
  ctx->mark(0, 3);
  const int qdim = d.n_q * d.head_dim;
  int n_proj = 0;                        // projections enqueued so far in this step
  auto normed = [&](GemmArgs& g) {       // g reads the normalised residual stream
    g.x = ctx->x;
    g.K = d.hidden;
    g.m_dev = bl.dyn;
    g.m_dev_settled = n_proj++ > 0;
    g.m_hint = m_hint;
    if (fold) { g.ss_in = ctx->ss; g.ss_slots = slots; g.ss_stride = Tm; g.norm_eps = d.rms_eps; }
  };
  auto residual = [&](GemmArgs& g, const void* next_gain) {   // g adds into the residual stream
    g.out = ctx->h;
    g.N = d.hidden;
    g.m_dev = bl.dyn;
    g.m_dev_settled = n_proj++ > 0;
    g.m_hint = m_hint;
    g.epi = fold ? EPI_RESIDUAL_NORM : EPI_RESIDUAL;
    if (fold) { g.x_out = ctx->x; g.gain = next_gain; g.ss_out = ctx->ss; g.ss_stride = Tm; }
  };
  const bool lbf = ctx->cfg.flags & RECG_FLAG_LOGITS_BF16;
  for (int l = 0; l < d.n_layers; ++l) {
    if (chain && l > 0) {
      // the QKV projection of this layer was the last op of the previous layer's chain
    } else {
    if (!fold) {
      launch_rmsnorm(ctx->h, ctx->attn_norm[l], ctx->x, T, d.hidden, d.rms_eps, st, bl.dyn);
      ctx->mark(1, 1);
    }
    GemmArgs a{};
    normed(a);
    a.w = ctx->wqkv[l]; a.out = ctx->q;
    a.M = T; a.N = (d.n_q + 2 * d.n_kv) * d.head_dim; a.epi = EPI_QKV_ROPE;
    a.tok_pos = bl.tok_pos; a.tok_slot = bl.tok_slot; a.kv_pool = kv_pool; a.n_pages = kv_pool_pages;
    a.layer = l; a.n_q = d.n_q; a.n_kv = d.n_kv; a.head_dim = d.head_dim; a.rope_cs = ctx->rope_cs;
    if ((s = run_gemm(ctx, a)) != RECG_OK) return s;
    ctx->mark(2, 1);
    }
    launch_attention(bl, d, l, ctx->q, ctx->o, kv_pool, kv_pool_pages, ctx->part_o, ctx->part_ml,
                     ctx->tok_per_tile, ctx->n_sm, ctx->d_status, st, !(ctx->cfg.flags & RECG_FLAG_SIMT_ATTENTION), true);
    CU(cudaGetLastError());
    ctx->mark(3, 2);
    if (chain) {
      const bool last = l + 1 == d.n_layers;
      const int slots_h = d.hidden / 128;      // sum-of-squares slots a residual op of the chain fills
      ChainOp ops[4] = {};
      ops[0].x = ctx->o; ops[0].w = ctx->wo[l]; ops[0].out = ctx->h; ops[0].N = d.hidden; ops[0].K = qdim;
      ops[0].epi = EPI_RESIDUAL_NORM; ops[0].x_out = ctx->x; ops[0].gain = ctx->ffn_norm[l];
      ops[1].x = ctx->x; ops[1].w = ctx->w_gate_up[l]; ops[1].out = ctx->act; ops[1].N = d.ffn; ops[1].K = d.hidden;
      ops[1].epi = EPI_SWIGLU; ops[1].scale_in = 1; ops[1].ss_slots_in = slots_h;
      ops[2].x = ctx->act; ops[2].w = ctx->w_down[l]; ops[2].out = ctx->h; ops[2].N = d.hidden; ops[2].K = d.ffn;
      ops[2].epi = EPI_RESIDUAL_NORM; ops[2].x_out = ctx->x; ops[2].gain = last ? ctx->final_norm : ctx->attn_norm[l + 1];
      ops[3].x = ctx->x; ops[3].K = d.hidden; ops[3].scale_in = 1; ops[3].ss_slots_in = slots_h;
      if (last) {
        ops[3].w = ctx->lm_head; ops[3].out = ctx->logits; ops[3].N = d.vocab; ops[3].epi = lbf ? EPI_PLAIN_BF16 : EPI_PLAIN_F32;
      } else {
        ops[3].w = ctx->wqkv[l + 1]; ops[3].out = ctx->q; ops[3].N = (d.n_q + 2 * d.n_kv) * d.head_dim; ops[3].epi = EPI_QKV_ROPE;
      }
      ChainCommon cm{};
      cm.ss = ctx->ss; cm.ss_stride = Tm; cm.eps = d.rms_eps; cm.tok_slot = bl.tok_slot; cm.rope_cs = ctx->rope_cs;
      cm.kv_pool = kv_pool; cm.n_pages = kv_pool_pages; cm.layer = l + 1; cm.n_q = d.n_q; cm.n_kv = d.n_kv; cm.head_dim = d.head_dim;
      if (!launch_gemm_chain(ctx->chain_state, ops, 4, T, cm, ctx->d_status, st)) {
        cudaGetLastError();
        return fail(ctx, RECG_ERR_INTERNAL, "projection chain: launch refused");
      }
      CU(cudaGetLastError());
      ctx->mark(5, 1);
      continue;
    }
    GemmArgs b{};
    residual(b, ctx->ffn_norm[l]);
    b.x = ctx->o; b.w = ctx->wo[l]; b.M = T; b.K = qdim;
    if ((s = run_gemm(ctx, b, &slots)) != RECG_OK) return s;
    ctx->mark(4, 1);
    if (!fold) {
      launch_rmsnorm(ctx->h, ctx->ffn_norm[l], ctx->x, T, d.hidden, d.rms_eps, st, bl.dyn);
      ctx->mark(1, 1);
    }
    GemmArgs c{};
    normed(c);
    c.w = ctx->w_gate_up[l]; c.out = ctx->act; c.M = T; c.N = d.ffn; c.epi = EPI_SWIGLU;
    if ((s = run_gemm(ctx, c)) != RECG_OK) return s;
    ctx->mark(5, 1);
    GemmArgs e{};
    residual(e, l + 1 < d.n_layers ? ctx->attn_norm[l + 1] : ctx->final_norm);
    e.x = ctx->act; e.w = ctx->w_down[l]; e.M = T; e.K = d.ffn;
    if ((s = run_gemm(ctx, e, &slots)) != RECG_OK) return s;
    ctx->mark(6, 1);
  }
  if (!chain) {      // (the chain of the last layer ends with the LM head)
    if (!fold) {
      launch_rmsnorm(ctx->h, ctx->final_norm, ctx->x, T, d.hidden, d.rms_eps, st, bl.dyn);
      ctx->mark(1, 1);
    }
    GemmArgs f{};
    normed(f);
    f.w = ctx->lm_head; f.out = ctx->logits; f.M = T; f.N = d.vocab;
    f.epi = lbf ? EPI_PLAIN_BF16 : EPI_PLAIN_F32;
    if ((s = run_gemm(ctx, f)) != RECG_OK) return s;
    ctx->mark(7, 1);
  }
  ctx->logits_valid = true;
  if (logits) {
    logits->data = ctx->logits;
    logits->dtype = lbf ? RECG_DTYPE_BF16 : RECG_DTYPE_F32;
    logits->n_rows = T;
    logits->vocab = d.vocab;
  }
  return RECG_OK;
}

recg_status recg_step(recg_ctx* ctx, const recg_batch* batch, recg_logits* logits) {
  if (!ctx) return RECG_ERR_INVALID_ARG;
  if (!ctx->has_weights) return fail(ctx, RECG_ERR_INVALID_ARG, "recg_step: the context was created without weights");
  ctx->logits_valid = false;
  ctx->mark(-1);
  recg_status s = upload_and_layout(ctx, batch, true);
  if (s != RECG_OK) return s;
  return run_forward(ctx, batch->kv_pool, batch->kv_pool_pages, 0, logits);
}

// ---- device-resident rounds ----
static recg_status check_device_batch(recg_ctx* ctx, const recg_device_batch* b, const char* who) {
  if (!b || b->n_req <= 0 || !b->ctx_len || !b->verify_len || !b->block_size || !b->verify_tokens || !b->page_table ||
      !b->kv_pool || b->kv_pool_pages <= 0)
    return fail(ctx, RECG_ERR_INVALID_ARG, std::string(who) + ": null array, n_req <= 0 or no KV pool");
  if (b->n_req > ctx->cfg.max_requests) return fail(ctx, RECG_ERR_CAPACITY, std::string(who) + ": n_req exceeds max_requests");
  if (b->max_verify < 1 || b->max_verify > ctx->cfg.max_tokens)
    return fail(ctx, RECG_ERR_INVALID_ARG, std::string(who) + ": max_verify must be 1 .. max_tokens");
  if (b->page_table_stride <= 0 || b->page_table_stride > ctx->cfg.max_pages_per_request)
    return fail(ctx, RECG_ERR_CAPACITY, std::string(who) + ": page_table_stride exceeds max_pages_per_request");
  return RECG_OK;
}

static DeviceRound device_round(const recg_ctx* ctx, const recg_device_batch* b) {
  DeviceRound dr;
  dr.n_req = b->n_req;
  dr.max_verify = b->max_verify;
  dr.pt_stride = b->page_table_stride;
  dr.max_tokens = ctx->cfg.max_tokens;
  dr.ctx_len = b->ctx_len;
  dr.verify_len = b->verify_len;
  dr.block_size = b->block_size;
  dr.verify_tokens = b->verify_tokens;
  return dr;
}

recg_status recg_step_device(recg_ctx* ctx, const recg_device_batch* b, recg_logits* logits) {
  if (!ctx) return RECG_ERR_INVALID_ARG;
  if (!ctx->has_weights) return fail(ctx, RECG_ERR_INVALID_ARG, "recg_step_device: the context was created without weights");
  if (ctx->cfg.flags & (RECG_FLAG_SIMT_GEMM | RECG_FLAG_FOLD_NORM))
    return fail(ctx, RECG_ERR_INVALID_ARG, "recg_step_device: not available with RECG_FLAG_SIMT_GEMM or RECG_FLAG_FOLD_NORM");
  recg_status s = check_device_batch(ctx, b, "recg_step_device");
  if (s != RECG_OK) return s;
  ctx->logits_valid = false;
  ctx->layout_valid = false;
  ctx->mark(-1);
  const int C = b->n_req;
  BatchLayout& bl = ctx->bl;
  int* d = ctx->d_desc;
  bl.dyn = ctx->d_dyn;
  bl.n_req = C;
  bl.n_tok = ctx->cfg.max_tokens;      // capacities: the true counts are in dyn
  bl.n_ver = ctx->cfg.max_tokens;
  bl.pt_stride = b->page_table_stride;
  bl.ctx_len = d;
  bl.verify_len = d + C;
  bl.block_size = d + 2 * C;
  bl.corr = d + 3 * C;
  bl.cu_tok = d + 9 * C;
  bl.cu_ver = bl.cu_tok + (C + 1);
  bl.verify_tokens = bl.cu_ver + (C + 1);
  bl.page_table = b->page_table;
  bl.risk_delta = 0.5f;
  launch_pack_device(device_round(ctx, b), ctx->d_desc, ctx->d_dyn, ctx->d_status, ctx->stream);
  launch_layout(bl, ctx->dm, ctx->tok_per_tile, ctx->target_items, b->kv_pool_pages, ctx->d_status, ctx->stream);
  CU(cudaGetLastError());
  ctx->layout_valid = true;
  ctx->layout_has_pages = true;
  ctx->last_pool = b->kv_pool;
  ctx->last_pool_pages = b->kv_pool_pages;
  return run_forward(ctx, b->kv_pool, b->kv_pool_pages, b->rows_hint, logits);
}

recg_status recg_next_round(recg_ctx* ctx, const recg_device_batch* b, const int32_t* next_block, const int32_t* planted_emitted,
                            const recg_round_log* log, int32_t round) {
  if (!ctx) return RECG_ERR_INVALID_ARG;
  recg_status s = check_device_batch(ctx, b, "recg_next_round");
  if (s != RECG_OK) return s;
  if (!ctx->layout_valid || !ctx->bl.dyn || ctx->bl.n_req != b->n_req)
    return fail(ctx, RECG_ERR_INVALID_ARG, "recg_next_round: no recg_step_device + recg_verify of this batch before");
  RoundLog lg{};
  if (log) {
    if (round < 0 || (log->accept_len && (!log->block_size || !log->verify_len || log->max_rounds <= 0)) ||
        (log->tokens && (!log->n_tokens || log->max_tokens_per_request <= 0)))
      return fail(ctx, RECG_ERR_INVALID_ARG, "recg_next_round: inconsistent log arrays");
    lg.tokens = log->tokens;
    lg.max_out = log->max_tokens_per_request;
    lg.n_tokens = log->n_tokens;
    lg.accept_len = log->accept_len;
    lg.block_size = log->block_size;
    lg.verify_len = log->verify_len;
    lg.max_rounds = log->max_rounds;
    lg.n_rounds = log->n_rounds;
    lg.entropy_mean = log->entropy_mean;
  }
  launch_next_round(device_round(ctx, b), ctx->bl, ctx->vws, next_block, planted_emitted, lg, round, ctx->d_status, ctx->stream);
  CU(cudaGetLastError());
  return RECG_OK;
}

recg_status recg_verify(recg_ctx* ctx, const recg_batch* batch, const void* logits, int32_t logits_dtype,
                        recg_verify_out* out) {
  if (!ctx || !out) return RECG_ERR_INVALID_ARG;
  if (out->mem != RECG_MEM_DEVICE && out->mem != RECG_MEM_HOST) return fail(ctx, RECG_ERR_INVALID_ARG, "recg_verify: bad out->mem");
  if (logits) {
    if (logits_dtype != RECG_DTYPE_BF16 && logits_dtype != RECG_DTYPE_F32)
      return fail(ctx, RECG_ERR_INVALID_ARG, "recg_verify: unknown logits dtype");
    if (batch) {
      recg_status s = upload_and_layout(ctx, batch, false);
      if (s != RECG_OK) return s;
      ctx->logits_valid = false;
    } else if (!ctx->layout_valid) {
      return fail(ctx, RECG_ERR_INVALID_ARG, "recg_verify: no batch given and none laid out before");
    }
  } else {
    if (!ctx->layout_valid || !ctx->logits_valid)
      return fail(ctx, RECG_ERR_INVALID_ARG, "recg_verify: no logits given and no recg_step before");
    if (batch && batch->n_req != ctx->bl.n_req)
      return fail(ctx, RECG_ERR_INVALID_ARG, "recg_verify: batch differs from the one of the last recg_step");
    logits = ctx->logits;
    logits_dtype = (ctx->cfg.flags & RECG_FLAG_LOGITS_BF16) ? RECG_DTYPE_BF16 : RECG_DTYPE_F32;
  }
  const BatchLayout& bl = ctx->bl;
  VerifyBuffers vb = ctx->vws;
  const bool dev = out->mem == RECG_MEM_DEVICE;
  if (bl.dyn && !dev)
    return fail(ctx, RECG_ERR_INVALID_ARG, "recg_verify: after recg_step_device the outputs stay on the device (RECG_MEM_DEVICE)");
  if (dev) {
#define PICK(f) if (out->f) vb.f = out->f
    PICK(accept_len); PICK(n_emitted); PICK(emitted); PICK(new_ctx_len); PICK(slot_state); PICK(freed_pages);
    PICK(next_draft); PICK(cont_hit); PICK(top1); PICK(top2); PICK(p1); PICK(p2); PICK(entropy); PICK(entropy_mean);
    PICK(corr_hit); PICK(risky_n); PICK(risky_index); PICK(risky_token); PICK(freed_page_ids);
#undef PICK
  }
  ctx->mark(-1);
  launch_verify(bl, logits, logits_dtype, ctx->dm.vocab, ctx->vpart, ctx->max_chunks_total, vb, ctx->n_sm, ctx->stream);
  CU(cudaGetLastError());
  ctx->mark(8, 2);
  if (!dev) {
    const size_t C = bl.n_req, T = bl.n_tok, Tv = bl.n_ver, Tb = T - Tv;
    if (ctx->h_vout) {
      // one copy of the whole output region into pinned memory, then plain host copies into the caller's arrays
      const uint8_t* region = ctx->arena.base + ctx->vout_off;
      CU(cudaMemcpyAsync(ctx->h_vout, region, ctx->vout_bytes, cudaMemcpyDeviceToHost, ctx->stream));
      CU(cudaStreamSynchronize(ctx->stream));
#define OUT(f, n) if (out->f && (n)) memcpy(out->f, ctx->h_vout + (reinterpret_cast<const uint8_t*>(vb.f) - region), (n) * 4)
      OUT(accept_len, C); OUT(n_emitted, C); OUT(emitted, Tv); OUT(new_ctx_len, C); OUT(slot_state, T);
      OUT(freed_pages, C); OUT(next_draft, Tb); OUT(cont_hit, C); OUT(top1, T); OUT(top2, T); OUT(p1, T); OUT(p2, T);
      OUT(entropy, T); OUT(entropy_mean, C);
      OUT(corr_hit, 2 * C); OUT(risky_n, 3 * C); OUT(risky_index, 6 * C); OUT(risky_token, 6 * C);
      OUT(freed_page_ids, T);
#undef OUT
      return RECG_OK;
    }
#define OUT(f, n) if (out->f && (n)) CU(cudaMemcpyAsync(out->f, vb.f, (n) * 4, cudaMemcpyDeviceToHost, ctx->stream))
    OUT(accept_len, C); OUT(n_emitted, C); OUT(emitted, Tv); OUT(new_ctx_len, C); OUT(slot_state, T);
    OUT(freed_pages, C); OUT(next_draft, Tb); OUT(cont_hit, C); OUT(top1, T); OUT(top2, T); OUT(p1, T); OUT(p2, T);
    OUT(entropy, T); OUT(entropy_mean, C);
    OUT(corr_hit, 2 * C); OUT(risky_n, 3 * C); OUT(risky_index, 6 * C); OUT(risky_token, 6 * C);
    OUT(freed_page_ids, T);
#undef OUT
    CU(cudaStreamSynchronize(ctx->stream));
  }
  return RECG_OK;
}

recg_status recg_policy_load(recg_ctx* ctx, const recg_policy_table* t) {
  if (!ctx) return RECG_ERR_INVALID_ARG;
  if (!t || !t->blocks || !t->value || !t->cost || (t->n_bins > 1 && !t->s_edges))
    return fail(ctx, RECG_ERR_INVALID_ARG, "recg_policy_load: null table array");
  if (t->n_blocks < 1 || t->n_blocks > RECG_POLICY_MAX_BLOCKS || t->n_bins < 1 || t->n_bins > RECG_POLICY_MAX_BINS)
    return fail(ctx, RECG_ERR_INVALID_ARG, "recg_policy_load: n_blocks must be 1..8 and n_bins 1..64");
  for (int j = 0; j < t->n_blocks; ++j)
    if (t->blocks[j] < 1 || (j > 0 && t->blocks[j] <= t->blocks[j - 1]))
      return fail(ctx, RECG_ERR_INVALID_ARG, "recg_policy_load: blocks must be positive and ascending");
  for (int i = 1; i < t->n_bins - 1; ++i)
    if (!(t->s_edges[i] >= t->s_edges[i - 1]))
      return fail(ctx, RECG_ERR_INVALID_ARG, "recg_policy_load: s_edges must be ascending");
  const size_t nv = (size_t)t->n_blocks * t->n_bins * t->n_blocks * 2;
  std::vector<int>& h = ctx->h_policy;
  h.assign(80 + nv, 0);
  memcpy(h.data(), t->blocks, t->n_blocks * sizeof(int));
  memcpy(h.data() + 8, t->cost, t->n_blocks * sizeof(float));
  if (t->n_bins > 1) memcpy(h.data() + 16, t->s_edges, (t->n_bins - 1) * sizeof(float));
  memcpy(h.data() + 80, t->value, nv * sizeof(float));
  CU(cudaMemcpyAsync(ctx->d_policy, h.data(), h.size() * sizeof(int), cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  ctx->policy.n_blocks = t->n_blocks;
  ctx->policy.n_bins = t->n_bins;
  ctx->policy.blocks = ctx->d_policy;
  ctx->policy.cost = reinterpret_cast<const float*>(ctx->d_policy + 8);
  ctx->policy.edges = reinterpret_cast<const float*>(ctx->d_policy + 16);
  ctx->policy.value = reinterpret_cast<const float*>(ctx->d_policy + 80);
  ctx->policy_loaded = true;
  return RECG_OK;
}

recg_status recg_policy_step(recg_ctx* ctx, const recg_policy_state* state, const float* entropy_mean,
                             const int32_t* accept_len, int32_t* next_block) {
  if (!ctx) return RECG_ERR_INVALID_ARG;
  if (!ctx->policy_loaded) return fail(ctx, RECG_ERR_INVALID_ARG, "recg_policy_step: no table loaded");
  if (!ctx->layout_valid) return fail(ctx, RECG_ERR_INVALID_ARG, "recg_policy_step: no batch laid out before");
  if (!state || !state->e1 || !state->e2 || !state->block_index || !state->full || !next_block)
    return fail(ctx, RECG_ERR_INVALID_ARG, "recg_policy_step: null state array or next_block");
  launch_policy(ctx->bl, ctx->policy, state->e1, state->e2, state->block_index, state->full,
                entropy_mean ? entropy_mean : ctx->vws.entropy_mean, accept_len ? accept_len : ctx->vws.accept_len,
                next_block, ctx->stream);
  CU(cudaGetLastError());
  return RECG_OK;
}

recg_status recg_attention(recg_ctx* ctx, const recg_batch* batch, int32_t layer, const void* q, void* o) {
  if (!ctx || !q || !o) return RECG_ERR_INVALID_ARG;
  if (layer < 0 || (ctx->cfg.n_layers > 0 && layer >= ctx->cfg.n_layers) ) return fail(ctx, RECG_ERR_INVALID_ARG, "recg_attention: layer out of range");
  if (batch) {
    recg_status s = upload_and_layout(ctx, batch, true, false);
    if (s != RECG_OK) return s;
    ctx->logits_valid = false;
  } else if (!ctx->layout_valid || !ctx->layout_has_pages || !ctx->last_pool) {
    return fail(ctx, RECG_ERR_INVALID_ARG, "recg_attention: no batch given and none with a KV pool laid out before");
  }
  launch_attention(ctx->bl, ctx->dm, layer, q, o, ctx->last_pool, ctx->last_pool_pages, ctx->part_o, ctx->part_ml,
                   ctx->tok_per_tile, ctx->n_sm, ctx->d_status, ctx->stream, !(ctx->cfg.flags & RECG_FLAG_SIMT_ATTENTION),
                   batch == nullptr);      // (a batch given with the call was laid out by the launch right before this one)
  CU(cudaGetLastError());
  return RECG_OK;
}

static recg_status kv_io(recg_ctx* ctx, bool write, void* pool, int64_t n_pool_pages, int32_t layer,
                         const int32_t* row, int32_t n_table, int32_t pos0, int32_t n_pos, void* k, void* v) {
  if (!ctx || !pool || !row || !k || !v) return RECG_ERR_INVALID_ARG;
  if (pos0 < 0 || n_pos < 0 || n_table <= 0 || n_table > ctx->cfg.max_pages_per_request || layer < 0 ||
      (ctx->cfg.n_layers > 0 && layer >= ctx->cfg.n_layers) || n_pool_pages <= 0)
    return fail(ctx, RECG_ERR_INVALID_ARG, "recg_kv_*: bad position range, layer or table length");
  if (n_pos == 0) return RECG_OK;
  if ((pos0 + n_pos - 1) / kPageSize >= n_table) return fail(ctx, RECG_ERR_CAPACITY, "recg_kv_*: positions beyond the page table row");
  for (int i = pos0 / kPageSize; i <= (pos0 + n_pos - 1) / kPageSize; ++i)
    if (row[i] < 0 || row[i] >= n_pool_pages) return fail(ctx, RECG_ERR_INVALID_ARG, "recg_kv_*: page id outside the pool");
  CU(cudaMemcpyAsync(ctx->d_page_row, row, n_table * sizeof(int), cudaMemcpyHostToDevice, ctx->stream));
  launch_kv_io(write, pool, n_pool_pages, layer, ctx->dm, ctx->d_page_row, pos0, n_pos, k, v, ctx->d_status, ctx->stream);
  CU(cudaGetLastError());
  return RECG_OK;
}

recg_status recg_kv_write(recg_ctx* ctx, void* kv_pool, int64_t kv_pool_pages, int32_t layer, const int32_t* page_table_row,
                          int32_t n_table, int32_t pos0, int32_t n_pos, const void* k, const void* v) {
  return kv_io(ctx, true, kv_pool, kv_pool_pages, layer, page_table_row, n_table, pos0, n_pos, const_cast<void*>(k),
               const_cast<void*>(v));
}
recg_status recg_kv_read(recg_ctx* ctx, const void* kv_pool, int64_t kv_pool_pages, int32_t layer, const int32_t* page_table_row,
                         int32_t n_table, int32_t pos0, int32_t n_pos, void* k, void* v) {
  return kv_io(ctx, false, const_cast<void*>(kv_pool), kv_pool_pages, layer, page_table_row, n_table, pos0, n_pos, k, v);
}

recg_status recg_linear(recg_ctx* ctx, const void* x, const void* w, void* y, int32_t M, int32_t N, int32_t K,
                        int32_t out_dtype) {
  if (!ctx || !x || !w || !y) return RECG_ERR_INVALID_ARG;
  if (M < 0 || N <= 0 || K <= 0 || N % 16 || K % 64) return fail(ctx, RECG_ERR_SHAPE, "recg_linear: N must be a multiple of 16 and K of 64");
  if (out_dtype != RECG_DTYPE_BF16 && out_dtype != RECG_DTYPE_F32) return fail(ctx, RECG_ERR_INVALID_ARG, "recg_linear: unknown out dtype");
  if (M == 0) return RECG_OK;
  GemmArgs a{};
  a.x = x; a.w = w; a.out = y; a.M = M; a.N = N; a.K = K;
  a.epi = out_dtype == RECG_DTYPE_BF16 ? EPI_PLAIN_BF16 : EPI_PLAIN_F32;
  return run_gemm(ctx, a);
}

recg_status recg_debug_gemm_config(recg_ctx* ctx, int32_t tile, int32_t stream_k) {
  if (!ctx) return RECG_ERR_INVALID_ARG;
  if (tile != 0 && tile != 64 && tile != 128 && tile != 256 && tile != 384 && tile != 512)
    return fail(ctx, RECG_ERR_INVALID_ARG, "recg_debug_gemm_config: tile must be 0, 64, 128, 256, 384 or 512");
  if (stream_k < 0 || stream_k > 2) return fail(ctx, RECG_ERR_INVALID_ARG, "recg_debug_gemm_config: stream_k must be 0, 1 or 2");
  tc_state_force(ctx->tc_state, tile, stream_k);
  return RECG_OK;
}

recg_status recg_debug_wait_timeout(recg_ctx* ctx, int32_t max_polls) {
  if (!ctx) return RECG_ERR_INVALID_ARG;
  if (max_polls < 1 || max_polls > (1 << 20)) return fail(ctx, RECG_ERR_INVALID_ARG, "recg_debug_wait_timeout: max_polls must be 1 .. 1048576");
  launch_wait_timeout((uint32_t)max_polls, ctx->d_status, ctx->stream);
  CU(cudaGetLastError());
  return RECG_OK;
}

int32_t recg_debug_map_cache_selftest(int32_t n_keys, int32_t* evictions) {
  int ev = 0;
  const int bad = tc_map_cache_selftest(n_keys, &ev);
  if (evictions) *evictions = ev;
  return bad;
}

recg_status recg_debug_buffer(recg_ctx* ctx, int32_t which, const void** ptr, int32_t* dtype, int32_t* rows, int32_t* cols) {
  if (!ctx || !ptr || !dtype || !rows || !cols) return RECG_ERR_INVALID_ARG;
  if (!ctx->has_weights || !ctx->logits_valid) return fail(ctx, RECG_ERR_INVALID_ARG, "recg_debug_buffer: no recg_step before");
  *rows = ctx->bl.n_tok;
  switch (which) {
    case 0: *ptr = ctx->h; *dtype = RECG_DTYPE_F32; *cols = ctx->dm.hidden; break;
    case 1: *ptr = ctx->o; *dtype = RECG_DTYPE_BF16; *cols = ctx->dm.n_q * ctx->dm.head_dim; break;
    case 2: *ptr = ctx->q; *dtype = RECG_DTYPE_BF16; *cols = ctx->dm.n_q * ctx->dm.head_dim; break;
    default: return fail(ctx, RECG_ERR_INVALID_ARG, "recg_debug_buffer: unknown buffer");
  }
  return RECG_OK;
}

}  // extern "C"

// Fused greedy verification: one pass over the logits (top-2 ids, softmax mass, entropy) split over
// vocab chunks, then a per-request finalize (accept-length scan, emitted tokens, continuation rule,
// mean verifier entropy, KV commit / rollback indices).
#include <string>

#include "../../include/recg.h"
#include "common.cuh"
#include "kernels.h"

namespace recg {

namespace {

constexpr int kVerifyThreads = 256;

struct Top2 {
  float m1, m2;
  int i1, i2;
};
__device__ __forceinline__ bool better(float av, int ai, float bv, int bi) { return av > bv || (av == bv && ai < bi); }
__device__ __forceinline__ void top2_insert(Top2& t, float x, int i) {
  if (better(x, i, t.m1, t.i1)) {
    t.m2 = t.m1; t.i2 = t.i1; t.m1 = x; t.i1 = i;
  } else if (better(x, i, t.m2, t.i2)) {
    t.m2 = x; t.i2 = i;
  }
}

// running softmax mass relative to a moving maximum m: s = sum e^(x-m), t = sum x e^(x-m)
// (entropy = ln s - t/s + m).  Logits of -inf contribute nothing: they are clamped to a finite value whose
// exponential underflows to zero, so that x * 0 stays 0.
struct Mass {
  float m, s, t;
};
constexpr float kLog2e = 1.4426950408889634f;
__device__ __forceinline__ void mass_rebase(Mass& a, float m_new) {
  if (m_new > a.m) {
    const float f = a.s > 0.f ? exp2f((a.m - m_new) * kLog2e) : 0.f;   // a.m may be -inf with s = t = 0
    a.s *= f;
    a.t *= f;
    a.m = m_new;
  }
}
// neg_m2 = -m * log2(e), hoisted by the caller
__device__ __forceinline__ void mass_add(Mass& a, float x, float neg_m2) {
  const float xc = fmaxf(x, -3.0e38f);
  const float e = exp2f(fmaf(xc, kLog2e, neg_m2));
  a.s += e;
  a.t = fmaf(xc, e, a.t);
}
__device__ __forceinline__ void mass_merge(Mass& a, const Mass& b) {
  if (b.s <= 0.f) return;
  Mass bb = b;
  const float m = fmaxf(a.m, b.m);
  mass_rebase(a, m);
  mass_rebase(bb, m);
  a.s += bb.s;
  a.t += bb.t;
}

template <typename T> struct Vec;
template <> struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void load(const __nv_bfloat16* p, float (&x)[8]) {
    uint4 u;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(u.x), "=r"(u.y), "=r"(u.z), "=r"(u.w)
                 : "l"(p));
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[2 * i] = __uint_as_float(w[i] << 16);
      x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static float one(const __nv_bfloat16* p) { return __bfloat162float(*p); }
};
template <> struct Vec<float> {
  static constexpr int N = 4;
  __device__ static void load(const float* p, float (&x)[4]) {
    float4 u = __ldg(reinterpret_cast<const float4*>(p));
    x[0] = u.x; x[1] = u.y; x[2] = u.z; x[3] = u.w;
  }
  __device__ static float one(const float* p) { return *p; }
};

// One-dimensional grid of rows x chunks_per_row CTAs, chunk-fastest (consecutive CTAs read consecutive memory; the
// row count is not bound by the 65535 limit of the other grid dimensions).  Each CTA scans [c0, c1) of one row.
template <typename T>
__global__ void __launch_bounds__(kVerifyThreads) verify_partial_kernel(const T* __restrict__ logits, int vocab,
                                                                        int chunk_len, int chunks_per_row,
                                                                        RowPartial* __restrict__ partials,
                                                                        const int* __restrict__ rows_dev) {
  constexpr int N = Vec<T>::N;
  griddep_launch();
  griddep_wait();
  const int row = blockIdx.x / chunks_per_row, chunk = blockIdx.x - row * chunks_per_row;
  if (rows_dev && row >= rows_dev[0]) return;      // (the grid was sized for the capacity)
  const T* base = logits + (size_t)row * vocab;
  const int c0 = chunk * chunk_len;
  const int c1 = min(vocab, c0 + chunk_len);
  Top2 tp = {-INFINITY, -INFINITY, 0x7fffffff, 0x7fffffff};
  Mass ms = {-INFINITY, 0.f, 0.f};
  const bool vec_ok = ((reinterpret_cast<uintptr_t>(base + c0) & 15) == 0);
  int done = c0;
  if (vec_ok) {
    const int nvec = (c1 - c0) / N;
    // Four 16-byte loads in flight per thread.  In the loop the top-2 bookkeeping is branch-free and per VECTOR:
    // each thread remembers its two vectors with the largest maximum (the two largest elements it has seen lie
    // in those two vectors; strict comparisons keep the earlier vector on ties), and only after the loop are
    // these two vectors re-read and searched element by element.  A per-element test would diverge in nearly
    // every warp and cost more issue slots than the arithmetic.
    float bv1 = -INFINITY, bv2 = -INFINITY;   // two largest vector maxima of this thread
    int bi1 = -1, bi2 = -1;                   // their vector indices
    auto track = [&](float vmax, int vec) {
      const bool g1 = vmax > bv1, g2 = vmax > bv2;
      bi2 = g1 ? bi1 : (g2 ? vec : bi2);
      bv2 = g1 ? bv1 : (g2 ? vmax : bv2);
      bi1 = g1 ? vec : bi1;
      bv1 = g1 ? vmax : bv1;
    };
    int i = threadIdx.x;
    for (; i + 3 * kVerifyThreads < nvec; i += 4 * kVerifyThreads) {
      float x[4][N];
#pragma unroll
      for (int u = 0; u < 4; ++u) Vec<T>::load(base + c0 + (size_t)(i + u * kVerifyThreads) * N, x[u]);
      float vm[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        vm[u] = x[u][0];
#pragma unroll
        for (int k = 1; k < N; ++k) vm[u] = fmaxf(vm[u], x[u][k]);
      }
      mass_rebase(ms, fmaxf(fmaxf(vm[0], vm[1]), fmaxf(vm[2], vm[3])));
      const float neg = ms.m > -INFINITY ? -ms.m * kLog2e : 0.f;   // all -inf so far: every term underflows to 0
#pragma unroll
      for (int k = 0; k < N; ++k) {
#pragma unroll
        for (int u = 0; u < 4; ++u) mass_add(ms, x[u][k], neg);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) track(vm[u], i + u * kVerifyThreads);
    }
    for (; i < nvec; i += kVerifyThreads) {
      float x[N];
      Vec<T>::load(base + c0 + (size_t)i * N, x);
      float vm = x[0];
#pragma unroll
      for (int k = 1; k < N; ++k) vm = fmaxf(vm, x[k]);
      mass_rebase(ms, vm);
      const float neg = ms.m > -INFINITY ? -ms.m * kLog2e : 0.f;   // all -inf so far: every term underflows to 0
#pragma unroll
      for (int k = 0; k < N; ++k) mass_add(ms, x[k], neg);
      track(vm, i);
    }
    // element-level search of the two remembered vectors (in index order, so that ties resolve to the lowest index)
    const int lo_vec = bi2 < 0 ? bi1 : min(bi1, bi2), hi_vec = bi2 < 0 ? -1 : max(bi1, bi2);
    const int cand[2] = {lo_vec, hi_vec};
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      if (cand[q] < 0) continue;
      float x[N];
      Vec<T>::load(base + c0 + (size_t)cand[q] * N, x);
#pragma unroll
      for (int k = 0; k < N; ++k) top2_insert(tp, x[k], c0 + cand[q] * N + k);
    }
    done = c0 + nvec * N;
  }
  for (int i = done + threadIdx.x; i < c1; i += kVerifyThreads) {
    const float x = Vec<T>::one(base + i);
    mass_rebase(ms, x);
    mass_add(ms, x, ms.m > -INFINITY ? -ms.m * kLog2e : 0.f);
    if (x >= tp.m2) top2_insert(tp, x, i);
  }
  // warp reduce, then across warps through shared memory
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    Top2 ot;
    ot.m1 = __shfl_xor_sync(0xffffffffu, tp.m1, o);
    ot.i1 = __shfl_xor_sync(0xffffffffu, tp.i1, o);
    ot.m2 = __shfl_xor_sync(0xffffffffu, tp.m2, o);
    ot.i2 = __shfl_xor_sync(0xffffffffu, tp.i2, o);
    top2_insert(tp, ot.m1, ot.i1);
    top2_insert(tp, ot.m2, ot.i2);
    Mass om;
    om.m = __shfl_xor_sync(0xffffffffu, ms.m, o);
    om.s = __shfl_xor_sync(0xffffffffu, ms.s, o);
    om.t = __shfl_xor_sync(0xffffffffu, ms.t, o);
    mass_merge(ms, om);
  }
  __shared__ Top2 s_tp[kVerifyThreads / 32];
  __shared__ Mass s_ms[kVerifyThreads / 32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) {
    s_tp[warp] = tp;
    s_ms[warp] = ms;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < kVerifyThreads / 32; ++w) {
      top2_insert(tp, s_tp[w].m1, s_tp[w].i1);
      top2_insert(tp, s_tp[w].m2, s_tp[w].i2);
      mass_merge(ms, s_ms[w]);
    }
    // express the mass relative to the chunk maximum m1 (== ms.m unless the chunk is empty)
    RowPartial p;
    p.m1 = tp.m1; p.m2 = tp.m2; p.i1 = tp.i1; p.i2 = tp.i2;
    p.s = ms.s; p.t = ms.t;
    partials[(size_t)row * chunks_per_row + chunk] = p;
  }
}

// One CTA per request: merge the chunk partials of its rows, then the accept scan and the index work.
__global__ void __launch_bounds__(128) verify_finalize_kernel(BatchLayout bl, const RowPartial* __restrict__ partials,
                                                              int chunks_per_row, VerifyBuffers vb) {
  griddep_launch();
  griddep_wait();
  const int r = blockIdx.x;
  const int t0 = bl.cu_tok[r];
  const int v = bl.verify_len[r], b = bl.block_size[r], L = bl.ctx_len[r];
  const int* cr = bl.corr + 6 * r;              // correction branches: count, mask tokens per branch, indices, tokens
  const int n_corr = cr[0], span = 1 + cr[1];
  const int n = bl.cu_tok[r + 1] - t0;          // v + b + n_corr * span
  for (int j = threadIdx.x; j < n; j += blockDim.x) {
    const RowPartial* p = partials + (size_t)(t0 + j) * chunks_per_row;
    Top2 tp = {-INFINITY, -INFINITY, 0x7fffffff, 0x7fffffff};
    Mass ms = {-INFINITY, 0.f, 0.f};
    for (int c = 0; c < chunks_per_row; ++c) {
      const RowPartial q = p[c];
      top2_insert(tp, q.m1, q.i1);
      top2_insert(tp, q.m2, q.i2);
      Mass o = {q.m1, q.s, q.t};
      mass_merge(ms, o);
    }
    const float inv = 1.f / ms.s;
    vb.top1[t0 + j] = tp.i1;
    vb.top2[t0 + j] = tp.i2;
    vb.p1[t0 + j] = inv;                             // e^(m1 - m1) / S
    vb.p2[t0 + j] = __expf(tp.m2 - tp.m1) * inv;
    vb.entropy[t0 + j] = logf(ms.s) - ms.t * inv + ms.m;   // ln S - (1/S) sum x e^(x-M) + M
  }
  __syncthreads();
  __shared__ int s_a, s_first_free, s_last;
  if (threadIdx.x == 0) {
    int a = 0;
    const int tv0 = bl.cu_ver[r];
    if (v > 0) {
      while (a < v - 1 && bl.verify_tokens[tv0 + a + 1] == vb.top1[t0 + a]) ++a;
      float es = 0.f;
      for (int i = 0; i <= a; ++i) es += vb.entropy[t0 + i];
      vb.entropy_mean[r] = es / (a + 1);
      for (int i = 0; i < v; ++i)
        vb.emitted[tv0 + i] = i < a ? bl.verify_tokens[tv0 + i + 1] : (i == a ? vb.top1[t0 + a] : -1);
    } else {
      vb.entropy_mean[r] = 0.f;
    }
    vb.accept_len[r] = a;
    vb.n_emitted[r] = v > 0 ? a + 1 : 0;
    const int new_L = L + (v > 0 ? a + 1 : 0);
    vb.new_ctx_len[r] = new_L;
    vb.cont_hit[r] = (v > 0 && b > 0 && a == v - 1 && vb.top1[t0 + v] == vb.top1[t0 + v - 1]) ? 1 : 0;
    const int first_free = (new_L + kPageSize - 1) / kPageSize;
    const int last = (L + n + kPageSize - 1) / kPageSize;
    vb.freed_pages[r] = bl.page_table ? last - first_free : 0;
    s_first_free = first_free;
    s_last = bl.page_table ? last : first_free;
    // a correction branch is confirmed when the verifier rejected exactly the draft it replaced and emitted the
    // replacement token there (Sec. 5.1)
    for (int k = 0; k < 2; ++k)
      vb.corr_hit[2 * r + k] = (k < n_corr && v > 0 && a == cr[2 + k] - 1 && vb.top1[t0 + a] == cr[4 + k]) ? 1 : 0;
    // risky drafts of every draft block, indexed as the verify tokens the block would become: the continuation's
    // mask row m is y'_m (row 0 only confirms the bonus token), a correction's mask row m is y'_{m+1}
    for (int j = 0; j < 3; ++j) {
      int row0 = 0, rows = 0, first_index = 1;
      if (j == 0) { row0 = t0 + v + 1; rows = b > 0 ? b - 1 : 0; }
      else if (j - 1 < n_corr) { row0 = t0 + v + b + (j - 1) * span + 1; rows = span - 1; }
      int cnt = 0;
      int* ri = vb.risky_index + 6 * r + 2 * j;
      int* rtk = vb.risky_token + 6 * r + 2 * j;
      ri[0] = ri[1] = rtk[0] = rtk[1] = -1;
      for (int m = 0; m < rows; ++m) {
        if (vb.p1[row0 + m] - vb.p2[row0 + m] < bl.risk_delta) {
          if (cnt < 2) { ri[cnt] = first_index + m; rtk[cnt] = vb.top2[row0 + m]; }
          ++cnt;
        }
      }
      vb.risky_n[3 * r + j] = cnt;
    }
    s_a = a;
  }
  __syncthreads();
  const int a = s_a;
  const int tb0 = t0 - bl.cu_ver[r];  // draft-token offset of this request: sum of b over earlier requests
  for (int j = threadIdx.x; j < n; j += blockDim.x) {
    if (j >= v) vb.next_draft[tb0 + (j - v)] = vb.top1[t0 + j];
    const int slot = bl.tok_slot[t0 + j];
    const bool committed = (j < v) && (j <= a);
    vb.slot_state[t0 + j] = slot < 0 ? 0 : (committed ? slot : -(slot + 1));
    // ids of the pages that hold no committed token any more, at the request's row offset (there are never more
    // of them than rows: each starts at a position of a row that was rolled back)
    if (vb.freed_page_ids) {
      const int e = s_first_free + j;
      vb.freed_page_ids[t0 + j] = e < s_last ? bl.page_table[(size_t)r * bl.pt_stride + e] : -1;
    }
  }
}

}  // namespace

int verify_chunks_per_row(int rows, int vocab, int n_sm) {
  int by_size = (vocab + 4095) / 4096;
  int by_rows = rows > 0 ? (n_sm * 4 + rows - 1) / rows : 1;
  int c = by_size < by_rows ? by_size : by_rows;
  if (c < 1) c = 1;
  if (c > 64) c = 64;
  return c;
}

void launch_verify(const BatchLayout& bl, const void* logits, int logits_dtype, int vocab, RowPartial* partials,
                   int max_chunks_total, const VerifyBuffers& vb, int n_sm, cudaStream_t st) {
  const int rows = bl.n_tok;
  if (rows <= 0) return;
  int chunks = verify_chunks_per_row(rows, vocab, n_sm);
  while (chunks > 1 && (long long)chunks * rows > max_chunks_total) --chunks;
  int chunk_len = (vocab + chunks - 1) / chunks;
  chunk_len = (chunk_len + 63) / 64 * 64;  // keeps every chunk start 16-byte aligned relative to the row
  chunks = (vocab + chunk_len - 1) / chunk_len;
  dim3 grid((unsigned)chunks * (unsigned)rows);
  if (logits_dtype == 0)
    launch_pdl(verify_partial_kernel<__nv_bfloat16>, grid, dim3(kVerifyThreads), 0, st,
               static_cast<const __nv_bfloat16*>(logits), vocab, chunk_len, chunks, partials, bl.dyn);
  else
    launch_pdl(verify_partial_kernel<float>, grid, dim3(kVerifyThreads), 0, st, static_cast<const float*>(logits), vocab,
               chunk_len, chunks, partials, bl.dyn);
  launch_pdl(verify_finalize_kernel, dim3(bl.n_req), dim3(128), 0, st, bl, (const RowPartial*)partials, chunks, vb);
}

}  // namespace recg

// ---------------------------------------------------------------------------------------------------
// Block-size rule of verification-guided drafting (Sec. 5.2): one thread per request.
// ---------------------------------------------------------------------------------------------------
namespace recg {
namespace {

__global__ void policy_kernel(BatchLayout bl, PolicyTable tb, float* __restrict__ e1, float* __restrict__ e2,
                              int* __restrict__ block_index, int* __restrict__ full,
                              const float* __restrict__ entropy_mean, const int* __restrict__ accept_len,
                              int* __restrict__ next_block) {
  griddep_launch();
  griddep_wait();
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= bl.n_req) return;
  const int v = bl.verify_len[r];
  float a1 = e1[r], a2 = e2[r];
  int f = full[r];
  if (v > 0) {   // the finished round verified something: shift its mean verifier entropy into the history
    a2 = a1;
    a1 = entropy_mean[r];
    f = (v > 1 && accept_len[r] == v - 1) ? 1 : 0;
    e1[r] = a1;
    e2[r] = a2;
    full[r] = f;
  }
  const float s = __fmul_rn(__fadd_rn(a1, a2), -0.5f);   // Eq. 2
  int k = 0;
  for (int i = 0; i < tb.n_bins - 1; ++i) k += tb.edges[i] <= s ? 1 : 0;
  int jp = block_index[r];
  jp = jp < 0 ? 0 : (jp >= tb.n_blocks ? tb.n_blocks - 1 : jp);
  int best = 0;
  float best_score = 0.f;
  for (int j = 0; j < tb.n_blocks; ++j) {   // Eq. 3; the first maximum wins
    const float score = __fsub_rn(tb.value[((j * tb.n_bins + k) * tb.n_blocks + jp) * 2 + f], tb.cost[j]);
    if (j == 0 || score > best_score) { best = j; best_score = score; }
  }
  block_index[r] = best;
  next_block[r] = tb.blocks[best];
}

}  // namespace

void launch_policy(const BatchLayout& bl, const PolicyTable& tb, float* e1, float* e2, int* block_index, int* full,
                   const float* entropy_mean, const int* accept_len, int* next_block, cudaStream_t st) {
  if (bl.n_req <= 0) return;
  launch_pdl(policy_kernel, dim3((bl.n_req + 127) / 128), dim3(128), 0, st, bl, tb, e1, e2, block_index, full,
             entropy_mean, accept_len, next_block);
}

}  // namespace recg

// ---------------------------------------------------------------------------------------------------
// Row statistics without any allocation: the chunk partials live in a file-scope device array.
// ---------------------------------------------------------------------------------------------------
namespace recg {
namespace {

constexpr int kStaticMaxPartials = 1 << 16;   // 65536 x 24 bytes = 1.5 MiB held by every GPU that loads the library
static __device__ __align__(256) RowPartial g_static_partials[kStaticMaxPartials];

RowPartial* g_static_ptr[kMaxDevices] = {nullptr};   // device address of the array, per device, set on first use
int g_static_sm[kMaxDevices] = {0};

thread_local std::string g_static_error;

// one thread per row: merge the row's chunk partials into the five per-row outputs
__global__ void row_stats_finalize_kernel(const RowPartial* __restrict__ partials, int rows, int chunks_per_row,
                                          int* __restrict__ top1, int* __restrict__ top2, float* __restrict__ p1,
                                          float* __restrict__ p2, float* __restrict__ entropy) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= rows) return;
  const RowPartial* p = partials + (size_t)r * chunks_per_row;
  Top2 tp = {-INFINITY, -INFINITY, 0x7fffffff, 0x7fffffff};
  Mass ms = {-INFINITY, 0.f, 0.f};
  for (int c = 0; c < chunks_per_row; ++c) {
    const RowPartial q = p[c];
    top2_insert(tp, q.m1, q.i1);
    top2_insert(tp, q.m2, q.i2);
    Mass o = {q.m1, q.s, q.t};
    mass_merge(ms, o);
  }
  const float inv = 1.f / ms.s;
  if (top1) top1[r] = tp.i1;
  if (top2) top2[r] = tp.i2;
  if (p1) p1[r] = inv;
  if (p2) p2[r] = __expf(tp.m2 - tp.m1) * inv;
  if (entropy) entropy[r] = logf(ms.s) - ms.t * inv + ms.m;
}

}  // namespace

const char* static_entry_error() { return g_static_error.c_str(); }

}  // namespace recg

extern "C" const char* recg_row_stats_static_error(void) { return recg::static_entry_error(); }

extern "C" recg_status recg_row_stats_static(const void* logits, int32_t logits_dtype, int32_t rows, int32_t vocab,
                                             int32_t* top1, int32_t* top2, float* p1, float* p2, float* entropy,
                                             void* cuda_stream) {
  using namespace recg;
  auto fail = [](recg_status s, const std::string& m) { g_static_error = m; return s; };
  if (!logits || rows < 0 || vocab <= 1) return fail(RECG_ERR_INVALID_ARG, "recg_row_stats_static: null logits or bad extent");
  if (logits_dtype != RECG_DTYPE_BF16 && logits_dtype != RECG_DTYPE_F32)
    return fail(RECG_ERR_INVALID_ARG, "recg_row_stats_static: unknown logits dtype");
  if (rows == 0) return RECG_OK;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
    return fail(RECG_ERR_CUDA, "recg_row_stats_static: no current CUDA device");
  if (!g_static_ptr[dev]) {
    // first call on this device: the array's name is only a host-side handle, so ask the runtime for the
    // device address (with this device current) and remember it
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_partials);
    if (e != cudaSuccess || !ptr)
      return fail(RECG_ERR_CUDA, std::string("recg_row_stats_static: cudaGetSymbolAddress: ") + cudaGetErrorString(e));
    int n_sm = 0;
    e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess || n_sm <= 0)
      return fail(RECG_ERR_CUDA, std::string("recg_row_stats_static: SM count: ") + cudaGetErrorString(e));
    g_static_sm[dev] = n_sm;
    g_static_ptr[dev] = static_cast<RowPartial*>(ptr);
  }
  if (rows > kStaticMaxPartials)
    return fail(RECG_ERR_CAPACITY, "recg_row_stats_static: more than 65536 rows; use recg_verify with a context");
  int chunks = verify_chunks_per_row(rows, vocab, g_static_sm[dev]);
  while (chunks > 1 && (long long)chunks * rows > kStaticMaxPartials) --chunks;
  int chunk_len = (vocab + chunks - 1) / chunks;
  chunk_len = (chunk_len + 63) / 64 * 64;
  chunks = (vocab + chunk_len - 1) / chunk_len;
  if ((long long)chunks * rows > kStaticMaxPartials)
    return fail(RECG_ERR_CAPACITY, "recg_row_stats_static: rows x vocab chunks exceed the static scratch (65536 partials)");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  RowPartial* scratch = g_static_ptr[dev];
  dim3 grid((unsigned)chunks * (unsigned)rows);
  if (logits_dtype == RECG_DTYPE_BF16)
    verify_partial_kernel<__nv_bfloat16>
        <<<grid, kVerifyThreads, 0, st>>>(static_cast<const __nv_bfloat16*>(logits), vocab, chunk_len, chunks, scratch, nullptr);
  else
    verify_partial_kernel<float><<<grid, kVerifyThreads, 0, st>>>(static_cast<const float*>(logits), vocab, chunk_len,
                                                                  chunks, scratch, nullptr);
  cudaError_t e = cudaGetLastError();   // nothing reads the scratch unless the scan was launched
  if (e != cudaSuccess) return fail(RECG_ERR_CUDA, std::string("recg_row_stats_static: launch: ") + cudaGetErrorString(e));
  row_stats_finalize_kernel<<<(rows + 127) / 128, 128, 0, st>>>(scratch, rows, chunks, top1, top2, p1, p2, entropy);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(RECG_ERR_CUDA, std::string("recg_row_stats_static: launch: ") + cudaGetErrorString(e));
  return RECG_OK;
}

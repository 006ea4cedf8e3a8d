// Ragged layout (per-token arrays + attention work list), embedding gather, RMSNorm, KV import/export.
#include "common.cuh"
#include "kernels.h"

namespace recg {

namespace {

__device__ __forceinline__ int upper_request(const int* cu, int n_req, int t) {
  // largest r with cu[r] <= t  (cu is an exclusive prefix sum with cu[n_req] = total)
  int lo = 0, hi = n_req;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (cu[mid] <= t) lo = mid; else hi = mid;
  }
  return lo;
}

// One CTA.  Shared: 8 arrays of n_req+1 ints, then n_ctas/2 + 1 and n_ctas + 1 ints.
//
// Attention work list.  A request with n new tokens has ceil(n / tok_per_tile) row tiles per kv head.  Row tiles
// 2 j and 2 j + 1 of a kv head are "siblings": they read the same K/V.  Two lines of 64-token KV blocks are built,
// every tile preceded by kItemCost virtual blocks that stand for the fixed cost of starting an item (fetching Q,
// refilling and draining the pipeline):
//   line A holds one segment per sibling PAIR and is cut into equal contiguous ranges, one per pair of CTAs
//          (2 p, 2 p + 1): the even CTA works on the first sibling and the odd CTA on the second sibling of the SAME
//          block ranges, at the same time, so that the second reader of a K/V block finds it in L2;
//   line B holds the tiles without a sibling and is cut into equal ranges, one per CTA.
// The CTAs are divided between the two lines in proportion to their work (line A: the first 2 n_pairs_a CTAs), so
// that every CTA walks ONE range and all carry about the same load.  Each piece that holds real blocks is an item;
// a tile whose blocks are cut by range boundaries gets one partial slot per piece.
// Items: [line A, first siblings | line A, second siblings (same order) | line B]; cta_off holds, per CTA, two
// index ranges it walks one after the other (the second one is empty in this division).
constexpr int kItemCost = 4;

__global__ void __launch_bounds__(1024) layout_kernel(BatchLayout bl, int n_kv, int mask_id, int tok_per_tile,
                                                      int n_ctas, int64_t n_pages, int* status) {
  extern __shared__ int sm[];
  const int C = bl.n_req;
  const int max_pairs = n_ctas / 2;
  int* off_a = sm;                       // first cost unit of request r in line A
  int* off_b = sm + (C + 1);             // ... in line B
  int* tile_off = sm + 2 * (C + 1);      // first tile entry of request r
  int* item_a = sm + 3 * (C + 1);        // first line-A piece of request r
  int* item_b = sm + 4 * (C + 1);        // first line-B piece of request r
  int* part_off = sm + 5 * (C + 1);      // first partial slot of request r
  int* req_nb = sm + 6 * (C + 1);        // blocks per tile of request r
  int* req_rt = sm + 7 * (C + 1);        // row tiles per kv head of request r
  int* a_off = sm + 8 * (C + 1);         // [max_pairs + 1] first line-A piece of every CTA pair
  int* b_off = a_off + (max_pairs + 1);  // [n_ctas + 1]  first line-B piece of every line-B CTA
  __shared__ int s_per_a, s_per_b, s_pairs_a;
  const int tid = threadIdx.x, nth = blockDim.x;
  griddep_launch();
  griddep_wait();   // the previous step's kernels may still be reading the arrays this kernel rewrites
  const int n_tok = bl.dyn ? bl.dyn[0] : bl.n_tok;

  // ---- per-token arrays ----
  for (int t = tid; t < n_tok; t += nth) {
    const int r = upper_request(bl.cu_tok, C, t);
    const int j = t - bl.cu_tok[r];
    const int L = bl.ctx_len[r], v = bl.verify_len[r], b = bl.block_size[r];
    const int idx = L + j;   // cache position of the token's K/V
    int pos, id, climit, lo, hi;
    if (j < v) {             // verifier: causal
      pos = idx; id = bl.verify_tokens[bl.cu_ver[r] + j]; climit = idx; lo = 0; hi = 0;
    } else if (j < v + b) {  // continuation block: the whole prefix and the block
      pos = idx; id = mask_id; climit = L + v - 1; lo = L + v; hi = L + v + b;
    } else {                 // correction branch k: replacement token, then its mask tokens
      const int* cr = bl.corr + 6 * r;
      const int span = 1 + cr[1], jj = j - v - b, k = jj / span, q = jj - k * span;
      const int i = cr[2 + k], first = L + v + b + k * span;
      pos = L + i + q;
      id = q == 0 ? cr[4 + k] : mask_id;
      climit = L + i - 1;
      lo = first;
      hi = q == 0 ? first + 1 : first + span;
    }
    bl.tok_req[t] = r;
    bl.tok_pos[t] = pos;
    bl.tok_id[t] = id;
    bl.tok_climit[t] = climit;
    bl.tok_lo[t] = lo;
    bl.tok_hi[t] = hi;
    int slot = -1;
    if (bl.page_table) {
      const int page = bl.page_table[(size_t)r * bl.pt_stride + idx / kPageSize];
      if (page < 0 || page >= n_pages) set_status(status, DEV_BAD_INDEX);
      else slot = page * kPageSize + idx % kPageSize;
    }
    bl.tok_slot[t] = slot;
  }

  // ---- attention work list ----
  for (int r = tid; r < C; r += nth) {
    const int n = bl.cu_tok[r + 1] - bl.cu_tok[r];
    req_nb[r] = (bl.ctx_len[r] + n + 63) / 64;
    req_rt[r] = (n + tok_per_tile - 1) / tok_per_tile;
  }
  __syncthreads();
  if (tid == 0) {
    off_a[0] = off_b[0] = tile_off[0] = 0;
    long long wa = 0, wb = 0;
    for (int r = 0; r < C; ++r) {
      const int rt = req_rt[r], seg = req_nb[r] + kItemCost;
      wa += (long long)n_kv * (rt / 2) * seg;
      wb += (long long)n_kv * (rt & 1) * seg;
      if (wa > 0x3fffffff) wa = 0x3fffffff;   // far beyond any pool; keeps the arithmetic in int
      if (wb > 0x3fffffff) wb = 0x3fffffff;
      off_a[r + 1] = (int)wa;
      off_b[r + 1] = (int)wb;
      tile_off[r + 1] = tile_off[r] + n_kv * rt;
    }
    // CTAs for line A in proportion to its CTA time (two CTAs work on every unit of it)
    int pairs_a = (2 * wa + wb) > 0 ? (int)(0.5 * n_ctas * (2.0 * wa) / (2.0 * wa + wb) + 0.5) : 0;
    if (wa > 0 && pairs_a < 1) pairs_a = 1;
    if (pairs_a > max_pairs) pairs_a = max_pairs;
    if (wb > 0 && n_ctas - 2 * pairs_a < 1) pairs_a = (n_ctas - 1) / 2;
    if (wa == 0) pairs_a = 0;
    const int ctas_b = n_ctas - 2 * pairs_a;
    const int pa = pairs_a > 0 ? (int)((wa + pairs_a - 1) / pairs_a) : 0x3fffffff;
    const int pb = ctas_b > 0 ? (int)((wb + ctas_b - 1) / ctas_b) : 0x3fffffff;
    s_per_a = pa < 1 ? 1 : pa;
    s_per_b = pb < 1 ? 1 : pb;
    s_pairs_a = pairs_a;
  }
  __syncthreads();
  const int per_a = s_per_a, per_b = s_per_b;
  const int n_pairs = s_pairs_a, n_ctas_b = n_ctas - 2 * s_pairs_a;
  // pieces of a segment whose real blocks occupy the cost range [g0, g0 + nb)
  auto n_pieces = [](int g0, int nb, int per) { return (g0 + nb - 1) / per - g0 / per + 1; };
  for (int r = tid; r < C; r += nth) {
    const int nb = req_nb[r], rt = req_rt[r], seg = nb + kItemCost;
    int ia = 0, ib = 0, parts = 0;
    for (int kvh = 0; kvh < n_kv; ++kvh) {
      for (int j = 0; j < rt / 2; ++j) {
        const int np = n_pieces(off_a[r] + (kvh * (rt / 2) + j) * seg + kItemCost, nb, per_a);
        ia += np;
        if (np > 1) parts += 2 * np;
      }
      if (rt & 1) {
        const int np = n_pieces(off_b[r] + kvh * seg + kItemCost, nb, per_b);
        ib += np;
        if (np > 1) parts += np;
      }
    }
    item_a[r + 1] = ia;
    item_b[r + 1] = ib;
    part_off[r + 1] = parts;
  }
  __syncthreads();
  if (tid == 0) {
    item_a[0] = item_b[0] = part_off[0] = 0;
    for (int r = 0; r < C; ++r) {
      item_a[r + 1] += item_a[r];
      item_b[r + 1] += item_b[r];
      part_off[r + 1] += part_off[r];
    }
    int n_items = 2 * item_a[C] + item_b[C];
    if (n_items > bl.max_items || part_off[C] > bl.max_parts) {
      set_status(status, DEV_BAD_INDEX);
      n_items = 0;
    }
    bl.counts[0] = n_items;
    bl.counts[1] = tile_off[C];
    bl.counts[2] = per_b;
    bl.counts[3] = per_a;
  }
  __syncthreads();
  const int n_items = bl.counts[0];
  const int na = n_items ? item_a[C] : 0, n_b = n_items ? item_b[C] : 0;
  for (int r = tid; r <= C; r += nth) bl.tile_off[r] = tile_off[r];
  for (int p = tid; p <= max_pairs; p += nth) a_off[p] = na;   // pairs after the last owner; the rest is filled below
  for (int c = tid; c <= n_ctas; c += nth) b_off[c] = n_b;
  __syncthreads();
  if (n_items) {
    for (int r = tid; r < C; r += nth) {
      const int n = bl.cu_tok[r + 1] - bl.cu_tok[r];
      const int kv_len = bl.ctx_len[r] + n;
      const int nb = req_nb[r], rt = req_rt[r], seg = nb + kItemCost;
      int ia = item_a[r], ib = item_b[r], part = part_off[r];
      // one tile's entry, and its items on one line: pieces [c_first, c_last] of the cost range [g0, g0 + nb)
      auto emit = [&](int kvh, int tile, int g0, int per, int item0, int* owner, int owner_base) {
        const int c_first = g0 / per, c_last = (g0 + nb - 1) / per;
        const int parts = c_last - c_first + 1;
        AttnTile tl;
        tl.part_begin = parts > 1 ? part : -1;
        tl.n_parts = parts;
        tl.tok0 = bl.cu_tok[r] + tile * tok_per_tile;
        tl.ntok = min(tok_per_tile, n - tile * tok_per_tile);
        tl.kv_head = kvh;
        bl.tiles[tile_off[r] + kvh * rt + tile] = tl;
        for (int c = c_first; c <= c_last; ++c) {
          const int gs = max(g0, c * per), ge = min(g0 + nb, (c + 1) * per);
          AttnItem a;
          a.req = r;
          a.kv_head = kvh;
          a.tok0 = tl.tok0;
          a.ntok = tl.ntok;
          a.blk_begin = gs - g0;
          a.blk_end = ge - g0;
          a.part = parts > 1 ? part++ : -1;
          a.kv_len = kv_len;
          bl.items[item0 + (c - c_first)] = a;
          if (owner) owner[owner_base + (c - c_first)] = c;
        }
        return parts;
      };
      for (int kvh = 0; kvh < n_kv; ++kvh) {
        for (int j = 0; j < rt / 2; ++j) {
          const int g0 = off_a[r] + (kvh * (rt / 2) + j) * seg + kItemCost;
          const int np = emit(kvh, 2 * j, g0, per_a, ia, bl.item_cta, ia);       // first sibling: even CTA of the pair
          emit(kvh, 2 * j + 1, g0, per_a, na + ia, nullptr, 0);                  // second sibling: odd CTA, same ranges
          ia += np;
        }
        if (rt & 1) {
          const int g0 = off_b[r] + kvh * seg + kItemCost;
          ib += emit(kvh, rt - 1, g0, per_b, 2 * na + ib, bl.item_cta, 2 * na + ib);
        }
      }
    }
    // first piece of every owner: pieces are in line order, so an owner's range starts where the owner changes
    __syncthreads();
    for (int it = tid; it < na; it += nth) {
      const int p = bl.item_cta[it];
      const int prev = it ? bl.item_cta[it - 1] : -1;
      for (int pp = prev + 1; pp <= p && pp <= max_pairs; ++pp) a_off[pp] = it;   // pairs between two owners have no items
    }
    for (int it = tid; it < n_b; it += nth) {
      const int c = bl.item_cta[2 * na + it];
      const int prev = it ? bl.item_cta[2 * na + it - 1] : -1;
      for (int cc = prev + 1; cc <= c && cc <= n_ctas; ++cc) b_off[cc] = it;
    }
  }
  __syncthreads();
  // the ranges of item indices every CTA walks: a CTA of line A its pair's pieces (first or second siblings), a CTA of
  // line B its own pieces
  for (int c = tid; c < n_ctas; c += nth) {
    int a0 = 0, a1 = 0, b0 = 0, b1 = 0;
    if (c < 2 * n_pairs) {
      const int p = c >> 1;
      a0 = ((c & 1) ? na : 0) + a_off[p];
      a1 = ((c & 1) ? na : 0) + a_off[p + 1];
    } else if (c - 2 * n_pairs < n_ctas_b) {
      b0 = 2 * na + b_off[c - 2 * n_pairs];
      b1 = 2 * na + b_off[c - 2 * n_pairs + 1];
    }
    bl.cta_off[4 * c + 0] = a0;
    bl.cta_off[4 * c + 1] = a1;
    bl.cta_off[4 * c + 2] = b0;
    bl.cta_off[4 * c + 3] = b1;
  }
}

__global__ void __launch_bounds__(256) embed_kernel(const int* __restrict__ tok_id, const __nv_bfloat16* __restrict__ embed,
                                                    float* __restrict__ h, int hidden, int vocab,
                                                    const __nv_bfloat16* __restrict__ gain, __nv_bfloat16* __restrict__ x,
                                                    float* __restrict__ ss, const int* __restrict__ rows_dev) {
  griddep_launch();
  griddep_wait();
  const int t = blockIdx.x;
  if (rows_dev && t >= rows_dev[0]) return;
  int id = tok_id[t];
  id = id < 0 ? 0 : (id >= vocab ? vocab - 1 : id);
  const __nv_bfloat162* src = reinterpret_cast<const __nv_bfloat162*>(embed + (size_t)id * hidden);
  float2* dst = reinterpret_cast<float2*>(h + (size_t)t * hidden);
  float sq = 0.f;
  for (int i = threadIdx.x; i < hidden / 2; i += blockDim.x) {
    const float2 v = __bfloat1622float2(src[i]);
    dst[i] = v;
    if (gain) {
      const float2 g = __bfloat1622float2(reinterpret_cast<const __nv_bfloat162*>(gain)[i]);
      reinterpret_cast<uint32_t*>(x + (size_t)t * hidden)[i] = pack_bf16(v.x * g.x, v.y * g.y);
      sq += v.x * v.x + v.y * v.y;
    }
  }
  if (gain) {
    __shared__ float red[8];
    for (int o = 16; o; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sq;
    __syncthreads();
    if (threadIdx.x == 0) {
      float tot = 0.f;
      for (int i = 0; i < 8; ++i) tot += red[i];
      ss[t] = tot;
    }
  }
}

// One CTA per row; fp32 in, bf16 out.  hidden a multiple of 4.  The row is read once and kept in registers
// when it fits (hidden <= 256 threads x kRegVecs float4), otherwise it is read a second time.
constexpr int kRegVecs = 8;
__global__ void __launch_bounds__(256) rmsnorm_kernel(const float* __restrict__ h, const __nv_bfloat16* __restrict__ g,
                                                      __nv_bfloat16* __restrict__ x, int hidden, float eps,
                                                      const int* __restrict__ rows_dev) {
  griddep_launch();
  griddep_wait();
  const int row = blockIdx.x;
  if (rows_dev && row >= rows_dev[0]) return;
  const int nvec = hidden / 4;
  const float4* src = reinterpret_cast<const float4*>(h + (size_t)row * hidden);
  const bool in_regs = nvec <= 256 * kRegVecs;
  float4 v[kRegVecs];
  float ss = 0.f;
  if (in_regs) {
#pragma unroll
    for (int u = 0; u < kRegVecs; ++u) {
      const int i = threadIdx.x + u * 256;
      v[u] = i < nvec ? src[i] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < kRegVecs; ++u) ss += v[u].x * v[u].x + v[u].y * v[u].y + v[u].z * v[u].z + v[u].w * v[u].w;
  } else {
    for (int i = threadIdx.x; i < nvec; i += 256) {
      const float4 t = src[i];
      ss += t.x * t.x + t.y * t.y + t.z * t.z + t.w * t.w;
    }
  }
  __shared__ float red[8];
  for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) tot += red[i];
  const float rstd = rsqrtf(tot / hidden + eps);
  uint2* dst = reinterpret_cast<uint2*>(x + (size_t)row * hidden);
  const uint2* gg = reinterpret_cast<const uint2*>(g);
  auto emit = [&](int i, const float4& t) {
    const uint2 gv = __ldg(gg + i);
    const float2 g0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gv.x));
    const float2 g1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gv.y));
    uint2 o;
    o.x = pack_bf16(t.x * rstd * g0.x, t.y * rstd * g0.y);
    o.y = pack_bf16(t.z * rstd * g1.x, t.w * rstd * g1.y);
    dst[i] = o;
  };
  if (in_regs) {
#pragma unroll
    for (int u = 0; u < kRegVecs; ++u) {
      const int i = threadIdx.x + u * 256;
      if (i < nvec) emit(i, v[u]);
    }
  } else {
    for (int i = threadIdx.x; i < nvec; i += 256) emit(i, src[i]);
  }
}

// grid (n_pos, n_kv), head_dim/8 threads: each moves one 16-byte chunk of K and of V.
__global__ void kv_io_kernel(bool write, __nv_bfloat16* pool, int64_t n_pages, int layer, int n_kv, int head_dim,
                             const int* __restrict__ page_row, int pos0, __nv_bfloat16* k, __nv_bfloat16* v,
                             int* status) {
  const int p = pos0 + blockIdx.x, hk = blockIdx.y, c = threadIdx.x;
  const int page = page_row[p / kPageSize];
  if (page < 0 || page >= n_pages) {
    set_status(status, DEV_BAD_INDEX);
    return;
  }
  const size_t base = kv_tile_base(n_pages, n_kv, head_dim, layer, page, hk);
  const int off = kv_tile_offset(p % kPageSize, c * 8, head_dim);
  uint4* pk = reinterpret_cast<uint4*>(pool + base + off);
  uint4* pv = reinterpret_cast<uint4*>(pool + base + kv_tile_elems(head_dim) + off);
  const size_t lin = ((size_t)blockIdx.x * n_kv + hk) * head_dim + c * 8;
  uint4* lk = reinterpret_cast<uint4*>(k + lin);
  uint4* lv = reinterpret_cast<uint4*>(v + lin);
  if (write) {
    *pk = *lk;
    *pv = *lv;
  } else {
    *lk = *pk;
    *lv = *pv;
  }
}

}  // namespace

size_t layout_smem_bytes(int n_req, int n_ctas) {
  return (8 * (size_t)(n_req + 1) + (size_t)(n_ctas / 2 + 1) + (size_t)(n_ctas + 1)) * sizeof(int);
}

void launch_layout(const BatchLayout& bl, const Dims& dm, int tok_per_tile, int n_ctas, int64_t n_pages,
                   int* status, cudaStream_t st) {
  const size_t smem = layout_smem_bytes(bl.n_req, n_ctas);
  static bool configured[kMaxDevices] = {false};
  if (first_use_on_device(configured))    // room for kMaxLayoutRequests requests (the default limit is 48 KB)
    cudaFuncSetAttribute(layout_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)layout_smem_bytes(kMaxLayoutRequests, 1024));
  launch_pdl(layout_kernel, dim3(1), dim3(1024), smem, st, bl, dm.n_kv, dm.mask_id, tok_per_tile, n_ctas, n_pages, status);
}

void launch_embed(const BatchLayout& bl, const Dims& dm, const void* embed, float* h, const void* gain, void* x, float* ss,
                  cudaStream_t st) {
  launch_pdl(embed_kernel, dim3(bl.n_tok), dim3(256), 0, st, (const int*)bl.tok_id, static_cast<const __nv_bfloat16*>(embed), h,
             dm.hidden, dm.vocab, static_cast<const __nv_bfloat16*>(gain), static_cast<__nv_bfloat16*>(x), ss, bl.dyn);
}

void launch_rmsnorm(const float* h, const void* gain, void* x, int rows, int hidden, float eps, cudaStream_t st,
                    const int* rows_dev) {
  launch_pdl(rmsnorm_kernel, dim3(rows), dim3(256), 0, st, h, static_cast<const __nv_bfloat16*>(gain),
             static_cast<__nv_bfloat16*>(x), hidden, eps, rows_dev);
}

void launch_kv_io(bool write, void* pool, int64_t n_pages, int layer, const Dims& dm, const int* page_row_dev, int pos0,
                  int n_pos, void* k, void* v, int* status, cudaStream_t st) {
  if (n_pos <= 0) return;
  dim3 grid(n_pos, dm.n_kv);
  kv_io_kernel<<<grid, dm.head_dim / 8, 0, st>>>(write, static_cast<__nv_bfloat16*>(pool), n_pages, layer, dm.n_kv,
                                                 dm.head_dim, page_row_dev, pos0, static_cast<__nv_bfloat16*>(k),
                                                 static_cast<__nv_bfloat16*>(v), status);
}

}  // namespace recg

namespace recg {
namespace {
__global__ void rope_table_kernel(const int* __restrict__ tok_pos, int n_tok, int half, double log_base,
                                  float2* __restrict__ cs, const int* __restrict__ n_tok_dev) {
  griddep_launch();
  griddep_wait();
  if (n_tok_dev) n_tok = n_tok_dev[0];     // (the grid was sized for the capacity)
  // frequency-major [half][n_tok]: the projection epilogue has one token per thread, so a warp reads 32 consecutive
  // tokens of one frequency in one 256-byte request
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_tok * half) return;
  const int i = idx / n_tok, t = idx % n_tok;
  const double theta = exp(-log_base * (double)i / (double)half);  // base^(-2i/d)
  const double ang = (double)tok_pos[t] * theta;
  cs[idx] = make_float2((float)cos(ang), (float)sin(ang));
}
}  // namespace

void launch_rope_table(const int* tok_pos, int n_tok, int head_dim, float rope_base, void* cs, cudaStream_t st,
                       const int* n_tok_dev) {
  const int half = head_dim / 2;
  const int total = n_tok * half;
  if (total <= 0) return;
  launch_pdl(rope_table_kernel, dim3((total + 255) / 256), dim3(256), 0, st, tok_pos, n_tok, half,
             log((double)rope_base), static_cast<float2*>(cs), n_tok_dev);
}
}  // namespace recg

// ---------------------------------------------------------------------------------------------------
// Debug checks: guard bands behind the workspace regions, and a wait that is meant to run out.
// ---------------------------------------------------------------------------------------------------
namespace recg {
namespace {
constexpr uint32_t kGuardWord = 0x5ca1ab1eu;

// grid = bands, 64 threads: 256 bytes each
__global__ void guard_fill_kernel(uint8_t* base, const size_t* __restrict__ offs) {
  reinterpret_cast<uint32_t*>(base + offs[blockIdx.x])[threadIdx.x] = kGuardWord;
}
__global__ void guard_check_kernel(const uint8_t* base, const size_t* __restrict__ offs, int* status) {
  if (reinterpret_cast<const uint32_t*>(base + offs[blockIdx.x])[threadIdx.x] != kGuardWord) set_status(status, DEV_GUARD);
}

// One CTA, one thread: waits on an mbarrier that nobody ever arrives on, with the same bounded wait the kernels
// use; when the polls are used up it records the timeout in the status word and returns.  Nothing else happens:
// no trap, no fault, the context stays usable.
__global__ void wait_timeout_kernel(uint32_t max_polls, int* status) {
  __shared__ uint64_t bar;
  mbar_init(&bar, 1);
  fence_barrier_init();
  if (!mbar_wait(&bar, 0, max_polls)) set_status(status, DEV_TIMEOUT_FULL);
}
}  // namespace

void launch_guard_fill(void* base, const size_t* offs_dev, int n, cudaStream_t st) {
  if (n > 0) guard_fill_kernel<<<n, 64, 0, st>>>(static_cast<uint8_t*>(base), offs_dev);
}
void launch_guard_check(const void* base, const size_t* offs_dev, int n, int* status, cudaStream_t st) {
  if (n > 0) guard_check_kernel<<<n, 64, 0, st>>>(static_cast<const uint8_t*>(base), offs_dev, status);
}
void launch_wait_timeout(uint32_t max_polls, int* status, cudaStream_t st) {
  wait_timeout_kernel<<<1, 1, 0, st>>>(max_polls, status);
}
}  // namespace recg

// ---------------------------------------------------------------------------------------------------
// Device-resident rounds (Sec. 5.2): descriptor of a round from device arrays, and the step from one round to the next.
// ---------------------------------------------------------------------------------------------------
namespace recg {
namespace {

// One CTA.  Writes the packed descriptor [ctx_len | verify_len | block_size | corr (all zero: no correction branches in
// this mode) | cu_tok | cu_ver | verify_tokens (ragged)] and {n_tok, n_ver}.  A request whose lengths break a capacity
// (negative, no rows, more verify tokens than max_verify, rows beyond its page-table row, or a total beyond max_tokens)
// flags the status word and the round becomes empty (n_tok = 0): later kernels then do nothing.
__global__ void __launch_bounds__(256) pack_device_kernel(DeviceRound dr, int* __restrict__ desc, int* __restrict__ dyn,
                                                          int* status) {
  griddep_launch();
  griddep_wait();
  const int C = dr.n_req;
  int* ctx = desc;
  int* ver = desc + C;
  int* blk = desc + 2 * C;
  int* corr = desc + 3 * C;
  int* cu_tok = desc + 9 * C;
  int* cu_ver = cu_tok + (C + 1);
  int* vt = cu_ver + (C + 1);
  __shared__ int s_bad, s_tok, s_ver;
  if (threadIdx.x == 0) s_bad = 0;
  __syncthreads();
  for (int r = threadIdx.x; r < C; r += blockDim.x) {
    const int L = dr.ctx_len[r], v = dr.verify_len[r], b = dr.block_size[r];
    if (L < 0 || v < 0 || b < 0 || v + b < 1 || v > dr.max_verify ||
        ((long long)L + v + b + kPageSize - 1) / kPageSize > dr.pt_stride)
      s_bad = 1;
    ctx[r] = L;
    ver[r] = v;
    blk[r] = b;
    for (int k = 0; k < 6; ++k) corr[6 * r + k] = 0;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int t = 0, tv = 0;
    cu_tok[0] = cu_ver[0] = 0;
    for (int r = 0; r < C; ++r) {
      t += ver[r] + blk[r];
      tv += ver[r];
      if (t > dr.max_tokens || t < 0) {
        s_bad = 1;
        t = tv = 0;
      }
      cu_tok[r + 1] = t;
      cu_ver[r + 1] = tv;
    }
    if (s_bad) {
      set_status(status, DEV_BAD_INDEX);
      t = tv = 0;
      for (int r = 0; r <= C; ++r) cu_tok[r] = cu_ver[r] = 0;
    }
    s_tok = t;
    s_ver = tv;
    dyn[0] = t;
    dyn[1] = tv;
  }
  __syncthreads();
  if (s_tok == 0) return;
  for (int r = threadIdx.x; r < C; r += blockDim.x)
    for (int j = 0; j < ver[r]; ++j) vt[cu_ver[r] + j] = dr.verify_tokens[(size_t)r * dr.max_verify + j];
}

// One thread per request: the bookkeeping between two rounds (Sec. 3.1, 5.1) from the verification results that are
// still on the device.  planted_emitted (may be null): synthetic acceptance -- the round is taken to have emitted
// min(planted_emitted[r], v) tokens, and its continuation block to be reusable exactly when all drafts were accepted.
__global__ void next_round_kernel(DeviceRound dr, BatchLayout bl, VerifyBuffers vb, const int* __restrict__ next_block,
                                  const int* __restrict__ planted_emitted, RoundLog log, int round, int* status) {
  griddep_launch();
  griddep_wait();
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r < dr.n_req) {
    const int L = bl.ctx_len[r], v = bl.verify_len[r], b = bl.block_size[r];
    const int t0 = bl.cu_tok[r], tv0 = bl.cu_ver[r];
    const bool ran = bl.cu_tok[dr.n_req] > 0;       // an empty round (a capacity was broken) changes nothing
    int a = 0, emitted = 0, cont = 0;
    if (ran && v > 0) {
      a = vb.accept_len[r];
      cont = vb.cont_hit[r];
      if (planted_emitted) {
        const int e = planted_emitted[r] < 1 ? 1 : (planted_emitted[r] > v ? v : planted_emitted[r]);
        a = e - 1;
        cont = (b > 0 && a == v - 1) ? 1 : 0;
      }
      emitted = a + 1;
    }
    if (log.accept_len && round < log.max_rounds) {
      log.accept_len[(size_t)round * dr.n_req + r] = a;
      log.block_size[(size_t)round * dr.n_req + r] = b;
      log.verify_len[(size_t)round * dr.n_req + r] = v;
      if (log.entropy_mean) log.entropy_mean[(size_t)round * dr.n_req + r] = (ran && v > 0) ? vb.entropy_mean[r] : 0.f;
    }
    if (ran && v > 0) {
      // emitted tokens: the accepted drafts y_1 .. y_a, then the verifier's token at row a
      const int last = vb.top1[t0 + a];
      if (log.tokens) {
        int n = log.n_tokens[r];
        for (int i = 1; i <= a && n < log.max_out; ++i) log.tokens[(size_t)r * log.max_out + n++] = bl.verify_tokens[tv0 + i];
        if (n < log.max_out) log.tokens[(size_t)r * log.max_out + n++] = last;
        log.n_tokens[r] = n;
      }
      int nb = next_block ? next_block[r] : b;
      int nv = 1;
      int* y = dr.verify_tokens + (size_t)r * dr.max_verify;
      y[0] = last;
      if (cont) {                      // the drafted block becomes the next verify tokens (its first token only
        nv = b < dr.max_verify ? b : dr.max_verify;   // confirmed the one just emitted)
        const int tb0 = t0 - tv0;      // offset of the request's draft rows in next_draft
        for (int j = 1; j < nv; ++j) y[j] = vb.next_draft[tb0 + j];
      }
      const int nL = L + emitted;
      // the next round must fit the page-table row; a request that has run out of room stops growing
      if (((long long)nL + nv + nb + kPageSize - 1) / kPageSize > dr.pt_stride) {
        nb = 0;
        nv = 1;
        if (((long long)nL + 1 + kPageSize - 1) / kPageSize > dr.pt_stride) set_status(status, DEV_BAD_INDEX);
      }
      dr.ctx_len[r] = nL;
      dr.verify_len[r] = nv;
      dr.block_size[r] = nb;
    } else if (ran && next_block) {
      dr.block_size[r] = next_block[r];
    }
  }
  if (r == 0 && log.n_rounds) log.n_rounds[0] = round + 1;     // rounds logged so far
}

}  // namespace

void launch_pack_device(const DeviceRound& dr, int* desc, int* dyn, int* status, cudaStream_t st) {
  launch_pdl(pack_device_kernel, dim3(1), dim3(256), 0, st, dr, desc, dyn, status);
}

void launch_next_round(const DeviceRound& dr, const BatchLayout& bl, const VerifyBuffers& vb, const int* next_block,
                       const int* planted_emitted, const RoundLog& log, int round, int* status, cudaStream_t st) {
  launch_pdl(next_round_kernel, dim3((dr.n_req + 127) / 128), dim3(128), 0, st, dr, bl, vb, next_block, planted_emitted, log,
             round, status);
}
}  // namespace recg

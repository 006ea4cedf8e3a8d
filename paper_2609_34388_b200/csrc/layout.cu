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

// One CTA.  Shared: 5 arrays of n_req+1 ints.
//
// Attention work list: the 64-token KV blocks of all (request, kv head, row tile) tiles form one line; every
// tile is preceded by kItemCost virtual blocks that stand for the fixed cost of starting an item (staging Q,
// refilling and draining the pipeline).  The line of W cost units is cut into n_ctas equal contiguous ranges,
// one per CTA of the persistent attention grid, and additionally at every tile boundary.  Each piece that holds
// real blocks is an item; a tile whose blocks are cut by CTA boundaries gets one partial slot per piece.
constexpr int kItemCost = 3;

__global__ void __launch_bounds__(1024) layout_kernel(BatchLayout bl, int n_kv, int mask_id, int tok_per_tile,
                                                      int n_ctas, int64_t n_pages, int* status) {
  extern __shared__ int sm[];
  const int C = bl.n_req;
  int* req_blk_off = sm;                 // first global block of request r
  int* tile_off = sm + (C + 1);          // first tile entry of request r
  int* item_off = sm + 2 * (C + 1);      // first item of request r
  int* part_off = sm + 3 * (C + 1);      // first partial slot of request r
  int* req_nb = sm + 4 * (C + 1);        // blocks per tile of request r
  __shared__ int s_per, s_total_blocks;
  const int tid = threadIdx.x, nth = blockDim.x;
  griddep_launch();
  griddep_wait();   // the previous step's kernels may still be reading the arrays this kernel rewrites

  // ---- per-token arrays ----
  for (int t = tid; t < bl.n_tok; t += nth) {
    const int r = upper_request(bl.cu_tok, C, t);
    const int j = t - bl.cu_tok[r];
    const int L = bl.ctx_len[r], v = bl.verify_len[r], b = bl.block_size[r];
    const int pos = L + j;
    const bool is_ver = j < v;
    bl.tok_req[t] = r;
    bl.tok_pos[t] = pos;
    bl.tok_id[t] = is_ver ? bl.verify_tokens[bl.cu_ver[r] + j] : mask_id;
    bl.tok_climit[t] = is_ver ? pos : L + v - 1;
    bl.tok_lo[t] = is_ver ? 0 : L + v;
    bl.tok_hi[t] = is_ver ? 0 : L + v + b;
    int slot = -1;
    if (bl.page_table) {
      const int page = bl.page_table[(size_t)r * bl.pt_stride + pos / kPageSize];
      if (page < 0 || page >= n_pages) set_status(status, DEV_BAD_INDEX);
      else slot = page * kPageSize + pos % kPageSize;
    }
    bl.tok_slot[t] = slot;
  }

  // ---- attention work list ----
  for (int r = tid; r < C; r += nth) {
    const int n = bl.verify_len[r] + bl.block_size[r];
    req_nb[r] = (bl.ctx_len[r] + n + 63) / 64;
    tile_off[r + 1] = n_kv * ((n + tok_per_tile - 1) / tok_per_tile);
  }
  __syncthreads();
  if (tid == 0) {
    req_blk_off[0] = 0;
    tile_off[0] = 0;
    long long w = 0;
    for (int r = 0; r < C; ++r) {
      w += (long long)tile_off[r + 1] * (req_nb[r] + kItemCost);
      if (w > 0x3fffffff) w = 0x3fffffff;   // far beyond any pool; keeps the arithmetic in int
      req_blk_off[r + 1] = (int)w;
      tile_off[r + 1] += tile_off[r];
    }
    s_total_blocks = (int)w;
    const int per = (int)((w + n_ctas - 1) / n_ctas);
    s_per = per < 1 ? 1 : per;
  }
  __syncthreads();
  const int per = s_per, W = s_total_blocks;
  for (int r = tid; r < C; r += nth) {
    const int nb = req_nb[r], nt = tile_off[r + 1] - tile_off[r];
    int items = 0, parts_split = 0;
    for (int k = 0; k < nt; ++k) {
      const int g0 = req_blk_off[r] + k * (nb + kItemCost) + kItemCost, g1 = g0 + nb;   // cost range of the real blocks
      const int parts = (g1 - 1) / per - g0 / per + 1;
      items += parts;
      if (parts > 1) parts_split += parts;
    }
    item_off[r + 1] = items;
    part_off[r + 1] = parts_split;
  }
  __syncthreads();
  if (tid == 0) {
    item_off[0] = part_off[0] = 0;
    for (int r = 0; r < C; ++r) {
      item_off[r + 1] += item_off[r];
      part_off[r + 1] += part_off[r];
    }
    int n_items = item_off[C];
    if (n_items > bl.max_items || part_off[C] > bl.max_parts) {
      set_status(status, DEV_BAD_INDEX);
      n_items = 0;
    }
    bl.counts[0] = n_items;
    bl.counts[1] = tile_off[C];
    bl.counts[2] = per;
  }
  __syncthreads();
  const int n_items = bl.counts[0];
  for (int r = tid; r <= C; r += nth) bl.tile_off[r] = tile_off[r];
  for (int c = tid; c <= n_ctas; c += nth)
    bl.cta_off[c] = -1;                                                      // filled below
  if (n_items == 0) return;
  for (int r = tid; r < C; r += nth) {
    const int n = bl.verify_len[r] + bl.block_size[r];
    const int kv_len = bl.ctx_len[r] + n;
    const int nb = req_nb[r], nt = tile_off[r + 1] - tile_off[r];
    const int tiles = nt / n_kv;
    int item = item_off[r], part = part_off[r];
    for (int k = 0; k < nt; ++k) {
      const int kvh = k / tiles, tile = k % tiles;
      const int g0 = req_blk_off[r] + k * (nb + kItemCost) + kItemCost, g1 = g0 + nb;
      const int c_first = g0 / per, c_last = (g1 - 1) / per;
      const int parts = c_last - c_first + 1;
      AttnTile tl;
      tl.part_begin = parts > 1 ? part : -1;
      tl.n_parts = parts;
      tl.tok0 = bl.cu_tok[r] + tile * tok_per_tile;
      tl.ntok = min(tok_per_tile, n - tile * tok_per_tile);
      tl.kv_head = kvh;
      bl.tiles[tile_off[r] + k] = tl;
      for (int c = c_first; c <= c_last; ++c, ++item) {
        const int gs = max(g0, c * per), ge = min(g1, (c + 1) * per);
        AttnItem a;
        a.req = r;
        a.kv_head = kvh;
        a.tok0 = tl.tok0;
        a.ntok = tl.ntok;
        a.blk_begin = gs - g0;
        a.blk_end = ge - g0;
        a.part = parts > 1 ? part++ : -1;
        a.kv_len = kv_len;
        bl.items[item] = a;
        bl.item_cta[item] = c;
      }
    }
  }
  // first item of every CTA: items are ordered by CTA, so a CTA's range starts where the owner changes
  __syncthreads();
  for (int it = tid; it < n_items; it += nth) {
    const int c = bl.item_cta[it];
    const int prev = it ? bl.item_cta[it - 1] : -1;
    for (int cc = prev + 1; cc <= c; ++cc) bl.cta_off[cc] = it;   // CTAs between two owners have no items
  }
  const int last_owner = bl.item_cta[n_items - 1];
  for (int c = last_owner + 1 + tid; c <= n_ctas; c += nth) bl.cta_off[c] = n_items;
}

__global__ void embed_kernel(const int* __restrict__ tok_id, const __nv_bfloat16* __restrict__ embed,
                             float* __restrict__ h, int hidden, int vocab) {
  griddep_launch();
  griddep_wait();
  const int t = blockIdx.x;
  int id = tok_id[t];
  id = id < 0 ? 0 : (id >= vocab ? vocab - 1 : id);
  const __nv_bfloat162* src = reinterpret_cast<const __nv_bfloat162*>(embed + (size_t)id * hidden);
  float2* dst = reinterpret_cast<float2*>(h + (size_t)t * hidden);
  for (int i = threadIdx.x; i < hidden / 2; i += blockDim.x) dst[i] = __bfloat1622float2(src[i]);
}

// One CTA per row; fp32 in, bf16 out.  hidden a multiple of 4.  The row is read once and kept in registers
// when it fits (hidden <= 256 threads x kRegVecs float4), otherwise it is read a second time.
constexpr int kRegVecs = 8;
__global__ void __launch_bounds__(256) rmsnorm_kernel(const float* __restrict__ h, const __nv_bfloat16* __restrict__ g,
                                                      __nv_bfloat16* __restrict__ x, int hidden, float eps) {
  griddep_launch();
  griddep_wait();
  const int row = blockIdx.x;
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

void launch_layout(const BatchLayout& bl, const Dims& dm, int tok_per_tile, int n_ctas, int64_t n_pages,
                   int* status, cudaStream_t st) {
  const size_t smem = 5 * (size_t)(bl.n_req + 1) * sizeof(int);
  launch_pdl(layout_kernel, dim3(1), dim3(1024), smem, st, bl, dm.n_kv, dm.mask_id, tok_per_tile, n_ctas, n_pages, status);
}

void launch_embed(const BatchLayout& bl, const Dims& dm, const void* embed, float* h, cudaStream_t st) {
  launch_pdl(embed_kernel, dim3(bl.n_tok), dim3(256), 0, st, (const int*)bl.tok_id, static_cast<const __nv_bfloat16*>(embed), h,
             dm.hidden, dm.vocab);
}

void launch_rmsnorm(const float* h, const void* gain, void* x, int rows, int hidden, float eps, cudaStream_t st) {
  launch_pdl(rmsnorm_kernel, dim3(rows), dim3(256), 0, st, h, static_cast<const __nv_bfloat16*>(gain),
             static_cast<__nv_bfloat16*>(x), hidden, eps);
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
                                  float2* __restrict__ cs) {
  griddep_launch();
  griddep_wait();
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_tok * half) return;
  const int t = idx / half, i = idx % half;
  const double theta = exp(-log_base * (double)i / (double)half);  // base^(-2i/d)
  const double ang = (double)tok_pos[t] * theta;
  cs[idx] = make_float2((float)cos(ang), (float)sin(ang));
}
}  // namespace

void launch_rope_table(const int* tok_pos, int n_tok, int head_dim, float rope_base, void* cs, cudaStream_t st) {
  const int half = head_dim / 2;
  const int total = n_tok * half;
  if (total <= 0) return;
  launch_pdl(rope_table_kernel, dim3((total + 255) / 256), dim3(256), 0, st, tok_pos, n_tok, half,
             log((double)rope_base), static_cast<float2*>(cs));
}
}  // namespace recg

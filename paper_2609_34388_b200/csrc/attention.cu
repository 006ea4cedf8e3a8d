// Hybrid-mask paged-KV attention (Eq. 1 over a shared prefix), split over KV ranges, plus the combine.
//
// A work item is (request, kv head, row tile of <=128 query rows = tokens x GQA group, KV block range).
// One producer warp streams the item's 64-token KV blocks page by page with 1-D bulk copies into a
// shared-memory ring (the pool tiles are stored pre-swizzled, so a linear copy lands fragment-ready);
// eight consumer warps hold 16 query rows each and, when the tile has fewer than 128 rows, share the
// rows and split the KV blocks among themselves instead.  Only blocks that reach past the committed
// context apply the visibility test; the prefix loop is mask-free.
#include <cstdlib>
#include "common.cuh"
#include "kernels.h"

namespace recg {

namespace {

constexpr int kStages = 4;
constexpr int kConsumerWarps = 8;
constexpr int kAttnThreads = (kConsumerWarps + 1) * 32;
constexpr int kBlockTokens = 64;
constexpr int kPagesPerBlock = kBlockTokens / kPageSize;
constexpr uint32_t kSpinLimit = 1u << 22;

template <int D>
struct AttnSmem {
  static constexpr int kPageBytes = 2 * kPageSize * D * 2;          // K tile + V tile
  static constexpr int kStageBytes = kPagesPerBlock * kPageBytes;
  static constexpr int kRingBytes = kStages * kStageBytes;
  static constexpr int kMergeFloats = (D / 8 * 4 + 4) * 32;         // per warp: o frags + m[2] + l[2]
  static constexpr int kMergeBytes = kConsumerWarps * kMergeFloats * 4;
  static constexpr int kBarOffset = kRingBytes + kMergeBytes;
  static constexpr int kTotal = kBarOffset + 2 * kStages * 8 + 16;
};

struct AttnParams {
  const AttnItem* items;
  const int* cta_off;
  const int* page_table;
  int pt_stride;
  const int* tok_climit;
  const int* tok_lo;
  const int* tok_hi;
  const __nv_bfloat16* q;
  __nv_bfloat16* o;
  const __nv_bfloat16* pool;
  int64_t n_pages;
  int layer, n_q, n_kv, group;
  float scale_log2;   // log2(e) / sqrt(d)
  float* part_o;      // [part][128][D]
  float* part_ml;     // [part][128][2]
  int* status;
};

__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1) attention_kernel(AttnParams P) {
  using SM = AttnSmem<D>;
  extern __shared__ __align__(1024) uint8_t smem[];
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + SM::kBarOffset);
  uint64_t* empty_bar = full_bar + kStages;
  float* merge = reinterpret_cast<float*>(smem + SM::kRingBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  griddep_launch();

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], kConsumerWarps);
    }
    fence_barrier_init();
  }
  __syncthreads();
  griddep_wait();

  // the CTA walks two ranges of the item list one after the other (see the layout kernel)
  const int4 r4 = *reinterpret_cast<const int4*>(P.cta_off + 4 * blockIdx.x);
  const int range_n0 = r4.y - r4.x;
  const int item_begin = 0, item_end = range_n0 + (r4.w - r4.z);
  auto item_at = [&](int i) { return i < range_n0 ? r4.x + i : r4.z + (i - range_n0); };
  uint32_t it = 0;  // running block counter, identical in producer and consumers
  bool aborted = false;

  if (warp == kConsumerWarps) {
    // ------------------------------ producer ------------------------------
    for (int item = item_begin; item < item_end && !aborted; ++item) {
      const AttnItem w = P.items[item_at(item)];
      const int n_req_pages = (w.kv_len + kPageSize - 1) / kPageSize;
      const int* pt = P.page_table + (size_t)w.req * P.pt_stride;
      // lanes 0..3 each own one page of the block; ids are fetched one block ahead of their use
      auto fetch_page = [&](int n) -> int {
        int pg = -1;
        if (lane < kPagesPerBlock && n < w.blk_end) {
          const int lp = n * kPagesPerBlock + lane;
          if (lp < n_req_pages) pg = __ldg(pt + lp);   // validated when used
        }
        return pg;
      };
      int pg_next = fetch_page(w.blk_begin);
      for (int n = w.blk_begin; n < w.blk_end; ++n, ++it) {
        const int s = it % kStages;
        int my_pg = pg_next;
        pg_next = fetch_page(n + 1);                   // in flight during this iteration
        if (my_pg >= P.n_pages) {
          set_status(P.status, DEV_BAD_INDEX);
          my_pg = -1;
        }
        if (!mbar_wait(&empty_bar[s], ((it / kStages) & 1) ^ 1, kSpinLimit)) {
          set_status(P.status, DEV_TIMEOUT_EMPTY);
          aborted = true;
          break;
        }
        const unsigned valid = __ballot_sync(0xffffffffu, my_pg >= 0);
        if (lane == 0) {
          if (valid == 0) mbar_arrive(&full_bar[s]);
          else mbar_arrive_expect_tx(&full_bar[s], __popc(valid) * SM::kPageBytes);
        }
        __syncwarp();
        if (my_pg >= 0) {
          const __nv_bfloat16* src = P.pool + kv_tile_base(P.n_pages, P.n_kv, D, P.layer, my_pg, w.kv_head);
          bulk_g2s(smem + s * SM::kStageBytes + lane * SM::kPageBytes, src, SM::kPageBytes, &full_bar[s]);
        }
        __syncwarp();
      }
    }
    if (aborted && lane == 0) {
      // let copies already in flight land before the CTA may exit
      for (int s = 0; s < kStages; ++s) {
        for (uint32_t i = 0; i < (1u << 16); ++i) {
          if (mbar_try_wait(&full_bar[s], 0) || mbar_try_wait(&full_bar[s], 1)) break;
          __nanosleep(64);
        }
      }
    }
    return;
  }

  // ------------------------------ consumers ------------------------------
  const int g = lane >> 2, q4 = lane & 3;
  const uint32_t ring = smem_u32(smem);

  for (int item = item_begin; item < item_end; ++item) {
    const AttnItem w = P.items[item_at(item)];
    const int R = w.ntok * P.group;
    const int RW = (R + 15) >> 4;
    const int KW = RW == 1 ? 8 : (RW == 2 ? 4 : (RW <= 4 ? 2 : 1));
    const int rw = warp % RW, kw = warp / RW;
    const bool active = kw < KW;

    // Q fragments and per-row visibility for this thread's two rows (g and g + 8 of the warp's 16)
    uint32_t qf[D / 16][4];
    int climit[2], vlo[2], vhi[2];
    int qrow_tok[2], qrow_head[2];
    bool rvalid[2];
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      const int rho = rw * 16 + g + hh * 8;
      rvalid[hh] = active && rho < R;
      const int j = rho / P.group, hg = rho % P.group;
      const int t = w.tok0 + (rvalid[hh] ? j : 0);
      qrow_tok[hh] = t;
      qrow_head[hh] = w.kv_head * P.group + hg;
      climit[hh] = rvalid[hh] ? P.tok_climit[t] : -1;
      vlo[hh] = rvalid[hh] ? P.tok_lo[t] : 0;
      vhi[hh] = rvalid[hh] ? P.tok_hi[t] : 0;
    }
#pragma unroll
    for (int k = 0; k < D / 16; ++k) {
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const uint32_t* src = reinterpret_cast<const uint32_t*>(
            P.q + ((size_t)qrow_tok[hh] * P.n_q + qrow_head[hh]) * D + k * 16 + q4 * 2);
        qf[k][hh] = rvalid[hh] ? __ldg(src) : 0u;
        qf[k][hh + 2] = rvalid[hh] ? __ldg(src + 4) : 0u;
      }
    }

    float o[D / 8][4];
#pragma unroll
    for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float m_run[2] = {-1e30f, -1e30f};
    float l_run[2] = {0.f, 0.f};
    const int ctx_first_new = w.kv_len;  // positions >= kv_len never exist

    for (int n = w.blk_begin; n < w.blk_end; ++n, ++it) {
      const int s = it % kStages;
      if (!aborted && !mbar_wait(&full_bar[s], (it / kStages) & 1, kSpinLimit)) {
        set_status(P.status, DEV_TIMEOUT_FULL);
        aborted = true;
      }
      if (!aborted && active && ((n - w.blk_begin) % KW) == kw) {
        const uint32_t stage = ring + s * SM::kStageBytes;
        // ---- S = Q K^T over the 64 tokens of the block ----
        float sc[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
        for (int j = 0; j < D / 32; ++j) {
#pragma unroll
          for (int nt = 0; nt < 8; ++nt) {
            const int token = nt * 8 + (lane & 7);
            const int pg = token >> 4, tok = token & 15;
            const int c = 4 * j + (lane >> 3);
            const uint32_t addr = stage + pg * SM::kPageBytes + ((tok >> 3) * (D / 64) + (c >> 3)) * 1024 +
                                  (tok & 7) * 128 + (((c & 7) ^ (tok & 7)) << 4);
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4(b0, b1, b2, b3, addr);
            mma_bf16_16816(sc[nt], qf[2 * j], b0, b1);
            mma_bf16_16816(sc[nt], qf[2 * j + 1], b2, b3);
          }
        }
        // ---- visibility (only blocks that reach past the mask-free prefix) ----
        const int pos0 = n * kBlockTokens;
        const int min_limit = min(climit[0], climit[1]);
        // every row of the tile sees all positions <= its climit; the block is mask-free when it ends
        // at or before the smallest climit of the warp's rows (invalid rows carry -1 and force the test)
        const bool need_mask = __any_sync(0xffffffffu, pos0 + kBlockTokens - 1 > min_limit);
        if (need_mask) {
#pragma unroll
          for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int hh = e >> 1;
              const int pos = pos0 + nt * 8 + q4 * 2 + (e & 1);
              const bool vis = pos <= climit[hh] || (pos >= vlo[hh] && pos < vhi[hh]);
              if (!vis) sc[nt][e] = -INFINITY;
            }
          }
        }
        // ---- online softmax in the log2 domain ----
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          float mx = -INFINITY;
#pragma unroll
          for (int nt = 0; nt < 8; ++nt) mx = fmaxf(mx, fmaxf(sc[nt][2 * hh], sc[nt][2 * hh + 1]));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
          const float m_new = fmaxf(m_run[hh], mx * P.scale_log2);
          const float alpha = exp2f(m_run[hh] - m_new);
          m_run[hh] = m_new;
          float ls = 0.f;
#pragma unroll
          for (int nt = 0; nt < 8; ++nt) {
            const float p0 = exp2f(sc[nt][2 * hh] * P.scale_log2 - m_new);
            const float p1 = exp2f(sc[nt][2 * hh + 1] * P.scale_log2 - m_new);
            sc[nt][2 * hh] = p0;
            sc[nt][2 * hh + 1] = p1;
            ls += p0 + p1;
          }
          l_run[hh] = l_run[hh] * alpha + ls;
#pragma unroll
          for (int i = 0; i < D / 8; ++i) {
            o[i][2 * hh] *= alpha;
            o[i][2 * hh + 1] *= alpha;
          }
        }
        // ---- O += P V ----
        const bool sanitize = pos0 + kBlockTokens > ctx_first_new;  // stale or unwritten V rows in the block
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          uint32_t a[4];
          a[0] = pack_bf16(sc[2 * kk][0], sc[2 * kk][1]);
          a[1] = pack_bf16(sc[2 * kk][2], sc[2 * kk][3]);
          a[2] = pack_bf16(sc[2 * kk + 1][0], sc[2 * kk + 1][1]);
          a[3] = pack_bf16(sc[2 * kk + 1][2], sc[2 * kk + 1][3]);
          uint32_t keep0 = 0xffffffffu, keep1 = 0xffffffffu;
          if (sanitize) {
            const int tb = pos0 + kk * 16 + q4 * 2;
            keep0 = (tb < ctx_first_new ? 0x0000ffffu : 0u) | (tb + 1 < ctx_first_new ? 0xffff0000u : 0u);
            keep1 = (tb + 8 < ctx_first_new ? 0x0000ffffu : 0u) | (tb + 9 < ctx_first_new ? 0xffff0000u : 0u);
          }
          const int mi = lane >> 3, r8 = lane & 7;
          const int tok = (mi & 1) * 8 + r8;
#pragma unroll
          for (int jj = 0; jj < D / 16; ++jj) {
            const int c = 2 * jj + (mi >> 1);
            const uint32_t addr = stage + kk * SM::kPageBytes + kPageSize * D * 2 +
                                  ((tok >> 3) * (D / 64) + (c >> 3)) * 1024 + (tok & 7) * 128 +
                                  (((c & 7) ^ (tok & 7)) << 4);
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4_trans(b0, b1, b2, b3, addr);
            if (sanitize) {
              b0 &= keep0; b1 &= keep1; b2 &= keep0; b3 &= keep1;
            }
            mma_bf16_16816(o[2 * jj], a, b0, b1);
            mma_bf16_16816(o[2 * jj + 1], a, b2, b3);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty_bar[s]);
    }

    // quad-reduce the row sums
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 1);
      l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 2);
    }

    // ---- merge the KV-split warps of the CTA ----
    if (KW > 1) {
      float* mine = merge + warp * SM::kMergeFloats;
      if (active && kw > 0) {
#pragma unroll
        for (int i = 0; i < D / 8; ++i)
#pragma unroll
          for (int e = 0; e < 4; ++e) mine[(i * 4 + e) * 32 + lane] = o[i][e];
        mine[(D / 2 + 0) * 32 + lane] = m_run[0];
        mine[(D / 2 + 1) * 32 + lane] = m_run[1];
        mine[(D / 2 + 2) * 32 + lane] = l_run[0];
        mine[(D / 2 + 3) * 32 + lane] = l_run[1];
      }
      consumer_bar();
      if (active && kw == 0) {
        for (int k2 = 1; k2 < KW; ++k2) {
          const float* oth = merge + (k2 * RW + rw) * SM::kMergeFloats;
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            const float mo = oth[(D / 2 + hh) * 32 + lane];
            const float lo_ = oth[(D / 2 + 2 + hh) * 32 + lane];
            const float m_new = fmaxf(m_run[hh], mo);
            const float fa = exp2f(m_run[hh] - m_new), fb = exp2f(mo - m_new);
            m_run[hh] = m_new;
            l_run[hh] = l_run[hh] * fa + lo_ * fb;
#pragma unroll
            for (int i = 0; i < D / 8; ++i) {
              o[i][2 * hh] = o[i][2 * hh] * fa + oth[(i * 4 + 2 * hh) * 32 + lane] * fb;
              o[i][2 * hh + 1] = o[i][2 * hh + 1] * fa + oth[(i * 4 + 2 * hh + 1) * 32 + lane] * fb;
            }
          }
        }
      }
      consumer_bar();  // scratch may be rewritten by the next item only after everyone has read it
    }

    // ---- write out ----
    if (active && kw == 0 && !aborted) {
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        if (!rvalid[hh]) continue;
        const int rho = rw * 16 + g + hh * 8;
        if (w.part < 0) {
          const float inv = l_run[hh] > 0.f ? 1.f / l_run[hh] : 0.f;
          uint32_t* dst = reinterpret_cast<uint32_t*>(P.o + ((size_t)qrow_tok[hh] * P.n_q + qrow_head[hh]) * D);
#pragma unroll
          for (int i = 0; i < D / 8; ++i)
            dst[i * 4 + q4] = pack_bf16(o[i][2 * hh] * inv, o[i][2 * hh + 1] * inv);
        } else {
          float2* dst = reinterpret_cast<float2*>(P.part_o + ((size_t)w.part * 128 + rho) * D);
#pragma unroll
          for (int i = 0; i < D / 8; ++i) dst[i * 4 + q4] = make_float2(o[i][2 * hh], o[i][2 * hh + 1]);
          if (q4 == 0) {
            P.part_ml[((size_t)w.part * 128 + rho) * 2 + 0] = m_run[hh];
            P.part_ml[((size_t)w.part * 128 + rho) * 2 + 1] = l_run[hh];
          }
        }
      }
    }
  }
}

// Merges the KV-range partials of the tiles that were split.  Tiles with a single part were written by the
// attention kernel itself and are skipped.  Work unit = 16 rows of a tile, one warp per query row, each lane D/32
// consecutive dims.  The kernel is latency bound (tile entry -> (max, sum) pairs -> partial rows), so every level
// is fetched for all parts at once and the grid is sized to hold all rows in one or two waves.
template <int D>
__global__ void __launch_bounds__(512, 3) attention_combine_kernel(const AttnTile* __restrict__ tiles,
                                                                const int* __restrict__ counts, int n_q, int group,
                                                                const float* __restrict__ part_o,
                                                                const float* __restrict__ part_ml,
                                                                __nv_bfloat16* __restrict__ o) {
  constexpr int E = D / 32;
  constexpr int kMaxP = 4;     // parts fetched together; longer lists go round by round
  griddep_launch();
  griddep_wait();
  const int n_tiles = counts[1];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int wu = blockIdx.x; wu < n_tiles * 8; wu += gridDim.x) {
    const AttnTile tl = tiles[wu >> 3];
    if (tl.n_parts <= 1) continue;
    const int rho = (wu & 7) * 16 + warp;
    if (rho >= tl.ntok * group) continue;
    float acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;
    float m = -1e30f, l = 0.f;
    for (int p0 = 0; p0 < tl.n_parts; p0 += kMaxP) {
      const int np = min(kMaxP, tl.n_parts - p0);
      float2 ml[kMaxP];
      float v[kMaxP][E];
#pragma unroll
      for (int p = 0; p < kMaxP; ++p) {
        ml[p] = make_float2(-1e30f, 0.f);
        if (p < np) {
          const size_t row = (size_t)(tl.part_begin + p0 + p) * 128 + rho;
          ml[p] = __ldcg(reinterpret_cast<const float2*>(part_ml) + row);
          if constexpr (E == 4) {
            const float4 t = __ldcg(reinterpret_cast<const float4*>(part_o + row * D) + lane);
            v[p][0] = t.x; v[p][1] = t.y; v[p][2] = t.z; v[p][3] = t.w;
          } else {
            const float2 t = __ldcg(reinterpret_cast<const float2*>(part_o + row * D) + lane);
            v[p][0] = t.x; v[p][1] = t.y;
          }
        }
      }
      float m_new = m;
#pragma unroll
      for (int p = 0; p < kMaxP; ++p) m_new = fmaxf(m_new, ml[p].x);
      const float f = exp2f(m - m_new);
      m = m_new;
      l *= f;
#pragma unroll
      for (int e = 0; e < E; ++e) acc[e] *= f;
#pragma unroll
      for (int p = 0; p < kMaxP; ++p)
        if (p < np) {
          const float wgt = exp2f(ml[p].x - m);
          l += wgt * ml[p].y;
#pragma unroll
          for (int e = 0; e < E; ++e) acc[e] += wgt * v[p][e];
        }
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;
    const int j = rho / group, hg = rho % group;
    __nv_bfloat16* dst = o + ((size_t)(tl.tok0 + j) * n_q + tl.kv_head * group + hg) * D + lane * E;
    if constexpr (E == 4) {
      uint2 pk;
      pk.x = pack_bf16(acc[0] * inv, acc[1] * inv);
      pk.y = pack_bf16(acc[2] * inv, acc[3] * inv);
      *reinterpret_cast<uint2*>(dst) = pk;
    } else {
      *reinterpret_cast<uint32_t*>(dst) = pack_bf16(acc[0] * inv, acc[1] * inv);
    }
  }
}

template <int D>
void launch_attention_t(const BatchLayout& bl, const Dims& dm, int layer, const void* q, void* o, const void* kv_pool,
                        int64_t n_pages, float* part_o, float* part_ml, int tok_per_tile, int n_sm, int* status,
                        cudaStream_t st) {
  static bool configured[kMaxDevices] = {false};
  if (first_use_on_device(configured))
    cudaFuncSetAttribute(attention_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<D>::kTotal);

  AttnParams P;
  P.items = bl.items;
  P.cta_off = bl.cta_off;
  P.page_table = bl.page_table;
  P.pt_stride = bl.pt_stride;
  P.tok_climit = bl.tok_climit;
  P.tok_lo = bl.tok_lo;
  P.tok_hi = bl.tok_hi;
  P.q = static_cast<const __nv_bfloat16*>(q);
  P.o = static_cast<__nv_bfloat16*>(o);
  P.pool = static_cast<const __nv_bfloat16*>(kv_pool);
  P.n_pages = n_pages;
  P.layer = layer;
  P.n_q = dm.n_q;
  P.n_kv = dm.n_kv;
  P.group = dm.n_q / dm.n_kv;
  P.scale_log2 = 1.4426950408889634f / sqrtf((float)D);
  P.part_o = part_o;
  P.part_ml = part_ml;
  P.status = status;
  launch_pdl(attention_kernel<D>, dim3(n_sm), dim3(kAttnThreads), AttnSmem<D>::kTotal, st, P);
  launch_pdl(attention_combine_kernel<D>, dim3(4 * n_sm), dim3(512), 0, st, (const AttnTile*)bl.tiles, (const int*)bl.counts,
             dm.n_q, P.group, (const float*)part_o, (const float*)part_ml, static_cast<__nv_bfloat16*>(o));
}

}  // namespace

size_t attention_smem_bytes(int head_dim) {
  return head_dim == 64 ? AttnSmem<64>::kTotal : AttnSmem<128>::kTotal;
}

void launch_attention(const BatchLayout& bl, const Dims& dm, int layer, const void* q, void* o, const void* kv_pool,
                      int64_t n_pages, float* part_o, float* part_ml, int tok_per_tile, int n_sm, int* status,
                      cudaStream_t st, bool use_tc, bool layout_settled) {
  if (use_tc && dm.head_dim == 128) {
    launch_attention_tc_main(bl, dm, layer, q, o, kv_pool, n_pages, part_o, part_ml, n_sm, status, st, layout_settled);
    launch_pdl(attention_combine_kernel<128>, dim3(4 * n_sm), dim3(512), 0, st, (const AttnTile*)bl.tiles,
               (const int*)bl.counts, dm.n_q, dm.n_q / dm.n_kv, (const float*)part_o, (const float*)part_ml,
               static_cast<__nv_bfloat16*>(o));
    return;
  }
  if (dm.head_dim == 64)
    launch_attention_t<64>(bl, dm, layer, q, o, kv_pool, n_pages, part_o, part_ml, tok_per_tile, n_sm, status, st);
  else
    launch_attention_t<128>(bl, dm, layer, q, o, kv_pool, n_pages, part_o, part_ml, tok_per_tile, n_sm, status, st);
}

}  // namespace recg

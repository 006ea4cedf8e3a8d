// Projection GEMM on the 5th-generation tensor cores: y = x . w^T, bf16 in, fp32 accumulate in TMEM.
//
// Persistent, warp-specialised CTA of 6 warps:
//   warp 0   producer: TMA tiled loads (128B swizzle) of the x tile [128 x 64] and the w tile [BN x 64]
//            into a shared-memory ring, completion on mbarriers;
//   warp 1   one elected lane issues tcgen05.mma (M = 128, N = BN, K = 16) from shared-memory descriptors
//            into one of two TMEM accumulators and commits to the ring's empty barriers;
//   warps 2-5  epilogue: tcgen05.ld of the finished accumulator (each warp its 32-lane quadrant), then the
//            fused epilogue straight from registers (residual add, SwiGLU, rotary + paged KV append, or
//            plain store) while the MMA warp already fills the other accumulator; output rows leave through
//            TMA box stores (add-reductions for the residual stream) from a small swizzled staging area.
// Tiles are walked m-fastest so that CTAs running together share the same weight tile through L2.
// Tiles can be cut over K (stream-K): partial tiles are parked in a workspace and reduced by the last part to arrive; for
// problems of one row tile (at most 128 rows) the parts of a tile form a thread-block cluster instead and hand their
// partial tiles to the cluster's leader through distributed shared memory.
// Every wait is bounded; on a timeout the kernel records a status code, drains and frees TMEM.
#include <cuda.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <cmath>
#include <mutex>
#include <unordered_map>

#include "common.cuh"
#include "epilogue.cuh"
#include "kernels.h"
#include "tc_ptx.cuh"

namespace recg {

namespace {

constexpr int BM = 128, BK = 64;
constexpr int kTcThreads = 192;
constexpr int kSmemBudget = 192 * 1024;     // operand ring (every configuration's stage size divides it)
constexpr int kStageOutBytes = 4 * 4096;      // per epilogue warp: two 2 KB boxes of output on their way to the TMA unit
// EPI_RESIDUAL_NORM kernels also stage the OLD residual rows (two 4 KB chunks per epilogue warp, fetched by the TMA unit
// ahead of their use) and the gains of the tile's columns (512 bytes per warp); their operand ring is that much shorter
constexpr int kNormHBytes = 4 * 2 * 4096;
constexpr int kNormGBytes = 4 * 512;
constexpr int kNormBytes = kNormHBytes + kNormGBytes + 6 * 1024;   // (rounded so that the ring budget stays a multiple of 8 KB)
constexpr uint32_t kSpin = 1u << 22;

template <int BN, bool PAIR = false, bool NORM = false> struct TcCfg {
  static constexpr int kBudget = NORM ? kSmemBudget - kNormBytes : kSmemBudget;
  static constexpr int kABytes = BM * BK * 2;
  static constexpr int kBBytes = (PAIR ? BN / 2 : BN) * BK * 2;     // per CTA: a pair splits the weight tile
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kStages = (kBudget / kStageBytes) > 8 ? 8 : (kBudget / kStageBytes);
  static constexpr int kMaxStages = 16;
  // thin problems (M <= 32) load only 32 rows of x per stage: the stage shrinks and more stages fit.  The MMA
  // still reads 128 rows; rows 32.. alias the bytes that follow (harmless: those accumulator rows are never
  // stored), so the ring is followed by a pad that keeps the last stage's read inside the allocation.
  static constexpr int kThinABytes = 32 * BK * 2;
  static constexpr int kThinStageBytes = kThinABytes + kBBytes;
  static constexpr int kThinStages =
      (kBudget / kThinStageBytes) > kMaxStages ? kMaxStages : (kBudget / kThinStageBytes);
  static constexpr int kRingBytes = kBudget + kABytes;     // either ring plus the pad
  static constexpr int kBarBytes = (2 * kMaxStages + 5 + 8) * 8 + 16;
  static constexpr int kNormOff = kRingBytes + kStageOutBytes;             // old residual rows, then gains (NORM only)
  static constexpr int kBarOff = kNormOff + (NORM ? kNormHBytes + kNormGBytes : 0);
  static constexpr int kSmemBytes = kBarOff + kBarBytes + 1024;  // + slack for 1024-byte alignment
  static constexpr int kTmemCols = 2 * BN < 32 ? 32 : 2 * BN;                  // power of two: 128, 256, 512
};

using namespace tc;   // the tcgen05 / TMA wrappers (tc_ptx.cuh)

// ---- CTA pairs (tcgen05 cta_group::2) ----------------------------------------------------------------
// With PAIR a cluster of two CTAs computes tiles of 256 rows: each CTA loads its own 128 rows of x and its own
// half of the weight tile per k-block (32 KB per stage instead of the 48 KB a single CTA needs for 128 x 256, so
// six stages fit and a third fewer operand bytes cross L2 -> shared memory per flop); the tensor cores of the
// pair read both halves of the weight tile, each CTA accumulates its 128 rows in its own TMEM.  Only the leader
// CTA (cluster rank 0) issues MMAs.
//   full barrier  (leader's):   the leader's producer arrives with the byte count of BOTH CTAs' loads; both CTAs'
//                               TMA loads (cta_group::2 form, no multicast) complete on it
//   empty barrier (per CTA):    tcgen05.commit multicast to both CTAs frees the stage in each
//   accumulator full (per CTA): commit multicast; accumulator empty (leader's): all eight epilogue warps of the
//                               pair arrive (the peer's remotely)
// The scheduling unit is the cluster; the two CTAs of a cluster park and reduce their halves of a cut tile
// independently (own slots, own counters).
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// the shared::cluster address of the same location in the CTA of rank `rank`
__device__ __forceinline__ uint32_t mapa_rank(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t smem_dst, const CUtensorMap* map, int x, int y, uint32_t bar_cluster) {
  asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               :
               : "r"(smem_dst), "l"(map), "r"(bar_cluster), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                               uint32_t accumulate) {
  const uint32_t z = 0;
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n}"
      :
      : "r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(z)
      : "memory");
}
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {   // arrives on this barrier in both CTAs
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
                   smem_u32(bar)),
               "h"(mask)
               : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* smem_slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_slot)), "r"(cols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}
__device__ __forceinline__ void st_cluster_f4(uint32_t addr_cluster, const float4& v) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr_cluster), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
               : "memory");
}

// ---- register epilogue: one thread owns one output row -------------------------------------------

// ---- epilogue through the TMA unit --------------------------------------------------------------------------------
// A warp's chunk (lane = row, 64 bytes per row: 32 bf16 or 16 fp32 columns) goes to one of the warp's two 2 KB staging
// buffers in the 64-byte-swizzle order of the output tensor map (16-byte piece c of row r at piece c ^ ((r >> 1) & 3):
// conflict free), and one lane hands it to the TMA unit as a 32-row box: the unit clips rows beyond M and columns
// beyond N, writes whole row segments, and with add = true adds into the fp32 destination (one addend per element and
// launch, hence the same single rounding as a load-add-store).  OutStage counts the boxes of the warp so that a
// buffer is only rewritten after the unit has read it.
struct OutStage {
  uint8_t* buf;     // this warp's 4 KB (two buffers)
  uint32_t k;       // boxes issued so far
};
__device__ __forceinline__ void tma_store_box(const CUtensorMap* map, OutStage& os, const uint4 (&piece)[4], int col, int row,
                                              bool add, bool active, int lane) {
  if (os.k >= 2) {
    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");   // the box before the last one has been read
    __syncwarp();
  }
  uint4* dst = reinterpret_cast<uint4*>(os.buf + (os.k & 1) * 2048) + lane * 4;
  const int x = (lane >> 1) & 3;
#pragma unroll
  for (int c = 0; c < 4; ++c) dst[c ^ x] = piece[c];
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncwarp();
  if (lane == 0) {
    const uint32_t src = smem_u32(os.buf + (os.k & 1) * 2048);
    if (active) {
      if (add)
        asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map),
                     "r"(src), "r"(col), "r"(row)
                     : "memory");
      else
        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map), "r"(src),
                     "r"(col), "r"(row)
                     : "memory");
    }
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
  }
  ++os.k;
}
// 32 columns of the thread's row as bf16 (one box) or fp32 (two boxes of 16 columns)
__device__ __forceinline__ void tma_store_rows_bf16(const CUtensorMap* map, OutStage& os, const float (&v)[32], int col, int row,
                                                    bool active, int lane) {
  uint4 piece[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    piece[q].x = pack_bf16(v[8 * q], v[8 * q + 1]);
    piece[q].y = pack_bf16(v[8 * q + 2], v[8 * q + 3]);
    piece[q].z = pack_bf16(v[8 * q + 4], v[8 * q + 5]);
    piece[q].w = pack_bf16(v[8 * q + 6], v[8 * q + 7]);
  }
  tma_store_box(map, os, piece, col, row, false, active, lane);
}
__device__ __forceinline__ void tma_store_rows_f32(const CUtensorMap* map, OutStage& os, const float (&v)[32], int col, int row,
                                                   bool add, bool active, int lane) {
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    uint4 piece[4];
#pragma unroll
    for (int q = 0; q < 4; ++q)
      piece[q] = make_uint4(__float_as_uint(v[16 * h + 4 * q]), __float_as_uint(v[16 * h + 4 * q + 1]),
                            __float_as_uint(v[16 * h + 4 * q + 2]), __float_as_uint(v[16 * h + 4 * q + 3]));
    tma_store_box(map, os, piece, col + 16 * h, row, add, active, lane);
  }
}
// the unit has read every box of the warp (its staging may be rewritten) / has written them all
__device__ __forceinline__ void tma_store_drain_reads(int lane) {
  if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
  __syncwarp();
}
__device__ __forceinline__ void tma_store_drain_all(int lane) {
  if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  __syncwarp();
}

// Where the epilogue takes the thread's accumulator row from: TMEM, or the sum over the K splits' partial tiles.
struct TmemLoader {
  uint32_t tacc;   // TMEM address of (lane quadrant, column 0)
  __device__ __forceinline__ void operator()(int col, float (&v)[32]) const { tmem_ld32(tacc + col, v); }
};
struct SplitLoader {
  const float* ws;        // partial-tile workspace; slot s holds a [BM][bn] fp32 tile
  int bn, row;            // tile width, this thread's row in the tile
  int slot0;              // slot of part 0
  int slot_next;          // slot of part 1; part p >= 1 is in slot_next + slot_stride (p - 1)
  int slot_stride;
  int n_parts;
  bool valid;             // rows beyond M were never parked
  __device__ __forceinline__ void operator()(int col, float (&v)[32]) const {
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = 0.f;
    if (!valid) return;
    // partial tiles are stored [column / 4][row][4]: a warp's 32 rows of one float4 column are 512 contiguous
    // bytes.  Parts are added in part order (the result does not depend on who arrived last); the loads of two
    // parts are issued together so that their latencies overlap.
    const float4* base = reinterpret_cast<const float4*>(ws) + (size_t)(col / 4) * BM + row;
    for (int p = 0; p < n_parts; p += 2) {
      const int sa = p == 0 ? slot0 : slot_next + slot_stride * (p - 1);
      const bool two = p + 1 < n_parts;
      const int sb = slot_next + slot_stride * p;   // slot of part p + 1 (>= 1)
      float4 a[8], b[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        a[i] = __ldcg(base + ((size_t)sa * (bn / 4) + i) * BM);
        b[i] = two ? __ldcg(base + ((size_t)sb * (bn / 4) + i) * BM) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        v[4 * i] += a[i].x; v[4 * i + 1] += a[i].y; v[4 * i + 2] += a[i].z; v[4 * i + 3] += a[i].w;
        v[4 * i] += b[i].x; v[4 * i + 1] += b[i].y; v[4 * i + 2] += b[i].z; v[4 * i + 3] += b[i].w;
      }
    }
  }
};

// The reducing CTA's own part comes from its TMEM accumulator, the other parts from copies in shared memory (the
// idle operand ring, one [BN/4][rows] float4 tile after the other in part order without the own part; rows = BM, or
// 32 for the parts that the CTAs of a cluster hand to their leader).  Parts are added in part order starting from
// zero, exactly like SplitLoader, so both give the same bits.
struct RingLoader {
  uint32_t tacc;
  const float4* ring;     // + row
  int bn, own, n_parts, rows;
  // Every lane takes part, also those whose row lies beyond M (the TMEM load is a warp-wide instruction; their
  // sums are never stored).
  __device__ __forceinline__ void operator()(int col, float (&v)[32]) const {
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = 0.f;
    int k = 0;
    for (int p = 0; p < n_parts; ++p) {
      if (p == own) {
        float t[32];
        tmem_ld32(tacc + col, t);
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] += t[i];
      } else {
        const float4* src = ring + ((size_t)k * (bn / 4) + col / 4) * rows;
        ++k;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float4 a = src[(size_t)i * rows];
          v[4 * i] += a.x; v[4 * i + 1] += a.y; v[4 * i + 2] += a.z; v[4 * i + 3] += a.w;
        }
      }
    }
  }
};

// Work decomposition ("stream-K"), done per COLUMN of output tiles (the mt row tiles that share one weight tile):
// the k-blocks of the columns form one line of n_cols * KB units, column after column; a TEAM of mt CTAs (CTA
// team * mt + i works on row tile i) owns the contiguous range [team * per, (team + 1) * per) and walks it in
// step, so that the members read the same weight k-blocks at the same time and share them through L2, exactly
// like the CTAs of a wave of whole tiles.  A column may be cut by team boundaries; each owner computes its K range
// of its row tile ("part").  Part p >= 1 of a tile is always the FIRST piece of its CTA, part 0 the last piece (or
// the first, when the range starts exactly at the column): that decides the workspace slot,
// 2 * cta + (first piece ? 0 : 1).
// The stream-K division of a problem of mt x (n_tiles / mt) tiles with KB k-blocks each over n_units scheduling units:
// all but the last one-to-two waves stay whole tiles (dp_tiles of them, done after the cut ones), the k-blocks of the
// remaining tile columns are spread evenly over teams of mt units.  Computed on the host, or in the kernel when the row
// count (hence mt) is only known on the device.  Needs mt <= n_units.
__host__ __device__ inline void stream_k_schedule(int n_tiles, int mt, int KB, int n_units, int* dp_tiles, long long* per,
                                                  int* used_units) {
  const int n_teams = n_units / mt;
  const int full = n_tiles / n_units;
  *dp_tiles = full >= 2 ? ((full - 1) * n_units / mt) * mt : 0;
  const long long total = (long long)((n_tiles - *dp_tiles) / mt) * KB;
  const long long teams = total < n_teams ? total : n_teams;
  long long p = teams > 0 ? (total + teams - 1) / teams : 1;
  if (p < 4 && total >= 4) p = 4;                     // keep pieces long enough to amortise their hand-over
  if (p < 1) p = 1;
  *per = p;
  const int used = (int)((total + p - 1) / p);        // teams that get a range
  *used_units = *dp_tiles ? n_units : used * mt;      // (with whole tiles behind, the grid stays at full size)
}

struct Piece {
  int tile, kb0, kb1;     // k-block range [kb0, kb1) of the tile
  int part, n_parts;      // which part of the tile this is
  int slot;               // workspace slot if n_parts > 1
  int slot0, slot_next;   // slots of part 0 and part 1 (for the reducing CTA)
};
// Next piece of this CTA: first its range of the stream-K line (pos advances by reference), then its whole tiles
// (jd counts them).  The cut tiles come first so that parking and reducing their partials overlaps the main loop
// of the whole tiles that follow, instead of happening in every CTA at once at the end of the kernel.
__device__ __forceinline__ Piece make_piece(int& jd, int dp_tiles, long long& pos, long long hi, int KB,
                                            long long per, int cta, int grid, int mt) {
  Piece p;
  if (pos >= hi) {
    p.tile = cta + jd * grid;
    ++jd;
    p.kb0 = 0;
    p.kb1 = KB;
    p.part = 0;
    p.n_parts = 1;
    p.slot = p.slot0 = p.slot_next = 0;
    return p;
  }
  const int team = cta / mt, member = cta % mt;
  const int col = (int)(pos / KB);
  p.kb0 = (int)(pos - (long long)col * KB);
  const long long room = hi - pos;
  p.kb1 = (int)(room < KB - p.kb0 ? p.kb0 + room : KB);
  const long long t0 = (long long)col * KB, t1 = t0 + KB;
  const int c_first = (int)(t0 / per), c_last = (int)((t1 - 1) / per);    // first and last team on this column
  p.n_parts = c_last - c_first + 1;
  p.part = team - c_first;
  const bool first_piece = pos == (long long)team * per;
  p.slot = 2 * cta + (first_piece ? 0 : 1);
  p.slot0 = 2 * (c_first * mt + member) + (((long long)c_first * per >= t0) ? 0 : 1);
  p.slot_next = 2 * ((c_first + 1) * mt + member);
  p.tile = dp_tiles + col * mt + member;
  pos += p.kb1 - p.kb0;
  return p;
}

// EPI_RESIDUAL_NORM: besides the accumulator a thread needs its row of the OLD residual stream and the gains of the
// next norm.  Both come through shared memory: the TMA unit fetches the old rows of a 32-column chunk as two boxes (the
// boxes of the output map: 32 rows x 16 columns, 64-byte swizzle) two chunks ahead of their use, completing on one
// mbarrier per slot, and the tile's gains are staged once per tile.  (Plain global loads in flight would be waited for
// by the proxy fence of every output box.)
struct NormStage {
  uint8_t* h;        // this warp's two 4 KB slots
  uint4* g;          // this warp's 32 x 16 bytes of gains
  uint64_t* bar;     // this warp's two barriers
  uint32_t count;    // chunks fetched so far by this warp (slot = count & 1, phase = (count >> 1) & 1)
};
__device__ __forceinline__ void norm_issue(NormStage& ns, const CUtensorMap* omap, uint32_t idx, int n, int m_base, int lane) {
  if (lane == 0) {
    uint64_t* bar = &ns.bar[idx & 1];
    uint8_t* dst = ns.h + (idx & 1) * 4096;
    mbar_arrive_expect_tx(bar, 4096);
    tma_load_2d(dst, omap, n, m_base, bar);
    tma_load_2d(dst + 2048, omap, n + 16, m_base, bar);
  }
}
// gains of the tile's columns and the first two chunks of old rows; returns the chunks the tile has
__device__ __forceinline__ int norm_prepare(const EpiParams& ep, NormStage& ns, const CUtensorMap* omap, int n0, int bn, int m_base,
                                            int lane) {
  const int left = ep.N - n0;
  const int nch = left <= 0 ? 0 : ((left < bn ? left : bn) + 31) / 32;
  if (lane * 8 < bn && n0 + lane * 8 < ep.N) ns.g[lane] = __ldg(reinterpret_cast<const uint4*>(ep.gain + n0) + lane);
  __syncwarp();
  for (int c = 0; c < 2 && c < nch; ++c) norm_issue(ns, omap, ns.count + c, n0 + c * 32, m_base, lane);
  return nch;
}

// Epilogue of one accumulator tile for the calling thread's row.
// stg: this warp's 4 KB of output staging (two boxes).  All 32 lanes of the warp call together.
// rstd: factor of this thread's row when the input of the projection was a residual stream that is normalised on the
// fly (1 otherwise); xmap: the tensor map over x_out of EPI_RESIDUAL_NORM; tile_col: index of the tile's column.
template <int BN, bool NORM, typename Loader>
__device__ __forceinline__ void row_epilogue(const EpiParams& ep, const Loader& load, int m, int n0, float* stg,
                                             const CUtensorMap* omap, const CUtensorMap* xmap, float rstd, int tile_col,
                                             NormStage& ns, bool prepared) {
  const bool row_ok = m < ep.M;
  const int lane = threadIdx.x & 31;
  const int m_base = m - lane;                                  // first row of this warp
  const int valid_rows = ep.M - m_base < 0 ? 0 : (ep.M - m_base > 32 ? 32 : ep.M - m_base);
  OutStage os{reinterpret_cast<uint8_t*>(stg), 0u};
  const bool active = valid_rows > 0;      // a box that starts beyond the last row is not issued at all
  if constexpr (NORM) {
    // The residual stream itself is updated by the TMA unit's add-reduction (one addend per element and launch: the
    // rounding of a load-add-store).  The new value is formed here as well, from the old rows staged in shared memory,
    // for the next norm's input x = bf16(h * gain) and the row's sum of squares over this tile's columns.
    const int nch = prepared ? (ep.N - n0 <= 0 ? 0 : ((ep.N - n0 < BN ? ep.N - n0 : BN) + 31) / 32)
                             : norm_prepare(ep, ns, omap, n0, BN, m_base, lane);
    const int sw = (lane >> 1) & 3;
    float ss = 0.f;
#pragma unroll 1
    for (int c = 0; c < nch; ++c) {
      const uint32_t idx = ns.count + c;
      if (!mbar_wait(&ns.bar[idx & 1], (idx >> 1) & 1, kSpin)) set_status(ep.status, DEV_TIMEOUT_FULL);
      float hv[32];
      const uint8_t* slot = ns.h + (idx & 1) * 4096 + lane * 64;
#pragma unroll
      for (int b = 0; b < 2; ++b)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float4 t = *reinterpret_cast<const float4*>(slot + b * 2048 + ((q ^ sw) << 4));
          hv[16 * b + 4 * q] = t.x; hv[16 * b + 4 * q + 1] = t.y; hv[16 * b + 4 * q + 2] = t.z; hv[16 * b + 4 * q + 3] = t.w;
        }
      __syncwarp();                 // every lane has read the slot: it may be refilled
      if (c + 2 < nch) norm_issue(ns, omap, idx + 2, n0 + (c + 2) * 32, m_base, lane);
      float v[32];
      load(c * 32, v);
      const int n = n0 + c * 32;
      tma_store_rows_f32(omap, os, v, n, m_base, true, active, lane);
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        v[i] += hv[i];
        ss = fmaf(v[i], v[i], ss);
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint4 gq = ns.g[c * 4 + q];
        const uint32_t w[4] = {gq.x, gq.y, gq.z, gq.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          v[8 * q + 2 * j] *= __uint_as_float(w[j] << 16);
          v[8 * q + 2 * j + 1] *= __uint_as_float(w[j] & 0xffff0000u);
        }
      }
      tma_store_rows_bf16(xmap, os, v, n, m_base, active, lane);
    }
    ns.count += nch;
    if (row_ok) ep.ss_out[(size_t)tile_col * ep.ss_stride + m] = ss;
    tma_store_drain_reads(lane);
    return;
  }
  if (ep.epi == EPI_SWIGLU) {
    // accumulator columns [0, BN/2) are gate, [BN/2, BN) up; n0 is the first output column
#pragma unroll 1
    for (int c = 0; c < BN / 64; ++c) {
      float g[32], u[32];
      load(c * 32, g);
      load(BN / 2 + c * 32, u);
      if (n0 + c * 32 < ep.N) {
#pragma unroll
        for (int i = 0; i < 32; ++i) g[i] = silu_f(g[i] * rstd) * (u[i] * rstd);
        tma_store_rows_bf16(omap, os, g, n0 + c * 32, m_base, active, lane);
      }
    }
    tma_store_drain_reads(lane);
    return;
  }
  if (ep.epi == EPI_QKV_ROPE) {
    const int D = ep.head_dim, half = D / 2;
    const int slot = row_ok ? ep.tok_slot[m] : -1;
#pragma unroll 1
    for (int hl = 0; hl < BN / D; ++hl) {        // heads in this tile
      const int head = n0 / D + hl;
      const bool is_q = head < ep.n_q, is_v = head >= ep.n_q + ep.n_kv;
      __nv_bfloat16* kv_base = nullptr;
      if (!is_q && slot >= 0) {
        const int64_t page = slot / kPageSize;
        if (page < ep.n_pages) {
          const int kvh = is_v ? head - ep.n_q - ep.n_kv : head - ep.n_q;
          kv_base = ep.kv_pool + kv_tile_base(ep.n_pages, ep.n_kv, D, ep.layer, page, kvh) + (is_v ? kv_tile_elems(D) : 0);
        } else {
          set_status(ep.status, DEV_BAD_INDEX);
        }
      }
      const int tok = slot >= 0 ? slot % kPageSize : 0;
#pragma unroll 1
      for (int c = 0; c < half / 32; ++c) {      // 32 low columns with their 32 partners half a head away
        float lo[32], hi[32];
        load(hl * D + c * 32, lo);
        load(hl * D + half + c * 32, hi);
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          lo[i] *= rstd;
          hi[i] *= rstd;
        }
        if (row_ok && !is_v) {
          const float2* cs = ep.rope_cs + (size_t)(c * 32) * ep.M + m;   // [frequency][token]
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float2 t = cs[(size_t)i * ep.M];
            const float a = lo[i] * t.x - hi[i] * t.y, b = hi[i] * t.x + lo[i] * t.y;
            lo[i] = a;
            hi[i] = b;
          }
        }
        if (is_q) {      // (the same for the whole warp): rows of the rotated queries [M, n_q * D] through the TMA unit
          tma_store_rows_bf16(omap, os, lo, head * D + c * 32, m_base, active, lane);
          tma_store_rows_bf16(omap, os, hi, head * D + half + c * 32, m_base, active, lane);
        } else if (kv_base) {
          // the pool tile is swizzled in 16-byte chunks: store chunk by chunk
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint4 a, b;
            a.x = pack_bf16(lo[8 * j], lo[8 * j + 1]); a.y = pack_bf16(lo[8 * j + 2], lo[8 * j + 3]);
            a.z = pack_bf16(lo[8 * j + 4], lo[8 * j + 5]); a.w = pack_bf16(lo[8 * j + 6], lo[8 * j + 7]);
            b.x = pack_bf16(hi[8 * j], hi[8 * j + 1]); b.y = pack_bf16(hi[8 * j + 2], hi[8 * j + 3]);
            b.z = pack_bf16(hi[8 * j + 4], hi[8 * j + 5]); b.w = pack_bf16(hi[8 * j + 6], hi[8 * j + 7]);
            *reinterpret_cast<uint4*>(kv_base + kv_tile_offset(tok, c * 32 + j * 8, D)) = a;
            *reinterpret_cast<uint4*>(kv_base + kv_tile_offset(tok, half + c * 32 + j * 8, D)) = b;
          }
        }
      }
    }
    tma_store_drain_reads(lane);
    return;
  }
#pragma unroll 1
  for (int c = 0; c < BN / 32; ++c) {
    float v[32];
    load(c * 32, v);
    const int n = n0 + c * 32;
    if (n >= ep.N) continue;
    if (ep.ss_in) {
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] *= rstd;
    }
    // the box is clipped at the right edge (N is a multiple of 16 but not always of 32) and at the last row
    if (ep.epi == EPI_PLAIN_BF16) tma_store_rows_bf16(omap, os, v, n, m_base, active, lane);
    else tma_store_rows_f32(omap, os, v, n, m_base, ep.epi == EPI_RESIDUAL, active, lane);
  }
  tma_store_drain_reads(lane);
}

template <int BN, bool PAIR, bool NORM>
__global__ void __launch_bounds__(kTcThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
               const __grid_constant__ CUtensorMap map_out, const __grid_constant__ CUtensorMap map_xout, int M_cap, int n_tiles_n,
               int K, int up_row_offset, int dp_tiles_in, long long per_in, int thin, int cl_parts, float* split_ws,
               int* split_counters, const int* __restrict__ m_dev, int m_dev_wait, EpiParams ep_in) {
  // Device-resident rounds: the row count comes from device memory; the tensor maps cover the capacity M_cap, and rows
  // between the count and the capacity hold stale data and are computed but never used.  The count is written by the
  // first kernel of the step, and the small kernels between it and the first projection signal their dependents before
  // they wait themselves, so the FIRST projection of a step can be running before that one has finished: it has to wait
  // for its predecessors before it reads the count (m_dev_wait; it gives up the early weight requests).  The first
  // projection signals its own dependents only after that wait, so for every kernel behind it the count is settled.
  if (m_dev && m_dev_wait) griddep_wait();
  const int M = m_dev ? *reinterpret_cast<const volatile int*>(m_dev) : M_cap;
  if (M <= 0) {                // an empty round (the same for every thread of the grid): nothing to do, nothing was set up yet
    griddep_wait();            // (this grid must not count as complete before the ones it follows are)
    return;
  }
  EpiParams ep = ep_in;
  ep.M = M;
  using Cfg = TcCfg<BN, PAIR, NORM>;
  constexpr int kRows = PAIR ? 2 * BM : BM;              // rows of a scheduling unit's tile
  constexpr int kSlotMul = PAIR ? 2 : 1;                 // the CTAs of a pair use separate slots and counters
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  const int unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;      // scheduling unit: CTA or cluster
  const int n_units = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  // Problems of one row tile (at most 128 rows) whose tiles are cut over K can run as CLUSTERS of cl CTAs per tile
  // (cl_parts > 1; single CTAs only): rank r computes k-blocks [r KB / cl, (r + 1) KB / cl) and hands its partial tile
  // (the rows in use, rounded up to 32) to the cluster's leader (rank 0) through distributed shared memory, into a
  // reserve at the top of the leader's ring budget; the leader adds the parts in rank order and runs the epilogue.  No
  // trip through global memory, no counter.
  const int cl = (!PAIR && cl_parts > 1) ? cl_parts : 0;
  const uint32_t crank = cl ? cluster_ctarank() : 0u;
  const int cl_rows = ((M < BM ? M : BM) + 31) & ~31;            // rows of a handed-over part
  const int cl_part_bytes = cl_rows * BN * 4;
  const int cl_reserve = cl ? (cl - 1) * cl_part_bytes : 0;
  const int a_bytes = thin ? Cfg::kThinABytes : Cfg::kABytes;
  const int stage_bytes = a_bytes + Cfg::kBBytes;
  const int cl_stages = (Cfg::kBudget - cl_reserve) / stage_bytes;
  const int n_stages = cl ? (cl_stages > Cfg::kMaxStages ? Cfg::kMaxStages : cl_stages) : (thin ? Cfg::kThinStages : Cfg::kStages);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + Cfg::kBarOff);
  uint64_t* empty_bar = full_bar + Cfg::kMaxStages;
  uint64_t* tfull_bar = empty_bar + Cfg::kMaxStages;
  uint64_t* tempty_bar = tfull_bar + 2;
  uint64_t* red_bar = tempty_bar + 2;      // completion of the partial tiles fetched into the idle ring (used once)
  uint64_t* h_bar = red_bar + 1;           // [4 epilogue warps][2 slots]: old residual rows have landed (NORM only)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(h_bar + 8);

  // Bounded waits.  The producer and the MMA issuer leave their loops when a wait runs out.  The four epilogue warps
  // must all keep meeting at the named barriers and must keep counting the arrivals of cut tiles (so that the counters
  // stay consistent for the next launch), so they never leave their loop: a wait of theirs that runs out records why
  // and raises a CTA-wide flag, after which their waits return at once; the outputs of such a launch are garbage and
  // the status word says so.  (The flag is only looked at between waits: polling it inside the producer's and the
  // issuer's per-k-block waits cost up to 40 % on narrow tiles.)
  __shared__ volatile int s_abort;
  auto wait_bar = [&](uint64_t* bar, uint32_t parity) -> bool {
    for (uint32_t i = 0; i < kSpin; ++i) {
      uint32_t ok;
      if constexpr (PAIR)
        asm volatile(
            "{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
            : "=r"(ok)
            : "r"(smem_u32(bar)), "r"(parity)
            : "memory");
      else
        ok = mbar_try_wait(bar, parity) ? 1u : 0u;
      if (ok) return true;
      if (i > 64) __nanosleep(32);
    }
    return false;
  };
  auto wait_or_abort = [&](uint64_t* bar, uint32_t parity, int code) {   // epilogue warps only
    if (s_abort) return;
    if (!wait_bar(bar, parity)) {
      set_status(ep.status, code);
      s_abort = 1;
    }
  };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_tiles_m = (M + kRows - 1) / kRows;
  const int n_tiles = n_tiles_m * n_tiles_n;
  const int KB = K / BK;
  // dp_tiles_in >= 0: the host's schedule; -1: whole tiles only; -2: stream-K, divided here from the device's row count
  int dp_tiles = dp_tiles_in < 0 ? n_tiles : dp_tiles_in;
  long long per = per_in;
  if (dp_tiles_in == -2) {
    if (n_tiles_m >= 1 && n_tiles_m <= n_units) {
      int used;
      stream_k_schedule(n_tiles, n_tiles_m, KB, n_units, &dp_tiles, &per, &used);
    } else {
      dp_tiles = n_tiles;
    }
  }
  const bool swiglu = ep.epi == EPI_SWIGLU;
  // schedule: the k-blocks of tiles [dp_tiles, n_tiles) as one line cut into equal ranges per CTA; then tiles
  // [0, dp_tiles) whole, strided over the grid (CTAs that run together share a weight tile through L2)
  const long long total = (long long)((n_tiles - dp_tiles) / n_tiles_m) * KB;
  const long long lo_raw = (long long)(unit / n_tiles_m) * per;
  const long long range_lo = cl ? 0 : (lo_raw < total ? lo_raw : total);
  const long long range_hi = cl ? 1 : (range_lo + per < total ? range_lo + per : total);
  const int dp_count = cl ? 0 : (unit < dp_tiles ? (dp_tiles - 1 - unit) / n_units + 1 : 0);
  // the next piece of this CTA (a cluster member has exactly one)
  auto next_piece = [&](int& jd, long long& pos) -> Piece {
    if (cl) {
      Piece p;
      p.tile = (int)blockIdx.x / cl;
      p.kb0 = (int)((long long)crank * KB / cl);
      p.kb1 = (int)((long long)(crank + 1) * KB / cl);
      p.part = (int)crank;
      p.n_parts = cl;
      p.slot = p.slot0 = p.slot_next = 0;
      pos = range_hi;
      return p;
    }
    return make_piece(jd, dp_tiles, pos, range_hi, KB, per, unit, n_units, n_tiles_m);
  };

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&tfull_bar[a], 1);
      mbar_init(&tempty_bar[a], PAIR ? 8 : 4);
    }
    mbar_init(red_bar, cl ? (cl - 1) * (cl_rows / 32) : 1);      // (cluster leader: one arrival per peer and 32 rows)
    for (int i = 0; i < 8; ++i) mbar_init(&h_bar[i], 1);
    fence_barrier_init();
    prefetch_tmap(&map_x);
    prefetch_tmap(&map_w);
  }
  if (warp == 1) {
    if constexpr (PAIR) {
      tmem_alloc_pair(tmem_slot, Cfg::kTmemCols);
      tmem_relinquish_pair();
    } else {
      tmem_alloc(tmem_slot, Cfg::kTmemCols);
      tmem_relinquish();
    }
  }
  tc_fence_before();
  __syncthreads();
  if constexpr (PAIR) cluster_sync_all();   // both CTAs' barriers are initialised before anyone signals across
  else if (cl) cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // (each role waits for the kernels before this one where it first needs their results)

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (elect_one()) {
      // of a pair, rank r loads rows [128 r, 128 r + 128) of the x tile and half r of the weight tile (SwiGLU: rank 0
      // the gate rows, rank 1 the up rows); all four loads of the pair complete on the leader's barrier
      auto expect = [&](int s) {
        if constexpr (PAIR) {
          if (rank == 0) mbar_arrive_expect_tx(&full_bar[s], 2 * stage_bytes);
        } else {
          mbar_arrive_expect_tx(&full_bar[s], stage_bytes);
        }
      };
      auto load_w = [&](int s, int kb, int tn) {
        uint8_t* b_dst = smem + s * stage_bytes + a_bytes;
        if constexpr (PAIR) {
          const uint32_t full0 = mapa_rank(smem_u32(&full_bar[s]), 0);
          const int w_row = swiglu ? (rank == 0 ? tn * (BN / 2) : up_row_offset + tn * (BN / 2)) : tn * BN + (int)rank * (BN / 2);
          tma_load_2d_pair(smem_u32(b_dst), &map_w, kb * BK, w_row, full0);
        } else if (swiglu) {
          tma_load_2d(b_dst, &map_w, kb * BK, tn * (BN / 2), &full_bar[s]);
          tma_load_2d(b_dst + Cfg::kBBytes / 2, &map_w, kb * BK, up_row_offset + tn * (BN / 2), &full_bar[s]);
        } else {
          tma_load_2d(b_dst, &map_w, kb * BK, tn * BN, &full_bar[s]);
        }
      };
      auto load_x = [&](int s, int kb, int tm) {
        uint8_t* a_dst = smem + s * stage_bytes;
        if constexpr (PAIR) tma_load_2d_pair(smem_u32(a_dst), &map_x, kb * BK, tm * kRows + (int)rank * BM, mapa_rank(smem_u32(&full_bar[s]), 0));
        else tma_load_2d(a_dst, &map_x, kb * BK, tm * BM, &full_bar[s]);
      };
      // The weights do not depend on the kernels before this one: the weight tiles of the first stages are requested
      // BEFORE waiting for those kernels, so the ring fills while they drain (or while a short kernel such as the
      // RMSNorm in front of this projection runs); the x tiles of those stages follow right after the wait.
      int n_pre = 0, pre_kb0 = 0, pre_tm = 0;
      if (dp_count > 0 || range_lo < range_hi) {
        long long p0 = range_lo;
        int j0 = 0;
        const Piece pc = next_piece(j0, p0);
        n_pre = pc.kb1 - pc.kb0 < n_stages ? pc.kb1 - pc.kb0 : n_stages;
        pre_kb0 = pc.kb0;
        pre_tm = pc.tile % n_tiles_m;
        for (int i = 0; i < n_pre; ++i) {
          expect(i);
          load_w(i, pre_kb0 + i, pc.tile / n_tiles_m);
        }
      }
      griddep_wait();
      for (int i = 0; i < n_pre; ++i) load_x(i, pre_kb0 + i, pre_tm);
      int st_idx = 0, issued = 0;
      uint32_t st_phase = 0;
      bool ok = true;
      long long pos = range_lo;
      for (int jd = 0; (jd < dp_count || pos < range_hi) && ok;) {
        const Piece pc = next_piece(jd, pos);
        const int tm = pc.tile % n_tiles_m, tn = pc.tile / n_tiles_m;
        const int kb0 = pc.kb0, kb1 = pc.kb1;
        for (int kb = kb0; kb < kb1; ++kb) {
          const int s = st_idx;
          const uint32_t ph = st_phase;
          if (++st_idx == n_stages) { st_idx = 0; st_phase ^= 1; }
          if (issued < n_pre) {       // requested above
            ++issued;
            continue;
          }
          if (!wait_bar(&empty_bar[s], ph ^ 1)) {
            set_status(ep.status, DEV_TIMEOUT_EMPTY);
            ok = false;
            break;
          }
          expect(s);
          load_x(s, kb, tm);
          load_w(s, kb, tn);
        }
      }
      if (!ok) {  // let loads already issued land before the CTA may exit
        for (int s = 0; s < n_stages; ++s)
          for (uint32_t i = 0; i < (1u << 14); ++i) {
            if (mbar_try_wait(&full_bar[s], 0) || mbar_try_wait(&full_bar[s], 1)) break;
            __nanosleep(64);
          }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (rank == 0 && elect_one()) {         // of a pair only the leader issues (it touches shared memory and TMEM only)
      constexpr uint32_t idesc = make_idesc(BN, kRows);
      const uint64_t desc0 = make_smem_desc(smem_u32(smem));
      int st_idx = 0;
      uint32_t st_phase = 0, tcount = 0;
      bool ok = true;
      long long pos = range_lo;
      for (int jd = 0; (jd < dp_count || pos < range_hi) && ok; ++tcount) {
        const Piece pc = next_piece(jd, pos);
        const int kb0 = pc.kb0, kb1 = pc.kb1;
        const int acc = tcount & 1;
        if (!wait_bar(&tempty_bar[acc], ((tcount >> 1) & 1) ^ 1)) {
          set_status(ep.status, DEV_TIMEOUT_MMA);
          break;
        }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = kb0; kb < kb1; ++kb) {
          const int s = st_idx;
          const uint32_t ph = st_phase;
          if (++st_idx == n_stages) { st_idx = 0; st_phase ^= 1; }
          if (!wait_bar(&full_bar[s], ph)) {
            set_status(ep.status, DEV_TIMEOUT_FULL);
            ok = false;
            break;
          }
          tc_fence_after();
          // descriptors are linear in the address (the ring lies inside the 14-bit address field without carry), so
          // the descriptor of a 16-column slice is the stage's descriptor plus 32 bytes >> 4
          const uint64_t da0 = desc0 + (uint64_t)((s * stage_bytes) >> 4);
          const uint64_t db0 = da0 + (uint64_t)(a_bytes >> 4);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            if constexpr (PAIR) umma_bf16_pair(d_tmem, da0 + 2 * k, db0 + 2 * k, idesc, ((kb - kb0) | k) ? 1u : 0u);
            else umma_bf16(d_tmem, da0 + 2 * k, db0 + 2 * k, idesc, ((kb - kb0) | k) ? 1u : 0u);
          }
          // frees the stage (in both CTAs of a pair) when these MMAs have read it
          if constexpr (PAIR) umma_commit_pair(&empty_bar[s]);
          else umma_commit(&empty_bar[s]);
        }
        if (ok) {                            // accumulator complete
          if constexpr (PAIR) umma_commit_pair(&tfull_bar[acc]);
          else umma_commit(&tfull_bar[acc]);
        }
      }
    }
  } else {
    // ------------------------------ epilogue warps ------------------------------
    const int quad = warp & 3;             // TMEM lane quadrant this warp may read
    float* stg = reinterpret_cast<float*>(smem + Cfg::kRingBytes) + (warp - 2) * 1024;
    uint32_t tcount = 0;
    __shared__ int s_last;
    NormStage ns{smem + Cfg::kNormOff + (warp - 2) * 8192, reinterpret_cast<uint4*>(smem + Cfg::kNormOff + kNormHBytes) + (warp - 2) * 32,
                 h_bar + (warp - 2) * 2, 0u};
    griddep_wait();                        // the epilogue reads and writes what earlier kernels produced
    long long pos = range_lo;
    for (int jd = 0; jd < dp_count || pos < range_hi; ++tcount) {
      const Piece pc = next_piece(jd, pos);
      const int tile = pc.tile, n_splits = pc.n_parts;
      const int tm = tile % n_tiles_m, tn = tile / n_tiles_m;
      const int acc = tcount & 1;
      const int row_in_tile = quad * 32 + lane;
      const int m = tm * kRows + (int)rank * BM + row_in_tile;
      // the row's normalisation factor, fetched while the accumulator is still being computed: the partial sums of
      // squares in slot order (the same bits in every tile of the row)
      float rstd = 1.f;
      if (ep.ss_in) {
        float sq = 0.f;
        if (m < ep.M)
          for (int k = 0; k < ep.ss_slots; ++k) sq += __ldcg(ep.ss_in + (size_t)k * ep.ss_stride + m);
        rstd = rsqrtf(sq * ep.norm_inv_n + ep.norm_eps);
      }
      // (likewise, for a whole tile, the gains and the first old residual rows)
      const bool prepared = NORM && n_splits == 1;
      if constexpr (NORM) {
        if (prepared) norm_prepare(ep, ns, &map_out, tn * BN, BN, m - lane, lane);
      }
      wait_or_abort(&tfull_bar[acc], (tcount >> 1) & 1, DEV_TIMEOUT_MMA);   // after a timeout: carry on without blocking
      tc_fence_after();
      const uint32_t tacc = tmem_base + ((uint32_t)(quad * 32) << 16) + acc * BN;
      // hands the accumulator back to the MMA issuer (of a pair: the leader's barrier collects both CTAs' warps)
      auto release_acc = [&]() {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if constexpr (PAIR) mbar_arrive_cluster(mapa_rank(smem_u32(&tempty_bar[acc]), 0));
          else mbar_arrive(&tempty_bar[acc]);
        }
      };
      const int n0 = swiglu ? tn * (BN / 2) : tn * BN;
      if (n_splits == 1) {
        row_epilogue<BN, NORM>(ep, TmemLoader{tacc}, m, n0, stg, &map_out, &map_xout, rstd, tn, ns, prepared);
        release_acc();
      } else if (cl) {
        uint8_t* reserve = smem + Cfg::kBudget - cl_reserve;       // the leader's: cl - 1 parts of [BN/4][cl_rows] float4
        if (crank != 0) {
          if (quad * 32 < cl_rows) {           // the warps that hold rows in use
            const uint32_t dst = mapa_rank(smem_u32(reserve + (crank - 1) * cl_part_bytes), 0) + row_in_tile * 16;
            const uint32_t col_stride = (uint32_t)cl_rows * 16u;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
              float v[32];
              tmem_ld32(tacc + c * 32, v);
#pragma unroll
              for (int i = 0; i < 8; ++i)
                st_cluster_f4(dst + (uint32_t)(c * 8 + i) * col_stride, make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]));
            }
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_rank(smem_u32(red_bar), 0));   // release: the warp's stores are visible
          }
          release_acc();
        } else {
          if (!s_abort) {            // the peers' parts have landed (acquire at cluster scope)
            bool ok = false;
            for (uint32_t i = 0; i < kSpin && !ok; ++i) {
              uint32_t got;
              asm volatile(
                  "{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                  : "=r"(got)
                  : "r"(smem_u32(red_bar)), "r"(0u)
                  : "memory");
              ok = got != 0;
              if (!ok && i > 64) __nanosleep(32);
            }
            if (!ok) {
              set_status(ep.status, DEV_TIMEOUT_FULL);
              s_abort = 1;
            }
          }
          RingLoader ld{tacc, reinterpret_cast<const float4*>(reserve) + row_in_tile, BN, 0, n_splits, cl_rows};
          row_epilogue<BN, NORM>(ep, ld, m, n0, stg, &map_out, &map_xout, rstd, tn, ns, false);
          release_acc();
        }
      } else {
        // park this split's partial tile and let the LAST split to arrive reduce all partials in split order
        // (deterministic) and run the fused epilogue
        // (the two CTAs of a pair park and reduce their 128-row halves independently: slot and counter index are
        // doubled and offset by the rank)
        const int slot_mine = pc.slot * kSlotMul + (int)rank, slot0 = pc.slot0 * kSlotMul + (int)rank;
        const int slot_next = pc.slot_next * kSlotMul + (int)rank, slot_stride = 2 * n_tiles_m * kSlotMul;
        const int counter = tile * kSlotMul + (int)rank;
        float4* mine = reinterpret_cast<float4*>(split_ws) + (size_t)slot_mine * (BN / 4) * BM + row_in_tile;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          float v[32];
          tmem_ld32(tacc + c * 32, v);
          if (m < ep.M) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
              __stcg(mine + (size_t)(c * 8 + i) * BM, make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]));
          }
        }
        // the accumulator may be handed back at once: the own part is read from TMEM again only when nothing follows
        // in this CTA, and then nobody overwrites it
        release_acc();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (warp == 2 && lane == 0) {
          __threadfence();   // cumulative: orders the partial rows all 128 threads wrote before the barrier
          const int old = atomicAdd(&split_counters[counter], 1);
          s_last = (old == n_splits - 1);
          if (old == n_splits - 1) split_counters[counter] = 0;   // ready for the next launch
          __threadfence();
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (s_last) {
          // When nothing follows in this CTA the operand ring is idle (every load was consumed before the accumulator
          // completed): the other parts are fetched into it with bulk copies at full bandwidth and the own part is
          // taken from TMEM.  Otherwise the parts are read from global memory while the next piece's main loop runs.
          constexpr int kPartBytes = BM * BN * 4;
          const bool final_piece = !(jd < dp_count || pos < range_hi);
          if (final_piece && (n_splits - 1) * kPartBytes <= Cfg::kBudget) {
            if (warp == 2 && lane == 0) {
              asm volatile("fence.proxy.async;" ::: "memory");   // the parts were written with ordinary stores
              mbar_arrive_expect_tx(red_bar, (uint32_t)((n_splits - 1) * kPartBytes));
              int k = 0;
              for (int p = 0; p < n_splits; ++p) {
                if (p == pc.part) continue;
                const int slot = p == 0 ? slot0 : slot_next + slot_stride * (p - 1);
                const uint8_t* src = reinterpret_cast<const uint8_t*>(split_ws) + (size_t)slot * kPartBytes;
                constexpr int kChunk = kPartBytes < 32768 ? kPartBytes : 32768;
                for (int off = 0; off < kPartBytes; off += kChunk)
                  bulk_g2s(smem + (size_t)k * kPartBytes + off, src + off, kChunk, red_bar);
                ++k;
              }
            }
            wait_or_abort(red_bar, 0, DEV_TIMEOUT_FULL);
            RingLoader ld{tacc, reinterpret_cast<const float4*>(smem) + row_in_tile, BN, pc.part, n_splits, BM};
            row_epilogue<BN, NORM>(ep, ld, m, n0, stg, &map_out, &map_xout, rstd, tn, ns, false);
          } else {
            SplitLoader ld{split_ws, BN, row_in_tile, slot0, slot_next, slot_stride, n_splits, m < ep.M};
            row_epilogue<BN, NORM>(ep, ld, m, n0, stg, &map_out, &map_xout, rstd, tn, ns, false);
          }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");       // s_last is reused by the next unit
      }
    }
  }

  if (warp >= 2) tma_store_drain_all(threadIdx.x & 31);   // the output boxes handed to the TMA unit have been written
  griddep_launch();   // this CTA's work is done: the next kernel's CTAs may be scheduled onto freed SMs
  tc_fence_before();
  __syncthreads();
  if constexpr (PAIR) cluster_sync_all();   // the peer may read this CTA's operands and signal its barriers until here
  // (a cluster of a thin problem needs no meeting here: only the leader's shared memory is written by others, and the
  // leader has waited for those stores; the peers are free to leave)
  if (warp == 1) {
    tc_fence_after();
    if constexpr (PAIR) tmem_dealloc_pair(tmem_base, Cfg::kTmemCols);
    else tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
}


// ---- host side -------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct MapKey {
  const void* ptr;
  uint64_t rows, cols;
  uint32_t box_rows;
  bool operator==(const MapKey& o) const { return ptr == o.ptr && rows == o.rows && cols == o.cols && box_rows == o.box_rows; }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    return std::hash<const void*>()(k.ptr) ^ (k.rows * 1000003u) ^ (k.cols * 7919u) ^ (size_t)k.box_rows << 40;
  }
};

constexpr size_t kSplitWsBytes = 96ull << 20;   // partial tiles of split-K launches
constexpr int kSplitCounters = 1 << 16;
constexpr size_t kMapCacheMax = 4096;           // entries; the keys include the row count, so a serving loop keeps adding

// Cache of encoded tensor maps (cached_map below).  Maps are handed out BY VALUE: a launch needs three maps at once,
// and a miss on the second or third lookup may empty the full cache, so nothing may point into it.
struct TcState {
  int n_sm = 0;
  int force_bn = 0, force_s = 0;
  float* split_ws = nullptr;
  int* split_counters = nullptr;
  EncodeTiledFn encode = nullptr;
  std::unordered_map<MapKey, CUtensorMap, MapKeyHash> maps;
  size_t evictions = 0;
  int last_tiles_n = 0;       // column tiles of the last launch
  bool configured[10] = {false, false, false, false, false, false, false, false, false, false};
  bool thin_clusters = true;  // problems of one row tile with cut tiles run as clusters that reduce through distributed shared memory
  int max_clusters[10][5];    // cached occupancy answers per kernel and cluster size (-1: not asked yet)
  TcState() {
    for (auto& row : max_clusters)
      for (int& v : row) v = -1;
  }
};

template <typename Encode>
bool cached_map(TcState* st, const MapKey& key, CUtensorMap* out, Encode&& encode) {
  auto it = st->maps.find(key);
  if (it != st->maps.end()) {
    *out = it->second;
    return true;
  }
  CUtensorMap m;
  if (!encode(&m)) return false;
  if (st->maps.size() >= kMapCacheMax) {   // emptied, never trimmed behind a caller's back: maps leave by value
    st->maps.clear();
    ++st->evictions;
  }
  st->maps.emplace(key, m);
  *out = m;
  return true;
}

// [rows, cols] bf16 row-major, box = [box_rows, 64 columns], 128-byte swizzle, zero fill out of bounds
bool get_map(TcState* st, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows, CUtensorMap* out) {
  return cached_map(st, MapKey{ptr, rows, cols, box_rows}, out, [&](CUtensorMap* m) {
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {BK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return st->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  });
}

// Output [rows, cols] of 2- or 4-byte elements, row-major: box = 32 rows x 64 bytes, 64-byte swizzle
bool get_out_map(TcState* st, const void* ptr, uint64_t rows, uint64_t cols, int elem_bytes, CUtensorMap* out) {
  return cached_map(st, MapKey{ptr, rows, cols, (uint32_t)(0x10000 + elem_bytes)}, out, [&](CUtensorMap* m) {
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * (uint64_t)elem_bytes};
    cuuint32_t box[2] = {(cuuint32_t)(64 / elem_bytes), 32};
    cuuint32_t estr[2] = {1, 1};
    return st->encode(m, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                      const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                      CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  });
}

template <int BN, bool PAIR, bool NORM>
bool launch_bn_t(TcState* st, int idx, const GemmArgs& a, const EpiParams& ep, bool stream_k, cudaStream_t stream);

template <int BN, bool PAIR>
bool launch_bn(TcState* st, int idx, const GemmArgs& a, const EpiParams& ep, bool stream_k, cudaStream_t stream) {
  return a.epi == EPI_RESIDUAL_NORM ? launch_bn_t<BN, PAIR, true>(st, idx + 5, a, ep, stream_k, stream)
                                    : launch_bn_t<BN, PAIR, false>(st, idx, a, ep, stream_k, stream);
}

template <int BN, bool PAIR, bool NORM>
int max_active_clusters(TcState* st, int idx, int n_tiles, int parts);

// Problems of one row tile (at most 128 rows) whose tiles would be cut over K: how many CTAs form the cluster that shares
// a tile (0: no clusters).  The whole grid has to be resident at once, which the occupancy query decides (cached).
template <int BN, bool PAIR, bool NORM>
int cluster_parts(TcState* st, int idx, int n_tiles, int KB, int rows) {
  if (PAIR || !st->thin_clusters || n_tiles <= 0) return 0;
  using Cfg = TcCfg<BN, PAIR, NORM>;
  int parts = st->n_sm / n_tiles;
  if (parts > 4) parts = 4;
  if (parts > KB) parts = KB;
  // the leader keeps the peers' parts at the top of its ring budget: at least four stages must remain
  const int part_bytes = ((rows + 31) & ~31) * BN * 4;
  const int stage_bytes = (rows <= 32 ? Cfg::kThinABytes : Cfg::kABytes) + Cfg::kBBytes;
  while (parts >= 2 && (Cfg::kBudget - (parts - 1) * part_bytes) / stage_bytes < 4) --parts;
  for (; parts >= 2; --parts) {
    if (max_active_clusters<BN, PAIR, NORM>(st, idx, n_tiles, parts) >= n_tiles) return parts;
  }
  return 0;
}

template <int BN, bool PAIR, bool NORM>
int max_active_clusters(TcState* st, int idx, int n_tiles, int parts) {
  int& cached = st->max_clusters[idx][parts];
  if (cached < 0) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_tiles * parts);
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = TcCfg<BN, PAIR, NORM>::kSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = parts;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_tc_kernel<BN, PAIR, NORM>, &cfg) != cudaSuccess) {
      cudaGetLastError();
      n = 0;
    }
    cached = n;
  }
  return cached;
}

template <int BN, bool PAIR, bool NORM>
bool launch_bn_t(TcState* st, int idx, const GemmArgs& a, const EpiParams& ep, bool stream_k, cudaStream_t stream) {
  st->last_tiles_n = (a.N + (a.epi == EPI_SWIGLU ? BN / 2 : BN) - 1) / (a.epi == EPI_SWIGLU ? BN / 2 : BN);
  using Cfg = TcCfg<BN, PAIR, NORM>;
  if (!st->configured[idx]) {
    if (cudaFuncSetAttribute(gemm_tc_kernel<BN, PAIR, NORM>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes) !=
        cudaSuccess)
      return false;
    st->configured[idx] = true;
  }
  constexpr int kRows = PAIR ? 2 * BM : BM;
  const bool swiglu = a.epi == EPI_SWIGLU;
  const uint64_t w_rows = swiglu ? 2ull * a.N : (uint64_t)a.N;
  const int thin = (!PAIR && a.M <= 32) ? 1 : 0;
  CUtensorMap mx, mw, mo;     // copies: see cached_map
  if (!get_map(st, a.x, a.M, a.K, thin ? 32 : BM, &mx)) return false;
  if (!get_map(st, a.w, w_rows, a.K, (swiglu || PAIR) ? BN / 2 : BN, &mw)) return false;
  // the epilogue stores through the TMA unit (of the rotary / KV-append epilogue: the rotated queries [M, n_q * d];
  // K and V are scattered into the paged pool by hand)
  const bool f32 = a.epi == EPI_PLAIN_F32 || a.epi == EPI_RESIDUAL || a.epi == EPI_RESIDUAL_NORM;
  CUtensorMap mxo = mx;       // only read by EPI_RESIDUAL_NORM
  if (a.epi == EPI_RESIDUAL_NORM && !get_out_map(st, a.x_out, a.M, (uint64_t)a.N, 2, &mxo)) return false;
  if (!get_out_map(st, a.out, a.M, a.epi == EPI_QKV_ROPE ? (uint64_t)a.n_q * a.head_dim : (uint64_t)a.N, f32 ? 4 : 2, &mo))
    return false;
  const int out_per_tile = swiglu ? BN / 2 : BN;
  const int n_tiles_n = (a.N + out_per_tile - 1) / out_per_tile;
  const int mt = (a.M + kRows - 1) / kRows;
  const int n_tiles = mt * n_tiles_n;
  const long long KB = a.K / BK;
  const int n_units = PAIR ? st->n_sm / 2 : st->n_sm;       // scheduling units: CTAs, or clusters of two
  int units = n_tiles < n_units ? n_tiles : n_units;
  int dp_tiles = n_tiles;       // whole tiles, strided
  long long per = 1;
  const int cl = (stream_k && mt == 1 && a.M <= BM) ? cluster_parts<BN, PAIR, NORM>(st, idx, n_tiles, (int)KB, a.M) : 0;
  if (cl) {
    units = n_tiles * cl;       // one cluster per tile; the kernel derives each member's k-blocks from its rank
  } else if (a.m_dev) {
    // the row count is on the device: the kernel counts the tiles and, for stream-K, divides the k-blocks itself; the
    // grid has every unit (units without work leave at once)
    dp_tiles = stream_k ? -2 : -1;
    units = n_units;
  } else if (stream_k) {
    stream_k_schedule(n_tiles, mt, (int)KB, n_units, &dp_tiles, &per, &units);     // the caller made sure that mt <= n_units
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(PAIR ? 2 * units : units);
  cfg.blockDim = dim3(kTcThreads);
  cfg.dynamicSmemBytes = Cfg::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  int n_attr = 0;
  if (PAIR || cl) {
    attr[n_attr].id = cudaLaunchAttributeClusterDimension;
    attr[n_attr].val.clusterDim.x = PAIR ? 2 : cl;
    attr[n_attr].val.clusterDim.y = 1;
    attr[n_attr].val.clusterDim.z = 1;
    ++n_attr;
  }
  // programmatic dependent launch, except inside a stream capture (see launch_pdl)
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(stream, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone) {
    attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
    ++n_attr;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n_attr;
  return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<BN, PAIR, NORM>, mx, mw, mo, mxo, a.M, n_tiles_n, a.K, a.N, dp_tiles, per, thin, cl,
                            st->split_ws, st->split_counters, a.m_dev, a.m_dev_settled ? 0 : 1, ep) == cudaSuccess;
}

}  // namespace

void* tc_state_create(int n_sm) {
  TcState* st = new TcState();
  st->n_sm = n_sm;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn) {
    delete st;
    return nullptr;
  }
  st->encode = reinterpret_cast<EncodeTiledFn>(fn);
  if (cudaMalloc(reinterpret_cast<void**>(&st->split_ws), kSplitWsBytes) != cudaSuccess ||
      cudaMalloc(reinterpret_cast<void**>(&st->split_counters), kSplitCounters * sizeof(int)) != cudaSuccess ||
      cudaMemset(st->split_counters, 0, kSplitCounters * sizeof(int)) != cudaSuccess) {
    if (st->split_ws) cudaFree(st->split_ws);
    if (st->split_counters) cudaFree(st->split_counters);
    delete st;
    return nullptr;
  }
  return st;
}

void tc_state_force(void* s, int bn, int stream_k) {
  TcState* st = static_cast<TcState*>(s);
  if (!st) return;
  st->force_bn = bn;
  st->force_s = stream_k != 0;
  st->thin_clusters = stream_k != 2;     // 2: cut tiles always go through the partial-tile workspace
}

void tc_state_reset(void* s, cudaStream_t stream) {
  TcState* st = static_cast<TcState*>(s);
  if (st && st->split_counters) cudaMemsetAsync(st->split_counters, 0, kSplitCounters * sizeof(int), stream);
}

// Host-only check of the map cache: n_keys distinct keys go through it three at a time, the way a launch takes its
// maps, with an encoder that writes the key into the map; every map handed out must still carry its own key after
// the later lookups of the same launch (which may have emptied the cache).  Returns the number of wrong maps.
int tc_map_cache_selftest(int n_keys, int* evictions) {
  TcState st;
  auto fake = [](const MapKey& k) {
    return [k](CUtensorMap* m) {
      memset(m, 0, sizeof(*m));
      memcpy(m, &k, sizeof(k));
      return true;
    };
  };
  auto key_of = [](int i) { return MapKey{reinterpret_cast<const void*>(static_cast<uintptr_t>(4096) * (i + 1)), (uint64_t)i, 64, 128}; };
  int bad = 0;
  for (int i = 0; i + 2 < n_keys; i += 3) {
    CUtensorMap m[3];
    for (int j = 0; j < 3; ++j)
      if (!cached_map(&st, key_of(i + j), &m[j], fake(key_of(i + j)))) ++bad;
    auto carries = [](const CUtensorMap& m, const MapKey& k) {   // (field by field: the key has padding bytes)
      MapKey got;
      memcpy(&got, &m, sizeof(got));
      return got == k;
    };
    for (int j = 0; j < 3; ++j)
      if (!carries(m[j], key_of(i + j))) ++bad;
    // an old key again: a hit, or a miss that re-encodes; either way the right map
    CUtensorMap again;
    const MapKey k0 = key_of(i / 2);
    if (!cached_map(&st, k0, &again, fake(k0)) || !carries(again, k0)) ++bad;
  }
  if (st.maps.size() > kMapCacheMax) ++bad;
  if (evictions) *evictions = (int)st.evictions;
  return bad;
}

void tc_state_destroy(void* s) {
  TcState* st = static_cast<TcState*>(s);
  if (!st) return;
  if (st->split_ws) cudaFree(st->split_ws);
  if (st->split_counters) cudaFree(st->split_counters);
  delete st;
}

static bool launch_gemm_tc_impl(const GemmArgs& a, TcState* st, int* status, cudaStream_t stream);

bool launch_gemm_tc(const GemmArgs& a, void* tc_state, int* status, cudaStream_t stream, int* ss_slots_out) {
  TcState* st = static_cast<TcState*>(tc_state);
  if (!st || a.M <= 0) return false;
  if (a.epi == EPI_RESIDUAL_NORM && (!a.x_out || !a.gain || !a.ss_out || a.N % 32)) return false;
  const bool ok = launch_gemm_tc_impl(a, st, status, stream);
  if (ok && ss_slots_out) *ss_slots_out = st->last_tiles_n;
  return ok;
}

static bool launch_gemm_tc_impl(const GemmArgs& a, TcState* st, int* status, cudaStream_t stream) {
  if (a.K % BK) return false;
  if ((reinterpret_cast<uintptr_t>(a.x) | reinterpret_cast<uintptr_t>(a.w)) & 15) return false;
  EpiParams ep;
  ep.epi = a.epi;
  ep.out = a.out;
  ep.M = a.M;
  ep.N = a.N;
  ep.tok_slot = a.tok_slot;
  ep.rope_cs = static_cast<const float2*>(a.rope_cs);
  ep.kv_pool = static_cast<__nv_bfloat16*>(a.kv_pool);
  ep.n_pages = a.n_pages;
  ep.layer = a.layer;
  ep.n_q = a.n_q;
  ep.n_kv = a.n_kv;
  ep.head_dim = a.head_dim;
  ep.status = status;
  ep.ss_in = a.ss_in;
  ep.ss_slots = a.ss_slots;
  ep.ss_stride = a.ss_stride;
  ep.norm_inv_n = 1.f / (float)a.K;
  ep.norm_eps = a.norm_eps;
  ep.gain = static_cast<const __nv_bfloat16*>(a.gain);
  ep.ss_out = a.ss_out;
  const bool swiglu = a.epi == EPI_SWIGLU;
  // Choose the tile width and the decomposition with a small cost model in microseconds, calibrated on B200:
  // whole tiles cost waves x k-blocks x (tensor time of one k-block at that width); the stream-K decomposition
  // spreads all k-blocks evenly over the SMs and pays a fixed hand-over for the cut tiles (park the partial,
  // fence, counter, reduction read).  Rotary tiles must hold whole heads.
  // (device-resident rounds: the configuration is chosen for the caller's hint of the row count, the launch covers the capacity)
  const int Mc = (a.m_dev && a.m_hint > 0 && a.m_hint < a.M) ? a.m_hint : a.M;
  const int mt = (Mc + BM - 1) / BM;
  const int KB = a.K / BK;
  int best_bn = 0;
  bool best_sk = false, best_pair = false;
  double best_t = 1e30;
  // configurations: single CTAs with 128-row tiles of width 256 / 128 / 64, and CTA pairs with 256 x 256 or 256 x 128
  // tiles (a k-block of a pair takes about 0.87 / 0.76 of the single CTA's, for twice the rows: the pair halves the
  // weight bytes each SM's tensor core pulls out of its own shared memory)
  constexpr int kConfigs = 5;
  const int bns[kConfigs] = {256, 128, 64, 256, 128};
  const double kb_tensor[kConfigs] = {0.44, 0.27, 0.22, 0.385, 0.205};
  const bool pair_ok = Mc > BM && (swiglu ? a.N % 128 == 0 : a.N % 256 == 0) && !(a.epi == EPI_QKV_ROPE && 256 % a.head_dim);
  const bool pair128_ok = Mc > BM && !swiglu && a.N % 128 == 0 && !(a.epi == EPI_QKV_ROPE && 128 % a.head_dim);
  for (int bi = 0; bi < kConfigs; ++bi) {
    const int bn = bns[bi];
    const bool pair = bi >= 3;
    if (bi == 3 && !pair_ok) continue;
    if (bi == 4 && !pair128_ok) continue;
    const int rows_tile = pair ? 2 * BM : BM;
    const int units = pair ? st->n_sm / 2 : st->n_sm;            // CTAs or clusters
    const int mtc = (Mc + rows_tile - 1) / rows_tile;
    const int per = swiglu ? bn / 2 : bn;
    if (a.epi == EPI_QKV_ROPE && (bn < a.head_dim || a.N % bn)) continue;
    if (swiglu && (a.N % per)) continue;
    const int tiles = mtc * ((a.N + per - 1) / per);
    if (tiles * (pair ? 2 : 1) > kSplitCounters) continue;
    const long long waves = (tiles + units - 1) / units;
    // a k-block costs its tensor time, or the time one SM needs to stream its share of the weight bytes (the
    // CTAs that work on one weight tile at the same time share them through L2)
    const double kbt = fmax(kb_tensor[bi], (bn * 128.0 / mt) / 35e3);
    const double rows = Mc < BM ? Mc : BM;
    const double t_plain = (double)waves * KB * kbt;
    const int sk_units = mtc <= units ? (units / mtc) * mtc : 1;     // teams of mtc units
    const double t_sk = ((double)tiles * KB / sk_units + 1.0) * kbt + 3.0 + rows * bn * 4.0 * 2.5 / 16e3;
    if (t_plain < best_t) { best_t = t_plain; best_bn = bn; best_sk = false; best_pair = pair; }
    const bool ws_fits = (size_t)2 * st->n_sm * BM * bn * 4 <= kSplitWsBytes && mtc <= units;
    const long long full = tiles / units, rem = tiles % units;
    if (ws_fits && full >= 2) {
      // a ragged last wave: the last (units + rem) tiles are cut evenly over the SMs and done FIRST, so that their
      // hand-over (park the partial, counter, reduction by the last arriver) hides under the whole tiles after it.
      // Measured: the cut tiles run a little slower than whole ones, so this only pays when the last wave would
      // leave a good part of the machine idle.
      const double idle = rem ? (double)(units - rem) / units / (double)(full + 1) : 0.0;
      const double t_h = (double)tiles * KB / units * kbt + 2.0;
      if (idle > 0.12 && t_h < best_t) { best_t = t_h; best_bn = bn; best_sk = true; best_pair = pair; }
    } else if (ws_fits && t_sk < best_t) {
      // no whole tiles to hide the hand-over under: it happens in every CTA at once at the end of the kernel and
      // costs about 3 us + 0.6 us per KB of partial tile, which t_sk charges
      best_t = t_sk; best_bn = bn; best_sk = true; best_pair = pair;
    }
  }
  if (st->force_bn == 384) {    // tuning aid: CTA pairs with 256 x 128 tiles, "384,<0 whole tiles | 1 stream-K>"
    if (pair128_ok && (a.M + 255) / 256 <= st->n_sm / 2) return launch_bn<128, true>(st, 4, a, ep, st->force_s != 0, stream);
  } else
  if (st->force_bn == 512) {    // tuning aid: the 256 x 256 CTA-pair kernel, "512,<0 whole tiles | 1 stream-K>"
    if (pair_ok && (a.M + 255) / 256 <= st->n_sm / 2) return launch_bn<256, true>(st, 3, a, ep, st->force_s != 0, stream);
  } else
  if (st->force_bn) {   // tuning aid (tc_state_force): tile width, 0 whole tiles | 1 stream-K; ignored where it does not fit
    const int bn = st->force_bn;
    const int per = swiglu ? bn / 2 : bn;
    const bool shape_ok = (bn == 256 || bn == 128 || bn == 64) &&
                          !(a.epi == EPI_QKV_ROPE && (bn < a.head_dim || a.N % bn)) && !(swiglu && (a.N % per)) &&
                          mt * ((a.N + per - 1) / per) <= kSplitCounters;
    if (shape_ok) {
      best_bn = bn;
      best_pair = false;
      best_sk = st->force_s != 0 && mt <= st->n_sm && (size_t)2 * st->n_sm * BM * bn * 4 <= kSplitWsBytes;
    }
  }
  if (!best_bn) return false;
  if (swiglu && (a.N % 32)) return false;
  if (best_pair && best_bn == 128) return launch_bn<128, true>(st, 4, a, ep, best_sk, stream);
  if (best_pair) return launch_bn<256, true>(st, 3, a, ep, best_sk, stream);
  switch (best_bn) {
    case 256: return launch_bn<256, false>(st, 0, a, ep, best_sk, stream);
    case 128: return launch_bn<128, false>(st, 1, a, ep, best_sk, stream);
    default: return launch_bn<64, false>(st, 2, a, ep, best_sk, stream);
  }
}

}  // namespace recg

// Hybrid-mask paged-KV attention on the 5th-generation tensor cores (head_dim 128).
//
// Work items are the same as in attention.cu: (request, kv head, row tile of <= 128 query rows, KV range).
// Per CTA (12 warps = 3 warpgroups, one CTA per SM, persistent over the work list):
//   warps 0, 2  producers: warp 0 streams the K operand and warp 2 the V operand of each 128-token KV block,
//             page by page, ONE 4 KB bulk copy per page, into a ring of 32 KB operand buffers (K and V of
//             a block are separate entries, so K is released early).  A page tile (8-row, 128-byte-swizzled
//             atoms ordered [token group][dim half]) lands exactly as stored, and tiles copied back to back
//             form one 128-token operand with a uniform 2 KB stride between token groups: K-major for
//             S = Q K^T, MN-major for O += P V.  The last, partly filled V page of a request is copied by
//             hand with the rows beyond its length zeroed, so stale pool contents never reach an accumulator.
//             Warp 0 also fetches the item's Q rows with two tiled TMA loads (box = 64 dims x the kv head's
//             query heads x 128 / group tokens, 128-byte swizzle) into one of two Q buffers, so the Q of the
//             next item is in place before the current item ends.
//   warp 1    one elected lane issues tcgen05.mma: S = Q K^T (M 128 rows, N 128 tokens, K = d, both operands
//             in shared memory) into one of two S buffers in TMEM (stage & 1), and per softmax group
//             O_g += P_g V_g (P read from TMEM, V from shared memory; N = d, K = the group's 64 tokens).  It runs
//             two stages ahead with S and into the next item while the softmax groups still write the previous
//             item's output.  Its per-instruction cost matters (it was the bottleneck once): descriptors are a
//             base plus constants, one product and one barrier per stage serve both groups.
//   warps 4-7 and 8-11: two softmax groups.  Group g takes tokens [64 g, 64 g + 64) of EVERY 128-token stage; it
//             has its own O accumulator in TMEM and its own running (reference maximum, sum), i.e. the two
//             groups are two independent partial attentions over interleaved 64-token chunks, merged once at
//             the end of the item.  Within a group ONE THREAD OWNS ONE QUERY ROW (= TMEM lane): its 64 scores
//             are read from TMEM once, probabilities are taken relative to a reference maximum that is only
//             moved (and O rescaled in TMEM) when the row maximum outgrows it by more than 2^8, and bf16 P is
//             written back over the first 32 of the group's 64 columns of the same S buffer (two tokens per
//             32-bit column), from where the P V product reads it.  Because S is double buffered, the S of
//             the next stage is already there when a group finishes a stage; the tensor pipe executes in issue
//             order, so a buffer's next S is produced after its P has been consumed.  No cross-thread
//             reductions are needed.  At the end of an item group 0 finishes output dims [0,64) and group 1
//             dims [64,128) of every row from both accumulators; partial results (items that cover part of
//             the KV range) go through a per-warp transposition in the item's Q buffer so that every global
//             store is a full 128-byte line.
//   All warps run with the kernel's 168 registers: moving registers from warpgroup 0 to the softmax groups
//   (setmaxnreg) made the compiler spill in the producer and MMA warps and measured 1.5 % slower.
// Only blocks that reach past a row's visibility limit evaluate the mask.  Every wait is bounded; a wait that
// runs out raises a CTA-wide flag after which no wait blocks, so the kernel always ends.
#include <cuda.h>
#include <cstdio>
#include <cstdlib>
#include <mutex>

#include "common.cuh"
#include "kernels.h"

namespace recg {

namespace {

constexpr int D = 128;
constexpr int kBT = 128;                       // tokens per KV block
constexpr int kPagesPerBT = kBT / kPageSize;   // 8
constexpr int kSubBytes = kPageSize * 128;     // 2 KB: [16 tokens][64 dims]
constexpr int kQBytes = 128 * D * 2;           // 32 KB
constexpr int kTileBytes = 2 * kSubBytes;        // 4 KB: the K (or V) tile of one page and head, as stored in the pool
constexpr int kKVStageBytes = kPagesPerBT * kTileBytes;  // one operand (K or V) of a 128-token block: 32 KB
constexpr int kKStages = 2;                      // K ring: a buffer is free after its Q K^T
constexpr int kVStages = 3;                      // V ring: a buffer is free after its P V.  The rings are separate so that a V
                                                 // buffer never holds the unsanitised rows of a partly filled K page
constexpr int kKVStages = kKStages + kVStages;
constexpr int kThreads = 384;                    // warpgroup 0: producer K, MMA, producer V, idle; warpgroups 1, 2: softmax
constexpr uint32_t kSpin = 1u << 22;
constexpr int kTmemCols = 512;                 // two S buffers of 128 columns (stage & 1); group g owns columns [64 g, 64 g + 64) of each
                                               // and overwrites the first 32 of them with its bf16 P; O of group g at 256 + 128 g
constexpr int kTmemO = 2 * kBT;

constexpr int kOffQ = 0;                       // two Q buffers: item i uses buffer i & 1
constexpr int kOffKV = kOffQ + 2 * kQBytes;
constexpr int kOffML = kOffKV + kKVStages * kKVStageBytes;   // float2 [2 groups][128 rows]: (reference max, sum)
constexpr int kOffBar = kOffML + 2 * 128 * 8;
constexpr int kNumBars = 2 * kKVStages + 2 + 2 + 2 + 4 + 1 + 1 + 1;
constexpr int kSmemBytes = kOffBar + kNumBars * 8 + 64;   // barriers, TMEM slot + flag, item ranges, first item
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

struct TcAttnParams {
  const AttnItem* items;
  const int* cta_off;
  const int* page_table;
  int pt_stride;
  const int* tok_climit;
  const int* tok_lo;
  const int* tok_hi;
  __nv_bfloat16* o;
  const __nv_bfloat16* pool;
  int64_t n_pages;
  int layer, n_q, n_kv, group;
  float scale_log2;
  float* part_o;
  float* part_ml;
  int* status;
  int early_desc;     // the work list is settled: it may be read before the wait for the kernel in front of this one
};

// ---- PTX wrappers (tcgen05) ------------------------------------------------------------------------
__device__ __forceinline__ bool elect_one() {
  uint32_t pred = 0;
  asm volatile("{\n .reg .b32 rx;\n .reg .pred px;\n elect.sync rx|px, %1;\n @px mov.s32 %0, 1;\n}"
               : "+r"(pred)
               : "r"(0xffffffffu));
  return pred != 0;
}
__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      :
      : "r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
// A operand (M x 16 bf16, two K elements per 32-bit column) read from TMEM instead of shared memory
__device__ __forceinline__ void umma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
      :
      : "r"(tmem_d), "r"(tmem_a), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_ld32_nowait(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,"
      "%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,"
      "%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// shared-memory operand descriptors, 128-byte swizzle, 8-row atoms of 1024 bytes
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t addr, uint32_t sbo_bytes = 1024) {
  return (uint64_t)((addr & 0x3ffff) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// MN-major: 64 contiguous MN elements per 128-byte row; LBO = stride between 64-wide MN groups, SBO = stride
// between 8-row K groups
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr & 0x3ffff) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// S / P column c of a 128-token block holds token c
__device__ __forceinline__ int col_token(int c) { return c; }
constexpr uint32_t kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBT >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
constexpr uint32_t kIdescPV =
    (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(D >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

__device__ __forceinline__ void tma_load_3d(uint32_t smem_dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
               :
               : "r"(smem_dst), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
               : "memory");
}
__device__ __forceinline__ void softmax_bar() { asm volatile("bar.sync 1, 256;" ::: "memory"); }


__global__ void __launch_bounds__(kThreads, 1) attention_tc_kernel(const __grid_constant__ CUtensorMap qmap, TcAttnParams P) {
  extern __shared__ __align__(1024) uint8_t smem[];
  if (smem_u32(smem) & 1023u) {          // the swizzled operand layouts need a 1 KB aligned base
    if (threadIdx.x == 0) set_status(P.status, DEV_BAD_INDEX);
    return;
  }
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kOffBar);
  uint64_t* kv_full = bars;                 // [kKVStages]: K ring first, then V ring
  uint64_t* kv_empty = bars + kKVStages;    // [kKVStages]
  uint64_t* q_full = bars + 2 * kKVStages;  // [2]  per Q buffer
  uint64_t* q_empty = q_full + 2;           // [2]
  uint64_t* s_full = q_full + 4;            // [2]  per S buffer (stage & 1); both groups wait on it
  uint64_t* p_full = q_full + 6;            // [4]  per (softmax group, S buffer): index 2 g + (stage & 1)
  uint64_t* pv_done = q_full + 10;          // both groups' P V products of a stage have completed
  uint64_t* o_full = q_full + 11;
  uint64_t* o_empty = q_full + 12;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kNumBars);
  float2* ml_smem = reinterpret_cast<float2*>(smem + kOffML);

  // A wait that runs out records why and raises this flag; from then on no wait in this CTA blocks any more, so
  // every warp still walks through its loops (and meets the others at the named barriers) and the kernel ends.
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  auto bwait = [&](uint64_t* bar, uint32_t parity, int code) {
    if (*abort_flag) return;
    if (!mbar_wait(bar, parity, kSpin)) {
      set_status(P.status, code);
      *abort_flag = 1;
    }
  };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Warp 0 waits for the kernels before this one and fetches the CTA's item range and first item while the other
  // warps set up barriers, the zeroed ring and TMEM: two dependent round trips off everybody's critical path.
  int* s_range = reinterpret_cast<int*>(tmem_slot + 2);
  AttnItem* s_first = reinterpret_cast<AttnItem*>(tmem_slot + 6);
  // the CTA walks two ranges of the item list one after the other (see the layout kernel): logical item i is
  // entry b0 + i for i < n0 and entry b1 + (i - n0) after that
  int range_b0 = 0, range_n0 = 0, range_b1 = 0;
  const int item_begin = 0;
  int item_end = 0;
  auto item_at = [&](int i) { return i < range_n0 ? range_b0 + i : range_b1 + (i - range_n0); };
  AttnItem w_next = {};
  if (warp == 0) {
    // (inside a step the work list was written many launches ago and the kernel in front of this one, the QKV
    // projection, only signals its dependents when its own work is done: the two dependent reads below then overlap
    // that kernel's tail instead of following it)
    if (!P.early_desc) griddep_wait();
    const int4 r4 = *reinterpret_cast<const int4*>(P.cta_off + 4 * blockIdx.x);
    range_b0 = r4.x;
    range_n0 = r4.y - r4.x;
    range_b1 = r4.z;
    item_end = range_n0 + (r4.w - r4.z);
    if (item_begin < item_end) w_next = P.items[item_at(0)];
    if (lane == 0) {
      s_range[0] = range_b0;
      s_range[1] = range_n0;
      s_range[2] = range_b1;
      s_range[3] = item_end;
      *s_first = w_next;
    }
    if (P.early_desc) griddep_wait();
  }
  if (threadIdx.x == 32) {
    *abort_flag = 0;
    for (int s = 0; s < kKVStages; ++s) {
      mbar_init(&kv_full[s], 1);
      mbar_init(&kv_empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&q_full[s], 1);
      mbar_init(&q_empty[s], 8);
      mbar_init(&s_full[s], 1);
    }
    for (int s = 0; s < 4; ++s) mbar_init(&p_full[s], 4);
    mbar_init(pv_done, 1);
    mbar_init(o_full, 1);
    mbar_init(o_empty, 8);
    fence_barrier_init();
    asm volatile("prefetch.tensormap [%0];" ::"l"(&qmap) : "memory");
  }
  // The operand ring starts out zeroed: later on a buffer only ever holds zeros, real K/V pages or hand-copied
  // pages, so V rows that no copy refreshes (pages beyond a request's end) are finite and 0 * V stays 0.
  if (warp != 0)
    for (int c = threadIdx.x - 32; c < kKVStages * kKVStageBytes / 16; c += kThreads - 32)
      reinterpret_cast<uint4*>(smem + kOffKV)[c] = make_uint4(0, 0, 0, 0);
  fence_proxy_async();
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (warp != 0) {
    griddep_wait();   // these warps touched only shared memory and TMEM so far
    range_b0 = s_range[0];
    range_n0 = s_range[1];
    range_b1 = s_range[2];
    item_end = s_range[3];
    w_next = *s_first;
  }
  const uint32_t smem_base = smem_u32(smem);

  if (warp < 4) {
    if (warp == 0 || warp == 2) {
      // ------------------------------------ producers: warp 0 streams Q and K, warp 2 streams V ------------------------------------
      const int part = warp == 0 ? 0 : 1;
      uint32_t blk = 0, item_cnt = 0;  // running KV-block and item counters
      for (int item = item_begin; item < item_end; ++item, ++item_cnt) {
        const AttnItem w = w_next;
        if (item + 1 < item_end) w_next = P.items[item_at(item + 1)];
        const int tok_begin = w.blk_begin * 64;
        const int tok_end = min(w.blk_end * 64, w.kv_len);
        const int nblk = (tok_end - tok_begin + kBT - 1) / kBT;
        const int n_req_pages = (w.kv_len + kPageSize - 1) / kPageSize;
        const int* pt = P.page_table + (size_t)w.req * P.pt_stride;
        // page ids are fetched by lanes 0..7 in parallel, one iteration ahead of their use
        auto fetch_page = [&](int n) -> int {
          int pg = -1;
          if (lane < kPagesPerBT && n < nblk) {
            const int lp = tok_begin / kPageSize + n * kPagesPerBT + lane;
            if (lp < n_req_pages && lp * kPageSize < tok_end) pg = __ldg(pt + lp);   // validated when used
          }
          return pg;
        };
        int pg_next = fetch_page(0);
        if (part == 0) {
          // Q rows of the item: (64 dims) x (the kv head's query heads) x (128 / group tokens from tok0); rows past the
          // tile's own tokens belong to other tokens or are zero-filled, and nobody reads their S / O rows
          const int buf = item_cnt & 1;
          bwait(&q_empty[buf], ((item_cnt >> 1) & 1) ^ 1, DEV_TIMEOUT_EMPTY);
          if (lane == 0) {
            // two boxes of 64 dims x group heads x 128 / group tokens (125 rows when the group is 5; the MMA reads 128)
            mbar_arrive_expect_tx(&q_full[buf], 2u * 128u * (uint32_t)(P.group * (128 / P.group)));
            const uint32_t dst = smem_base + kOffQ + buf * kQBytes;
            tma_load_3d(dst, &qmap, 0, w.kv_head * P.group, w.tok0, &q_full[buf]);
            tma_load_3d(dst + kQBytes / 2, &qmap, 64, w.kv_head * P.group, w.tok0, &q_full[buf]);
          }
          __syncwarp();
        }
        for (int n = 0; n < nblk; ++n, ++blk) {
          int my_pg = pg_next;
          pg_next = fetch_page(n + 1);                 // in flight during this iteration
          if (my_pg >= P.n_pages) {
            set_status(P.status, DEV_BAD_INDEX);
            my_pg = -1;
          }
          // lane p < 8 owns page p of the block: full pages go by bulk copy, the rest by hand
          const int first_tok = tok_begin + (n * kPagesPerBT + lane) * kPageSize;
          const int my_valid = (lane < kPagesPerBT && my_pg >= 0) ? min(kPageSize, w.kv_len - first_tok) : 0;
          // K: every existing page goes by bulk copy (rows beyond the request's end are masked in S).
          // V: full pages by bulk copy; the one partly filled page by hand with its stale rows zeroed (0 * stale
          // could be NaN); pages beyond the end are not touched (the buffer holds finite data, see the start).
          const bool my_bulk = part == 0 ? my_valid > 0 : my_valid == kPageSize;
          const unsigned bulk_mask = __ballot_sync(0xffffffffu, my_bulk);
          const unsigned hand_mask = part == 0 ? 0u : __ballot_sync(0xffffffffu, my_valid > 0 && my_valid < kPageSize);
          const int ring = part == 0 ? kKStages : kVStages;
          const int s = (part == 0 ? 0 : kKStages) + blk % ring;
          bwait(&kv_empty[s], ((blk / ring) & 1) ^ 1, DEV_TIMEOUT_EMPTY);
          uint8_t* stage = smem + kOffKV + s * kKVStageBytes;
          if (hand_mask) {
            const int p = __ffs(hand_mask) - 1;            // at most one partly filled page per request
            const int pg = __shfl_sync(0xffffffffu, my_pg, p);
            const int valid_tok = __shfl_sync(0xffffffffu, my_valid, p);
            const uint4* src = reinterpret_cast<const uint4*>(
                                   P.pool + kv_tile_base(P.n_pages, P.n_kv, D, P.layer, pg, w.kv_head)) + part * 256;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const int c = u * 32 + lane;
              const uint4 v = (((c >> 7) * 8 + ((c >> 3) & 7)) < valid_tok) ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
              *reinterpret_cast<uint4*>(stage + p * kTileBytes + c * 16) = v;
            }
            fence_proxy_async();
          }
          __syncwarp();
          if (lane == 0) {
            if (bulk_mask == 0) mbar_arrive(&kv_full[s]);
            else mbar_arrive_expect_tx(&kv_full[s], __popc(bulk_mask) * kTileBytes);
          }
          __syncwarp();
          if (my_bulk) {
            const uint8_t* src = reinterpret_cast<const uint8_t*>(
                                     P.pool + kv_tile_base(P.n_pages, P.n_kv, D, P.layer, my_pg, w.kv_head)) +
                                 part * kTileBytes;
            bulk_g2s(stage + lane * kTileBytes, src, kTileBytes, &kv_full[s]);
          }
          __syncwarp();
        }
      }
      if (*abort_flag && lane == 0) {     // gave up somewhere: let this warp's copies in flight land before exiting
        for (int s = 0; s < kKVStages; ++s)
          for (uint32_t i = 0; i < (1u << 14); ++i) {
            if (mbar_try_wait(&kv_full[s], 0) || mbar_try_wait(&kv_full[s], 1)) break;
            __nanosleep(64);
          }
      }
    } else if (warp == 1) {
      // ------------------------------------ MMA issuer ------------------------------------
      if (elect_one()) {
        uint32_t blk = 0, item_cnt = 0;      // running stage (128-token KV block) and item counters
        // Group g works on tokens [64 g, 64 g + 64) of EVERY stage.  S of stage b = Q K^T goes to S buffer b & 1 (one
        // N = 128 product for both groups), so the S of stage b + 1 is ready while the groups still work on stage b;
        // the tensor pipe executes in issue order, which puts it after the P V products that read the buffer's
        // previous P.  Shared-memory descriptors are linear in the address (no carry out of the 14-bit field
        // within the operand areas), so the per-instruction descriptors are a base plus constants.
        auto issue_qk = [&](uint32_t b, uint64_t dq0) {
          const int s = b % kKStages;
          bwait(&kv_full[s], (b / kKStages) & 1, DEV_TIMEOUT_FULL);
          tc_fence_after();
          // K block: 16 token groups (2 per page) 2 KB apart; the dim half selects the atom next door
          const uint64_t dk0 = desc_kmajor(smem_base + kOffKV + s * kKVStageBytes, 2048);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk)
            umma_bf16(tmem_base + (b & 1) * kBT, dq0 + (uint64_t)((((kk >> 2) * (128 * 128)) + (kk & 3) * 32) >> 4),
                      dk0 + (uint64_t)((((kk >> 2) * 1024) + (kk & 3) * 32) >> 4), kIdescQK, kk ? 1u : 0u);
          umma_commit(&s_full[b & 1]);
          umma_commit(&kv_empty[s]);   // the K buffer is free once these MMAs have read it
        };
        for (int item = item_begin; item < item_end; ++item, ++item_cnt) {
          const AttnItem w = w_next;
          if (item + 1 < item_end) w_next = P.items[item_at(item + 1)];
          const int tok_begin = w.blk_begin * 64;
          const int tok_end = min(w.blk_end * 64, w.kv_len);
          const int nblk = (tok_end - tok_begin + kBT - 1) / kBT;
          const int buf = item_cnt & 1;
          const uint64_t dq0 = desc_kmajor(smem_base + kOffQ + buf * kQBytes);
          bwait(&q_full[buf], (item_cnt >> 1) & 1, DEV_TIMEOUT_FULL);
          tc_fence_after();
          issue_qk(blk, dq0);
          if (nblk > 1) issue_qk(blk + 1, dq0);
          for (int n = 0; n < nblk; ++n, ++blk) {
            const int s = kKStages + blk % kVStages;
            // V block: tokens [16 j, 16 j + 16) = page j: two token groups 2 KB apart, the dim halves 1 KB apart
            const uint64_t dv0 = desc_mnmajor(smem_base + kOffKV + s * kKVStageBytes, 1024, 2048);
#pragma unroll
            for (int g = 0; g < 2; ++g) {
              // O of group g (+)= P V over its 64 tokens of stage n: P (bf16, two tokens per 32-bit column) from TMEM
              bwait(&p_full[2 * g + (blk & 1)], (blk >> 1) & 1, DEV_TIMEOUT_MMA);
              if (g == 0) {
                // the previous item's accumulators must have been read out before this item's products overwrite them
                if (n == 0) bwait(o_empty, (item_cnt & 1) ^ 1, DEV_TIMEOUT_MMA);
                bwait(&kv_full[s], (blk / kVStages) & 1, DEV_TIMEOUT_FULL);
              }
              tc_fence_after();
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                umma_bf16_ts(tmem_base + kTmemO + g * D, tmem_base + (blk & 1) * kBT + g * 64 + kk * 8,
                             dv0 + (uint64_t)(((4 * g + kk) * kTileBytes) >> 4), kIdescPV, (n | kk) ? 1u : 0u);
            }
            umma_commit(pv_done);
            umma_commit(&kv_empty[s]);
            if (n == nblk - 1) umma_commit(o_full);
            if (n + 2 < nblk) issue_qk(blk + 2, dq0);
          }
        }
      }
    }
  } else {
    // ------------------------------------ softmax ------------------------------------
    const int g = (warp - 4) >> 2;             // softmax group: takes tokens [64 g, 64 g + 64) of every stage
    const int quad = warp & 3;
    const int row = quad * 32 + lane;          // query row of the tile = TMEM lane
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const uint32_t s_addr = lane_addr + g * 64, o_addr = lane_addr + kTmemO + g * D;
    uint32_t cs = 0, item_cnt = 0;   // stages and items so far
    // visibility triple of this thread's row, fetched one item ahead
    auto row_vis = [&](const AttnItem& it, int& cl, int& lo, int& hi) {
      cl = -1; lo = 0; hi = 0;
      if (row < it.ntok * P.group) {
        const int t = it.tok0 + row / P.group;
        cl = P.tok_climit[t];
        lo = P.tok_lo[t];
        hi = P.tok_hi[t];
      }
    };
    int nx_cl = -1, nx_lo = 0, nx_hi = 0;
    if (item_begin < item_end) row_vis(w_next, nx_cl, nx_lo, nx_hi);
    for (int item = item_begin; item < item_end; ++item) {
      const AttnItem w = w_next;
      if (item + 1 < item_end) w_next = P.items[item_at(item + 1)];
      const int R = w.ntok * P.group;
      const int tok_begin = w.blk_begin * 64;
      const int tok_end = min(w.blk_end * 64, w.kv_len);
      const int nblk = (tok_end - tok_begin + kBT - 1) / kBT;
      const bool rvalid = row < R;
      const bool warp_valid = quad * 32 < R;
      const int climit = nx_cl, vlo = nx_lo, vhi = nx_hi;
      float m_ref = -1e30f, l_run = 0.f;
      bool first = true;

      for (int n = 0; n < nblk; ++n, ++cs) {
        // this group's 64 tokens of stage n: S buffer cs & 1 (cs = running stage count, the same in every role)
        const uint32_t s_buf = s_addr + (cs & 1) * kBT;
        bwait(&s_full[cs & 1], (cs >> 1) & 1, DEV_TIMEOUT_MMA);
        tc_fence_after();
        const int pos0 = tok_begin + n * kBT + g * 64;
        uint32_t sr[2][32];   // the S row of this thread: 64 scores
        float mx = -INFINITY;
        if (warp_valid) {
#pragma unroll
          for (int c = 0; c < 2; ++c) tmem_ld32_nowait(s_buf + c * 32, sr[c]);
          tmem_ld_wait();
          const int lim = min(climit, tok_end - 1);
          const bool need_mask = __any_sync(0xffffffffu, rvalid && (pos0 + 63 > lim));
          if (need_mask) {
            // visible tokens of this row within the 64: [0, a] and [b, c), as a 64-bit mask over tokens
            const int a = lim - pos0, b = vlo - pos0, cc = min(vhi, tok_end) - pos0;
            auto ones = [](int n) -> unsigned long long {      // n lowest bits set, n clamped to [0, 64]
              return n <= 0 ? 0ull : (n >= 64 ? ~0ull : ((1ull << n) - 1ull));
            };
            const unsigned long long m0 = ones(a + 1) | (ones(cc) & ~ones(b));
#pragma unroll
            for (int c = 0; c < 2; ++c)
#pragma unroll
              for (int i = 0; i < 32; ++i) {
                const int t = col_token(c * 32 + i);        // compile-time constant after unrolling
                if (((m0 >> t) & 1ull) == 0ull) sr[c][i] = 0xff800000u;   // -inf
              }
          }
          {  // four independent chains instead of one long dependent one
            float mxa[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int c = 0; c < 2; ++c)
#pragma unroll
              for (int i = 0; i < 32; i += 4) {
                mxa[2 * c] = fmaxf(mxa[2 * c], fmaxf(__uint_as_float(sr[c][i]), __uint_as_float(sr[c][i + 1])));
                mxa[2 * c + 1] = fmaxf(mxa[2 * c + 1], fmaxf(__uint_as_float(sr[c][i + 2]), __uint_as_float(sr[c][i + 3])));
              }
            mx = fmaxf(fmaxf(mxa[0], mxa[1]), fmaxf(mxa[2], mxa[3]));
          }
          const float m_blk = mx * P.scale_log2;
          // move the reference maximum only when the row maximum outgrows it by more than 2^8 (or at the first
          // stage): probabilities stay below 256 relative to the reference, well inside bf16 and fp32 range
          const bool grow = rvalid && (m_blk > m_ref + 8.f);
          if (n == 0) {
            if (rvalid && m_blk > m_ref) m_ref = m_blk;
          } else if (__any_sync(0xffffffffu, grow)) {
            // rare: O is rescaled in TMEM, once the group's P V of the previous stage has completed
            bwait(pv_done, (cs - 1) & 1, DEV_TIMEOUT_MMA);
            tc_fence_after();
            const float m_new = grow ? m_blk : m_ref;
            const float f = exp2f(m_ref - m_new);
            m_ref = m_new;
            l_run *= f;
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
              uint32_t r[32];
              tmem_ld32_nowait(o_addr + c * 32, r);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f);
              tmem_st32(o_addr + c * 32, r);
            }
            tmem_st_wait();
          }
          float lsa[4] = {0.f, 0.f, 0.f, 0.f};
          uint32_t pk[32];     // 64 tokens -> 32 packed columns over the start of this S buffer
#pragma unroll
          for (int c = 0; c < 2; ++c) {
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              const float p0 = exp2f(__uint_as_float(sr[c][i]) * P.scale_log2 - m_ref);   // exp2(-inf) = 0 for masked
              const float p1 = exp2f(__uint_as_float(sr[c][i + 1]) * P.scale_log2 - m_ref);
              lsa[(i >> 1) & 3] += p0 + p1;
              pk[c * 16 + (i >> 1)] = pack_bf16(p0, p1);
            }
          }
          tmem_st32(s_buf, pk);
          l_run += (lsa[0] + lsa[1]) + (lsa[2] + lsa[3]);
          tmem_st_wait();
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[2 * g + (cs & 1)]);
        if (first) {      // the next item's descriptor has arrived by now: fetch its rows' visibility for later
          first = false;
          if (item + 1 < item_end) row_vis(w_next, nx_cl, nx_lo, nx_hi);
        }
      }

      // ---- merge the two groups' partial attentions and write out: this group finishes dims [64 g, 64 g + 64) ----
      const bool two = true;                      // both groups take part in every stage
      const int buf = item_cnt & 1;
      bwait(o_full, item_cnt & 1, DEV_TIMEOUT_MMA);
      tc_fence_after();
      ml_smem[g * 128 + row] = make_float2(m_ref, l_run);
      softmax_bar();
      if (warp_valid) {
        const float2 a0 = ml_smem[row];
        const float2 a1 = two ? ml_smem[128 + row] : make_float2(-1e30f, 0.f);
        const float m_all = fmaxf(a0.x, a1.x);
        float f0 = exp2f(a0.x - m_all), f1 = two ? exp2f(a1.x - m_all) : 0.f;
        const float l_all = a0.y * f0 + a1.y * f1;
        const float inv = (w.part < 0) ? (l_all > 0.f ? 1.f / l_all : 0.f) : 1.f;
        f0 *= inv;
        f1 *= inv;
        const int j = row / P.group, hg = row % P.group;
        // all MMAs of the item are complete, so its Q buffer is free: 4 KB of it per warp serve as transposition space
        float* stg = reinterpret_cast<float*>(smem + kOffQ + buf * kQBytes) + (warp - 4) * 1024;
        const int nrow = min(32, R - quad * 32);
#pragma unroll 1
        for (int cc = 0; cc < 2; ++cc) {
          const int c = 2 * g + cc;               // 32-dim chunk of the output row
          uint32_t r[32];
          tmem_ld32_nowait(lane_addr + kTmemO + c * 32, r);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f0);
          if (two) {
            uint32_t r1[32];
            tmem_ld32_nowait(lane_addr + kTmemO + D + c * 32, r1);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(fmaf(__uint_as_float(r1[i]), f1, __uint_as_float(r[i])));
          }
          if (w.part < 0) {
            if (rvalid) {
              uint4* dst = reinterpret_cast<uint4*>(P.o + ((size_t)(w.tok0 + j) * P.n_q + w.kv_head * P.group + hg) * D + c * 32);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                uint4 v;
                v.x = pack_bf16(__uint_as_float(r[8 * i]), __uint_as_float(r[8 * i + 1]));
                v.y = pack_bf16(__uint_as_float(r[8 * i + 2]), __uint_as_float(r[8 * i + 3]));
                v.z = pack_bf16(__uint_as_float(r[8 * i + 4]), __uint_as_float(r[8 * i + 5]));
                v.w = pack_bf16(__uint_as_float(r[8 * i + 6]), __uint_as_float(r[8 * i + 7]));
                dst[i] = v;
              }
            }
          } else {
            // fp32 partial rows: the thread's 32 values go to shared memory as eight 16-byte chunks (chunk q of row
            // `lane` at position q ^ (lane & 7): conflict free within every quarter warp, both ways); then each store
            // instruction writes four whole 128-byte row segments
            float4* s4 = reinterpret_cast<float4*>(stg);
#pragma unroll
            for (int q = 0; q < 8; ++q)
              s4[lane * 8 + (q ^ (lane & 7))] = make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]),
                                                            __uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3]));
            __syncwarp();
            const int rq = lane >> 3, q = lane & 7;
            float4* dst = reinterpret_cast<float4*>(P.part_o + ((size_t)w.part * 128 + quad * 32) * D + c * 32) + q;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int rr = 4 * j + rq;
              const float4 t = s4[rr * 8 + (q ^ (rr & 7))];
              if (rr < nrow) __stcg(dst + (size_t)rr * (D / 4), t);
            }
            __syncwarp();
          }
        }
        if (g == 0 && rvalid && w.part >= 0) {
          P.part_ml[((size_t)w.part * 128 + row) * 2 + 0] = m_all;
          P.part_ml[((size_t)w.part * 128 + row) * 2 + 1] = l_all;
        }
      }
      tc_fence_before();
      fence_proxy_async();    // the Q buffer goes back to the TMA unit
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(o_empty);
        mbar_arrive(&q_empty[buf]);
      }
      ++item_cnt;
      softmax_bar();          // the (max, sum) exchange area may be rewritten
    }
  }

  // this CTA's work is done: let the next kernel's CTAs be scheduled (they run their prologue and then wait for
  // this whole grid).  Signalling earlier would park their warps on the SMs while the softmax warps still need
  // every issue slot.
  griddep_launch();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---- host side: the tensor map over q -------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
struct QMapEntry {
  const void* q;
  int n_tok, n_q, group, device;
  CUtensorMap map;
};

// q is bf16 [n_tok][n_q][128]; box = 64 dims x group heads x (128 / group) tokens, 128-byte swizzle, zero fill.
// The map is copied out under a lock: contexts on several host threads share the small cache.
bool q_tensor_map(const void* q, int n_tok, int n_q, int group, CUtensorMap* out) {
  static std::mutex mu;
  static EncodeTiledFn encode = nullptr;
  static QMapEntry cache[16];
  static int n_cached = 0, next_slot = 0;
  int device = 0;
  cudaGetDevice(&device);   // an address means something else on another device
  std::lock_guard<std::mutex> lock(mu);
  for (int i = 0; i < n_cached; ++i)
    if (cache[i].q == q && cache[i].n_tok == n_tok && cache[i].n_q == n_q && cache[i].group == group &&
        cache[i].device == device) {
      *out = cache[i].map;
      return true;
    }
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn)
      return false;
    encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  QMapEntry& e = cache[next_slot];
  cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)n_q, (cuuint64_t)n_tok};
  cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)n_q * D * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)group, (cuuint32_t)(128 / group)};
  cuuint32_t estr[3] = {1, 1, 1};
  e.q = nullptr;   // the slot is invalid until the new map is in place
  if (encode(&e.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(q), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  e.q = q; e.n_tok = n_tok; e.n_q = n_q; e.group = group; e.device = device;
  next_slot = (next_slot + 1) % 16;
  if (n_cached < 16) ++n_cached;
  *out = e.map;
  return true;
}

}  // namespace

void launch_attention_tc_main(const BatchLayout& bl, const Dims& dm, int layer, const void* q, void* o,
                              const void* kv_pool, int64_t n_pages, float* part_o, float* part_ml, int n_sm, int* status,
                              cudaStream_t st, bool layout_settled) {
  static bool configured[kMaxDevices] = {false};
  if (first_use_on_device(configured))
    cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);

  TcAttnParams P;
  P.items = bl.items;
  P.cta_off = bl.cta_off;
  P.page_table = bl.page_table;
  P.pt_stride = bl.pt_stride;
  P.tok_climit = bl.tok_climit;
  P.tok_lo = bl.tok_lo;
  P.tok_hi = bl.tok_hi;
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
  P.early_desc = layout_settled ? 1 : 0;
  CUtensorMap qmap;
  if (!q_tensor_map(q, bl.n_tok, dm.n_q, P.group, &qmap)) {
    // nothing is launched; the status word makes the next recg_sync() fail instead of returning stale outputs
    fprintf(stderr, "recg: cannot encode the tensor map over q\n");
    static const int code = DEV_BAD_INDEX;
    if (status) cudaMemcpyAsync(status, &code, sizeof(int), cudaMemcpyHostToDevice, st);
    return;
  }
  launch_pdl(attention_tc_kernel, dim3(n_sm), dim3(kThreads), kSmemBytes, st, qmap, P);
}

}  // namespace recg

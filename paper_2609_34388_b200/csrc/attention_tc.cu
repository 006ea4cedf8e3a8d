// Hybrid-mask paged-KV attention on the 5th-generation tensor cores (head_dim 128).
//
// Work items are the same as in attention.cu: (request, kv head, row tile of <= 128 query rows, KV range).
// Per CTA (6 warps, one CTA per SM, persistent over the work list):
//   warp 0    producer: streams 128-token KV blocks page by page, ONE 4 KB bulk copy per page and operand,
//             into a ring of five 32 KB operand buffers (K and V of a block are separate entries, so K is
//             released early).  A page tile (8-row, 128-byte-swizzled atoms ordered [token group][dim half])
//             lands exactly as stored, and tiles copied back to back form one 128-token operand with a
//             uniform 2 KB stride between token groups: K-major for S = Q K^T, MN-major for O += P V.
//             The last, partly filled page of a request is copied by hand with the rows beyond its length
//             zeroed, so stale pool contents can never reach an accumulator.
//   warp 1    one elected lane issues tcgen05.mma: S = Q K^T (M 128 rows, N 128 tokens, K = d) into one
//             of two TMEM buffers, and O += P V (N = d, K = 128 tokens) into a third, which accumulates
//             over all blocks of the item.
//   warps 2-5 softmax, ONE THREAD PER QUERY ROW (= TMEM lane): the S row is read from TMEM once, the
//             probabilities are taken relative to a reference maximum that is only moved (and O rescaled
//             in TMEM) when the row maximum outgrows it by more than 2^8, and bf16 P is written to shared
//             memory in operand layout.  No cross-thread reductions are needed.  O is read once per item.
// Only blocks that reach past a row's visibility limit evaluate the mask.  Every wait is bounded.
#include "common.cuh"
#include "kernels.h"

namespace recg {

namespace {

constexpr int D = 128;
constexpr int kBT = 128;                       // tokens per KV block
constexpr int kPagesPerBT = kBT / kPageSize;   // 8
constexpr int kSubBytes = kPageSize * 128;     // 2 KB: [16 tokens][64 dims]
constexpr int kOperandHalf = kPagesPerBT * kSubBytes;  // 16 KB: one 64-wide half of a 128-token operand
constexpr int kQBytes = 128 * D * 2;           // 32 KB
constexpr int kPBytes = 128 * kBT * 2;         // 32 KB
constexpr int kTileBytes = 2 * kSubBytes;        // 4 KB: the K (or V) tile of one page and head, as stored in the pool
constexpr int kKVStageBytes = kPagesPerBT * kTileBytes;  // one operand (K or V) of a 128-token block: 32 KB
constexpr int kKVStages = 4;                     // ring K0 V0 K1 V1 K2 ...: a K buffer is free after Q K^T, a V buffer after P V
constexpr int kThreads = 224;                    // producer K, MMA, 4 softmax warps, producer V
constexpr uint32_t kSpin = 1u << 22;
constexpr int kTmemCols = 512;                 // S0 [0,128) S1 [128,256) O_blk [256,384)

constexpr int kOffQ = 0;
constexpr int kOffP = kOffQ + kQBytes;
constexpr int kOffKV = kOffP + 2 * kPBytes;    // P is double buffered: softmax of block n+1 overlaps P V of block n
constexpr int kOffBar = kOffKV + kKVStages * kKVStageBytes;
constexpr int kNumBars = 2 * kKVStages + 1 + 2 + 2 + 2 + 2 + 1 + 1;
constexpr int kSmemBytes = kOffBar + kNumBars * 8 + 16 + 1024;

struct TcAttnParams {
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
  float scale_log2;
  float* part_o;
  float* part_ml;
  int* status;
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

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void softmax_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

__global__ void __launch_bounds__(kThreads, 1) attention_tc_kernel(TcAttnParams P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kOffBar);
  uint64_t* kv_full = bars;                 // [kKVStages]
  uint64_t* kv_empty = bars + kKVStages;    // [kKVStages]
  uint64_t* q_full = bars + 2 * kKVStages;
  uint64_t* s_full = q_full + 1;            // [2]
  uint64_t* s_empty = q_full + 3;           // [2]
  uint64_t* p_full = q_full + 5;            // [2]
  uint64_t* p_empty = q_full + 7;           // [2]
  uint64_t* o_full = q_full + 9;
  uint64_t* o_empty = q_full + 10;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kNumBars);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kKVStages; ++s) {
      mbar_init(&kv_full[s], 1);
      mbar_init(&kv_empty[s], 1);
    }
    mbar_init(q_full, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&s_full[s], 1);
      mbar_init(&s_empty[s], 4);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&p_full[s], 4);
      mbar_init(&p_empty[s], 1);
    }
    mbar_init(o_full, 1);
    mbar_init(o_empty, 4);
    fence_barrier_init();
  }
  // The operand ring starts out zeroed: later on a buffer only ever holds zeros, real K/V pages or hand-copied
  // pages, so V rows that no copy refreshes (pages beyond a request's end) are finite and 0 * V stays 0.
  for (int c = threadIdx.x; c < kKVStages * kKVStageBytes / 16; c += kThreads)
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
  griddep_wait();   // everything above touched only shared memory and TMEM
  const int item_begin = P.cta_off[blockIdx.x], item_end = P.cta_off[blockIdx.x + 1];
  const uint32_t smem_base = smem_u32(smem);

  if (warp == 0 || warp == 6) {
    // ------------------------------------ producers: warp 0 streams K, warp 6 streams V ------------------------------------
    const int my_part = warp == 0 ? 0 : 1;
    uint32_t blk = 0;  // running KV-block counter
    bool ok = true;
    for (int item = item_begin; item < item_end && ok; ++item) {
      const AttnItem w = P.items[item];
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
      for (int n = 0; n < nblk && ok; ++n, ++blk) {
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
        const bool my_bulk = my_part == 0 ? my_valid > 0 : my_valid == kPageSize;
        const unsigned bulk_mask = __ballot_sync(0xffffffffu, my_bulk);
        const unsigned hand_mask = my_part == 0 ? 0u : __ballot_sync(0xffffffffu, my_valid > 0 && my_valid < kPageSize);
        for (int part = my_part; part <= my_part; ++part) {       // 0: the K operand, 1: the V operand
          const uint32_t qi = 2 * blk + part;
          const int s = qi % kKVStages;
          if (!mbar_wait(&kv_empty[s], ((qi / kKVStages) & 1) ^ 1, kSpin)) {
            set_status(P.status, DEV_TIMEOUT_EMPTY);
            ok = false;
            break;
          }
          uint8_t* stage = smem + kOffKV + s * kKVStageBytes;
          if (hand_mask) {
            const int p = __ffs(hand_mask) - 1;            // at most one partly filled page per request
            const int pg = __shfl_sync(0xffffffffu, my_pg, p);
            const int valid_tok = __shfl_sync(0xffffffffu, my_valid, p);
            const uint4* src = reinterpret_cast<const uint4*>(
                                   P.pool + kv_tile_base(P.n_pages, P.n_kv, D, P.layer, pg, w.kv_head)) + part * 256;
            uint4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const int c = u * 32 + lane;
              v[u] = (((c >> 7) * 8 + ((c >> 3) & 7)) < valid_tok) ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) *reinterpret_cast<uint4*>(stage + p * kTileBytes + (u * 32 + lane) * 16) = v[u];
          }
          if (hand_mask) fence_proxy_async();
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
    }
    if (!ok && lane == 0) {
      for (int s = 0; s < kKVStages; ++s)
        for (uint32_t i = 0; i < (1u << 14); ++i) {
          if (mbar_try_wait(&kv_full[s], 0) || mbar_try_wait(&kv_full[s], 1)) break;
          __nanosleep(64);
        }
    }
  } else if (warp == 1) {
    // ------------------------------------ MMA issuer ------------------------------------
    if (elect_one()) {
      uint32_t blk = 0, item_cnt = 0, pv_cnt = 0;
      bool ok = true;
      const uint32_t q_addr = smem_base + kOffQ, p_addr = smem_base + kOffP;
      auto issue_qk = [&](uint32_t b) -> bool {   // S[b & 1] = Q K^T for running block b
        const uint32_t qi = 2 * b;
        const int s = qi % kKVStages, sb = b & 1;
        if (!mbar_wait(&kv_full[s], (qi / kKVStages) & 1, kSpin)) { set_status(P.status, DEV_TIMEOUT_FULL); return false; }
        if (!mbar_wait(&s_empty[sb], ((b >> 1) & 1) ^ 1, kSpin)) { set_status(P.status, DEV_TIMEOUT_MMA); return false; }
        tc_fence_after();
        const uint32_t k_addr = smem_base + kOffKV + s * kKVStageBytes;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint64_t da = desc_kmajor(q_addr + (kk >> 2) * (128 * 128) + (kk & 3) * 32);
          // K block: 16 token groups (2 per page) 2 KB apart; the dim half selects the atom next door
          const uint64_t db = desc_kmajor(k_addr + (kk >> 2) * 1024 + (kk & 3) * 32, 2048);
          umma_bf16(tmem_base + sb * kBT, da, db, kIdescQK, kk ? 1u : 0u);
        }
        umma_commit(&kv_empty[s]);   // the K buffer is free once these MMAs have read it
        umma_commit(&s_full[sb]);
        return true;
      };
      for (int item = item_begin; item < item_end && ok; ++item, ++item_cnt) {
        const AttnItem w = P.items[item];
        const int tok_begin = w.blk_begin * 64;
        const int tok_end = min(w.blk_end * 64, w.kv_len);
        const int nblk = (tok_end - tok_begin + kBT - 1) / kBT;
        if (!mbar_wait(q_full, item_cnt & 1, kSpin)) { set_status(P.status, DEV_TIMEOUT_FULL); break; }
        // the previous item's O must have been read out before this item's first P V overwrites it
        if (!mbar_wait(o_empty, (item_cnt & 1) ^ 1, kSpin)) { set_status(P.status, DEV_TIMEOUT_MMA); break; }
        tc_fence_after();
        if (!(ok = issue_qk(blk))) break;
        for (int n = 0; n < nblk && ok; ++n, ++blk, ++pv_cnt) {
          if (n + 1 < nblk && !(ok = issue_qk(blk + 1))) break;
          // O (+)= P V for block n
          const int pb = pv_cnt & 1;
          if (!mbar_wait(&p_full[pb], (pv_cnt >> 1) & 1, kSpin)) {
            set_status(P.status, DEV_TIMEOUT_MMA);
            ok = false;
            break;
          }
          const uint32_t qv = 2 * blk + 1;
          const int s = qv % kKVStages;
          if (!mbar_wait(&kv_full[s], (qv / kKVStages) & 1, kSpin)) {
            set_status(P.status, DEV_TIMEOUT_FULL);
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t v_addr = smem_base + kOffKV + s * kKVStageBytes;
#pragma unroll
          for (int kk = 0; kk < kBT / 16; ++kk) {
            const uint64_t da = desc_kmajor(p_addr + pb * kPBytes + (kk >> 2) * (128 * 128) + (kk & 3) * 32);
            // tokens [16 kk, 16 kk + 16) = page kk: two token groups 2 KB apart, the dim halves 1 KB apart
            const uint64_t db = desc_mnmajor(v_addr + kk * kTileBytes, 1024, 2048);
            umma_bf16(tmem_base + 2 * kBT, da, db, kIdescPV, (n | kk) ? 1u : 0u);
          }
          umma_commit(&kv_empty[s]);
          umma_commit(&p_empty[pb]);
          if (n == nblk - 1) umma_commit(o_full);
        }
      }
    }
  } else if (warp < 6) {
    // ------------------------------------ softmax ------------------------------------
    const int quad = warp & 3;
    const int row = quad * 32 + lane;          // query row of the tile = TMEM lane
    const int sthread = (warp - 2) * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    uint32_t blk = 0, pv_cnt = 0, item_cnt = 0;
    bool ok = true;
    for (int item = item_begin; item < item_end && ok; ++item) {
      const AttnItem w = P.items[item];
      const int R = w.ntok * P.group;
      const int tok_begin = w.blk_begin * 64;
      const int tok_end = min(w.blk_end * 64, w.kv_len);
      const int nblk = (tok_end - tok_begin + kBT - 1) / kBT;
      // ---- stage Q in operand layout: [2 halves][128 rows][128 B], 16-byte chunks swizzled by row & 7 ----
      // only the R valid rows are staged: the other rows of the M = 128 operand yield S / O rows nobody reads.
      // Loads are issued in batches of 8 before any store so that their latencies overlap.
      for (int c0 = 0; c0 < R * 16; c0 += 128 * 8) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int c = c0 + u * 128 + sthread;
          v[u] = make_uint4(0, 0, 0, 0);
          if (c < R * 16) {
            const int r = c >> 4, ch = c & 15;
            const int j = r / P.group, hg = r % P.group;
            v[u] = __ldg(reinterpret_cast<const uint4*>(P.q + ((size_t)(w.tok0 + j) * P.n_q + w.kv_head * P.group + hg) * D) + ch);
          }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int c = c0 + u * 128 + sthread;
          if (c < R * 16) {
            const int r = c >> 4, ch = c & 15;
            *reinterpret_cast<uint4*>(smem + kOffQ + (ch >> 3) * (128 * 128) + r * 128 + (((ch & 7) ^ (r & 7)) << 4)) = v[u];
          }
        }
      }
      fence_proxy_async();
      softmax_bar();
      if (sthread == 0) mbar_arrive(q_full);

      const bool rvalid = row < R;
      const bool warp_valid = quad * 32 < R;
      int climit = -1, vlo = 0, vhi = 0;
      if (rvalid) {
        const int t = w.tok0 + row / P.group;
        climit = P.tok_climit[t];
        vlo = P.tok_lo[t];
        vhi = P.tok_hi[t];
      }
      float m_ref = -1e30f, l_run = 0.f;
      const uint32_t p_row0 = smem_base + kOffP + row * 128;

      for (int n = 0; n < nblk && ok; ++n, ++blk, ++pv_cnt) {
        const int sb = blk & 1;
        if (!mbar_wait(&s_full[sb], (blk >> 1) & 1, kSpin)) { set_status(P.status, DEV_TIMEOUT_MMA); ok = false; break; }
        tc_fence_after();
        const int pos0 = tok_begin + n * kBT;
        uint32_t sr[4][32];   // the S row of this thread: 128 scores
        float mx = -INFINITY;
        bool need_mask = false;
        if (warp_valid) {
#pragma unroll
          for (int c = 0; c < 4; ++c) tmem_ld32_nowait(lane_addr + sb * kBT + c * 32, sr[c]);
          tmem_ld_wait();
          const int lim = min(climit, tok_end - 1);
          need_mask = __any_sync(0xffffffffu, rvalid && (pos0 + kBT - 1 > lim));
          if (need_mask) {
            // visible tokens of this row within the block: [0, a] and [b, c), as a 128-bit mask over tokens
            const int a = lim - pos0, b = vlo - pos0, cc = min(vhi, tok_end) - pos0;
            auto ones = [](int n) -> unsigned long long {      // n lowest bits set, n clamped to [0, 64]
              return n <= 0 ? 0ull : (n >= 64 ? ~0ull : ((1ull << n) - 1ull));
            };
            const unsigned long long m0 = ones(a + 1) | (ones(cc) & ~ones(b));
            const unsigned long long m1 = ones(a + 1 - 64) | (ones(cc - 64) & ~ones(b - 64));
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
              for (int i = 0; i < 32; ++i) {
                const int t = col_token(c * 32 + i);        // compile-time constant after unrolling
                const bool vis = ((t < 64 ? (m0 >> t) : (m1 >> (t - 64))) & 1ull) != 0ull;
                if (!vis) sr[c][i] = 0xff800000u;   // -inf
              }
          }
          {  // four independent chains instead of one 128-long dependent one
            float mxa[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
              for (int i = 0; i < 32; i += 2)
                mxa[c] = fmaxf(mxa[c], fmaxf(__uint_as_float(sr[c][i]), __uint_as_float(sr[c][i + 1])));
            mx = fmaxf(fmaxf(mxa[0], mxa[1]), fmaxf(mxa[2], mxa[3]));
          }
        }
        // S has been read: the MMA warp may overwrite this buffer with the block after next
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&s_empty[sb]);
        // the P V that last read this P buffer (two blocks ago) must be complete before it is overwritten
        const int pb = pv_cnt & 1;
        const uint32_t p_row = p_row0 + pb * kPBytes;
        if (!mbar_wait(&p_empty[pb], ((pv_cnt >> 1) & 1) ^ 1, kSpin)) { set_status(P.status, DEV_TIMEOUT_MMA); ok = false; break; }
        if (warp_valid) {
          const float m_blk = mx * P.scale_log2;
          // move the reference maximum only when the row maximum outgrows it by more than 2^8 (or at the first
          // block): probabilities stay below 256 relative to the reference, well inside bf16 and fp32 range
          const bool grow = rvalid && (m_blk > m_ref + 8.f);
          if (n == 0) {
            if (rvalid && m_blk > m_ref) m_ref = m_blk;
          } else if (__any_sync(0xffffffffu, grow)) {
            // rare: O is rescaled in TMEM, which needs EVERY earlier P V complete (the previous one may still run)
            if (!mbar_wait(&p_empty[pb ^ 1], (((pv_cnt - 1) >> 1) & 1), kSpin)) { set_status(P.status, DEV_TIMEOUT_MMA); ok = false; break; }
            const float m_new = grow ? m_blk : m_ref;
            const float f = exp2f(m_ref - m_new);
            m_ref = m_new;
            l_run *= f;
            tc_fence_after();
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
              uint32_t r[32];
              tmem_ld32_nowait(lane_addr + 2 * kBT + c * 32, r);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f);
              tmem_st32(lane_addr + 2 * kBT + c * 32, r);
            }
            tmem_st_wait();
          }
          float lsa[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int c = 0; c < 4; ++c) {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const float p = exp2f(__uint_as_float(sr[c][i]) * P.scale_log2 - m_ref);   // exp2(-inf) = 0 for masked
              sr[c][i] = __float_as_uint(p);
              lsa[i & 3] += p;
            }
            if (rvalid) {
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int ch = c * 4 + j;   // 16-byte chunk (8 tokens) of the row: half = ch >> 3
                st_shared_v4(p_row + (ch >> 3) * (128 * 128) + (((ch & 7) ^ (row & 7)) << 4),
                             pack_bf16(__uint_as_float(sr[c][8 * j]), __uint_as_float(sr[c][8 * j + 1])),
                             pack_bf16(__uint_as_float(sr[c][8 * j + 2]), __uint_as_float(sr[c][8 * j + 3])),
                             pack_bf16(__uint_as_float(sr[c][8 * j + 4]), __uint_as_float(sr[c][8 * j + 5])),
                             pack_bf16(__uint_as_float(sr[c][8 * j + 6]), __uint_as_float(sr[c][8 * j + 7])));
              }
            }
          }
          l_run += (lsa[0] + lsa[1]) + (lsa[2] + lsa[3]);
        }
        tc_fence_before();
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[pb]);
      }
      if (!ok) break;

      // ---- read O once, write out: one row per thread ----
      if (!mbar_wait(o_full, item_cnt & 1, kSpin)) { set_status(P.status, DEV_TIMEOUT_MMA); ok = false; break; }
      tc_fence_after();
      if (warp_valid) {
        const int j = row / P.group, hg = row % P.group;
        const float inv = (w.part < 0) ? (l_run > 0.f ? 1.f / l_run : 0.f) : 1.f;
#pragma unroll 1
        for (int c = 0; c < D / 32; ++c) {
          uint32_t r[32];
          tmem_ld32_nowait(lane_addr + 2 * kBT + c * 32, r);
          tmem_ld_wait();
          if (!rvalid) continue;
          if (w.part < 0) {
            uint4* dst = reinterpret_cast<uint4*>(P.o + ((size_t)(w.tok0 + j) * P.n_q + w.kv_head * P.group + hg) * D + c * 32);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              uint4 v;
              v.x = pack_bf16(__uint_as_float(r[8 * i]) * inv, __uint_as_float(r[8 * i + 1]) * inv);
              v.y = pack_bf16(__uint_as_float(r[8 * i + 2]) * inv, __uint_as_float(r[8 * i + 3]) * inv);
              v.z = pack_bf16(__uint_as_float(r[8 * i + 4]) * inv, __uint_as_float(r[8 * i + 5]) * inv);
              v.w = pack_bf16(__uint_as_float(r[8 * i + 6]) * inv, __uint_as_float(r[8 * i + 7]) * inv);
              dst[i] = v;
            }
          } else {
            uint4* dst = reinterpret_cast<uint4*>(P.part_o + ((size_t)w.part * 128 + row) * D + c * 32);
#pragma unroll
            for (int i = 0; i < 8; ++i) dst[i] = make_uint4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
          }
        }
        if (rvalid && w.part >= 0) {
          P.part_ml[((size_t)w.part * 128 + row) * 2 + 0] = m_ref;
          P.part_ml[((size_t)w.part * 128 + row) * 2 + 1] = l_run;
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(o_empty);
      ++item_cnt;
      // all MMAs of this item have completed (the last o_full tracked them), so Q may be restaged
      softmax_bar();
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

}  // namespace

void launch_attention_tc_main(const BatchLayout& bl, const Dims& dm, int layer, const void* q, void* o,
                              const void* kv_pool, int64_t n_pages, float* part_o, float* part_ml, int n_sm, int* status,
                              cudaStream_t st) {
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    configured = true;
  }
  TcAttnParams P;
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
  launch_pdl(attention_tc_kernel, dim3(n_sm), dim3(kThreads), kSmemBytes, st, P);
}

}  // namespace recg

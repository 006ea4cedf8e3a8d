// A chain of projections in ONE persistent kernel, for steps with few rows (low concurrency).
//
// With at most 128 rows every projection of a layer is bound by streaming its weights, and a kernel of its own per
// projection spends 7-9 us on launch, prologue, the first operand round trip, the hand-over of cut tiles and the drain,
// during which HBM idles.  Here the projections between two attention calls -- output projection, gate|up, down, and the
// QKV projection of the next layer (or the LM head) -- run as one grid of one CTA per SM, and the weight stream never
// stops: the producer warp requests the weight tiles of the next projection as soon as ring slots free up, across the
// grid-wide barriers that separate the projections.
//
// Per projection ("op"):
//   phase A  the k-blocks of all column tiles (128 accumulator columns each) form one line that is cut into equal ranges,
//            one per CTA, so every CTA streams the same number of weight bytes.  A CTA's range touches one to a few
//            column tiles; for each it accumulates its K range in TMEM (tcgen05.mma, M = 128, N = 128) and parks the rows
//            that exist as an fp32 partial tile in a workspace slot;
//   barrier  all CTAs have parked (grid-wide: one counter in global memory, bounded polling);
//   phase B  the column tiles are dealt out over the CTAs; the four epilogue warps of a CTA add the partial tiles of its
//            tiles in part order (deterministic) and apply the epilogue: residual add with the next RMSNorm's input and
//            row sums of squares, SwiGLU, rotary embedding + paged K/V append, or a plain store, each with the row's
//            RMSNorm factor where the input was an un-normalised residual stream (see EpiParams in epilogue.cuh);
//   barrier  all outputs are written: the next projection may load them as its A operand.
// The A operand of the next projection is only requested after the second barrier, its weight tiles long before.
//
// All CTAs of the grid must be resident at the same time (the grid is one CTA per SM and a CTA takes an SM's shared
// memory, so they are once the kernels before this one have drained); every wait is bounded and a wait that runs out
// sets the status word, after which nothing in this CTA blocks any more.
#include <cuda.h>

#include "common.cuh"
#include "epilogue.cuh"
#include "kernels.h"
#include "tc_ptx.cuh"

namespace recg {

namespace {

using namespace tc;

constexpr int BN = 128, BK = 64;
constexpr int kThreads = 192;
constexpr int kRing = 192 * 1024;
constexpr int kMaxStages = 12;
constexpr uint32_t kSpin = 1u << 22;
constexpr uint32_t kGridSpin = 1u << 18;     // polls of the grid barrier, each a round trip to L2 (0.5 - 1 us): at least 0.1 s

struct ChainMaps {
  CUtensorMap x[kChainMaxOps];
  CUtensorMap w[kChainMaxOps];
};

struct ChainDev {            // what the kernel needs of a ChainOp
  int N, K, epi, up_row_offset, scale_in, ss_slots_in;
  void* out;
  void* x_out;
  const __nv_bfloat16* gain;
};

struct ChainParams {
  int n_ops, M, m_pad, a_rows;     // rows, rows padded to 32 / 64 / 128, rows of the A operand's TMA box (32 or 128)
  ChainDev op[kChainMaxOps];
  float* ss;
  int ss_stride;
  float eps;
  float* ws;
  unsigned* bar;
  unsigned bar_base;
  const int* tok_slot;
  const float2* rope_cs;
  __nv_bfloat16* kv_pool;
  int64_t n_pages;
  int layer, n_q, n_kv, head_dim;
  int* status;
};

// the stream-K line of one op
struct OpSched {
  int n_tiles, KB, per, max_pieces;
  long long total;
};
__device__ __forceinline__ OpSched op_sched(const ChainDev& o, int grid) {
  OpSched s;
  const int out_per_tile = o.epi == EPI_SWIGLU ? BN / 2 : BN;
  s.n_tiles = (o.N + out_per_tile - 1) / out_per_tile;
  s.KB = o.K / BK;
  s.total = (long long)s.n_tiles * s.KB;
  s.per = (int)((s.total + grid - 1) / grid);
  s.max_pieces = s.per / s.KB + 2;
  return s;
}

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

__global__ void __launch_bounds__(kThreads, 1) gemm_chain_kernel(const __grid_constant__ ChainMaps maps, const ChainParams P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int a_bytes = P.a_rows * BK * 2;
  const int stage_bytes = a_bytes + BN * BK * 2;
  const int n_stages = kRing / stage_bytes > kMaxStages ? kMaxStages : kRing / stage_bytes;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + kRing);
  uint64_t* empty_bar = full_bar + kMaxStages;
  uint64_t* tfull_bar = empty_bar + kMaxStages;
  uint64_t* tempty_bar = tfull_bar + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + 2);
  __shared__ volatile int s_abort;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, grid = gridDim.x;

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&tfull_bar[a], 1);
      mbar_init(&tempty_bar[a], 4);
    }
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 2 * BN);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // grid barrier k is passed when the counter has reached base + (k + 1) * grid (wrap-around safe)
  auto barrier_passed = [&](int k) -> bool {
    const unsigned target = P.bar_base + (unsigned)(k + 1) * (unsigned)grid;
    return (int)(ld_acquire(P.bar) - target) >= 0;
  };
  auto barrier_wait = [&](int k) -> bool {       // bounded; false (and the CTA-wide flag) when it gives up
    if (s_abort) return false;
    for (uint32_t i = 0; i < kGridSpin; ++i) {
      if (barrier_passed(k)) return true;
    }
    set_status(P.status, DEV_TIMEOUT_FULL);
    s_abort = 1;
    return false;
  };

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (elect_one()) {
      struct Pending { int stage, kb, op; };
      Pending pend[kMaxStages];
      int p_head = 0, p_tail = 0;          // (indices grow; slot = index % kMaxStages)
      int ready_op = -1;                   // A operands of ops <= ready_op may be loaded
      bool waited_dep = false;
      // mode 0: while slots are free (the weights keep going out); 1: no slot is free; 2: everything has been requested
      auto ready = [&](int op, int mode) -> bool {
        if (op <= ready_op) return true;
        if (op == 0) {                     // the first A operand comes from the kernels before this one: wait for them only
          if (mode == 0) return false;     // when nothing else can be requested (the ring fills with weights meanwhile)
          if (!waited_dep) {
            griddep_wait();
            waited_dep = true;
          }
          ready_op = 0;
          return true;
        }
        const int k = 2 * (op - 1) + 1;    // outputs of the previous op are written
        if (mode == 2 ? barrier_wait(k) : barrier_passed(k)) {
          ready_op = op;
          return true;
        }
        return false;
      };
      auto flush = [&](int mode) {
        while (p_head != p_tail) {
          const Pending& q = pend[p_head % kMaxStages];
          if (!ready(q.op, mode)) break;
          tma_load_2d(smem + q.stage * stage_bytes, &maps.x[q.op], q.kb * BK, 0, &full_bar[q.stage]);
          ++p_head;
        }
      };
      int st_idx = 0;
      uint32_t st_phase = 0;
      bool ok = true;
      for (int op = 0; op < P.n_ops && ok; ++op) {
        const ChainDev& o = P.op[op];
        const OpSched sc = op_sched(o, grid);
        const long long lo = (long long)cta * sc.per < sc.total ? (long long)cta * sc.per : sc.total;
        const long long hi = lo + sc.per < sc.total ? lo + sc.per : sc.total;
        const bool swiglu = o.epi == EPI_SWIGLU;
        for (long long u = lo; u < hi && ok; ++u) {
          const int tile = (int)(u / sc.KB), kb = (int)(u - (long long)tile * sc.KB);
          const int s = st_idx;
          const uint32_t ph = st_phase;
          if (++st_idx == n_stages) { st_idx = 0; st_phase ^= 1; }
          uint32_t spins = 0;
          while (!mbar_try_wait(&empty_bar[s], ph ^ 1)) {      // a free slot; meanwhile A operands that became loadable go out
            flush(1);
            if (s_abort || ++spins > kSpin) {
              if (!s_abort) set_status(P.status, DEV_TIMEOUT_EMPTY);
              s_abort = 1;
              ok = false;
              break;
            }
            if (spins > 64) __nanosleep(32);
          }
          if (!ok) break;
          mbar_arrive_expect_tx(&full_bar[s], stage_bytes);
          uint8_t* b_dst = smem + s * stage_bytes + a_bytes;
          if (swiglu) {
            tma_load_2d(b_dst, &maps.w[op], kb * BK, tile * (BN / 2), &full_bar[s]);
            tma_load_2d(b_dst + BN * BK, &maps.w[op], kb * BK, o.up_row_offset + tile * (BN / 2), &full_bar[s]);
          } else {
            tma_load_2d(b_dst, &maps.w[op], kb * BK, tile * BN, &full_bar[s]);
          }
          pend[p_tail % kMaxStages] = Pending{s, kb, op};
          ++p_tail;
          flush(0);
        }
      }
      if (ok) flush(2);
      if (!ok || s_abort) {   // let loads already issued land before the CTA may exit
        for (int s = 0; s < n_stages; ++s)
          for (uint32_t i = 0; i < (1u << 14); ++i) {
            if (mbar_try_wait(&full_bar[s], 0) || mbar_try_wait(&full_bar[s], 1)) break;
            __nanosleep(64);
          }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (elect_one()) {
      constexpr uint32_t idesc = make_idesc(BN, 128);
      const uint64_t desc0 = make_smem_desc(smem_u32(smem));
      int st_idx = 0;
      uint32_t st_phase = 0, tcount = 0;
      bool ok = true;
      for (int op = 0; op < P.n_ops && ok; ++op) {
        const OpSched sc = op_sched(P.op[op], grid);
        const long long lo = (long long)cta * sc.per < sc.total ? (long long)cta * sc.per : sc.total;
        const long long hi = lo + sc.per < sc.total ? lo + sc.per : sc.total;
        for (long long u = lo; u < hi && ok; ++tcount) {
          const int tile = (int)(u / sc.KB);
          const long long t_end = (long long)(tile + 1) * sc.KB;
          const long long u_end = hi < t_end ? hi : t_end;
          const int acc = tcount & 1;
          if (!mbar_wait(&tempty_bar[acc], ((tcount >> 1) & 1) ^ 1, kSpin)) {
            set_status(P.status, DEV_TIMEOUT_MMA);
            s_abort = 1;
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + acc * BN;
          bool first = true;
          for (; u < u_end; ++u) {
            const int s = st_idx;
            const uint32_t ph = st_phase;
            if (++st_idx == n_stages) { st_idx = 0; st_phase ^= 1; }
            if (!mbar_wait(&full_bar[s], ph, kSpin)) {
              set_status(P.status, DEV_TIMEOUT_FULL);
              s_abort = 1;
              ok = false;
              break;
            }
            tc_fence_after();
            const uint64_t da0 = desc0 + (uint64_t)((s * stage_bytes) >> 4);
            const uint64_t db0 = da0 + (uint64_t)(a_bytes >> 4);
#pragma unroll
            for (int k = 0; k < BK / 16; ++k) {
              umma_bf16(d_tmem, da0 + 2 * k, db0 + 2 * k, idesc, (first && k == 0) ? 0u : 1u);
            }
            first = false;
            umma_commit(&empty_bar[s]);
          }
          if (ok) umma_commit(&tfull_bar[acc]);
        }
      }
    }
  } else {
    // ------------------------------ epilogue warps ------------------------------
    const int quad = warp & 3;                 // TMEM lane quadrant this warp may read
    const int e = threadIdx.x - 64;            // 0 .. 127
    const int tpr = 128 / P.m_pad;             // threads per row in phase B: 4, 2 or 1
    const int b_row = e / tpr, b_q = e % tpr;
    uint32_t tcount = 0;
    griddep_wait();
    auto ewait = [&](uint64_t* bar, uint32_t parity) {
      if (s_abort) return;
      if (!mbar_wait(bar, parity, kSpin)) {
        set_status(P.status, DEV_TIMEOUT_MMA);
        s_abort = 1;
      }
    };
    for (int op = 0; op < P.n_ops; ++op) {
      const ChainDev& o = P.op[op];
      const OpSched sc = op_sched(o, grid);
      const size_t slot_floats = (size_t)P.m_pad * BN;
      // ---- phase A: park the partial tiles of this CTA's pieces ----
      {
        const long long lo = (long long)cta * sc.per < sc.total ? (long long)cta * sc.per : sc.total;
        const long long hi = lo + sc.per < sc.total ? lo + sc.per : sc.total;
        const int first_tile = (int)(lo / sc.KB);
        for (long long u = lo; u < hi; ++tcount) {
          const int tile = (int)(u / sc.KB);
          const long long t_end = (long long)(tile + 1) * sc.KB;
          u = hi < t_end ? hi : t_end;
          const int acc = tcount & 1;
          ewait(&tfull_bar[acc], (tcount >> 1) & 1);
          tc_fence_after();
          const int row = quad * 32 + lane;
          float* dst = P.ws + ((size_t)cta * sc.max_pieces + (tile - first_tile)) * slot_floats + (size_t)row * BN;
          if (quad * 32 < P.m_pad) {           // (warp-uniform: every lane of the warp takes part in the TMEM loads)
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
              float v[32];
              tmem_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + acc * BN + c * 32, v);
              if (row < P.M) {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                  __stcg(reinterpret_cast<float4*>(dst + c * 32) + i, make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]));
              }
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tempty_bar[acc]);
        }
      }
      // ---- grid barrier: everybody has parked ----
      // One counter serves all barriers, so no CTA may arrive at barrier k + 1 before barrier k has been passed: a CTA
      // whose range of this op is empty gets here without having waited for the previous op's outputs, and its early
      // arrival would let the previous barrier pass with a slower CTA still missing.
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (e == 0) {
        if (op > 0) barrier_wait(2 * op - 1);
        __threadfence();
        atomicAdd(P.bar, 1u);
      }
      if (lane == 0) {
        barrier_wait(2 * op);
        __threadfence();
      }
      __syncwarp();
      // ---- phase B: this CTA's column tiles: add the parts in part order, apply the epilogue ----
      // the row's RMSNorm factor: the slots are added in a fixed grouping (the tpr threads of a row take every tpr-th
      // slot, eight loads in flight each, then the threads' sums are added by shuffles), the same in every CTA
      float rstd = 1.f;
      if (o.scale_in) {
        float sq = 0.f;
        if (b_row < P.M) {
          for (int k0 = b_q; k0 < o.ss_slots_in; k0 += 8 * tpr) {
            float t[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int k = k0 + j * tpr;
              t[j] = k < o.ss_slots_in ? __ldcg(P.ss + (size_t)k * P.ss_stride + b_row) : 0.f;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) sq += t[j];
          }
        }
        for (int off = 1; off < tpr; off <<= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
        rstd = rsqrtf(sq / (float)o.K + P.eps);
      }
      for (int tile = cta; tile < sc.n_tiles; tile += grid) {
        const long long t0 = (long long)tile * sc.KB, t1 = t0 + sc.KB;
        const int c_first = (int)(t0 / sc.per), c_last = (int)((t1 - 1) / sc.per);
        float ssum = 0.f;
#pragma unroll 1
        for (int pc = b_q; pc < 4; pc += tpr) {          // pair chunk: tile columns [16 pc, 16 pc + 16) and 64 + the same
          float lo[16], hi[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) lo[i] = hi[i] = 0.f;
          if (b_row < P.M) {
            // parts are added in part order; the loads of two parts are in flight together
            for (int c = c_first; c <= c_last; c += 2) {
              float4 a[2][4], b[2][4];
#pragma unroll
              for (int u = 0; u < 2; ++u) {
                const int cc = c + u;
                const bool on = cc <= c_last;
                const int piece = tile - (int)(((long long)cc * sc.per) / sc.KB);
                const float* src = P.ws + ((size_t)(on ? cc : c) * sc.max_pieces + (on ? piece : 0)) * slot_floats + (size_t)b_row * BN + 16 * pc;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  a[u][i] = on ? __ldcg(reinterpret_cast<const float4*>(src) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                  b[u][i] = on ? __ldcg(reinterpret_cast<const float4*>(src + 64) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
              }
#pragma unroll
              for (int u = 0; u < 2; ++u)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  lo[4 * i] += a[u][i].x; lo[4 * i + 1] += a[u][i].y; lo[4 * i + 2] += a[u][i].z; lo[4 * i + 3] += a[u][i].w;
                  hi[4 * i] += b[u][i].x; hi[4 * i + 1] += b[u][i].y; hi[4 * i + 2] += b[u][i].z; hi[4 * i + 3] += b[u][i].w;
                }
            }
          }
          if (b_row >= P.M) continue;
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            lo[i] *= rstd;
            hi[i] *= rstd;
          }
          const int m = b_row;
          if (o.epi == EPI_RESIDUAL_NORM) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              float* v = half ? hi : lo;
              const int n = tile * BN + 64 * half + 16 * pc;
              if (n >= o.N) continue;
              float* hp = static_cast<float*>(o.out) + (size_t)m * o.N + n;
              uint32_t xo[8];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                float4 h = __ldcg(reinterpret_cast<const float4*>(hp) + i);
                h.x += v[4 * i]; h.y += v[4 * i + 1]; h.z += v[4 * i + 2]; h.w += v[4 * i + 3];
                reinterpret_cast<float4*>(hp)[i] = h;
                ssum = fmaf(h.x, h.x, fmaf(h.y, h.y, fmaf(h.z, h.z, fmaf(h.w, h.w, ssum))));
                const uint2 g = __ldg(reinterpret_cast<const uint2*>(o.gain + n) + i);
                xo[2 * i] = pack_bf16(h.x * __uint_as_float(g.x << 16), h.y * __uint_as_float(g.x & 0xffff0000u));
                xo[2 * i + 1] = pack_bf16(h.z * __uint_as_float(g.y << 16), h.w * __uint_as_float(g.y & 0xffff0000u));
              }
              uint4* xp = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(o.x_out) + (size_t)m * o.N + n);
              xp[0] = make_uint4(xo[0], xo[1], xo[2], xo[3]);
              xp[1] = make_uint4(xo[4], xo[5], xo[6], xo[7]);
            }
          } else if (o.epi == EPI_SWIGLU) {
            const int n = tile * (BN / 2) + 16 * pc;
            if (n < o.N) {
              uint32_t a[8];
#pragma unroll
              for (int i = 0; i < 8; ++i)
                a[i] = pack_bf16(silu_f(lo[2 * i]) * hi[2 * i], silu_f(lo[2 * i + 1]) * hi[2 * i + 1]);
              uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(o.out) + (size_t)m * o.N + n);
              dst[0] = make_uint4(a[0], a[1], a[2], a[3]);
              dst[1] = make_uint4(a[4], a[5], a[6], a[7]);
            }
          } else if (o.epi == EPI_QKV_ROPE) {
            const int head = tile;             // one head per tile: head_dim = 128
            const bool is_q = head < P.n_q, is_v = head >= P.n_q + P.n_kv;
            if (!is_v) {
              const float2* cs = P.rope_cs + (size_t)(16 * pc) * P.M + m;      // [frequency][token]
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                const float2 t = cs[(size_t)i * P.M];
                const float a = lo[i] * t.x - hi[i] * t.y, b = hi[i] * t.x + lo[i] * t.y;
                lo[i] = a;
                hi[i] = b;
              }
            }
            uint4 pl[2], phh[2];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
              pl[j] = make_uint4(pack_bf16(lo[8 * j], lo[8 * j + 1]), pack_bf16(lo[8 * j + 2], lo[8 * j + 3]),
                                 pack_bf16(lo[8 * j + 4], lo[8 * j + 5]), pack_bf16(lo[8 * j + 6], lo[8 * j + 7]));
              phh[j] = make_uint4(pack_bf16(hi[8 * j], hi[8 * j + 1]), pack_bf16(hi[8 * j + 2], hi[8 * j + 3]),
                                  pack_bf16(hi[8 * j + 4], hi[8 * j + 5]), pack_bf16(hi[8 * j + 6], hi[8 * j + 7]));
            }
            if (is_q) {
              uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(o.out) + ((size_t)m * P.n_q + head) * 128 + 16 * pc);
              dst[0] = pl[0];
              dst[1] = pl[1];
              dst[8] = phh[0];                 // + 64 elements
              dst[9] = phh[1];
            } else {
              const int slot = P.tok_slot[m];
              if (slot >= 0) {
                const int64_t page = slot / kPageSize;
                if (page < P.n_pages) {
                  const int kvh = is_v ? head - P.n_q - P.n_kv : head - P.n_q;
                  __nv_bfloat16* base = P.kv_pool + kv_tile_base(P.n_pages, P.n_kv, 128, P.layer, page, kvh) +
                                        (is_v ? kv_tile_elems(128) : 0);
                  const int tok = slot % kPageSize;
#pragma unroll
                  for (int j = 0; j < 2; ++j) {
                    *reinterpret_cast<uint4*>(base + kv_tile_offset(tok, 16 * pc + 8 * j, 128)) = pl[j];
                    *reinterpret_cast<uint4*>(base + kv_tile_offset(tok, 64 + 16 * pc + 8 * j, 128)) = phh[j];
                  }
                } else {
                  set_status(P.status, DEV_BAD_INDEX);
                }
              }
            }
          } else {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const float* v = half ? hi : lo;
              const int n = tile * BN + 64 * half + 16 * pc;
              if (n >= o.N) continue;
              if (o.epi == EPI_PLAIN_F32) {
                float4* dst = reinterpret_cast<float4*>(static_cast<float*>(o.out) + (size_t)m * o.N + n);
#pragma unroll
                for (int i = 0; i < 4; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
              } else {
                uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(o.out) + (size_t)m * o.N + n);
                dst[0] = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
                dst[1] = make_uint4(pack_bf16(v[8], v[9]), pack_bf16(v[10], v[11]), pack_bf16(v[12], v[13]), pack_bf16(v[14], v[15]));
              }
            }
          }
        }
        if (o.epi == EPI_RESIDUAL_NORM) {
          // the row's sum of squares over this tile: the tpr threads of a row are neighbours in the warp
          for (int off = 1; off < tpr; off <<= 1) ssum += __shfl_xor_sync(0xffffffffu, ssum, off);
          if (b_q == 0 && b_row < P.M) P.ss[(size_t)tile * P.ss_stride + b_row] = ssum;
        }
      }
      // ---- grid barrier: the outputs of this op are written ----
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (e == 0) {
        __threadfence();
        atomicAdd(P.bar, 1u);
      }
    }
  }

  griddep_launch();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 2 * BN);
  }
}

// ---- host side ---------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct ChainState {
  int n_sm = 0;
  EncodeTiledFn encode = nullptr;
  float* ws = nullptr;
  size_t ws_bytes = 0;
  unsigned* bar = nullptr;
  unsigned bar_base = 0;
  bool configured = false;
};

bool encode_map(ChainState* st, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows, CUtensorMap* out) {
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {BK, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return st->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kSmemBytes = kRing + (2 * kMaxStages + 4) * 8 + 16 + 1024;

}  // namespace

void* chain_state_create(int n_sm) {
  ChainState* st = new ChainState();
  st->n_sm = n_sm;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn) {
    delete st;
    return nullptr;
  }
  st->encode = reinterpret_cast<EncodeTiledFn>(fn);
  if (cudaMalloc(reinterpret_cast<void**>(&st->bar), 256) != cudaSuccess || cudaMemset(st->bar, 0, 256) != cudaSuccess) {
    delete st;
    return nullptr;
  }
  return st;
}

void chain_state_destroy(void* s) {
  ChainState* st = static_cast<ChainState*>(s);
  if (!st) return;
  if (st->ws) cudaFree(st->ws);
  if (st->bar) cudaFree(st->bar);
  delete st;
}

void chain_state_reset(void* s, cudaStream_t stream) {
  ChainState* st = static_cast<ChainState*>(s);
  if (!st) return;
  cudaMemsetAsync(st->bar, 0, 256, stream);
  st->bar_base = 0;
}

// workspace for the largest op of the model at this row count: (SMs) x (pieces per CTA) x (padded rows x 128 floats)
bool chain_state_reserve(void* s, int max_rows, long long max_total_kblocks, int min_kb) {
  ChainState* st = static_cast<ChainState*>(s);
  if (!st) return false;
  const int m_pad = max_rows <= 32 ? 32 : (max_rows <= 64 ? 64 : 128);
  const long long per = (max_total_kblocks + st->n_sm - 1) / st->n_sm;
  const long long pieces = per / min_kb + 2;
  const size_t need = (size_t)st->n_sm * (size_t)pieces * m_pad * BN * sizeof(float);
  if (need <= st->ws_bytes) return true;
  if (st->ws) cudaFree(st->ws);
  st->ws = nullptr;
  st->ws_bytes = 0;
  if (cudaMalloc(reinterpret_cast<void**>(&st->ws), need) != cudaSuccess) return false;
  st->ws_bytes = need;
  return true;
}

bool launch_gemm_chain(void* s, const ChainOp* ops, int n_ops, int M, const ChainCommon& cm, int* status, cudaStream_t stream) {
  ChainState* st = static_cast<ChainState*>(s);
  if (!st || !st->ws || n_ops < 1 || n_ops > kChainMaxOps || M < 1 || M > 128) return false;
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) return false;   // the barrier
  // counter's base is a launch argument: a captured launch would replay a stale one
  if (!st->configured) {
    if (cudaFuncSetAttribute(gemm_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return false;
    st->configured = true;
  }
  ChainMaps maps;
  ChainParams P{};
  P.n_ops = n_ops;
  P.M = M;
  P.m_pad = M <= 32 ? 32 : (M <= 64 ? 64 : 128);
  P.a_rows = M <= 32 ? 32 : 128;
  for (int i = 0; i < n_ops; ++i) {
    const ChainOp& o = ops[i];
    const bool swiglu = o.epi == EPI_SWIGLU;
    if (o.K % BK || o.N % 16 || (swiglu && o.N % 64) || (o.epi == EPI_QKV_ROPE && (cm.head_dim != 128 || o.N % 128)) ||
        (o.epi == EPI_RESIDUAL_NORM && o.N % 128))
      return false;
    const int out_per_tile = swiglu ? BN / 2 : BN;
    const long long total = (long long)((o.N + out_per_tile - 1) / out_per_tile) * (o.K / BK);
    const long long per = (total + st->n_sm - 1) / st->n_sm;
    const size_t need = (size_t)st->n_sm * (size_t)(per / (o.K / BK) + 2) * P.m_pad * BN * sizeof(float);
    if (need > st->ws_bytes) return false;
    const uint64_t w_rows = swiglu ? 2ull * o.N : (uint64_t)o.N;
    if (!encode_map(st, o.x, M, o.K, P.a_rows, &maps.x[i])) return false;
    if (!encode_map(st, o.w, w_rows, o.K, swiglu ? BN / 2 : BN, &maps.w[i])) return false;
    P.op[i].N = o.N;
    P.op[i].K = o.K;
    P.op[i].epi = o.epi;
    P.op[i].up_row_offset = o.N;
    P.op[i].scale_in = o.scale_in;
    P.op[i].ss_slots_in = o.ss_slots_in;
    P.op[i].out = o.out;
    P.op[i].x_out = o.x_out;
    P.op[i].gain = static_cast<const __nv_bfloat16*>(o.gain);
  }
  P.ss = cm.ss;
  P.ss_stride = cm.ss_stride;
  P.eps = cm.eps;
  P.ws = st->ws;
  P.bar = st->bar;
  P.bar_base = st->bar_base;
  P.tok_slot = cm.tok_slot;
  P.rope_cs = static_cast<const float2*>(cm.rope_cs);
  P.kv_pool = static_cast<__nv_bfloat16*>(cm.kv_pool);
  P.n_pages = cm.n_pages;
  P.layer = cm.layer;
  P.n_q = cm.n_q;
  P.n_kv = cm.n_kv;
  P.head_dim = cm.head_dim;
  P.status = status;
  const int grid = st->n_sm;
  st->bar_base += (unsigned)(2 * n_ops) * (unsigned)grid;
  return launch_pdl(gemm_chain_kernel, dim3(grid), dim3(kThreads), kSmemBytes, stream, maps, P) == cudaSuccess;
}

}  // namespace recg

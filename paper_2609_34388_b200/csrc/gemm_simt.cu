// Legacy tensor path: bf16 mma.sync GEMM, y = x . w^T with the projection epilogues.
// Kept as the A/B baseline for the tcgen05 kernel and for shapes that kernel does not take.
// CTA tile 128 x 128 x 32, 8 warps (2 x 4, each 64 x 32), 3-stage cp.async ring, padded rows.
#include "common.cuh"
#include "epilogue.cuh"
#include "kernels.h"

namespace recg {

namespace {

constexpr int BM = 128, BN = 128, BK = 32, STAGES = 3, THREADS = 256;
constexpr int LDS = BK + 8;                      // padded row stride (bf16 elements): 80 bytes
constexpr int STAGE_ELEMS = (BM + BN) * LDS;
constexpr int PIPE_BYTES = STAGES * STAGE_ELEMS * 2;
constexpr int EPI_LD = BN + 4;
constexpr int EPI_BYTES = BM * EPI_LD * 4;
constexpr int SMEM_BYTES = PIPE_BYTES > EPI_BYTES ? PIPE_BYTES : EPI_BYTES;

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// W rows for the tile: plain -> n0 + r ; SwiGLU -> 64 gate rows then 64 up rows
__device__ __forceinline__ int w_row(int r, int n0_tile, int epi, int F) {
  if (epi == EPI_SWIGLU) return r < BN / 2 ? n0_tile + r : F + n0_tile + (r - BN / 2);
  return n0_tile + r;
}

__global__ void __launch_bounds__(THREADS) gemm_simt_kernel(const __nv_bfloat16* __restrict__ X,
                                                            const __nv_bfloat16* __restrict__ W, int M, int Nw, int K,
                                                            EpiParams ep) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  __nv_bfloat16* sm = reinterpret_cast<__nv_bfloat16*>(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  griddep_launch();
  griddep_wait();
  const int wm = warp >> 2, wn = warp & 3;
  const int m0 = blockIdx.y * BM;
  const bool swiglu = ep.epi == EPI_SWIGLU;
  const int n0_tile = swiglu ? blockIdx.x * (BN / 2) : blockIdx.x * BN;  // first output column
  const int w_rows = swiglu ? 2 * ep.N : Nw;

  float acc[4][4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j][0] = acc[i][j][1] = acc[i][j][2] = acc[i][j][3] = 0.f;

  const int KT = K / BK;
  auto load_stage = [&](int kt, int s) {
    __nv_bfloat16* a = sm + s * STAGE_ELEMS;
    __nv_bfloat16* b = a + BM * LDS;
    const int k0 = kt * BK;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int idx = tid + i * THREADS;       // 0..511: row = idx / 4, chunk = idx % 4
      const int r = idx >> 2, c = (idx & 3) * 8;
      const int m = m0 + r;
      cp_async16(smem_u32(a + r * LDS + c), X + (size_t)(m < M ? m : 0) * K + k0 + c, m < M);
      const int wr = w_row(r, n0_tile, ep.epi, ep.N);
      const bool ok = swiglu ? (n0_tile + (r % (BN / 2)) < ep.N) : (wr < w_rows);
      cp_async16(smem_u32(b + r * LDS + c), W + (size_t)(ok ? wr : 0) * K + k0 + c, ok);
    }
  };

  for (int s = 0; s < STAGES - 1; ++s) {
    if (s < KT) load_stage(s, s);
    cp_async_commit();
  }
  for (int kt = 0; kt < KT; ++kt) {
    cp_async_wait<STAGES - 2>();
    __syncthreads();
    if (kt + STAGES - 1 < KT) load_stage(kt + STAGES - 1, (kt + STAGES - 1) % STAGES);
    cp_async_commit();
    const __nv_bfloat16* a = sm + (kt % STAGES) * STAGE_ELEMS;
    const __nv_bfloat16* b = a + BM * LDS;
#pragma unroll
    for (int ks = 0; ks < BK / 16; ++ks) {
      uint32_t af[4][4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int r = wm * 64 + i * 16 + (lane & 15);
        const int c = ks * 16 + (lane >> 4) * 8;
        ldmatrix_x4(af[i][0], af[i][1], af[i][2], af[i][3], smem_u32(a + r * LDS + c));
      }
#pragma unroll
      for (int jp = 0; jp < 2; ++jp) {
        const int r = wn * 32 + jp * 16 + (lane & 7) + (lane >> 4) * 8;
        const int c = ks * 16 + ((lane >> 3) & 1) * 8;
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4(b0, b1, b2, b3, smem_u32(b + r * LDS + c));
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          mma_bf16_16816(acc[i][2 * jp], af[i], b0, b1);
          mma_bf16_16816(acc[i][2 * jp + 1], af[i], b2, b3);
        }
      }
    }
  }
  cp_async_wait<0>();
  __syncthreads();

  // stage the accumulators, then the shared epilogue
  float* tile = reinterpret_cast<float*>(smem_raw);
  const int g = lane >> 2, q4 = lane & 3;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int r = wm * 64 + i * 16 + g, c = wn * 32 + j * 8 + q4 * 2;
      *reinterpret_cast<float2*>(tile + r * EPI_LD + c) = make_float2(acc[i][j][0], acc[i][j][1]);
      *reinterpret_cast<float2*>(tile + (r + 8) * EPI_LD + c) = make_float2(acc[i][j][2], acc[i][j][3]);
    }
  __syncthreads();
  tile_epilogue<THREADS>(ep, tile, EPI_LD, BM, BN, m0, n0_tile);
}

}  // namespace

void launch_gemm_simt(const GemmArgs& a, int* status, cudaStream_t st) {
  static bool configured[kMaxDevices] = {false};
  if (first_use_on_device(configured))
    cudaFuncSetAttribute(gemm_simt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);

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
  const int out_per_tile = a.epi == EPI_SWIGLU ? BN / 2 : BN;
  dim3 grid((a.N + out_per_tile - 1) / out_per_tile, (a.M + BM - 1) / BM);
  if (a.M <= 0) return;
  launch_pdl(gemm_simt_kernel, grid, dim3(THREADS), SMEM_BYTES, st, static_cast<const __nv_bfloat16*>(a.x),
             static_cast<const __nv_bfloat16*>(a.w), a.M, a.N, a.K, ep);
}

}  // namespace recg

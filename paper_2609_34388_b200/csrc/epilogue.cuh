// Projection epilogues shared by the two GEMM kernels.  Both stage the fp32 accumulator tile in
// shared memory ([rows][cols] with a padded row stride) and then call tile_epilogue(), which maps
// threads over the tile so that global stores are contiguous along a row.
#pragma once
#include "common.cuh"
#include "kernels.h"

namespace recg {

struct EpiParams {
  int epi;
  void* out;
  int M, N;       // logical output extent (EPI_SWIGLU: N = F)
  // EPI_QKV_ROPE
  const int* tok_slot;
  const float2* rope_cs;  // [head_dim/2][M] (cos, sin) of each token's position, frequency-major
  __nv_bfloat16* kv_pool;
  int64_t n_pages;
  int layer, n_q, n_kv, head_dim;
  int* status;
  // RMSNorm folded into the projections.  A projection whose input is a normalised residual stream reads
  // x = bf16(h * g) (not yet divided by the row's root mean square) and multiplies its accumulator rows by
  // rstd = rsqrt(sum_k ss_in[k][row] / norm_n + eps); EPI_RESIDUAL_NORM writes that x and the partial sums of squares
  // of the rows it updates, one slot per column tile, for the projection that follows.
  const float* ss_in;      // [ss_slots][ss_stride] partial sums of h^2 per row, or null: no scaling
  int ss_slots, ss_stride;
  float norm_inv_n, norm_eps;
  const __nv_bfloat16* gain;   // EPI_RESIDUAL_NORM: gain of the NEXT norm, [N]
  float* ss_out;               // EPI_RESIDUAL_NORM: [n column tiles][ss_stride]
};

__device__ __forceinline__ float silu_f(float z) { return z / (1.f + __expf(-z)); }

// tile: fp32 [tile_rows][ld]; covers output rows m0.. and accumulator columns n0.. (tile_cols wide).
// For EPI_SWIGLU the tile holds tile_cols/2 gate columns followed by tile_cols/2 up columns and
// n0 is the first OUTPUT column.
template <int kThreads>
__device__ __forceinline__ void tile_epilogue(const EpiParams& ep, const float* tile, int ld, int tile_rows,
                                              int tile_cols, int m0, int n0) {
  const int tid = threadIdx.x;
  if (ep.epi == EPI_SWIGLU) {
    const int oc = tile_cols / 2;
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(ep.out);
    for (int idx = tid; idx < tile_rows * (oc / 2); idx += kThreads) {
      const int r = idx / (oc / 2), c = (idx % (oc / 2)) * 2;
      const int m = m0 + r;
      if (m >= ep.M || n0 + c >= ep.N) continue;
      const float* row = tile + (size_t)r * ld;
      const float a0 = silu_f(row[c]) * row[oc + c];
      const float a1 = silu_f(row[c + 1]) * row[oc + c + 1];
      *reinterpret_cast<uint32_t*>(out + (size_t)m * ep.N + n0 + c) = pack_bf16(a0, a1);
    }
    return;
  }
  if (ep.epi == EPI_QKV_ROPE) {
    const int D = ep.head_dim, half = D / 2;
    __nv_bfloat16* q = static_cast<__nv_bfloat16*>(ep.out);
    // pairs (i, i + D/2) of one head: a thread handles two adjacent i
    const int heads_in_tile = tile_cols / D;
    const int per_row = heads_in_tile * (half / 2);
    for (int idx = tid; idx < tile_rows * per_row; idx += kThreads) {
      const int r = idx / per_row, rem = idx % per_row;
      const int hl = rem / (half / 2), i = (rem % (half / 2)) * 2;
      const int m = m0 + r;
      if (m >= ep.M) continue;
      const int head = n0 / D + hl;
      const float* x = tile + (size_t)r * ld + hl * D;
      float lo0 = x[i], lo1 = x[i + 1], hi0 = x[i + half], hi1 = x[i + half + 1];
      if (head < ep.n_q + ep.n_kv) {
        const float2 cs0 = ep.rope_cs[(size_t)i * ep.M + m], cs1 = ep.rope_cs[(size_t)(i + 1) * ep.M + m];
        const float a0 = lo0 * cs0.x - hi0 * cs0.y, b0 = hi0 * cs0.x + lo0 * cs0.y;
        const float a1 = lo1 * cs1.x - hi1 * cs1.y, b1 = hi1 * cs1.x + lo1 * cs1.y;
        lo0 = a0; hi0 = b0; lo1 = a1; hi1 = b1;
      }
      const uint32_t plo = pack_bf16(lo0, lo1), phi = pack_bf16(hi0, hi1);
      if (head < ep.n_q) {
        __nv_bfloat16* dst = q + ((size_t)m * ep.n_q + head) * D;
        *reinterpret_cast<uint32_t*>(dst + i) = plo;
        *reinterpret_cast<uint32_t*>(dst + i + half) = phi;
      } else {
        const int slot = ep.tok_slot[m];
        if (slot < 0) continue;
        const bool is_v = head >= ep.n_q + ep.n_kv;
        const int kvh = is_v ? head - ep.n_q - ep.n_kv : head - ep.n_q;
        const int64_t page = slot / kPageSize;
        const int tok = slot % kPageSize;
        if (page >= ep.n_pages) {
          set_status(ep.status, DEV_BAD_INDEX);
          continue;
        }
        __nv_bfloat16* base = ep.kv_pool + kv_tile_base(ep.n_pages, ep.n_kv, D, ep.layer, page, kvh) +
                              (is_v ? kv_tile_elems(D) : 0);
        *reinterpret_cast<uint32_t*>(base + kv_tile_offset(tok, i, D)) = plo;
        *reinterpret_cast<uint32_t*>(base + kv_tile_offset(tok, i + half, D)) = phi;
      }
    }
    return;
  }
  // plain / residual: 4 consecutive columns per thread
  for (int idx = tid; idx < tile_rows * (tile_cols / 4); idx += kThreads) {
    const int r = idx / (tile_cols / 4), c = (idx % (tile_cols / 4)) * 4;
    const int m = m0 + r, n = n0 + c;
    if (m >= ep.M || n >= ep.N) continue;
    const float4 v = *reinterpret_cast<const float4*>(tile + (size_t)r * ld + c);
    if (ep.epi == EPI_RESIDUAL) {
      float4* dst = reinterpret_cast<float4*>(static_cast<float*>(ep.out) + (size_t)m * ep.N + n);
      float4 h = *dst;
      h.x += v.x; h.y += v.y; h.z += v.z; h.w += v.w;
      *dst = h;
    } else if (ep.epi == EPI_PLAIN_F32) {
      *reinterpret_cast<float4*>(static_cast<float*>(ep.out) + (size_t)m * ep.N + n) = v;
    } else {
      uint2 o;
      o.x = pack_bf16(v.x, v.y);
      o.y = pack_bf16(v.z, v.w);
      *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(ep.out) + (size_t)m * ep.N + n) = o;
    }
  }
}

}  // namespace recg

// Shared device helpers for the recg kernels (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace recg {

// Codes a kernel may leave in the device status word (first writer wins).
enum : int {
  DEV_OK = 0,
  DEV_TIMEOUT_FULL = 1,   // consumer gave up waiting for a loaded stage
  DEV_TIMEOUT_EMPTY = 2,  // producer gave up waiting for a free stage
  DEV_TIMEOUT_MMA = 3,    // epilogue gave up waiting for an accumulator
  DEV_BAD_INDEX = 4,      // a page id or slot was out of range (access skipped)
  DEV_GUARD = 5           // a guard band behind a workspace region was overwritten (debug checks)
};

__device__ __forceinline__ void set_status(int* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- programmatic dependent launch ------------------------------------------------------------------
// Every kernel of a step is launched with programmatic stream serialisation: it signals at once that its
// dependent may be scheduled (launch_dependents), runs its own prologue (barrier init, TMEM allocation, shared
// memory clearing), and only then waits for the kernels before it to complete and flush (griddep_wait).  No
// kernel reads or writes global memory before its wait, so the launch latency and prologue of kernel n+1 overlap
// the tail of kernel n and nothing else changes.  Without the launch attribute both instructions do nothing.
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---- mbarrier ---------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.shared::cta.b64 st, [%0];\n}" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n}" ::"r"(smem_u32(bar)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: returns false (and the caller must bail out) after ~max_iter polls.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint32_t max_iter = (1u << 24)) {
  for (uint32_t i = 0; i < max_iter; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (i > 64) __nanosleep(32);
  }
  return false;
}

// ---- 1-D bulk copy global -> shared, completion on an mbarrier --------------------------------
// Both addresses 16-byte aligned, size a multiple of 16 bytes.
__device__ __forceinline__ void bulk_g2s(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(smem_dst)),
               "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

// ---- warp-level matrix fragments (legacy tensor path used by attention and the SIMT GEMM) ------
__device__ __forceinline__ void ldmatrix_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3,
                                                  uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
// D(16x8, f32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }

// ---- KV pool addressing ------------------------------------------------------------------------
// Pool = [layer][page][kv_head][K tile | V tile]; a tile holds 16 tokens x head_dim bf16 as 8-row atoms
// [token group g = tok / 8][dim half h = dim / 64][8 tokens][64 elements = 128 bytes], the eight 16-byte chunks
// of a row XOR-swizzled with (token & 7).  An atom is exactly the tensor core's canonical 128-byte-swizzle atom
// (K-major for K, MN-major for V), and because the token groups of consecutive pages are a constant
// 2 * (head_dim / 64) atoms apart, tiles copied back to back into shared memory form a multi-page operand
// with one uniform stride; row-wise and transposed ldmatrix loads from the same bytes are conflict free.
constexpr int kPageSize = 16;

__host__ __device__ __forceinline__ size_t kv_tile_elems(int head_dim) { return (size_t)kPageSize * head_dim; }
// element offset of (token-in-page, dim) inside a tile
__host__ __device__ __forceinline__ int kv_tile_offset(int tok, int dim, int head_dim) {
  const int atom = (tok >> 3) * (head_dim >> 6) + (dim >> 6), c = (dim >> 3) & 7, e = dim & 7, r = tok & 7;
  return atom * 512 + r * 64 + ((c ^ r) << 3) + e;
}
// element offset of the K tile of (layer, page, kv_head); the V tile follows it
__host__ __device__ __forceinline__ size_t kv_tile_base(int64_t n_pages, int n_kv, int head_dim, int layer,
                                                        int64_t page, int kv_head) {
  return ((((size_t)layer * n_pages + page) * n_kv + kv_head) * 2) * kv_tile_elems(head_dim);
}

// Host side.  Opt-in attributes of a kernel (its dynamic shared memory size) are per device: a call site keeps one
// flag per device and sets the attribute on first use there.  Setting it twice from two threads is harmless.
constexpr int kMaxDevices = 64;
inline bool first_use_on_device(bool (&seen)[kMaxDevices]) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return true;
  if (seen[dev]) return false;
  seen[dev] = true;
  return true;
}

// Host side: launch with the programmatic-serialisation attribute.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  // inside a stream capture the kernels become graph nodes, where plain edges measured faster than programmatic
  // ones (21.4 vs 24.6 us for the attention + combine pair), so the attribute is only used on live streams
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  if (cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone) {
    cfg.attrs = attr;
    cfg.numAttrs = 1;
  }
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace recg

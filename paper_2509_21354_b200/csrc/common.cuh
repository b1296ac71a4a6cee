// Shared device helpers for the libkve kernels (sm_100a): bf16 bit handling, mbarrier and bulk-copy
// (TMA engine) PTX wrappers with bounded waits, and the device status word.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace kve {

constexpr int D = 128;                 // head dim (elements); one K or V row = 256 bytes
constexpr int ROW_BYTES = D * 2;

// mirrors kvE_status in include/kve.h
constexpr int ERR_CAPACITY = -3;
constexpr int ERR_TIMEOUT = -6;

__device__ __forceinline__ void set_status(int32_t* status_word, int code) {
  if (status_word) atomicCAS(status_word, 0, code);   // first error sticks
}

// ---- bf16 <-> fp32 on raw bit patterns ----------------------------------------------------------
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// round to nearest even; finite inputs (NaN maps to a quiet NaN pattern)
__device__ __forceinline__ uint32_t f32_to_bf16_bits(float f) {
  uint32_t u = __float_as_uint(f);
  if ((u & 0x7fffffffu) > 0x7f800000u) return 0x7fc0u;
  u += 0x7fffu + ((u >> 16) & 1u);
  return u >> 16;
}
// two fp32 -> packed bf16 pair (lo in bits 0..15), round to nearest even, one conversion instruction
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
// exact split of two fp32 values into three bf16 pieces each (x = p0 + p1 + p2), packed pairwise:
// w[pl] holds piece pl of `a` in bits 0..15 and of `b` in bits 16..31
__device__ __forceinline__ void split3_pair(float a, float b, uint32_t (&w)[3]) {
  w[0] = pack_bf16x2(a, b);
  const float ra = a - bf16lo(w[0]), rb = b - bf16hi(w[0]);
  w[1] = pack_bf16x2(ra, rb);
  const float sa = ra - bf16lo(w[1]), sb = rb - bf16hi(w[1]);
  w[2] = pack_bf16x2(sa, sb);
}

// ---- shared-memory addresses, mbarriers, bulk copies --------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// non-blocking poll: has the phase of the given parity completed?
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after `limit` polls (each try_wait already blocks for a hardware-defined
// slice), returns false on give-up.  The caller records KVE_ERR_TIMEOUT and unwinds.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint32_t limit = (1u << 20)) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (i > 64) __nanosleep(64);
  }
  return false;
}

// 1-D bulk copy global -> this CTA's shared memory through the TMA engine, completion counted in
// bytes on `bar`.  dst, src 16-byte aligned; bytes a multiple of 16.  No multicast.
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(dst_smem)),
      "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}

// 16-byte asynchronous copy global -> shared (bypassing L1); `live` false writes 16 zero bytes instead
__device__ __forceinline__ void cp_async16(void* dst_smem, const void* src_gmem, bool live) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst_smem)), "l"(src_gmem),
               "r"(live ? 16 : 0)
               : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// ---- programmatic dependent launch ----------------------------------------------------------------
// Every kernel of the library is launched so that it may start while its predecessor on the stream is
// still draining.  A kernel calls pdl_launch_dependents() first thing (its successor may then be
// scheduled as soon as all of this grid's CTAs are resident), does whatever does not depend on
// earlier kernels (weights into shared memory or registers, barriers, tensor-memory allocation),
// and calls pdl_wait() before it touches anything an earlier kernel writes or still reads.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// 2^x by the special-function unit alone (2 ulp; results below 2^-126 flush to zero, -inf gives 0)
__device__ __forceinline__ float ex2_fast(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// D += A * B, m16n8k16, bf16 inputs, fp32 accumulate (warp-level tensor-core op)
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// A launch whose position comes from the DEVICE (a trigger replayed from a CUDA graph): the chunk to work on is the one
// right behind the keep list's coverage, and it is due once the stored length says it has left the window.
struct NextChunk { int t; bool due; };
__device__ __forceinline__ NextChunk next_chunk(const int32_t* n_listed, const int32_t* seq_len, int C, int window, int max_chunks) {
  NextChunk nx;
  nx.t = *n_listed;
  const int n = seq_len[0];      // lengths are uniform over the sequences of a layer
  const int stale = n > window ? (n - window) / C : 0;
  nx.due = nx.t >= 0 && nx.t < stale && nx.t < max_chunks;
  return nx;
}

// host side: launch with the programmatic-serialisation attribute
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace kve

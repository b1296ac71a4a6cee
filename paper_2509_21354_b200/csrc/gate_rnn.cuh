// Pieces shared by the LSTM recurrence kernels: launch arguments, cluster addressing, stores and bulk
// copies into a peer CTA's shared memory that count bytes on the peer's mbarrier, bounded cluster
// waits, the fast activations and the exact 3-way bf16 split of an fp32 value.
#pragma once
#include "common.cuh"
#include "kernels.h"

namespace kve {

constexpr int RNN_WARPS = 8;
constexpr int RNN_THREADS = RNN_WARPS * 32;

struct RnnArgs {
  const float* P;          // [S * n_range][4 d_g], column 4 u + gate: the pre-activations W_ih x + b of unit u
  float* H;                // [S * n_range][d_g]: h_t for the score kernel
  const uint16_t* W_hh;    // bf16 [4 d_g][d_g]
  const float* w_s;        // [d_g] (score kernel)
  float b_s;
  float* scores;           // [S][max_chunks]
  float* lstm_h;           // [S][d_g]
  float* lstm_c;
  int32_t* status;
  int S, max_chunks, t0, n_range, reset;
};

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
// stores into the shared memory of a CTA of the cluster (address from mapa) that count their bytes
// on an mbarrier of the same CTA when they land
__device__ __forceinline__ void st_async_u32(uint32_t addr, uint32_t val, uint32_t bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.u32 [%0], %1, [%2];" ::"r"(addr), "r"(val),
               "r"(bar)
               : "memory");
}
__device__ __forceinline__ void st_async_v4(uint32_t addr, const uint4& v, uint32_t bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.u32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(addr),
               "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"(bar)
               : "memory");
}
// bulk copy from this CTA's shared memory into a peer's (addresses from mapa), bytes counted on the peer's barrier
__device__ __forceinline__ void bulk_s2cluster(uint32_t dst, uint32_t src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "r"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// bounded: gives up `deadline_ns` (one second unless told otherwise) after the quick polls ran out, then false
__device__ __forceinline__ bool mbar_wait_cluster_bounded(uint64_t* bar, uint32_t parity,
                                                          unsigned long long deadline_ns = 1000000000ull) {
  for (int i = 0; i < 4096; ++i)
    if (mbar_try_wait_cluster(bar, parity)) return true;
  unsigned long long t_start, t_now;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_start));
  do {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    __nanosleep(128);
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_now));
  } while (t_now - t_start < deadline_ns);
  return false;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ float fast_sigmoid(float x) { return __fdividef(1.f, 1.f + __expf(-x)); }
__device__ __forceinline__ float fast_tanh(float x) { return 2.f * fast_sigmoid(2.f * x) - 1.f; }
// four 8 x 8 b16 blocks of shared memory as mma fragments (lane l gives the address of row l & 7 of block l >> 3)
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}

// exact 3-way split of an fp32 value into bf16 pieces: x = p0 + p1 + p2
__device__ __forceinline__ void split3(float x, uint32_t (&p)[3]) {
  p[0] = f32_to_bf16_bits(x);
  const float r1 = x - __uint_as_float(p[0] << 16);
  p[1] = f32_to_bf16_bits(r1);
  const float r2 = r1 - __uint_as_float(p[1] << 16);
  p[2] = f32_to_bf16_bits(r2);
}

}  // namespace kve

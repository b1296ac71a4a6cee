// kvE_append / kvE_set_len kernels: place new (k, v) rows at the tail of every sequence's paged
// cache, in temporal order (Sec. 3.2), and keep the device-side length in step.
#include "common.cuh"
#include "kernels.h"

namespace kve {

// One thread moves 16 bytes.  idx -> (row of k_new/v_new, K-or-V, 16-byte lane within the 256-byte row).
// pos0 = tokens stored before the call (the handle tracks it on the host, so no device read sits in
// front of the page-table look-up); the first threads also publish the new length.
__global__ void __launch_bounds__(256) kve_append_kernel(LayerView v, const uint4* __restrict__ k_new,
                                                         const uint4* __restrict__ v_new, int n_new, int pos0) {
  pdl_launch_dependents();
  pdl_wait();
  const long long total = (long long)v.S * n_new * 32;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int lane16 = (int)(idx & 15);
    const int is_v = (int)((idx >> 4) & 1);
    const long long row = idx >> 5;              // s * n_new + i
    const int s = (int)(row / n_new);
    const int i = (int)(row - (long long)s * n_new);
    const int pos = pos0 + i;
    if (pos < 0 || pos >= v.max_tokens) { set_status(v.status, ERR_CAPACITY); continue; }
    const int chunk = pos / v.C;
    const int r = pos - chunk * v.C;
    const long long page = v.page_table[(long long)s * v.max_chunks + chunk];
    if (page < 0 || page >= v.n_pages) { set_status(v.status, ERR_CAPACITY); continue; }
    uint4* dst = reinterpret_cast<uint4*>((is_v ? v.v_pages : v.k_pages) + (page * v.C + r) * D) + lane16;
    const uint4* src = (is_v ? v_new : k_new) + row * 16 + lane16;
    *dst = __ldg(src);
  }
  if (blockIdx.x == 0)
    for (int b = threadIdx.x; b < v.B; b += blockDim.x) v.seq_len[b] = pos0 + n_new;
}

// n_new tokens per sequence from the position the DEVICE holds in seq_len (replayable from a CUDA graph: nothing
// about the position is baked into the launch).  Every CTA reads the old length before it writes; the
// last CTA to finish (atomic ticket, nobody spins) advances the length and resets the ticket, so no CTA
// can see the new length while it is still placing rows.
__global__ void __launch_bounds__(256) kve_append_next_kernel(LayerView v, const uint4* __restrict__ k_new,
                                                              const uint4* __restrict__ v_new, int n_new, int32_t* ticket) {
  pdl_launch_dependents();
  pdl_wait();
  const long long total = (long long)v.S * n_new * 32;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int lane16 = (int)(idx & 15);
    const int is_v = (int)((idx >> 4) & 1);
    const long long row = idx >> 5;              // s * n_new + i
    const int s = (int)(row / n_new);
    const int n0 = v.seq_len[s / v.H];
    if (n0 < 0 || n0 + n_new > v.max_tokens) continue;  // no room: flagged below, nothing written
    const int pos = n0 + (int)(row - (long long)s * n_new);
    const int chunk = pos / v.C;
    const int r = pos - chunk * v.C;
    const long long page = v.page_table[(long long)s * v.max_chunks + chunk];
    if (page < 0 || page >= v.n_pages) { set_status(v.status, ERR_CAPACITY); continue; }
    uint4* dst = reinterpret_cast<uint4*>((is_v ? v.v_pages : v.k_pages) + (page * v.C + r) * D) + lane16;
    const uint4* src = (is_v ? v_new : k_new) + row * 16 + lane16;
    *dst = __ldg(src);
  }
  __shared__ int last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) last = (atomicAdd(ticket, 1) == (int)gridDim.x - 1) ? 1 : 0;
  __syncthreads();
  if (!last) return;
  for (int b = threadIdx.x; b < v.B; b += blockDim.x) {
    const int n = v.seq_len[b];
    if (n < 0 || n + n_new > v.max_tokens) set_status(v.status, ERR_CAPACITY);      // no room: nothing was written
    else v.seq_len[b] = n + n_new;
  }
  if (threadIdx.x == 0) *ticket = 0;      // clean for the next launch
}

__global__ void kve_set_len_kernel(int32_t* seq_len, int B, int n, int32_t* n_listed, int listed) {
  pdl_launch_dependents();
  pdl_wait();
  int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < B) seq_len[b] = n;
  if (b == 0 && listed >= 0) *n_listed = listed;
}

cudaError_t launch_append(const LayerView& v, const void* k_new, const void* v_new, int n_new, int pos0, cudaStream_t st) {
  const long long total = (long long)v.S * n_new * 32;
  long long blocks = (total + 255) / 256;
  if (blocks > sm_count() * 32LL) blocks = sm_count() * 32LL;   // grid-stride beyond 32 CTAs per SM
  if (blocks < 1) blocks = 1;
  return launch_pdl(kve_append_kernel, dim3((unsigned)blocks), dim3(256), 0, st, v, static_cast<const uint4*>(k_new),
                    static_cast<const uint4*>(v_new), n_new, pos0);
}

cudaError_t launch_append_next(const LayerView& v, const void* k_new, const void* v_new, int n_new, int32_t* ticket,
                               cudaStream_t st) {
  long long blocks = ((long long)v.S * n_new * 32 + 255) / 256;
  if (blocks > sm_count() * 32LL) blocks = sm_count() * 32LL;
  return launch_pdl(kve_append_next_kernel, dim3((unsigned)blocks), dim3(256), 0, st, v, static_cast<const uint4*>(k_new),
                    static_cast<const uint4*>(v_new), n_new, ticket);
}

__global__ void kve_set_listed_kernel(int32_t* n_listed, int listed) {
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x == 0) *n_listed = listed;
}

cudaError_t launch_set_listed(const LayerView& v, int n_listed, cudaStream_t st) {
  return launch_pdl(kve_set_listed_kernel, dim3(1), dim3(32), 0, st, v.n_listed, n_listed);
}

cudaError_t launch_set_len(const LayerView& v, int n, int n_listed, cudaStream_t st) {
  return launch_pdl(kve_set_len_kernel, dim3((v.B + 127) / 128), dim3(128), 0, st, v.seq_len, v.B, n, v.n_listed, n_listed);
}

}  // namespace kve

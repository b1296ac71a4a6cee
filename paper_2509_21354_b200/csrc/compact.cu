// kvE_compact kernel: the retention rule of Sec. 3.2, "keep chunk t iff s_t >= tau", turned into an
// ascending list of kept chunk ids per sequence.  One warp per sequence: 32 scores per round, a
// ballot gives the keep mask, popcount of the lower lanes gives each kept chunk its slot.
#include "common.cuh"
#include "kernels.h"

namespace kve {

constexpr int COMPACT_WARPS = 4;

__global__ void __launch_bounds__(COMPACT_WARPS * 32) kve_compact_kernel(LayerView v, int n_chunks, float tau) {
  pdl_launch_dependents();
  pdl_wait();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int s = blockIdx.x * COMPACT_WARPS + warp;
  if (s >= v.S) return;
  const float* sc = v.scores + (long long)s * v.max_chunks;
  int32_t* idx = v.keep_idx + (long long)s * v.max_chunks;
  int base = 0;
  for (int t0 = 0; t0 < n_chunks; t0 += 32) {
    const int t = t0 + lane;
    const bool keep = (t < n_chunks) && (sc[t] >= tau);
    const unsigned mask = __ballot_sync(0xffffffffu, keep);
    if (keep) idx[base + __popc(mask & ((1u << lane) - 1u))] = t;
    base += __popc(mask);
  }
  for (int t = base + lane; t < v.max_chunks; t += 32) idx[t] = -1;
  if (lane == 0) v.keep_cnt[s] = base;
}

cudaError_t launch_compact(const LayerView& v, int n_chunks, float tau, cudaStream_t st) {
  return launch_pdl(kve_compact_kernel, dim3((v.S + COMPACT_WARPS - 1) / COMPACT_WARPS), dim3(COMPACT_WARPS * 32), 0, st, v, n_chunks, tau);
}

}  // namespace kve

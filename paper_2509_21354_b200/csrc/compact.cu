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
  if (s == 0 && lane == 0) *v.n_listed = n_chunks;      // what the attention kernel reads: the list covers chunks [0, n_chunks)
}

// ---- what attention wants from a fresh keep list ---------------------------------------------------------
// The kept chunks' summary rows, copied into one contiguous run per sequence ("compacted chunk tokens",
// Sec. 3.3): attention then fetches a sequence's kept rows with one bulk copy per 64 rows instead of one
// per row, on every decode step until the next trigger.  One warp moves 8 kept rows: lanes 0-15 the K
// row, lanes 16-31 the V row, 16 bytes each, all 8 loads in flight.
constexpr int GATHER_ROWS = 8;

__global__ void __launch_bounds__(COMPACT_WARPS * 32) kve_keep_gather_kernel(LayerView v, int n_chunks, int groups,
                                                                            uint4* __restrict__ kkept, uint4* __restrict__ vkept) {
  pdl_launch_dependents();
  pdl_wait();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long unit = (long long)blockIdx.x * COMPACT_WARPS + warp;
  const int s = (int)(unit / groups), gi = (int)(unit - (long long)s * groups);
  if (s >= v.S) return;
  const int M = min(max(v.keep_cnt[s], 0), n_chunks);
  const int i0 = gi * GATHER_ROWS;
  if (i0 >= M) return;
  const long long sb = (long long)s * v.max_chunks;
  const int is_v = lane >> 4, l16 = lane & 15;
  const uint4* src = reinterpret_cast<const uint4*>(is_v ? v.vsum_bf16 : v.ksum_bf16);
  uint4* dst = is_v ? vkept : kkept;
  int t[GATHER_ROWS];
#pragma unroll
  for (int r = 0; r < GATHER_ROWS; ++r) {
    t[r] = (i0 + r < M) ? v.keep_idx[sb + i0 + r] : -1;
    if (t[r] >= n_chunks) { set_status(v.status, ERR_CAPACITY); t[r] = -1; }
  }
  uint4 w[GATHER_ROWS];
#pragma unroll
  for (int r = 0; r < GATHER_ROWS; ++r)
    if (t[r] >= 0) w[r] = __ldg(src + (sb + t[r]) * 16 + l16);
#pragma unroll
  for (int r = 0; r < GATHER_ROWS; ++r)
    if (t[r] >= 0) dst[(sb + i0 + r) * 16 + l16] = w[r];
}

// after either retention rule: the kept rows, compacted
static cudaError_t launch_keep_gather(const LayerView& v, int n_chunks, void* kkept, void* vkept, cudaStream_t st) {
  if (n_chunks <= 0) return cudaSuccess;
  const int groups = (n_chunks + GATHER_ROWS - 1) / GATHER_ROWS;
  const long long units = (long long)v.S * groups;
  return launch_pdl(kve_keep_gather_kernel, dim3((unsigned)((units + COMPACT_WARPS - 1) / COMPACT_WARPS)), dim3(COMPACT_WARPS * 32), 0, st,
                    v, n_chunks, groups, static_cast<uint4*>(kkept), static_cast<uint4*>(vkept));
}

cudaError_t launch_compact(const LayerView& v, int n_chunks, float tau, void* kkept, void* vkept, cudaStream_t st) {
  cudaError_t e = launch_pdl(kve_compact_kernel, dim3((v.S + COMPACT_WARPS - 1) / COMPACT_WARPS), dim3(COMPACT_WARPS * 32), 0, st, v,
                             n_chunks, tau);
  return e == cudaSuccess ? launch_keep_gather(v, n_chunks, kkept, vkept, st) : e;
}

// ---- kvE_compact_topk kernel: keep the k highest-scoring chunks of every sequence --------------------------
// One warp per sequence.  Chunk t is kept iff fewer than k chunks rank before it; u ranks before t when
// s_u > s_t, or s_u == s_t and u < t (the older chunk first), so the result is unique.  Each lane counts
// the chunks ranking before its own by walking the sequence's scores - in shared memory while a sequence's scores
// fit there (STAGED), straight from global memory beyond that; the kept ids are then written in ascending order
// with the same ballot + popcount as the threshold rule.
constexpr int TOPK_STAGED_CHUNKS = 2048;      // scores of one sequence staged per warp up to here

template <bool STAGED>
__global__ void __launch_bounds__(COMPACT_WARPS * 32) kve_compact_topk_kernel(LayerView v, int n_chunks, int k) {
  extern __shared__ float topk_scores[];   // STAGED: [COMPACT_WARPS][n_chunks]
  pdl_launch_dependents();
  pdl_wait();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int s = blockIdx.x * COMPACT_WARPS + warp;
  if (s >= v.S) return;
  const float* sc = v.scores + (long long)s * v.max_chunks;
  const float* mine = sc;
  int32_t* idx = v.keep_idx + (long long)s * v.max_chunks;
  if (STAGED) {
    float* stage = topk_scores + warp * n_chunks;
    for (int t = lane; t < n_chunks; t += 32) stage[t] = sc[t];
    __syncwarp();
    mine = stage;
  }
  int base = 0;
  for (int t0 = 0; t0 < n_chunks; t0 += 32) {
    const int t = t0 + lane;
    bool keep = false;
    if (t < n_chunks) {
      const float st = mine[t];
      int before = 0;
      for (int u = 0; u < n_chunks; ++u) {
        const float su = mine[u];
        before += (su > st || (su == st && u < t)) ? 1 : 0;
      }
      keep = before < k;
    }
    const unsigned mask = __ballot_sync(0xffffffffu, keep);
    if (keep) idx[base + __popc(mask & ((1u << lane) - 1u))] = t;
    base += __popc(mask);
  }
  for (int t = base + lane; t < v.max_chunks; t += 32) idx[t] = -1;
  if (lane == 0) v.keep_cnt[s] = base;
  if (s == 0 && lane == 0) *v.n_listed = n_chunks;
}

cudaError_t launch_compact_topk(const LayerView& v, int n_chunks, int k, void* kkept, void* vkept, cudaStream_t st) {
  const dim3 grid((v.S + COMPACT_WARPS - 1) / COMPACT_WARPS), block(COMPACT_WARPS * 32);
  cudaError_t e;
  if (n_chunks <= TOPK_STAGED_CHUNKS) {
    const size_t smem = sizeof(float) * (size_t)COMPACT_WARPS * (n_chunks > 0 ? n_chunks : 1);
    static DeviceFlags opted;
    e = smem_opt_in(opted, kve_compact_topk_kernel<true>, (int)(sizeof(float) * COMPACT_WARPS * TOPK_STAGED_CHUNKS));
    if (e == cudaSuccess) e = launch_pdl(kve_compact_topk_kernel<true>, grid, block, smem, st, v, n_chunks, k);
  } else {
    e = launch_pdl(kve_compact_topk_kernel<false>, grid, block, 0, st, v, n_chunks, k);
  }
  return e == cudaSuccess ? launch_keep_gather(v, n_chunks, kkept, vkept, st) : e;
}

// ---- kvE_reclaim_pages kernels (Sec. 3.3, memory ratio n / (W + M)): pages of gated chunks go back to the caller ----
// A chunk gives its page back if it was discarded (score < tau) or, with mode 1, in any case (retained
// chunks live on as their summary row).  Free-list order: sequences in order, chunks ascending, so the
// result is unique.  count -> scan -> scatter; the scatter does nothing if the list would overflow.
__device__ __forceinline__ bool reclaimable(const LayerView& v, int s, int t, float tau, int mode) {
  const long long i = (long long)s * v.max_chunks + t;
  return (mode == 1 || !(v.scores[i] >= tau)) && v.page_table[i] >= 0;
}

__global__ void __launch_bounds__(COMPACT_WARPS * 32) kve_reclaim_count_kernel(LayerView v, int t0, int t1, float tau, int mode,
                                                                              int32_t* counts) {
  pdl_launch_dependents();
  pdl_wait();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int s = blockIdx.x * COMPACT_WARPS + warp;
  if (s >= v.S) return;
  int n = 0;
  for (int tb = t0; tb < t1; tb += 32) {
    const int t = tb + lane;
    n += __popc(__ballot_sync(0xffffffffu, t < t1 && reclaimable(v, s, t, tau, mode)));
  }
  if (lane == 0) counts[s] = n;
}

// one CTA: exclusive prefix sum of counts[0..S) -> offsets[0..S); offsets[S] = 1 if the total fits, else 0
__global__ void __launch_bounds__(1024) kve_reclaim_scan_kernel(const int32_t* counts, int S, int32_t* offsets, long long capacity,
                                                                int32_t* free_count, int32_t* status) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ int warp_tot[32];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int per = (S + 1023) / 1024;
  const int lo = min(S, tid * per), hi = min(S, lo + per);
  int mine = 0;
  for (int i = lo; i < hi; ++i) mine += counts[i];
  int incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int x = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += x;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = warp_tot[lane], wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int x = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += x;
    }
    warp_tot[lane] = wi - w;      // exclusive
  }
  __syncthreads();
  int run = warp_tot[warp] + incl - mine;
  for (int i = lo; i < hi; ++i) {
    offsets[i] = run;
    run += counts[i];
  }
  if (tid == 1023) {
    const bool fits = (long long)run <= capacity;
    offsets[S] = fits ? 1 : 0;
    *free_count = fits ? run : 0;
    if (!fits) set_status(status, ERR_CAPACITY);
  }
}

__global__ void __launch_bounds__(COMPACT_WARPS * 32) kve_reclaim_scatter_kernel(LayerView v, int t0, int t1, float tau, int mode,
                                                                                const int32_t* offsets, int32_t* free_list) {
  pdl_launch_dependents();
  pdl_wait();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int s = blockIdx.x * COMPACT_WARPS + warp;
  if (s >= v.S || offsets[v.S] == 0) return;
  int32_t* table = const_cast<int32_t*>(v.page_table) + (long long)s * v.max_chunks;
  int base = offsets[s];
  for (int tb = t0; tb < t1; tb += 32) {
    const int t = tb + lane;
    const bool give = t < t1 && reclaimable(v, s, t, tau, mode);
    const unsigned mask = __ballot_sync(0xffffffffu, give);
    if (give) {
      free_list[base + __popc(mask & ((1u << lane) - 1u))] = table[t];
      table[t] = -1;
    }
    base += __popc(mask);
  }
}

cudaError_t launch_reclaim(const LayerView& v, int t0, int t1, float tau, int mode, int32_t* scratch, int32_t* free_list,
                           long long capacity, int32_t* free_count, cudaStream_t st) {
  int32_t* counts = scratch;
  int32_t* offsets = scratch + v.S;
  const dim3 grid((v.S + COMPACT_WARPS - 1) / COMPACT_WARPS), block(COMPACT_WARPS * 32);
  cudaError_t e = launch_pdl(kve_reclaim_count_kernel, grid, block, 0, st, v, t0, t1, tau, mode, counts);
  if (e == cudaSuccess)
    e = launch_pdl(kve_reclaim_scan_kernel, dim3(1), dim3(1024), 0, st, (const int32_t*)counts, v.S, offsets, capacity, free_count,
                   v.status);
  if (e == cudaSuccess)
    e = launch_pdl(kve_reclaim_scatter_kernel, grid, block, 0, st, v, t0, t1, tau, mode, (const int32_t*)offsets, free_list);
  return e;
}

}  // namespace kve

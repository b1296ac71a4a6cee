// kvE_summarize_chunks kernels (Eq. 2): per (sequence, chunk) the mean of the chunk's C key rows and
// of its C value rows, then (AGG_MLP) a 2-layer GELU MLP on each mean.
//
// chunk_mean: HBM-bound.  One warp per (sequence, chunk): lanes 0-15 stream the K page, lanes 16-31 the
// V page, 16 bytes per lane per row, rows added in temporal order in fp32 (so the sum has the same
// rounding as a plain sequential loop), divided by C with an IEEE division.
#include "common.cuh"
#include "kernels.h"

namespace kve {

constexpr int MEAN_WARPS = 8;
constexpr int MEAN_UNROLL = 8;

__device__ __forceinline__ void add_row(float (&acc)[8], const uint4& w) {
  acc[0] += bf16lo(w.x); acc[1] += bf16hi(w.x);
  acc[2] += bf16lo(w.y); acc[3] += bf16hi(w.y);
  acc[4] += bf16lo(w.z); acc[5] += bf16hi(w.z);
  acc[6] += bf16lo(w.w); acc[7] += bf16hi(w.w);
}

__global__ void __launch_bounds__(MEAN_WARPS * 32) kve_chunk_mean_kernel(LayerView v, int t0, int n_range,
                                                                        long long n_units, int final_output) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long unit = (long long)blockIdx.x * MEAN_WARPS + warp;
  if (unit >= n_units) return;
  const int s = (int)(unit / n_range);
  const int t = t0 + (int)(unit - (long long)s * n_range);
  const int is_v = lane >> 4, l16 = lane & 15;
  const long long page = v.page_table[(long long)s * v.max_chunks + t];
  if (page < 0 || page >= v.n_pages) {
    if (lane == 0) set_status(v.status, ERR_CAPACITY);
    return;
  }
  const uint4* src = reinterpret_cast<const uint4*>((is_v ? v.v_pages : v.k_pages) + page * v.C * D) + l16;
  float acc[8];
#pragma unroll
  for (int x = 0; x < 8; ++x) acc[x] = 0.f;
  int j = 0;
  for (; j + MEAN_UNROLL <= v.C; j += MEAN_UNROLL) {
    uint4 w[MEAN_UNROLL];
#pragma unroll
    for (int u = 0; u < MEAN_UNROLL; ++u) w[u] = __ldcs(src + (long long)(j + u) * 16);
#pragma unroll
    for (int u = 0; u < MEAN_UNROLL; ++u) add_row(acc, w[u]);
  }
  for (; j < v.C; ++j) add_row(acc, __ldcs(src + (long long)j * 16));
  const float fc = (float)v.C;
#pragma unroll
  for (int x = 0; x < 8; ++x) acc[x] = __fdiv_rn(acc[x], fc);

  const long long o = ((long long)s * v.max_chunks + t) * D + l16 * 8;
  float4* of = reinterpret_cast<float4*>((is_v ? v.vsum_f32 : v.ksum_f32) + o);
  of[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
  of[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
  if (final_output) {
    uint4 b;
    b.x = pack_bf16x2(acc[0], acc[1]);
    b.y = pack_bf16x2(acc[2], acc[3]);
    b.z = pack_bf16x2(acc[4], acc[5]);
    b.w = pack_bf16x2(acc[6], acc[7]);
    *reinterpret_cast<uint4*>((is_v ? v.vsum_bf16 : v.ksum_bf16) + o) = b;
  }
}

cudaError_t launch_chunk_mean(const LayerView& v, int t0, int t1, bool final_output, cudaStream_t st) {
  const int n_range = t1 - t0;
  const long long n_units = (long long)v.S * n_range;
  if (n_units <= 0) return cudaSuccess;
  const long long blocks = (n_units + MEAN_WARPS - 1) / MEAN_WARPS;
  kve_chunk_mean_kernel<<<(unsigned)blocks, MEAN_WARPS * 32, 0, st>>>(v, t0, n_range, n_units, final_output ? 1 : 0);
  return cudaGetLastError();
}

// ---- aggregator MLP (Eq. 2 read as mean -> d_sum -> d, exact-erf GELU), fp32 FMA ------------------
// A CTA takes MLP_ROWS (sequence, chunk) units of one side (blockIdx.y: 0 = keys, 1 = values).
// The unit's mean sits in ksum_f32 / vsum_f32 (written by chunk_mean); the MLP output overwrites it
// and its bf16 rounding goes to ksum_bf16 / vsum_bf16.
constexpr int MLP_ROWS = 32;
constexpr int MLP_THREADS = 256;

__device__ __forceinline__ float gelu_erf(float x) { return 0.5f * x * (1.f + erff(x * 0.70710678118654752440f)); }

__device__ __forceinline__ void unpack8(const uint4& w, float (&f)[8]) {
  f[0] = bf16lo(w.x); f[1] = bf16hi(w.x); f[2] = bf16lo(w.y); f[3] = bf16hi(w.y);
  f[4] = bf16lo(w.z); f[5] = bf16hi(w.z); f[6] = bf16lo(w.w); f[7] = bf16hi(w.w);
}

__global__ void __launch_bounds__(MLP_THREADS) kve_chunk_mlp_kernel(LayerView v, int t0, int n_range, long long n_units,
                                                                   MlpWeights w, int d_sum) {
  extern __shared__ __align__(16) float smem[];
  float* Xs = smem;                    // [MLP_ROWS][128]
  float* Hs = smem + MLP_ROWS * D;     // [MLP_ROWS][d_sum]
  const int tid = threadIdx.x;
  const int side = blockIdx.y;
  const uint16_t* W1 = side ? w.W1V : w.W1K;
  const uint16_t* W2 = side ? w.W2V : w.W2K;
  const float* b1 = side ? w.b1V : w.b1K;
  const float* b2 = side ? w.b2V : w.b2K;
  float* sum_f32 = side ? v.vsum_f32 : v.ksum_f32;
  uint16_t* sum_b16 = side ? v.vsum_bf16 : v.ksum_bf16;
  const long long unit0 = (long long)blockIdx.x * MLP_ROWS;

  // stage the means
  for (int i = tid; i < MLP_ROWS * (D / 4); i += MLP_THREADS) {
    const int r = i / (D / 4), c4 = i % (D / 4);
    const long long unit = unit0 + r;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    if (unit < n_units) {
      const int s = (int)(unit / n_range);
      const int t = t0 + (int)(unit - (long long)s * n_range);
      x = *reinterpret_cast<const float4*>(sum_f32 + ((long long)s * v.max_chunks + t) * D + c4 * 4);
    }
    reinterpret_cast<float4*>(Xs)[i] = x;
  }
  __syncthreads();

  // layer 1: thread owns hidden unit u, accumulates all rows
  for (int u = tid; u < d_sum; u += MLP_THREADS) {
    float acc[MLP_ROWS];
    const float bias = b1[u];
#pragma unroll
    for (int r = 0; r < MLP_ROWS; ++r) acc[r] = bias;
    const uint4* wrow = reinterpret_cast<const uint4*>(W1 + (long long)u * D);
    for (int x8 = 0; x8 < D / 8; ++x8) {
      float wf[8];
      unpack8(__ldg(wrow + x8), wf);
#pragma unroll
      for (int r = 0; r < MLP_ROWS; ++r) {
        const float4 a = *reinterpret_cast<const float4*>(Xs + r * D + x8 * 8);
        const float4 b = *reinterpret_cast<const float4*>(Xs + r * D + x8 * 8 + 4);
        acc[r] = fmaf(wf[0], a.x, acc[r]); acc[r] = fmaf(wf[1], a.y, acc[r]);
        acc[r] = fmaf(wf[2], a.z, acc[r]); acc[r] = fmaf(wf[3], a.w, acc[r]);
        acc[r] = fmaf(wf[4], b.x, acc[r]); acc[r] = fmaf(wf[5], b.y, acc[r]);
        acc[r] = fmaf(wf[6], b.z, acc[r]); acc[r] = fmaf(wf[7], b.w, acc[r]);
      }
    }
#pragma unroll
    for (int r = 0; r < MLP_ROWS; ++r) Hs[r * d_sum + u] = gelu_erf(acc[r]);
  }
  __syncthreads();

  // layer 2: thread owns output dim x for half of the rows
  {
    const int x = tid & (D - 1);
    const int r0 = (tid >> 7) * (MLP_ROWS / 2);
    float acc[MLP_ROWS / 2];
    const float bias = b2[x];
#pragma unroll
    for (int r = 0; r < MLP_ROWS / 2; ++r) acc[r] = bias;
    const uint4* wrow = reinterpret_cast<const uint4*>(W2 + (long long)x * d_sum);
    for (int u8 = 0; u8 < d_sum / 8; ++u8) {
      float wf[8];
      unpack8(__ldg(wrow + u8), wf);
#pragma unroll
      for (int r = 0; r < MLP_ROWS / 2; ++r) {
        const float4 a = *reinterpret_cast<const float4*>(Hs + (r0 + r) * d_sum + u8 * 8);
        const float4 b = *reinterpret_cast<const float4*>(Hs + (r0 + r) * d_sum + u8 * 8 + 4);
        acc[r] = fmaf(wf[0], a.x, acc[r]); acc[r] = fmaf(wf[1], a.y, acc[r]);
        acc[r] = fmaf(wf[2], a.z, acc[r]); acc[r] = fmaf(wf[3], a.w, acc[r]);
        acc[r] = fmaf(wf[4], b.x, acc[r]); acc[r] = fmaf(wf[5], b.y, acc[r]);
        acc[r] = fmaf(wf[6], b.z, acc[r]); acc[r] = fmaf(wf[7], b.w, acc[r]);
      }
    }
#pragma unroll
    for (int r = 0; r < MLP_ROWS / 2; ++r) {
      const long long unit = unit0 + r0 + r;
      if (unit < n_units) {
        const int s = (int)(unit / n_range);
        const int t = t0 + (int)(unit - (long long)s * n_range);
        const long long o = ((long long)s * v.max_chunks + t) * D + x;
        sum_f32[o] = acc[r];
        sum_b16[o] = (uint16_t)f32_to_bf16_bits(acc[r]);
      }
    }
  }
}

cudaError_t launch_chunk_mlp(const LayerView& v, int t0, int t1, const MlpWeights& w, int d_sum, cudaStream_t st) {
  const int n_range = t1 - t0;
  const long long n_units = (long long)v.S * n_range;
  if (n_units <= 0) return cudaSuccess;
  const size_t smem = sizeof(float) * (size_t)MLP_ROWS * (D + d_sum);
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(kve_chunk_mlp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)(sizeof(float) * MLP_ROWS * (D + 1024)));
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  dim3 grid((unsigned)((n_units + MLP_ROWS - 1) / MLP_ROWS), 2);
  kve_chunk_mlp_kernel<<<grid, MLP_THREADS, smem, st>>>(v, t0, n_range, n_units, w, d_sum);
  return cudaGetLastError();
}

}  // namespace kve

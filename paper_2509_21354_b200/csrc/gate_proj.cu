// Gate input projection (Eq. 3, the W_ih x_t term for all chunks at once):
//   P[s, t, :] = W_ih [Kbar_t ; Vbar_t] + b_ih + b_hh      a GEMM [S * n_range, 256] x [256, 4 d_g]
// bf16 operands (the rounded summaries and bf16 weights, so every product is exact), fp32 accumulate
// on the tensor cores, bias fused in the epilogue.  Rows are gathered straight from the summary
// store: columns 0..127 of a row come from ksum_bf16, columns 128..255 from vsum_bf16.
#include "common.cuh"
#include "kernels.h"

namespace kve {

constexpr int PJ_TM = 64, PJ_TN = 64, PJ_K = 2 * D, PJ_LD = PJ_K + 8;   // padded row: conflict-free fragments
constexpr int PJ_THREADS = 128;

__global__ void __launch_bounds__(PJ_THREADS) kve_gate_proj_kernel(LayerView v, int t0, int n_range, long long n_rows,
                                                                   const uint16_t* __restrict__ W_ih,
                                                                   const float* __restrict__ b_ih,
                                                                   const float* __restrict__ b_hh, int n_cols,
                                                                   float* __restrict__ P) {
  extern __shared__ __align__(16) uint16_t sm16[];
  uint16_t* As = sm16;                    // [PJ_TM][PJ_LD]
  uint16_t* Bs = sm16 + PJ_TM * PJ_LD;    // [PJ_TN][PJ_LD]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, tig = lane & 3;
  const long long row0 = (long long)blockIdx.x * PJ_TM;
  const int col0 = blockIdx.y * PJ_TN;

  for (int i = tid; i < PJ_TM * 32; i += PJ_THREADS) {
    const int r = i >> 5, c = i & 31;             // c: 16-byte piece of the 512-byte row
    const long long gr = row0 + r;
    uint4 val = make_uint4(0, 0, 0, 0);
    if (gr < n_rows) {
      const int s = (int)(gr / n_range);
      const int t = t0 + (int)(gr - (long long)s * n_range);
      const uint16_t* src = (c < 16 ? v.ksum_bf16 : v.vsum_bf16) + ((long long)s * v.max_chunks + t) * D + (c & 15) * 8;
      val = *reinterpret_cast<const uint4*>(src);
    }
    *reinterpret_cast<uint4*>(As + r * PJ_LD + c * 8) = val;
  }
  for (int i = tid; i < PJ_TN * 32; i += PJ_THREADS) {
    const int r = i >> 5, c = i & 31;
    uint4 val = make_uint4(0, 0, 0, 0);
    if (col0 + r < n_cols) val = __ldg(reinterpret_cast<const uint4*>(W_ih + (long long)(col0 + r) * PJ_K + c * 8));
    *reinterpret_cast<uint4*>(Bs + r * PJ_LD + c * 8) = val;
  }
  __syncthreads();

  const int wm = warp >> 1, wn = warp & 1;
  float acc[2][4][4];
#pragma unroll
  for (int mi = 0; mi < 2; ++mi)
#pragma unroll
    for (int ni = 0; ni < 4; ++ni)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[mi][ni][e] = 0.f;

  const uint32_t* A32 = reinterpret_cast<const uint32_t*>(As);
  const uint32_t* B32 = reinterpret_cast<const uint32_t*>(Bs);
  constexpr int LDW = PJ_LD / 2;
#pragma unroll 4
  for (int kt = 0; kt < PJ_K / 16; ++kt) {
    uint32_t a[2][4];
#pragma unroll
    for (int mi = 0; mi < 2; ++mi) {
      const int r = wm * 32 + mi * 16 + g;
      a[mi][0] = A32[r * LDW + kt * 8 + tig];
      a[mi][1] = A32[(r + 8) * LDW + kt * 8 + tig];
      a[mi][2] = A32[r * LDW + kt * 8 + 4 + tig];
      a[mi][3] = A32[(r + 8) * LDW + kt * 8 + 4 + tig];
    }
#pragma unroll
    for (int ni = 0; ni < 4; ++ni) {
      const int n = wn * 32 + ni * 8 + g;
      const uint32_t b0 = B32[n * LDW + kt * 8 + tig];
      const uint32_t b1 = B32[n * LDW + kt * 8 + 4 + tig];
#pragma unroll
      for (int mi = 0; mi < 2; ++mi) mma_bf16_16816(acc[mi][ni], a[mi], b0, b1);
    }
  }

#pragma unroll
  for (int ni = 0; ni < 4; ++ni) {
    const int col = col0 + wn * 32 + ni * 8 + tig * 2;
    if (col >= n_cols) continue;
    const float bias0 = b_ih[col] + b_hh[col], bias1 = b_ih[col + 1] + b_hh[col + 1];
#pragma unroll
    for (int mi = 0; mi < 2; ++mi) {
      const long long r = row0 + wm * 32 + mi * 16 + g;
      if (r < n_rows)
        *reinterpret_cast<float2*>(P + r * n_cols + col) = make_float2(acc[mi][ni][0] + bias0, acc[mi][ni][1] + bias1);
      if (r + 8 < n_rows)
        *reinterpret_cast<float2*>(P + (r + 8) * n_cols + col) = make_float2(acc[mi][ni][2] + bias0, acc[mi][ni][3] + bias1);
    }
  }
}

cudaError_t launch_gate_proj(const LayerView& v, int t0, int t1, const uint16_t* W_ih, const float* b_ih,
                             const float* b_hh, int d_g, float* P, cudaStream_t st) {
  const int n_range = t1 - t0;
  const long long n_rows = (long long)v.S * n_range;
  if (n_rows <= 0) return cudaSuccess;
  const int n_cols = 4 * d_g;
  constexpr int smem = (PJ_TM + PJ_TN) * PJ_LD * 2;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(kve_gate_proj_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  dim3 grid((unsigned)((n_rows + PJ_TM - 1) / PJ_TM), (unsigned)((n_cols + PJ_TN - 1) / PJ_TN));
  kve_gate_proj_kernel<<<grid, PJ_THREADS, smem, st>>>(v, t0, n_range, n_rows, W_ih, b_ih, b_hh, n_cols, P);
  return cudaGetLastError();
}

}  // namespace kve

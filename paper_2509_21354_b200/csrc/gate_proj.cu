// Gate input projection (Eq. 3, the W_ih x_t term for all chunks at once):
//   P[s, t, :] = W_ih [Kbar_t ; Vbar_t] + b_ih + b_hh      a GEMM [S * n_range, 256] x [256, 4 d_g]
// bf16 operands (the rounded summaries and bf16 weights, so every product is exact), fp32
// accumulation in tensor memory (tcgen05.mma, M = 128, N = 256 per instruction), bias fused in the
// epilogue.
//
//  * A CTA owns one 256-column slice of W_ih^T for its whole life: the slice (128 KB, K-major,
//    128-byte swizzle) is written to shared memory once.
//  * It then walks over 128-row tiles of X.  The rows are gathered straight from the summary store
//    (columns 0..127 of a row from ksum_bf16, 128..255 from vsum_bf16) into the swizzled A tile
//    (64 KB), one thread issues the 16 MMAs of the tile (K = 256 in steps of 16) and commits them
//    to an mbarrier; all eight warps then read the 128 x 256 fp32 accumulator out of tensor
//    memory (warp w: lanes 32 (w % 4) .., column half w / 4), add the bias and store P.
//  * The only wait (on the MMA commit) is bounded; on give-up the status word gets KVE_ERR_TIMEOUT.
#include "common.cuh"
#include "kernels.h"
#include "umma.cuh"

namespace kve {

constexpr int PJ_M = 128, PJ_N = 256, PJ_K = 2 * D;
constexpr int PJ_KB = PJ_K / umma::KBLOCK_ELEMS;            // 4 K-blocks of 64
constexpr int PJ_THREADS = 256;
constexpr int PJ_A_KB_BYTES = PJ_M * umma::KBLOCK_ROW_BYTES;   // 16 KB
constexpr int PJ_B_KB_BYTES = PJ_N * umma::KBLOCK_ROW_BYTES;   // 32 KB
constexpr int PJ_SMEM_B = 0;
constexpr int PJ_SMEM_A = PJ_SMEM_B + PJ_KB * PJ_B_KB_BYTES;   // 128 KB
constexpr int PJ_SMEM_BIAS = PJ_SMEM_A + PJ_KB * PJ_A_KB_BYTES;   // +64 KB
constexpr int PJ_SMEM_BAR = PJ_SMEM_BIAS + PJ_N * 4;
constexpr int PJ_SMEM_BYTES = PJ_SMEM_BAR + 16 + 1024;         // + slack to reach a 1024-byte boundary

__global__ void __launch_bounds__(PJ_THREADS, 1) kve_gate_proj_kernel(LayerView v, int t0, int n_range, long long n_rows,
                                                                      const uint16_t* __restrict__ W_ih,
                                                                      const float* __restrict__ b_ih,
                                                                      const float* __restrict__ b_hh, int n_cols,
                                                                      float* __restrict__ P) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* Bs = smem + PJ_SMEM_B;
  unsigned char* As = smem + PJ_SMEM_A;
  float* bias = reinterpret_cast<float*>(smem + PJ_SMEM_BIAS);
  uint64_t* bar = reinterpret_cast<uint64_t*>(smem + PJ_SMEM_BAR);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + PJ_SMEM_BAR + 8);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int col0 = blockIdx.x * PJ_N;
  const long long n_tiles = (n_rows + PJ_M - 1) / PJ_M;

  // ---- one-time set-up: weight slice, bias, tensor memory, barrier ---------------------------------
  for (int i = tid; i < PJ_N * 32; i += PJ_THREADS) {
    const int r = i >> 5, p = i & 31;                 // p: 16-byte piece of the 512-byte weight row
    const uint4 val = __ldg(reinterpret_cast<const uint4*>(W_ih + (long long)(col0 + r) * PJ_K) + p);
    *reinterpret_cast<uint4*>(Bs + (p >> 3) * PJ_B_KB_BYTES + umma::piece_offset(r, p & 7)) = val;
  }
  for (int i = tid; i < PJ_N; i += PJ_THREADS) bias[i] = b_ih[col0 + i] + b_hh[col0 + i];
  if (warp == 0) umma::tmem_alloc(tmem_slot, PJ_N);
  if (tid == 0) {
    mbar_init(bar, 1);
    mbar_fence_init();
  }
  umma::fence_before_sync();
  __syncthreads();
  umma::fence_after_sync();
  const uint32_t tmem_d = *tmem_slot;
  constexpr uint32_t idesc = umma::instr_desc_bf16(PJ_M, PJ_N);
  const uint32_t a_base = smem_u32(As), b_base = smem_u32(Bs);

  uint32_t phase = 0;
  bool ok = true;
  for (long long tile = blockIdx.y; tile < n_tiles; tile += gridDim.y) {
    const long long row0 = tile * PJ_M;
    // ---- gather the A tile ------------------------------------------------------------------------
#pragma unroll 4
    for (int i = tid; i < PJ_M * 32; i += PJ_THREADS) {
      const int r = i >> 5, p = i & 31;
      const long long gr = row0 + r;
      uint4 val = make_uint4(0, 0, 0, 0);
      if (gr < n_rows) {
        const int s = (int)(gr / n_range);
        const int t = t0 + (int)(gr - (long long)s * n_range);
        const uint16_t* src = (p < 16 ? v.ksum_bf16 : v.vsum_bf16) + ((long long)s * v.max_chunks + t) * D + (p & 15) * 8;
        val = *reinterpret_cast<const uint4*>(src);
      }
      *reinterpret_cast<uint4*>(As + (p >> 3) * PJ_A_KB_BYTES + umma::piece_offset(r, p & 7)) = val;
    }
    umma::fence_smem_to_async();
    __syncthreads();

    // ---- 16 MMAs, one issuing thread -----------------------------------------------------------------
    if (tid == 0) {
      umma::fence_after_sync();
#pragma unroll
      for (int kb = 0; kb < PJ_KB; ++kb) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint64_t da = umma::smem_desc(a_base + kb * PJ_A_KB_BYTES + k * 32);
          const uint64_t db = umma::smem_desc(b_base + kb * PJ_B_KB_BYTES + k * 32);
          umma::mma_bf16(tmem_d, da, db, idesc, (kb | k) != 0);
        }
      }
      umma::commit(bar);
    }
    ok = mbar_wait_bounded(bar, phase);
    phase ^= 1;
    if (__syncthreads_or(!ok)) {
      if (tid == 0) set_status(v.status, ERR_TIMEOUT);
      break;
    }
    umma::fence_after_sync();

    // ---- epilogue: accumulator + bias -> P ----------------------------------------------------------------
    {
      const int lg = warp & 3, half = warp >> 2;
      const long long row = row0 + lg * 32 + lane;
#pragma unroll 1
      for (int cc = 0; cc < 4; ++cc) {
        const int c = half * 128 + cc * 32;
        float acc[32];
        umma::tmem_ld32(tmem_d + ((uint32_t)(lg * 32) << 16) + (uint32_t)c, acc);
        if (row < n_rows) {
          float4* dst = reinterpret_cast<float4*>(P + row * n_cols + col0 + c);
#pragma unroll
          for (int j = 0; j < 8; ++j)
            dst[j] = make_float4(acc[4 * j] + bias[c + 4 * j], acc[4 * j + 1] + bias[c + 4 * j + 1],
                                 acc[4 * j + 2] + bias[c + 4 * j + 2], acc[4 * j + 3] + bias[c + 4 * j + 3]);
        }
      }
    }
    umma::fence_before_sync();
    __syncthreads();     // the accumulator and the A tile are free again
  }

  umma::fence_before_sync();
  __syncthreads();
  if (warp == 0) umma::tmem_dealloc(tmem_d, PJ_N);
}

cudaError_t launch_gate_proj(const LayerView& v, int t0, int t1, const uint16_t* W_ih, const float* b_ih,
                             const float* b_hh, int d_g, float* P, cudaStream_t st) {
  const int n_range = t1 - t0;
  const long long n_rows = (long long)v.S * n_range;
  if (n_rows <= 0) return cudaSuccess;
  const int n_cols = 4 * d_g;                     // 256, 512 or 1024: whole 256-column slices
  if (n_cols % PJ_N != 0) return cudaErrorInvalidValue;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(kve_gate_proj_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PJ_SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const int col_slices = n_cols / PJ_N;
  const long long n_tiles = (n_rows + PJ_M - 1) / PJ_M;
  long long row_ctas = 148 / col_slices;          // one CTA per SM (shared memory), every slice equally served
  if (row_ctas > n_tiles) row_ctas = n_tiles;
  if (row_ctas < 1) row_ctas = 1;
  dim3 grid((unsigned)col_slices, (unsigned)row_ctas);
  kve_gate_proj_kernel<<<grid, PJ_THREADS, PJ_SMEM_BYTES, st>>>(v, t0, n_range, n_rows, W_ih, b_ih, b_hh, n_cols, P);
  return cudaGetLastError();
}

}  // namespace kve

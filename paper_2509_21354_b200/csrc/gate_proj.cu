// Gate input projection (Eq. 3, the W_ih x_t term for all chunks at once):
//   P[s, t, :] = W_ih [Kbar_t ; Vbar_t] + b_ih + b_hh      a GEMM [S * n_range, 256] x [256, 4 d_g]
// stored with the four gates of a hidden unit side by side (column 4 u + gate)
// bf16 operands (the rounded summaries and bf16 weights, so every product is exact), fp32
// accumulation in tensor memory (tcgen05.mma, M = 128, N = 256 per instruction), bias fused in the
// epilogue.
//
//  * A CTA owns one 256-column slice of W_ih^T for its whole life: the slice (128 KB, K-major,
//    128-byte swizzle) goes to shared memory once, by cp.async.
//  * It then walks over 128-row tiles of X.  The rows are gathered straight from the summary store
//    (columns 0..127 of a row from ksum_bf16, 128..255 from vsum_bf16) into the swizzled A tile
//    (64 KB) by cp.async copies that are all in flight at once; one thread issues the 16 MMAs of
//    the tile (K = 256 in steps of 16) and commits them to an mbarrier.
//  * Two accumulators in tensor memory: while the eight warps read tile i out of one (warp w: lanes
//    32 (w % 4) .., column half w / 4), add the bias and store P, the A tile of tile i+1 is gathered
//    and its MMAs run into the other.  The epilogue turns each 32 x 32 block through shared memory
//    so that a store instruction writes whole 128-byte row segments.
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
constexpr int PJ_SMEM_STG = PJ_SMEM_BAR + 16;                  // per warp: a 32 x 32 fp32 block on its way out
constexpr int PJ_SMEM_BYTES = PJ_SMEM_STG + (PJ_THREADS / 32) * 4096 + 1024;   // + slack to reach a 1024-byte boundary

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
  float* stg = reinterpret_cast<float*>(smem + PJ_SMEM_STG) + (threadIdx.x >> 5) * 1024;

  pdl_launch_dependents();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int col0 = blockIdx.x * PJ_N;
  const long long n_tiles = (n_rows + PJ_M - 1) / PJ_M;

  // ---- one-time set-up: weight slice, bias, tensor memory, barrier ---------------------------------
  for (int i = tid; i < PJ_N * 32; i += PJ_THREADS) {
    const int r = i >> 5, p = i & 31;                 // p: 16-byte piece of the 512-byte weight row
    // column c of P holds gate c & 3 of hidden unit c >> 2 (the four pre-activations of a unit side by side: the
    // recurrence fetches them with one 16-byte load): row (c & 3) d_g + (c >> 2) of W_ih
    const int c = col0 + r, d_g = n_cols >> 2;
    cp_async16(Bs + (p >> 3) * PJ_B_KB_BYTES + umma::piece_offset(r, p & 7),
               reinterpret_cast<const uint4*>(W_ih + (long long)((c & 3) * d_g + (c >> 2)) * PJ_K) + p, true);
  }
  for (int i = tid; i < PJ_N; i += PJ_THREADS) {
    const int c = col0 + i, row = (c & 3) * (n_cols >> 2) + (c >> 2);
    bias[i] = b_ih[row] + b_hh[row];
  }
  if (warp == 0) umma::tmem_alloc(tmem_slot, 2 * PJ_N);      // two accumulators: MMAs of tile i+1 overlap the epilogue of tile i
  if (tid == 0) {
    mbar_init(bar, 1);
    mbar_fence_init();
  }
  const uint32_t a_base = smem_u32(As), b_base = smem_u32(Bs);
  constexpr uint32_t idesc = umma::instr_desc_bf16(PJ_M, PJ_N);

  // gathers the A tile of `tile` (asynchronous copies, zero fill beyond the last row).  A thread
  // keeps its 16-byte column p and walks down 16 rows; 32-bit index arithmetic, one division per row
  // (the host checks that S * n_range and S * max_chunks fit 31 bits).
  auto gather_a = [&](long long tile) {
    const uint32_t row0 = (uint32_t)tile * PJ_M, nr = (uint32_t)n_range, total = (uint32_t)n_rows;
    const int p = tid & 31;
    const uint16_t* base = (p < 16 ? v.ksum_bf16 : v.vsum_bf16) + (p & 15) * 8;
    unsigned char* dst0 = As + (p >> 3) * PJ_A_KB_BYTES;
#pragma unroll 8
    for (int r = tid >> 5; r < PJ_M; r += PJ_THREADS / 32) {
      const uint32_t gr = row0 + r;
      const bool live = gr < total;
      const uint32_t grc = live ? gr : 0u;
      const uint32_t s = grc / nr;
      const uint32_t t = (uint32_t)t0 + (grc - s * nr);
      cp_async16(dst0 + umma::piece_offset(r, p & 7), base + (size_t)(s * (uint32_t)v.max_chunks + t) * D, live);
    }
  };
  // one thread: the 16 MMAs of a tile into accumulator `acc_sel`, then commit to the barrier
  auto issue_mma = [&](uint32_t tmem_acc) {
    umma::fence_after_sync();
#pragma unroll
    for (int kb = 0; kb < PJ_KB; ++kb) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint64_t da = umma::smem_desc(a_base + kb * PJ_A_KB_BYTES + k * 32);
        const uint64_t db = umma::smem_desc(b_base + kb * PJ_B_KB_BYTES + k * 32);
        umma::mma_bf16(tmem_acc, da, db, idesc, (kb | k) != 0);
      }
    }
    umma::commit(bar);
  };
  // half of the accumulator columns of this warp's lanes + bias -> P.  tcgen05.ld hands a thread one
  // row (32 columns); the block is turned through the staging area (16-byte groups, group q of row
  // r at position q ^ (r & 7): conflict-free both ways) so that a store instruction covers four
  // rows with 128 contiguous bytes each.
  auto epilogue_half = [&](uint32_t tmem_acc, long long row0, int part) {
    const int lg = warp & 3, half = warp >> 2;
#pragma unroll 1
    for (int cc = 2 * part; cc < 2 * part + 2; ++cc) {
      const int c = half * 128 + cc * 32;
      float acc[32];
      umma::tmem_ld32(tmem_acc + ((uint32_t)(lg * 32) << 16) + (uint32_t)c, acc);
#pragma unroll
      for (int q = 0; q < 8; ++q)
        *reinterpret_cast<float4*>(stg + lane * 32 + ((q ^ (lane & 7)) << 2)) =
            make_float4(acc[4 * q] + bias[c + 4 * q], acc[4 * q + 1] + bias[c + 4 * q + 1],
                        acc[4 * q + 2] + bias[c + 4 * q + 2], acc[4 * q + 3] + bias[c + 4 * q + 3]);
      __syncwarp();
      const int q = lane & 7;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int rr = i * 4 + (lane >> 3);
        const float4 val = *reinterpret_cast<const float4*>(stg + rr * 32 + ((q ^ (rr & 7)) << 2));
        const long long row = row0 + lg * 32 + rr;
        if (row < n_rows) *reinterpret_cast<float4*>(P + row * n_cols + col0 + c + q * 4) = val;
      }
      __syncwarp();
    }
  };

  pdl_wait();      // the weight slice is on its way; the summaries come from the previous kernel
  long long tile = blockIdx.y;
  if (tile < n_tiles) gather_a(tile);
  cp_async_wait_all();
  umma::fence_smem_to_async();
  umma::fence_before_sync();
  __syncthreads();
  umma::fence_after_sync();
  const uint32_t tmem_d = *tmem_slot;
  if (tile < n_tiles && tid == 0) issue_mma(tmem_d);

  uint32_t phase = 0, sel = 0;
  for (; tile < n_tiles; tile += gridDim.y) {
    const long long next = tile + gridDim.y;
    const bool ok = mbar_wait_bounded(bar, phase);      // this tile's MMAs are done: the A tile is free
    phase ^= 1;
    if (__syncthreads_or(!ok)) {
      if (tid == 0) set_status(v.status, ERR_TIMEOUT);
      break;
    }
    umma::fence_after_sync();
    if (next < n_tiles) gather_a(next);                 // in flight during the first half of the epilogue
    epilogue_half(tmem_d + sel * PJ_N, tile * PJ_M, 0);
    if (next < n_tiles) {
      cp_async_wait_all();
      umma::fence_smem_to_async();
      umma::fence_before_sync();
      __syncthreads();                                  // also: the other accumulator was drained an iteration ago
      if (tid == 0) issue_mma(tmem_d + (sel ^ 1) * PJ_N);
    }
    epilogue_half(tmem_d + sel * PJ_N, tile * PJ_M, 1);
    sel ^= 1;
  }

  umma::fence_before_sync();
  __syncthreads();
  if (warp == 0) umma::tmem_dealloc(tmem_d, 2 * PJ_N);
}

cudaError_t launch_gate_proj(const LayerView& v, int t0, int t1, const uint16_t* W_ih, const float* b_ih,
                             const float* b_hh, int d_g, float* P, cudaStream_t st) {
  const int n_range = t1 - t0;
  const long long n_rows = (long long)v.S * n_range;
  if (n_rows <= 0) return cudaSuccess;
  const int n_cols = 4 * d_g;                     // 256, 512 or 1024: whole 256-column slices
  if (n_cols % PJ_N != 0) return cudaErrorInvalidValue;
  if (n_rows + PJ_M >= (1LL << 31) || (long long)v.S * v.max_chunks >= (1LL << 31)) return cudaErrorInvalidValue;
  static DeviceFlags opted;
  {
    cudaError_t e = smem_opt_in(opted, kve_gate_proj_kernel, PJ_SMEM_BYTES);
    if (e != cudaSuccess) return e;
  }
  const int col_slices = n_cols / PJ_N;
  const long long n_tiles = (n_rows + PJ_M - 1) / PJ_M;
  long long row_ctas = sm_count() / col_slices;          // one CTA per SM (shared memory), every slice equally served
  if (row_ctas > n_tiles) row_ctas = n_tiles;
  if (row_ctas < 1) row_ctas = 1;
  dim3 grid((unsigned)col_slices, (unsigned)row_ctas);
  return launch_pdl(kve_gate_proj_kernel, grid, dim3(PJ_THREADS), PJ_SMEM_BYTES, st, v, t0, n_range, n_rows, W_ih, b_ih, b_hh, n_cols, P);
}

}  // namespace kve

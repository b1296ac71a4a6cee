// kvE_summarize_chunks kernels (Eq. 2): per (sequence, chunk) the mean of the chunk's C key rows and
// of its C value rows, then (AGG_MLP) a 2-layer GELU MLP on each mean.
//
// chunk_mean: HBM-bound.  One warp per (sequence, chunk): lanes 0-15 stream the K page, lanes 16-31 the
// V page, 16 bytes per lane per row, rows added in temporal order in fp32 (so the sum has the same
// rounding as a plain sequential loop), divided by C with an IEEE division.
#include "common.cuh"
#include "kernels.h"
#include "umma.cuh"
#include "gelu.cuh"

namespace kve {

constexpr int MEAN_WARPS = 8;
constexpr int MEAN_UNROLL = 8;

__device__ __forceinline__ void add_row(float (&acc)[8], const uint4& w) {
  acc[0] += bf16lo(w.x); acc[1] += bf16hi(w.x);
  acc[2] += bf16lo(w.y); acc[3] += bf16hi(w.y);
  acc[4] += bf16lo(w.z); acc[5] += bf16hi(w.z);
  acc[6] += bf16lo(w.w); acc[7] += bf16hi(w.w);
}

__device__ __forceinline__ void max_row(float (&acc)[8], const uint4& w) {
  acc[0] = fmaxf(acc[0], bf16lo(w.x)); acc[1] = fmaxf(acc[1], bf16hi(w.x));
  acc[2] = fmaxf(acc[2], bf16lo(w.y)); acc[3] = fmaxf(acc[3], bf16hi(w.y));
  acc[4] = fmaxf(acc[4], bf16lo(w.z)); acc[5] = fmaxf(acc[5], bf16hi(w.z));
  acc[6] = fmaxf(acc[6], bf16lo(w.w)); acc[7] = fmaxf(acc[7], bf16hi(w.w));
}

// POOL_MAX: element-wise maximum of the chunk instead of its mean (the "pooling" aggregator of Sec. 3.1)
template <bool POOL_MAX>
__global__ void __launch_bounds__(MEAN_WARPS * 32) kve_chunk_mean_kernel(LayerView v, int t0, int n_range,
                                                                        long long n_units, int final_output, int dev_window) {
  pdl_launch_dependents();
  pdl_wait();
  if (dev_window >= 0) {      // one chunk per sequence, found on the device
    const NextChunk nx = next_chunk(v.n_listed, v.seq_len, v.C, dev_window, v.max_chunks);
    if (!nx.due) return;
    t0 = nx.t;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // persistent warps: unit = global warp id, then strides of the whole grid
  for (long long unit = (long long)blockIdx.x * MEAN_WARPS + warp; unit < n_units; unit += (long long)gridDim.x * MEAN_WARPS) {
  const int s = (int)(unit / n_range);
  const int t = t0 + (int)(unit - (long long)s * n_range);
  const int is_v = lane >> 4, l16 = lane & 15;
  const long long page = v.page_table[(long long)s * v.max_chunks + t];
  if (page < 0 || page >= v.n_pages) {
    if (lane == 0) set_status(v.status, ERR_CAPACITY);
    continue;
  }
  const uint4* src = reinterpret_cast<const uint4*>((is_v ? v.v_pages : v.k_pages) + page * v.C * D) + l16;
  float acc[8];
#pragma unroll
  for (int x = 0; x < 8; ++x) acc[x] = POOL_MAX ? -INFINITY : 0.f;
  int j = 0;
  for (; j + MEAN_UNROLL <= v.C; j += MEAN_UNROLL) {
    uint4 w[MEAN_UNROLL];
#pragma unroll
    for (int u = 0; u < MEAN_UNROLL; ++u) w[u] = __ldcs(src + (long long)(j + u) * 16);
#pragma unroll
    for (int u = 0; u < MEAN_UNROLL; ++u) {
      if (POOL_MAX) max_row(acc, w[u]); else add_row(acc, w[u]);
    }
  }
  for (; j < v.C; ++j) {
    const uint4 w1 = __ldcs(src + (long long)j * 16);
    if (POOL_MAX) max_row(acc, w1); else add_row(acc, w1);
  }
  if (!POOL_MAX) {
    const float fc = (float)v.C;
#pragma unroll
    for (int x = 0; x < 8; ++x) acc[x] = __fdiv_rn(acc[x], fc);
  }

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
}

// CTAs of the mean kernel that are resident per SM (registers decide), looked up once per device
template <bool POOL_MAX>
static int mean_ctas_per_sm() {
  static std::atomic<int> cached[MAX_DEVICES];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return 4;
  int n = cached[dev].load(std::memory_order_acquire);
  if (n > 0) return n;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kve_chunk_mean_kernel<POOL_MAX>, MEAN_WARPS * 32, 0) != cudaSuccess || n <= 0) n = 4;
  cached[dev].store(n, std::memory_order_release);
  return n;
}

// The grid is exactly one resident wave and every warp strides over the units, so all SMs carry the same share.
// That only holds if the CTAs land on an empty GPU: the kernel is therefore launched WITHOUT the programmatic edge the
// other kernels use.  (Launched early, beside the tail of its predecessor, its CTAs spread unevenly over the SMs
// and the static striding turns that into a tail: measured +25 % on 4 GB of stale KV.)
cudaError_t launch_chunk_mean(const LayerView& v, int t0, int t1, bool final_output, bool pool_max, cudaStream_t st, int dev_window) {
  const int n_range = dev_window >= 0 ? 1 : t1 - t0;
  const long long n_units = (long long)v.S * n_range;
  if (n_units <= 0) return cudaSuccess;
  long long blocks = (n_units + MEAN_WARPS - 1) / MEAN_WARPS;
  const long long wave = (long long)sm_count() * (pool_max ? mean_ctas_per_sm<true>() : mean_ctas_per_sm<false>());
  if (blocks > wave) blocks = wave;
  if (pool_max) kve_chunk_mean_kernel<true><<<dim3((unsigned)blocks), dim3(MEAN_WARPS * 32), 0, st>>>(v, t0, n_range, n_units, 1, dev_window);
  else kve_chunk_mean_kernel<false><<<dim3((unsigned)blocks), dim3(MEAN_WARPS * 32), 0, st>>>(v, t0, n_range, n_units, final_output ? 1 : 0, dev_window);
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
                                                                   MlpWeights w, int d_sum, int dev_window) {
  pdl_launch_dependents();
  pdl_wait();
  if (dev_window >= 0) {      // one chunk per sequence, found on the device
    const NextChunk nx = next_chunk(v.n_listed, v.seq_len, v.C, dev_window, v.max_chunks);
    if (!nx.due) return;
    t0 = nx.t;
  }
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

// ---- the same MLP on the 5th-generation tensor cores (d_sum a multiple of 64, at most 256) ----------------
// Both layers are GEMMs over a tile of 128 (sequence, chunk) units:
//   H = M W1^T  (128 x d_sum, K = 128),   Y = gelu(H + b1) W2^T  (128 x 128, K = d_sum).
// The left operands (the chunk means, the activations) are fp32.  Each is split exactly into three
// bf16 planes (x = p0 + p1 + p2), the weights are bf16 by definition, so every product the tensor
// core forms is exact and the result differs from a plain fp32 loop only in summation order.
//  * A CTA serves one side (keys or values) and keeps that side's W1 and W2 (64 KB each, K-major,
//    128-byte swizzle) in shared memory for all its tiles.
//  * Layer 1: 24 tcgen05.mma (3 planes x K/16) of shape 128 x d_sum accumulate H in tensor memory.
//  * Layer 2 runs in slices of 64 hidden units: the eight warps read a slice of H from tensor
//    memory, add b1, apply the erf GELU, split into planes and store them as the next A operand
//    (double-buffered, 48 KB per slice, in the space the layer-1 planes have left); one thread
//    issues the slice's 12 MMAs into the second accumulator while the warps prepare the next slice.
//  * Epilogue: Y + b2 -> fp32 summary and its bf16 rounding.
// Every mbarrier wait is bounded; on give-up the status word gets KVE_ERR_TIMEOUT.
constexpr int MT_M = 128;
constexpr int MT_THREADS = 512;   // 16 warps: four per scheduler, to hide the latency of the GELU / split phases
constexpr int MT_MAX_DSUM = 256;
constexpr int MT_PLANE_KB_BYTES = MT_M * umma::KBLOCK_ROW_BYTES;          // 16 KB: one plane, one K-block of 64
constexpr int MT_SMEM_A = 0;                                              // 96 KB: 3 planes x 2 K-blocks, later 2 x (3 planes x 1)
constexpr int MT_SMEM_W1 = MT_SMEM_A + 6 * MT_PLANE_KB_BYTES;
constexpr int MT_SMEM_W2 = MT_SMEM_W1 + MT_MAX_DSUM * D * 2;
constexpr int MT_SMEM_B1 = MT_SMEM_W2 + D * MT_MAX_DSUM * 2;
constexpr int MT_SMEM_B2 = MT_SMEM_B1 + MT_MAX_DSUM * 4;
constexpr int MT_SMEM_BAR = MT_SMEM_B2 + D * 4;
constexpr int MT_SMEM_BYTES = MT_SMEM_BAR + 64 + 1024;                    // + slack to reach a 1024-byte boundary
constexpr int MT_TMEM_COLS = 512;                                         // H: columns [0, d_sum), Y: columns [256, 384)
constexpr int MT_TMEM_Y = 256;

// splits 8 consecutive fp32 values and stores the three 16-byte pieces at dst + pl * plane_stride
__device__ __forceinline__ void store_split8(const float (&x)[8], unsigned char* dst, int plane_stride) {
  uint32_t w[4][3];
#pragma unroll
  for (int e = 0; e < 4; ++e) split3_pair(x[2 * e], x[2 * e + 1], w[e]);
#pragma unroll
  for (int pl = 0; pl < 3; ++pl)
    *reinterpret_cast<uint4*>(dst + pl * plane_stride) = make_uint4(w[0][pl], w[1][pl], w[2][pl], w[3][pl]);
}

__global__ void __launch_bounds__(MT_THREADS, 1) kve_chunk_mlp_tc_kernel(LayerView v, int t0, int n_range, long long n_units,
                                                                         MlpWeights w, int d_sum, int dev_window) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* As = smem + MT_SMEM_A;
  unsigned char* W1s = smem + MT_SMEM_W1;
  unsigned char* W2s = smem + MT_SMEM_W2;
  float* b1s = reinterpret_cast<float*>(smem + MT_SMEM_B1);
  float* b2s = reinterpret_cast<float*>(smem + MT_SMEM_B2);
  uint64_t* bar_h = reinterpret_cast<uint64_t*>(smem + MT_SMEM_BAR);       // layer-1 MMAs done
  uint64_t* bar_buf = bar_h + 1;                                            // [2]: slice MMAs that read buffer b done
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + MT_SMEM_BAR + 32);

  pdl_launch_dependents();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int side = blockIdx.y;
  const uint16_t* W1 = side ? w.W1V : w.W1K;
  const uint16_t* W2 = side ? w.W2V : w.W2K;
  const float* b1 = side ? w.b1V : w.b1K;
  const float* b2 = side ? w.b2V : w.b2K;
  float* sum_f32 = side ? v.vsum_f32 : v.ksum_f32;
  uint16_t* sum_b16 = side ? v.vsum_bf16 : v.ksum_bf16;
  const int n_slices = d_sum / 64;
  const long long n_tiles = (n_units + MT_M - 1) / MT_M;

  // ---- one-time set-up -----------------------------------------------------------------------------
  for (int i = tid; i < d_sum * 16; i += MT_THREADS) {              // W1 [d_sum][128]: rows of 16 pieces, 2 K-blocks
    const int r = i >> 4, p = i & 15;
    cp_async16(W1s + (p >> 3) * (d_sum * umma::KBLOCK_ROW_BYTES) + umma::piece_offset(r, p & 7),
               reinterpret_cast<const uint4*>(W1 + (long long)r * D) + p, true);
  }
  const int w2_pieces = d_sum / 8;
  for (int i = tid; i < D * w2_pieces; i += MT_THREADS) {           // W2 [128][d_sum]: n_slices K-blocks of 16 KB
    const int r = i / w2_pieces, p = i - r * w2_pieces;
    cp_async16(W2s + (p >> 3) * MT_PLANE_KB_BYTES + umma::piece_offset(r, p & 7),
               reinterpret_cast<const uint4*>(W2 + (long long)r * d_sum) + p, true);
  }
  for (int i = tid; i < d_sum; i += MT_THREADS) b1s[i] = b1[i];
  for (int i = tid; i < D; i += MT_THREADS) b2s[i] = b2[i];
  if (warp == 0) umma::tmem_alloc(tmem_slot, MT_TMEM_COLS);
  if (tid == 0) {
    mbar_init(bar_h, 1);
    mbar_init(&bar_buf[0], 1);
    mbar_init(&bar_buf[1], 1);
    mbar_fence_init();
  }
  cp_async_wait_all();
  umma::fence_smem_to_async();
  umma::fence_before_sync();
  __syncthreads();
  umma::fence_after_sync();
  const uint32_t tmem_h = *tmem_slot, tmem_y = tmem_h + MT_TMEM_Y;
  const uint32_t idesc1 = umma::instr_desc_bf16(MT_M, d_sum), idesc2 = umma::instr_desc_bf16(MT_M, D);
  const uint32_t a_base = smem_u32(As), w1_base = smem_u32(W1s), w2_base = smem_u32(W2s);
  const int lg = warp & 3, part = warp >> 2;      // tensor-memory lanes 32 lg .., column part (0..3) of whatever is read
  const int row_in_tile = lg * 32 + lane;
  const uint32_t tmem_lane = (uint32_t)(lg * 32) << 16;

  pdl_wait();      // weights, barriers and tensor memory are set up; the chunk means come from the previous kernel
  uint32_t ph_h = 0, ph_buf[2] = {0, 0};
  bool failed = false, due = true;
  if (dev_window >= 0) {      // one chunk per sequence, found on the device
    const NextChunk nx = next_chunk(v.n_listed, v.seq_len, v.C, dev_window, v.max_chunks);
    due = nx.due;
    t0 = nx.t;
  }
  for (long long tile = blockIdx.x; tile < n_tiles && !failed && due; tile += gridDim.x) {
    const long long unit0 = tile * MT_M;
    // ---- chunk means -> three bf16 planes (layer-1 A operand) ------------------------------------------
    {
      // a thread keeps its 32-byte column pc and walks down 4 rows: all 8 loads first, then the splits
      // (32-bit index arithmetic, one division per row; the host checks the ranges)
      const int pc = tid & 15;
      const uint32_t u0 = (uint32_t)unit0, nr = (uint32_t)n_range, total = (uint32_t)n_units;
      float4 lo[4], hi[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t unit = u0 + (tid >> 4) + 32 * i;
        lo[i] = hi[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (unit < total) {
          const uint32_t s = unit / nr;
          const uint32_t t = (uint32_t)t0 + (unit - s * nr);
          const float4* src = reinterpret_cast<const float4*>(sum_f32 + (size_t)(s * (uint32_t)v.max_chunks + t) * D + pc * 8);
          lo[i] = src[0];
          hi[i] = src[1];
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int r = (tid >> 4) + 32 * i;
        const float x[8] = {lo[i].x, lo[i].y, lo[i].z, lo[i].w, hi[i].x, hi[i].y, hi[i].z, hi[i].w};
        // plane pl, K-block kb at (pl * 2 + kb) * 16 KB
        store_split8(x, As + (pc >> 3) * MT_PLANE_KB_BYTES + umma::piece_offset(r, pc & 7), 2 * MT_PLANE_KB_BYTES);
      }
    }
    umma::fence_smem_to_async();
    __syncthreads();
    if (tid == 0) {
      umma::fence_after_sync();
      bool acc = false;
#pragma unroll 1
      for (int pl = 2; pl >= 0; --pl)                 // smallest plane first
#pragma unroll
        for (int kb = 0; kb < 2; ++kb)
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            umma::mma_bf16(tmem_h, umma::smem_desc(a_base + (pl * 2 + kb) * MT_PLANE_KB_BYTES + k * 32),
                           umma::smem_desc(w1_base + kb * (d_sum * umma::KBLOCK_ROW_BYTES) + k * 32), idesc1, acc);
            acc = true;
          }
      umma::commit(bar_h);
    }
    {
      const bool ok = mbar_wait_bounded(bar_h, ph_h);
      ph_h ^= 1;
      if (__syncthreads_or(!ok)) { failed = true; break; }
    }
    umma::fence_after_sync();

    // ---- layer 2 in slices of 64 hidden units ------------------------------------------------------------
    for (int j = 0; j < n_slices; ++j) {
      const int buf = j & 1;
      if (j >= 2) {        // the MMAs of slice j - 2 still read this buffer
        const bool ok = mbar_wait_bounded(&bar_buf[buf], ph_buf[buf]);
        ph_buf[buf] ^= 1;
        if (__syncthreads_or(!ok)) { failed = true; break; }
      }
      float h[16];
      umma::tmem_ld16(tmem_h + tmem_lane + (uint32_t)(j * 64 + part * 16), h);
      unsigned char* abuf = As + buf * 3 * MT_PLANE_KB_BYTES;
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        float g[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) g[e] = gelu_tc(h[q * 8 + e] + b1s[j * 64 + part * 16 + q * 8 + e]);
        store_split8(g, abuf + umma::piece_offset(row_in_tile, part * 2 + q), MT_PLANE_KB_BYTES);
      }
      umma::fence_smem_to_async();
      umma::fence_before_sync();
      __syncthreads();
      if (tid == 0) {
        umma::fence_after_sync();
        const uint32_t ab = a_base + buf * 3 * MT_PLANE_KB_BYTES;
#pragma unroll 1
        for (int pl = 2; pl >= 0; --pl)
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma::mma_bf16(tmem_y, umma::smem_desc(ab + pl * MT_PLANE_KB_BYTES + k * 32),
                           umma::smem_desc(w2_base + j * MT_PLANE_KB_BYTES + k * 32), idesc2, !(j == 0 && pl == 2 && k == 0));
        umma::commit(&bar_buf[buf]);
      }
    }
    if (failed) break;
    // drain: one outstanding commit per buffer that was used (the later one covers every MMA before it)
    {
      bool ok = true;
      const int first = (n_slices >= 2) ? (n_slices & 1) : 0;     // older buffer first
      for (int u = 0; u < (n_slices >= 2 ? 2 : 1); ++u) {
        const int b = (first + u) & 1;
        ok = mbar_wait_bounded(&bar_buf[b], ph_buf[b]) && ok;
        ph_buf[b] ^= 1;
      }
      if (__syncthreads_or(!ok)) { failed = true; break; }
    }
    umma::fence_after_sync();

    // ---- epilogue: Y + b2 -> fp32 summary and its bf16 rounding ----------------------------------------------
    // The operand space is idle now: it holds the output row table and, per warp, a 32 x 32 block on
    // its way out.  tcgen05.ld hands a thread one row; the block is turned through shared memory
    // (16-byte groups, group q of row r at position q ^ (r & 7)) so that every store instruction
    // writes whole 128-byte (fp32) / 64-byte (bf16) row segments.
    {
      int* row_tab = reinterpret_cast<int*>(As + (MT_THREADS / 32) * 4096);       // [128] summary row, -1 beyond the end
      float* stg = reinterpret_cast<float*>(As) + warp * 1024;
      if (tid < MT_M) {
        const long long unit = unit0 + tid;
        int o = -1;
        if (unit < n_units) {
          const uint32_t s = (uint32_t)unit / (uint32_t)n_range;
          o = (int)(s * (uint32_t)v.max_chunks + (uint32_t)t0 + ((uint32_t)unit - s * (uint32_t)n_range));
        }
        row_tab[tid] = o;
      }
      __syncthreads();
      {
        const int c = part * 32;
        float y[32];
        umma::tmem_ld32(tmem_y + tmem_lane + (uint32_t)c, y);
#pragma unroll
        for (int q = 0; q < 8; ++q)
          *reinterpret_cast<float4*>(stg + lane * 32 + ((q ^ (lane & 7)) << 2)) =
              make_float4(y[4 * q] + b2s[c + 4 * q], y[4 * q + 1] + b2s[c + 4 * q + 1], y[4 * q + 2] + b2s[c + 4 * q + 2],
                          y[4 * q + 3] + b2s[c + 4 * q + 3]);
        __syncwarp();
        const int q = lane & 7;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int rr = i * 4 + (lane >> 3);
          const float4 val = *reinterpret_cast<const float4*>(stg + rr * 32 + ((q ^ (rr & 7)) << 2));
          const int orow = row_tab[lg * 32 + rr];
          if (orow >= 0) {
            const size_t o = (size_t)orow * D + c + q * 4;
            *reinterpret_cast<float4*>(sum_f32 + o) = val;
            *reinterpret_cast<uint2*>(sum_b16 + o) = make_uint2(pack_bf16x2(val.x, val.y), pack_bf16x2(val.z, val.w));
          }
        }
        __syncwarp();
      }
    }
    umma::fence_before_sync();
    __syncthreads();     // accumulators and operand space are free for the next tile
  }
  if (failed && tid == 0) set_status(v.status, ERR_TIMEOUT);

  umma::fence_before_sync();
  __syncthreads();
  if (warp == 0) umma::tmem_dealloc(tmem_h, MT_TMEM_COLS);
}

cudaError_t launch_chunk_mlp(const LayerView& v, int t0, int t1, const MlpWeights& w, int d_sum, cudaStream_t st, int dev_window) {
  const int n_range = dev_window >= 0 ? 1 : t1 - t0;
  const long long n_units = (long long)v.S * n_range;
  if (n_units <= 0) return cudaSuccess;
  if (d_sum % 64 == 0 && d_sum <= MT_MAX_DSUM && n_units + MT_M < (1LL << 31) &&
      (long long)v.S * v.max_chunks < (1LL << 31)) {
    static DeviceFlags opted_tc;
    {
      cudaError_t e = smem_opt_in(opted_tc, kve_chunk_mlp_tc_kernel, MT_SMEM_BYTES);
      if (e != cudaSuccess) return e;
    }
    const long long n_tiles = (n_units + MT_M - 1) / MT_M;
    const long long half = sm_count() / 2;
    const long long per_side = n_tiles < half ? n_tiles : half;  // one CTA per SM: half of the SMs per side
    dim3 grid((unsigned)per_side, 2);
    return launch_pdl(kve_chunk_mlp_tc_kernel, grid, dim3(MT_THREADS), MT_SMEM_BYTES, st, v, t0, n_range, n_units, w, d_sum, dev_window);
  }
  const size_t smem = sizeof(float) * (size_t)MLP_ROWS * (D + d_sum);
  static DeviceFlags opted;
  {
    cudaError_t e = smem_opt_in(opted, kve_chunk_mlp_kernel, (int)(sizeof(float) * MLP_ROWS * (D + 1024)));
    if (e != cudaSuccess) return e;
  }
  dim3 grid((unsigned)((n_units + MLP_ROWS - 1) / MLP_ROWS), 2);
  return launch_pdl(kve_chunk_mlp_kernel, grid, dim3(MLP_THREADS), smem, st, v, t0, n_range, n_units, w, d_sum, dev_window);
}

}  // namespace kve

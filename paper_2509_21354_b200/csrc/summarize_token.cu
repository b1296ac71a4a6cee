// KVE_AGG_TOKEN_MLP: Eq. 2 with the MLP acting on every token of the chunk, the C outputs mean-pooled:
//   Kbar = (1/C) sum_j [ W2 gelu(W1 k_j + b1) + b2 ]  =  W2 [ (1/C) sum_j gelu(W1 k_j + b1) ] + b2
// (the last layer is affine and the mean is linear, so the activations are pooled and the second layer
// runs once per chunk).  Two kernels:
//
//  kve_token_mlp_pool_kernel - the contraction [tokens, 128] x [128, d_sum] over EVERY stale token on the
//    5th-generation tensor cores, activation and pooling in the epilogue, one pass over the stale KV.
//    * A CTA serves one side (keys or values) and keeps that side's W1 (d_sum x 128 bf16, K-major,
//      128-byte swizzle) in shared memory.
//    * Tile = 128 consecutive tokens of one sequence's stale range (one or several whole chunks, or a
//      128-token slice of a longer chunk).  The token rows are bf16 already, so they are the A operand as
//      they stand: 16-byte asynchronous copies put a page's rows into the swizzled layout; 8 tcgen05.mma
//      (M 128, N d_sum, K 16 each) accumulate the pre-activations in tensor memory.
//    * Two A buffers and two accumulators: while the sixteen warps read tile i out of tensor memory (a thread
//      owns one token), add b1, apply the erf GELU and sum each column over the tokens of a chunk with a
//      butterfly of shuffles (lane l ends up with column l), tile i + 1 is gathered and multiplied.
//    * The pooled activations (1/C) sum_j gelu(...) go to a scratch row per (side, sequence, chunk).
//    Bound by the activation arithmetic (about 20 instructions per activation and 256 activations per
//    token and side), not by HBM or the tensor pipe.
//  kve_token_mlp_out_kernel - the second layer on the pooled activations, fp32 FMA: Kbar = W2 g + b2, written
//    as the fp32 summary and its bf16 rounding.
// The only wait (on the MMA commit) is bounded; on give-up the status word gets KVE_ERR_TIMEOUT.
#include "common.cuh"
#include "kernels.h"
#include "umma.cuh"
#include "gelu.cuh"

namespace kve {

constexpr int TM_M = 128;                                   // tokens per tile
constexpr int TM_THREADS = 512;                             // 16 warps: four per scheduler hide the latency of the activation chains
constexpr int TM_MAX_DSUM = 256;
constexpr int TM_KB_BYTES = TM_M * umma::KBLOCK_ROW_BYTES;  // 16 KB: 128 rows x 64 head dims
constexpr int TM_SMEM_W1 = 0;                               // 2 K-blocks of [d_sum rows][64]: up to 64 KB
constexpr int TM_SMEM_A = TM_SMEM_W1 + 2 * TM_MAX_DSUM * umma::KBLOCK_ROW_BYTES;   // 2 buffers x 2 K-blocks: 64 KB
constexpr int TM_SMEM_B1 = TM_SMEM_A + 2 * 2 * TM_KB_BYTES;
constexpr int TM_SMEM_POOL = TM_SMEM_B1 + TM_MAX_DSUM * 4;  // [4 chunks of a tile][d_sum] running column sums
constexpr int TM_SMEM_ROWS = TM_SMEM_POOL + 4 * TM_MAX_DSUM * 4;       // [128] source row of every tile row (-1: none)
constexpr int TM_SMEM_BAR = TM_SMEM_ROWS + TM_M * 8;
constexpr int TM_SMEM_BYTES = TM_SMEM_BAR + 32 + 1024;      // + slack to reach a 1024-byte boundary
constexpr int TM_TMEM_COLS = 512;                           // two accumulators of up to 256 columns
static_assert(TM_SMEM_BYTES > 116 * 1024, "one CTA per SM: each allocates all of tensor memory");

struct TokenMlpArgs {
  LayerView v;
  int t0, n_range;           // chunks [t0, t0 + n_range) of every sequence
  int d_sum;
  int tiles_per_item;        // max(1, C / 128): 128-token tiles of one chunk
  int units_per_item;        // max(1, 128 / C): chunks in one tile
  long long n_units, n_items;
  MlpWeights w;
  float* hid;                // [2][n_units][d_sum] pooled activations (side, unit = s * n_range + (t - t0))
};

__global__ void __launch_bounds__(TM_THREADS, 1) kve_token_mlp_pool_kernel(TokenMlpArgs a) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* W1s = smem + TM_SMEM_W1;
  unsigned char* As = smem + TM_SMEM_A;
  float* b1s = reinterpret_cast<float*>(smem + TM_SMEM_B1);
  float* pool = reinterpret_cast<float*>(smem + TM_SMEM_POOL);
  long long* row_src = reinterpret_cast<long long*>(smem + TM_SMEM_ROWS);
  uint64_t* bar = reinterpret_cast<uint64_t*>(smem + TM_SMEM_BAR);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + TM_SMEM_BAR + 8);

  pdl_launch_dependents();
  const LayerView& v = a.v;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int side = blockIdx.y, d_sum = a.d_sum;
  const uint16_t* W1 = side ? a.w.W1V : a.w.W1K;
  const float* b1 = side ? a.w.b1V : a.w.b1K;
  const uint16_t* pages = side ? v.v_pages : v.k_pages;

  // ---- one-time set-up: W1 of this side, b1, cleared pools, tensor memory, barrier -----------------------
  for (int i = tid; i < d_sum * 16; i += TM_THREADS) {              // W1 [d_sum][128]: rows of 16 pieces, 2 K-blocks
    const int r = i >> 4, p = i & 15;
    cp_async16(W1s + (p >> 3) * (d_sum * umma::KBLOCK_ROW_BYTES) + umma::piece_offset(r, p & 7),
               reinterpret_cast<const uint4*>(W1 + (long long)r * D) + p, true);
  }
  for (int i = tid; i < d_sum; i += TM_THREADS) b1s[i] = b1[i];
  for (int i = tid; i < 4 * TM_MAX_DSUM; i += TM_THREADS) pool[i] = 0.f;
  if (warp == 0) umma::tmem_alloc(tmem_slot, TM_TMEM_COLS);
  if (tid == 0) {
    mbar_init(bar, 1);
    mbar_fence_init();
  }
  const uint32_t a_base = smem_u32(As), w1_base = smem_u32(W1s);
  const uint32_t idesc = umma::instr_desc_bf16(TM_M, d_sum);

  // A CTA walks whole items (a chunk longer than a tile keeps all its 128-token slices on one CTA, in a row): its
  // q-th tile is slice q % tiles_per_item of item blockIdx.x + (q / tiles_per_item) gridDim.x
  const long long my_items = a.n_items > (long long)blockIdx.x ? (a.n_items - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  const long long n_tiles = my_items * a.tiles_per_item;      // of this CTA
  // source row (element offset into the page pool) of every row of this CTA's tile q, or -1 beyond the last unit
  auto rows_of = [&](long long q) {
    if (tid < TM_M) {
      const long long item = blockIdx.x + (q / a.tiles_per_item) * gridDim.x;
      const int slice = (int)(q % a.tiles_per_item);
      const int u_in = tid / v.C;                                  // chunk of the tile this row belongs to (0 when C >= 128)
      const long long unit = item * a.units_per_item + (a.tiles_per_item > 1 ? 0 : u_in);
      long long src = -1;
      if (unit < a.n_units) {
        const int s = (int)(unit / a.n_range);
        const int t = a.t0 + (int)(unit - (long long)s * a.n_range);
        const int r = (a.tiles_per_item > 1) ? slice * TM_M + tid : tid - u_in * v.C;     // row inside the chunk
        const long long page = v.page_table[(long long)s * v.max_chunks + t];
        if (page < 0 || page >= v.n_pages) set_status(v.status, ERR_CAPACITY);
        else src = (page * v.C + r) * D;
      }
      row_src[tid] = src;
    }
  };
  // 16-byte asynchronous copies of the tile's rows into A buffer `buf` (zeros where there is no row)
  auto gather = [&](int buf) {
    const int p = tid & 15;
    unsigned char* dst0 = As + buf * 2 * TM_KB_BYTES + (p >> 3) * TM_KB_BYTES;
#pragma unroll
    for (int i = 0; i < TM_M / (TM_THREADS / 16); ++i) {
      const int r = (tid >> 4) + i * (TM_THREADS / 16);
      const long long src = row_src[r];
      cp_async16(dst0 + umma::piece_offset(r, p & 7), pages + (src < 0 ? 0 : src) + p * 8, src >= 0);
    }
  };
  auto issue_mma = [&](uint32_t tmem_acc, int buf) {
    umma::fence_after_sync();
#pragma unroll
    for (int kb = 0; kb < 2; ++kb)
#pragma unroll
      for (int k = 0; k < 4; ++k)
        umma::mma_bf16(tmem_acc, umma::smem_desc(a_base + (buf * 2 + kb) * TM_KB_BYTES + k * 32),
                       umma::smem_desc(w1_base + kb * (d_sum * umma::KBLOCK_ROW_BYTES) + k * 32), idesc, (kb | k) != 0);
    umma::commit(bar);
  };
  // Columns [c, c + 32) of this warp's 32 tokens: + b1, GELU, summed over the tokens; lane l adds the sum of
  // column c + l to the running sum of the chunk the warp's tokens belong to.
  const int lg = warp & 3, quarter = warp >> 2;      // tensor-memory lanes 32 lg .., columns [quarter d_sum / 4, ..)
  const int cols_q = d_sum >> 2;                     // 32 or 64 columns per warp
  auto epilogue_cols = [&](uint32_t tmem_acc, int c, float* pool_row) {
    float h[32];
    umma::tmem_ld32(tmem_acc + ((uint32_t)(lg * 32) << 16) + (uint32_t)c, h);
    float part[32];
#pragma unroll
    for (int e = 0; e < 32; ++e) part[e] = gelu_tc(h[e] + b1s[c + e]);
    // butterfly: after the round with offset o a lane keeps the columns whose bit o matches its own
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
      const bool upper = (lane & o) != 0;
#pragma unroll
      for (int j = 0; j < o; ++j) {
        const float send = upper ? part[j] : part[j + o];
        const float keep = upper ? part[j + o] : part[j];
        part[j] = keep + __shfl_xor_sync(0xffffffffu, send, o);
      }
    }
    atomicAdd(pool_row + c + lane, part[0]);
  };

  pdl_wait();      // W1 is on its way; the pages come from earlier kernels
  long long tile = 0;
  if (tile < n_tiles) rows_of(tile);
  cp_async_wait_all();
  __syncthreads();
  if (tile < n_tiles) gather(0);
  cp_async_wait_all();
  umma::fence_smem_to_async();
  umma::fence_before_sync();
  __syncthreads();
  umma::fence_after_sync();
  const uint32_t tmem_d = *tmem_slot;
  if (tile < n_tiles && tid == 0) issue_mma(tmem_d, 0);

  uint32_t phase = 0;
  int sel = 0;
  const float inv_c = 1.f / (float)v.C;
  for (; tile < n_tiles; ++tile) {
    const long long next = tile + 1;
    const long long item = blockIdx.x + (tile / a.tiles_per_item) * gridDim.x;
    const int slice = (int)(tile % a.tiles_per_item);
    float* pool_item = pool;
    // rows of this warp's tokens belong to chunk (lg * 32) / C of the tile (0 when C >= 128)
    float* pool_row = pool_item + (a.tiles_per_item > 1 ? 0 : (lg * 32) / v.C) * TM_MAX_DSUM;
    if (next < n_tiles) rows_of(next);
    __syncthreads();
    if (next < n_tiles) gather(sel ^ 1);                             // in flight while this tile's MMAs finish
    const bool ok = mbar_wait_bounded(bar, phase);
    phase ^= 1;
    if (__syncthreads_or(!ok)) {
      if (tid == 0) set_status(v.status, ERR_TIMEOUT);
      break;
    }
    umma::fence_after_sync();
    const uint32_t acc = tmem_d + (uint32_t)sel * TM_MAX_DSUM;
    epilogue_cols(acc, quarter * cols_q, pool_row);
    if (next < n_tiles) {
      cp_async_wait_all();
      umma::fence_smem_to_async();
      umma::fence_before_sync();
      __syncthreads();                                               // also: the other accumulator was drained a tile ago
      if (tid == 0) issue_mma(tmem_d + (uint32_t)(sel ^ 1) * TM_MAX_DSUM, sel ^ 1);
    }
    if (cols_q > 32) epilogue_cols(acc, quarter * cols_q + 32, pool_row);
    sel ^= 1;
    // the chunk(s) of this item are complete with its last slice: pooled activations out, pool cleared (the barrier at
    // the top of the next round separates the clearing from the next tile's sums)
    if (slice == a.tiles_per_item - 1) {
      umma::fence_before_sync();
      __syncthreads();
      for (int i = tid; i < a.units_per_item * d_sum; i += TM_THREADS) {
        const int u_in = i / d_sum, col = i - u_in * d_sum;
        const long long unit = item * a.units_per_item + u_in;
        float* pr = pool_item + u_in * TM_MAX_DSUM + col;
        if (unit < a.n_units) a.hid[((long long)side * a.n_units + unit) * d_sum + col] = *pr * inv_c;
        *pr = 0.f;
      }
    }
  }

  umma::fence_before_sync();
  __syncthreads();
  if (warp == 0) umma::tmem_dealloc(tmem_d, TM_TMEM_COLS);
}

// ---- second layer on the pooled activations: Kbar = W2 g + b2 (fp32 FMA) ------------------------------------
constexpr int TO_ROWS = 32;
constexpr int TO_THREADS = 256;

__global__ void __launch_bounds__(TO_THREADS) kve_token_mlp_out_kernel(LayerView v, int t0, int n_range, long long n_units,
                                                                      MlpWeights w, int d_sum, const float* __restrict__ hid) {
  pdl_launch_dependents();
  pdl_wait();
  extern __shared__ __align__(16) float hs[];      // [TO_ROWS][d_sum]
  const int tid = threadIdx.x, side = blockIdx.y;
  const uint16_t* W2 = side ? w.W2V : w.W2K;
  const float* b2 = side ? w.b2V : w.b2K;
  float* sum_f32 = side ? v.vsum_f32 : v.ksum_f32;
  uint16_t* sum_b16 = side ? v.vsum_bf16 : v.ksum_bf16;
  const long long unit0 = (long long)blockIdx.x * TO_ROWS;
  const float* src = hid + ((long long)side * n_units + unit0) * d_sum;
  const long long live = min((long long)TO_ROWS, n_units - unit0);
  for (int i = tid; i < TO_ROWS * d_sum / 4; i += TO_THREADS) {
    const int r = i / (d_sum / 4);
    reinterpret_cast<float4*>(hs)[i] = (r < live) ? reinterpret_cast<const float4*>(src)[i] : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  __syncthreads();
  const int x = tid & (D - 1);
  const int r0 = (tid >> 7) * (TO_ROWS / 2);
  float acc[TO_ROWS / 2];
  const float bias = b2[x];
#pragma unroll
  for (int r = 0; r < TO_ROWS / 2; ++r) acc[r] = bias;
  const uint4* wrow = reinterpret_cast<const uint4*>(W2 + (long long)x * d_sum);
  for (int u8 = 0; u8 < d_sum / 8; ++u8) {
    const uint4 wv = __ldg(wrow + u8);
    const float wf[8] = {bf16lo(wv.x), bf16hi(wv.x), bf16lo(wv.y), bf16hi(wv.y), bf16lo(wv.z), bf16hi(wv.z), bf16lo(wv.w), bf16hi(wv.w)};
#pragma unroll
    for (int r = 0; r < TO_ROWS / 2; ++r) {
      const float4 p = *reinterpret_cast<const float4*>(hs + (r0 + r) * d_sum + u8 * 8);
      const float4 q = *reinterpret_cast<const float4*>(hs + (r0 + r) * d_sum + u8 * 8 + 4);
      acc[r] = fmaf(wf[0], p.x, acc[r]); acc[r] = fmaf(wf[1], p.y, acc[r]);
      acc[r] = fmaf(wf[2], p.z, acc[r]); acc[r] = fmaf(wf[3], p.w, acc[r]);
      acc[r] = fmaf(wf[4], q.x, acc[r]); acc[r] = fmaf(wf[5], q.y, acc[r]);
      acc[r] = fmaf(wf[6], q.z, acc[r]); acc[r] = fmaf(wf[7], q.w, acc[r]);
    }
  }
#pragma unroll
  for (int r = 0; r < TO_ROWS / 2; ++r) {
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

bool token_mlp_supported(int C, int d_sum) {
  if (d_sum <= 0 || d_sum % 128 != 0 || d_sum > TM_MAX_DSUM) return false;      // the epilogue hands out 32-column groups
  if (C < 32 || C % 32 != 0) return false;
  return C <= 128 ? (128 % C == 0) : (C % 128 == 0);
}

cudaError_t launch_chunk_token_mlp(const LayerView& v, int t0, int t1, const MlpWeights& w, int d_sum, float* hid, cudaStream_t st) {
  const int n_range = t1 - t0;
  const long long n_units = (long long)v.S * n_range;
  if (n_units <= 0) return cudaSuccess;
  if (!token_mlp_supported(v.C, d_sum)) return cudaErrorInvalidValue;
  static DeviceFlags opted;
  {
    cudaError_t e = smem_opt_in(opted, kve_token_mlp_pool_kernel, TM_SMEM_BYTES);
    if (e != cudaSuccess) return e;
  }
  TokenMlpArgs a;
  a.v = v; a.t0 = t0; a.n_range = n_range; a.d_sum = d_sum;
  a.tiles_per_item = v.C > TM_M ? v.C / TM_M : 1;
  a.units_per_item = v.C < TM_M ? TM_M / v.C : 1;
  a.n_units = n_units;
  a.n_items = (n_units + a.units_per_item - 1) / a.units_per_item;
  a.w = w; a.hid = hid;
  // one CTA per SM, half of the SMs per side; a CTA walks whole items (all 128-token slices of a chunk in a row)
  long long per_side = sm_count() / 2;
  if (per_side > a.n_items) per_side = a.n_items;
  if (per_side < 1) per_side = 1;
  cudaError_t e = launch_pdl(kve_token_mlp_pool_kernel, dim3((unsigned)per_side, 2), dim3(TM_THREADS), TM_SMEM_BYTES, st, a);
  if (e != cudaSuccess) return e;
  static DeviceFlags opted_out;
  const int smem_out = TO_ROWS * d_sum * 4;
  e = smem_opt_in(opted_out, kve_token_mlp_out_kernel, TO_ROWS * TM_MAX_DSUM * 4);
  if (e != cudaSuccess) return e;
  return launch_pdl(kve_token_mlp_out_kernel, dim3((unsigned)((n_units + TO_ROWS - 1) / TO_ROWS), 2), dim3(TO_THREADS), smem_out, st, v, t0,
                    n_range, n_units, w, d_sum, (const float*)hid);
}

}  // namespace kve

// Internal launch interface between the host API (api.cu) and the kernel files.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <atomic>

namespace kve {

// ---- per-device launch state ------------------------------------------------------------------------
// A process may drive several GPUs.  The opt-in for more than 48 KB of dynamic shared memory is a
// property of (kernel, device), and grids are sized from the SM count of the device that runs them,
// so both are looked up once per device (the device that is current when the launch is issued).
constexpr int MAX_DEVICES = 64;
int sm_count();                                   // SMs of the current device (cached per device; 148 on a B200)
struct DeviceFlags { std::atomic<unsigned char> done[MAX_DEVICES]; };
template <typename Kernel>
inline cudaError_t smem_opt_in(DeviceFlags& f, Kernel kernel, int bytes) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
  if (f.done[dev].load(std::memory_order_acquire)) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) f.done[dev].store(1, std::memory_order_release);
  return e;
}

// Device pointers of ONE layer plus the geometry the kernels need.
struct LayerView {
  uint16_t* k_pages;          // bf16 [n_pages][C][128]
  uint16_t* v_pages;
  int64_t n_pages;
  const int32_t* page_table;  // [S][max_chunks]
  int32_t* seq_len;           // [B]
  float* ksum_f32;            // [S][max_chunks][128]
  float* vsum_f32;
  uint16_t* ksum_bf16;
  uint16_t* vsum_bf16;
  float* scores;              // [S][max_chunks]
  int32_t* keep_idx;          // [S][max_chunks]
  int32_t* keep_cnt;          // [S]
  float* lstm_h;              // [S][d_g]
  float* lstm_c;
  int32_t* status;
  int32_t* n_listed;          // one int: chunks [0, *n_listed) are covered by the keep list (device copy of the handle's count)
  int32_t* step_ticket;       // one int, zero between launches: arrivals of the gate-step kernel's clusters
  int B, H, S, C, max_chunks, max_tokens;
};

struct MlpWeights {
  const uint16_t *W1K, *W2K, *W1V, *W2V;   // bf16
  const float *b1K, *b2K, *b1V, *b2V;
};

enum AttnMode { ATTN_SUMMARY = 0, ATTN_RAW = 1, ATTN_DENSE = 2 };

// split geometry of the block-of-queries attention, chosen on the host
struct AttnPlan {
  int rows_per_split;   // multiple of the kernel's tile height
  int max_splits;       // grid.x: upper bound of splits any sequence can need
};
constexpr int ATTN_TILE_ROWS = 64;
constexpr int ATTN_PARTIAL_FLOATS = 132;       // acc[128], m, l, 2 pad: keeps every record 16-byte aligned

cudaError_t launch_append(const LayerView& v, const void* k_new, const void* v_new, int n_new, int pos0, cudaStream_t st);
cudaError_t launch_set_listed(const LayerView& v, int n_listed, cudaStream_t st);      // the device copy of the keep list's coverage
// n_listed >= 0: also set the device copy of the keep list's coverage to it
cudaError_t launch_set_len(const LayerView& v, int n, int n_listed, cudaStream_t st);
cudaError_t launch_append_next(const LayerView& v, const void* k_new, const void* v_new, int n_new, int32_t* ticket,
                               cudaStream_t st);
// dev_window < 0: chunks [t0, t1).  dev_window >= 0 (the window size W): ONE chunk per sequence whose index the kernel
// finds on the device - the chunk behind the keep list's coverage, if the stored length says it has left the window,
// else the launch does nothing (a trigger that is replayed from a CUDA graph)
cudaError_t launch_chunk_mean(const LayerView& v, int t0, int t1, bool final_output, bool pool_max, cudaStream_t st, int dev_window);
cudaError_t launch_chunk_mlp(const LayerView& v, int t0, int t1, const MlpWeights& w, int d_sum, cudaStream_t st, int dev_window);
// per-token MLP aggregator: hid = scratch of 2 * S * (t1 - t0) * d_sum floats
bool token_mlp_supported(int C, int d_sum);
cudaError_t launch_chunk_token_mlp(const LayerView& v, int t0, int t1, const MlpWeights& w, int d_sum, float* hid, cudaStream_t st);
cudaError_t launch_gate_proj(const LayerView& v, int t0, int t1, const uint16_t* W_ih, const float* b_ih,
                             const float* b_hh, int d_g, float* P, cudaStream_t st);
// planes: bf16 planes of the fp32 state h that enter the recurrent product (2, or 3 = exact products)
cudaError_t launch_gate_rnn(const LayerView& v, int t0, int t1, const uint16_t* W_hh, const float* w_s, float b_s,
                            int d_g, const float* P, float* H, bool reset_state, int planes, cudaStream_t st);
// one LSTM step on chunk t with the carried state, its score, and chunk t appended to the keep list for tau (which must
// cover chunks [0, t)), its summary rows appended to kkept / vkept, the device's coverage count set to t + 1.
// dev_window >= 0: t is found on the device as above (the argument t is ignored), nothing happens if no chunk is due
cudaError_t launch_gate_step(const LayerView& v, int t, const uint16_t* W_ih, const uint16_t* W_hh, const float* b_ih,
                             const float* b_hh, const float* w_s, float b_s, float tau, int d_g, int planes,
                             uint16_t* kept_k, uint16_t* kept_v, int dev_window, cudaStream_t st);
// both also leave the kept chunks' summary rows compacted in kkept / vkept [S][max_chunks][128] bf16, which is
// what attention reads until the next keep list
cudaError_t launch_compact(const LayerView& v, int n_chunks, float tau, void* kkept, void* vkept, cudaStream_t st);
cudaError_t launch_compact_topk(const LayerView& v, int n_chunks, int k, void* kkept, void* vkept, cudaStream_t st);
cudaError_t launch_reclaim(const LayerView& v, int t0, int t1, float tau, int mode, int32_t* scratch, int32_t* free_list,
                           long long capacity, int32_t* free_count, cudaStream_t st);
// parts_per_seq: equal parts every sequence is cut into; grid: CTAs that share the S * parts_per_seq parts;
// partials: S + grid records of ATTN_PARTIAL_FLOATS
// k_new, v_new ([S][128] bf16) non-null: fused append of one token per sequence at the device-held length; ticket: one
// int32 (zero between launches) through which the last CTA publishes the new length
cudaError_t launch_attn(const LayerView& v, AttnMode mode, int n_chunks, int parts_per_seq, int grid, const void* q, void* out,
                        float* lse, float scale, const void* kkept, const void* vkept, float* partials, int32_t* counters,
                        const void* k_new, const void* v_new, int32_t* ticket, cudaStream_t st);
int attn_smem_bytes();
cudaError_t launch_selftest_timeout(int which, int32_t* status, cudaStream_t st);

// block-of-queries attention (grouped query heads x query tokens), tensor-map fed
constexpr int ATTN_BLOCK_MAX_ROWS = 128;       // query rows (tokens x heads per KV head) per KV sequence
constexpr int ATTN_BLOCK_MAP_BYTES = 128;      // one tensor map; a handle keeps four (K pages, V pages, kept K summaries, kept V summaries)
constexpr int ATTN_BLOCK_SUM_BOX = 16;         // rows per box of the maps over the compacted kept summary rows
int attn_block_hp(int C);                      // rows per page box: largest power of two <= 64 dividing C
cudaError_t encode_attn_block_maps(void* maps, const void* k_pages, const void* v_pages, long long page_rows, int hp,
                                   const void* ksum, const void* vsum, long long sum_rows);
cudaError_t launch_attn_block(const LayerView& v, const void* maps, AttnMode mode, int n_chunks, AttnPlan plan, int T, int G,
                              int causal, int hp, long long sum_row0, const void* q, void* out, float* lse, float scale, float* partials,
                              int32_t* counters, cudaStream_t st);

}  // namespace kve

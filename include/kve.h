/*
 * kve.h — C ABI of libkve: the RNN-gated chunked KV cache decode path on one B200 (sm_100a).
 *
 * The paper's module replaces a transformer layer's KV cache (Sec. 1, Sec. 3.1): history outside a
 * recent window is cut into chunks of C tokens, each chunk is reduced to one summary key/value
 * (Eq. 2), an LSTM scores the summaries in temporal order (Eq. 3), chunks with s_t >= tau are kept
 * (Sec. 3.2), and decode attention (Eq. 1) runs over the kept chunks plus the raw window
 * (Sec. 3.3, n' = W + M).
 *
 * Conventions for every entry point
 *   - returns KVE_OK (0) or a negative kvE_status; never throws, never aborts.
 *   - work is enqueued on the given CUDA stream (passed as void*, a cudaStream_t); the call does not
 *     wait for it.  kvE_poll_status and kvE_create are the only calls that synchronise.
 *   - no entry point allocates or frees device memory.  Every device buffer is owned by the caller
 *     (allocate it with any allocator, e.g. PyTorch) and only borrowed; the handle owns host metadata.
 *   - argument and geometry errors are found on the host before any launch.  Device-side problems
 *     (a page id out of range, a wait that ran out) set *status_word to a kvE_status and the kernel
 *     skips the access; nothing traps and no wait is unbounded.
 *   - one stream at a time per handle; calls on one handle are not thread-safe.
 *   - a handle belongs to the device that was current at kvE_create (where its buffers live); a call
 *     made with another device current returns KVE_ERR_STATE.  Several handles on several devices
 *     may live in one process.
 *   - "bf16" is the 16-bit brain float bit pattern; matrices are row-major; S = B * Hkv sequences,
 *     sequence index s = b * Hkv + h.  d (head dim) must be 128.
 */
#ifndef KVE_H_
#define KVE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  KVE_OK = 0,
  KVE_ERR_ARG = -1,       /* null pointer, negative size, unknown enum value */
  KVE_ERR_GEOMETRY = -2,  /* a size combination the kernels do not support (d != 128, d_g, ...) */
  KVE_ERR_CAPACITY = -3,  /* append beyond max_tokens, workspace too small, page id out of range */
  KVE_ERR_STATE = -4,     /* call order: chunk range not yet summarised / gated, ... */
  KVE_ERR_CUDA = -5,      /* a CUDA runtime call failed (launch error text via kvE_last_cuda_error) */
  KVE_ERR_TIMEOUT = -6    /* a bounded device-side wait ran out (reported through status_word) */
} kvE_status;

/* Eq. 2 aggregator.  MEAN: chunk mean; MLP: 2-layer GELU MLP on the chunk mean; IDENTITY: C == 1; MAX: max-pool
 * (Sec. 3.1); TOKEN_MLP: Eq. 2 taken literally, the MLP on every token of the chunk, the C outputs mean-pooled. */
enum { KVE_AGG_MEAN = 0, KVE_AGG_MLP = 1, KVE_AGG_IDENTITY = 2, KVE_AGG_MAX = 3, KVE_AGG_TOKEN_MLP = 4 };
enum { KVE_ATTEND_SUMMARY = 0, KVE_ATTEND_RAW = 1 };                /* what a kept chunk contributes */

/* Geometry, fixed at kvE_create. */
typedef struct {
  int32_t B;           /* batch */
  int32_t Hq, Hkv;     /* query heads, KV heads, Hq a multiple of Hkv (query head hq reads KV head hq / (Hq / Hkv));
                          Hq > Hkv: attention only through kvE_decode_attn_block */
  int32_t d;           /* head dim, 128 */
  int32_t C;           /* chunk size in tokens, 1..1024 (Sec. 3.2) */
  int32_t W;           /* recent window in tokens, >= 0 (Sec. 3.3): never summarised */
  int32_t max_tokens;  /* capacity of one sequence */
  int32_t n_layers;    /* independent layers sharing the handle */
  int32_t agg;         /* KVE_AGG_* ; IDENTITY needs C == 1; MAX: element-wise maximum of the chunk */
  int32_t d_sum;       /* MLP hidden size: KVE_AGG_MLP: multiple of 8, <= 1024; KVE_AGG_TOKEN_MLP: 128 or 256, and C
                          must be 32, 64, 128 or a multiple of 128 */
  int32_t d_g;         /* LSTM hidden size: 64, 128 or 256 */
  int32_t attend;      /* KVE_ATTEND_* */
  int32_t max_query_tokens; /* most query tokens per kvE_decode_attn_block call; 0: that entry point is not used.
                               max_query_tokens * (Hq / Hkv) <= 128, and C must be a multiple of 8 */
} kvE_config;

/* max_chunks = ceil(max_tokens / C) is the chunk stride of every per-chunk array below. */

/* Caller-owned DEVICE buffers. */
typedef struct {
  void* k_pages;        /* bf16 [n_pages][C][d]: one page = one chunk of one (layer, b, h) */
  void* v_pages;        /* bf16 [n_pages][C][d] */
  int64_t n_pages;
  int32_t* page_table;  /* [n_layers][S][max_chunks] page ids, filled by the caller; kvE_reclaim_pages writes -1 */
  int32_t* seq_len;     /* [n_layers][B] tokens stored; written by kvE_append / kvE_set_len */
  float* ksum_f32;      /* [n_layers][S][max_chunks][d] chunk summaries, fp32 */
  float* vsum_f32;
  void* ksum_bf16;      /* same, rounded to bf16: what the gate and attention read */
  void* vsum_bf16;
  float* scores;        /* [n_layers][S][max_chunks] gate scores s_t */
  int32_t* keep_idx;    /* [n_layers][S][max_chunks] ascending kept chunk ids, rest -1 */
  int32_t* keep_cnt;    /* [n_layers][S] */
  float* lstm_h;        /* [n_layers][S][d_g] carried hidden state */
  float* lstm_c;        /* [n_layers][S][d_g] carried cell state */
  void* workspace;      /* kvE_workspace_bytes(cfg) bytes, 256-byte aligned, zeroed by kvE_create */
  size_t workspace_bytes;
  int32_t* status_word; /* one int32, zeroed by kvE_create; first device-side error sticks */
} kvE_buffers;

/* Aggregator MLP_K / MLP_V of Eq. 2 (KVE_AGG_MLP: y = W2 gelu(W1 m + b1) + b2, m the chunk mean; KVE_AGG_TOKEN_MLP:
 * the same MLP applied to every token of the chunk, the outputs averaged).
 * DEVICE pointers; W1 [d_sum][d], W2 [d][d_sum] bf16; b1 [d_sum], b2 [d] fp32; matrices on 16-byte boundaries. */
typedef struct {
  const void *W1K, *W2K, *W1V, *W2V;
  const float *b1K, *b2K, *b1V, *b2V;
} kvE_agg_weights;

/* LSTM gate of Eq. 3.  DEVICE pointers; W_ih [4 d_g][2 d], W_hh [4 d_g][d_g] bf16, gate rows in the
 * order i, f, g, o; b_ih, b_hh [4 d_g], w_s [d_g] fp32; b_s by value.  Matrices and w_s start on 16-byte boundaries
 * (the kernels fetch them 16 bytes at a time). */
typedef struct {
  const void *W_ih, *W_hh;
  const float *b_ih, *b_hh, *w_s;
  float b_s;
} kvE_lstm_weights;

typedef struct kvE_store kvE_store;

/* Bytes of workspace the handle needs: the gate projection buffer and the h_t rows of one kvE_gate call, the split-K partial records and tickets of
 * the attention kernels (those of kvE_decode_attn_block only when cfg.max_query_tokens > 0), staging rows of the
 * host-buffer step, scratch of kvE_reclaim_pages.  0 if the geometry is not supported. */
size_t kvE_workspace_bytes(const kvE_config* cfg);

/* Host-side handle.  Validates the geometry, zeroes workspace, status_word, seq_len and keep_cnt
 * (synchronous memsets on the current device).  All layers start empty. */
int kvE_create(const kvE_config* cfg, const kvE_buffers* buf, kvE_store** out);
int kvE_destroy(kvE_store* st);

/* Sec. 3.2 "stores the key-value pairs in temporal order": append n_new tokens to every sequence
 * of `layer`.  k_new, v_new: DEVICE bf16 [S][n_new][d].  *n_ready (nullable, host) receives how
 * many completed chunks now lie outside the window and have not been gated yet (the trigger of
 * Sec. 3.3).  KVE_ERR_CAPACITY if the layer would exceed max_tokens. */
int kvE_append(kvE_store* st, int layer, const void* k_new, const void* v_new, int n_new,
               int* n_ready, void* stream);

/* kvE_append of n_new tokens per sequence at the length the DEVICE holds (seq_len), which the call advances by
 * n_new: nothing about the position is fixed at launch, so the call can be captured in a CUDA graph and every
 * replay appends the next n_new tokens (k_new, v_new: DEVICE bf16 [S][n_new][d], read at replay time).  This is the decode
 * loop between two gate triggers of Sec. 3.3 without a host round trip per token.
 *   n_reserve: how many further tokens such appends (replays included) may add before the next kvE_set_len or
 *   kvE_append.  kvE_decode_attn / kvE_decode_attn_dense cut their work into pieces on the device from the length
 *   they find there, so a replayed launch follows the cache however far it grows; kvE_decode_attn_block launches
 *   issued after this call are sized for n_reserve more tokens, and one replayed past that sets KVE_ERR_CAPACITY in
 *   the status word instead of dropping rows.  The handle's own length advances by n_new per call, not per replay:
 *   after replaying, give it the true length with kvE_set_len(layer, n) before summarising or gating the chunks
 *   that have completed meanwhile (attention keeps reading them as raw rows until then, which is exact).
 *   Device side: a sequence without room for n_new more tokens is left alone and KVE_ERR_CAPACITY is set in the
 *   status word. */
int kvE_append_next(kvE_store* st, int layer, const void* k_new, const void* v_new, int n_new, int n_reserve,
                    void* stream);

/* Set the stored length of `layer` (all sequences) to n tokens, n <= max_tokens; the pages keep
 * their contents.  Chunks at or beyond the new stale range lose their summarised mark; if the new
 * stale range is shorter than the gated range, the carried LSTM state is past the cut, so the gated mark
 * returns to 0 (gate again from chunk 0); if it is shorter than the range the keep list covers, the
 * keep list is dropped (attention then reads every stored row, which is exact, until the next
 * kvE_compact).  Used to load a prefilled cache and to roll a decode step back. */
int kvE_set_len(kvE_store* st, int layer, int n, void* stream);

/* Switch what a kept chunk contributes to attention (cfg.attend) for all later calls on this handle:
 * its one summary row (KVE_ATTEND_SUMMARY, the method of Sec. 3.3) or its C raw rows (KVE_ATTEND_RAW).
 * Host-side only; summaries, scores and keep lists do not depend on it.  Pages handed back with
 * KVE_RECLAIM_GATED are gone for KVE_ATTEND_RAW (reading them flags KVE_ERR_CAPACITY). */
int kvE_set_attend(kvE_store* st, int attend);

/* Precision of the recurrent product W_hh h of Eq. 3 for all later kvE_gate calls on this handle.  W_hh is bf16 and
 * the state h is fp32; the tensor cores take h as a sum of bf16 planes.  planes == 2 (default): h = hi + lo to
 * 2^-17 |h| (16 of its 24 significant bits), the faster form; planes == 3: h = p0 + p1 + p2 exactly, every product
 * exact, the sum differing from a plain fp32 loop only in summation order.  Host-side only. */
int kvE_set_gate_planes(kvE_store* st, int planes);

/* Eq. 2: summaries of chunks [chunk_begin, chunk_end) of every sequence of `layer`;
 * chunk_end <= floor((n - W) / C).  w is NULL unless agg is KVE_AGG_MLP or KVE_AGG_TOKEN_MLP. */
int kvE_summarize_chunks(kvE_store* st, int layer, int chunk_begin, int chunk_end,
                         const kvE_agg_weights* w, void* stream);

/* Eq. 3: run the LSTM over summaries [chunk_begin, chunk_end) oldest first and write scores.
 * chunk_begin == 0 starts from h = c = 0; otherwise chunk_begin must equal the number of chunks
 * already gated (state carried in lstm_h / lstm_c).  The range must have been summarised. */
int kvE_gate(kvE_store* st, int layer, int chunk_begin, int chunk_end,
             const kvE_lstm_weights* w, void* stream);

/* Sec. 3.3, the gate's part of a trigger while decoding: ONE more chunk per sequence has left the window and has been
 * summarised.  Gates chunk t = (number of chunks gated so far) with the carried (h, c) (Eq. 3), writes scores[t] and
 * brings the keep list for `tau` up to date (Sec. 3.2): like kvE_gate(t, t + 1) + kvE_compact(tau).  When the keep
 * list already covers chunks [0, t) under the same tau (kvE_compact, kvE_refresh or earlier calls of this one; t > 0)
 * all of it is ONE launch: the LSTM step on the new summary, the score, and chunk t appended to keep_idx / keep_cnt
 * and to the compacted summary rows; otherwise it runs the two calls.  The single launch sums in another order than
 * kvE_gate: its scores agree with kvE_gate's to rounding (1e-6), not bit for bit.  KVE_ERR_STATE if chunk t has not
 * been summarised.  Timed under KVE_K_GATE_RNN. */
int kvE_gate_next(kvE_store* st, int layer, const kvE_lstm_weights* w, float tau, void* stream);

/* Sec. 3.3, the trigger with nothing about the position fixed at launch, so that it can sit in a captured CUDA graph
 * behind the decode steps (kvE_decode_step) and be replayed: every execution looks on the DEVICE for the chunk right
 * behind the keep list's coverage and, if the stored length says that chunk has left the window, summarises it (Eq. 2),
 * gates it with the carried (h, c) (Eq. 3) and appends it to the keep list for `tau` (Sec. 3.2), as kvE_summarize_chunks
 * + kvE_gate_next do; if no chunk is due the launches return at once.  A graph of C decode steps followed by this call
 * replays for as long as the cache has room, with no host work besides the replay.  Needs, at the call: a keep list under
 * the same tau that covers every gated chunk (at least one), and nothing summarised beyond it; else KVE_ERR_STATE.
 * KVE_ERR_GEOMETRY for KVE_AGG_TOKEN_MLP.  The handle's own counters advance as for one execution on the state it
 * knows; after replays, kvE_adopt_device_state brings them up to date.  Sequences of a layer have one common length. */
int kvE_refresh_next(kvE_store* st, int layer, const kvE_agg_weights* aw, const kvE_lstm_weights* lw, float tau, void* stream);

/* Read the stored length and the keep list's coverage of `layer` back from the device (waits for `stream`) and make them
 * the handle's: the token count, and - when the keep list covered every gated chunk before - the counts of summarised,
 * gated and listed chunks.  For use after replaying captured kvE_append_next / kvE_decode_step / kvE_refresh_next
 * launches, which move the device's counters without the host.  KVE_ERR_STATE if the device holds impossible values. */
int kvE_adopt_device_state(kvE_store* st, int layer, void* stream);

/* Sec. 3.2 retention rule: keep chunk t iff scores[t] >= tau, over all gated chunks of `layer`;
 * writes keep_idx / keep_cnt.  Attention then treats tokens from (gated chunks) * C on as raw.  Also copies the kept
 * chunks' summary rows into one contiguous run per sequence (workspace), which is what attention reads, and records
 * on the device how many chunks the list covers: kvE_decode_attn / kvE_decode_step read that count from the device,
 * so one of their launches captured in a CUDA graph keeps serving after later triggers without a new capture. */
int kvE_compact(kvE_store* st, int layer, float tau, void* stream);

/* Sec. 3.3, the whole aggregation-and-gating step of `layer` from scratch in one call: summaries of every chunk
 * outside the window (Eq. 2), the gate over all of them starting from h = c = 0 (Eq. 3), the keep list for `tau`
 * (Sec. 3.2): kvE_summarize_chunks(0, Nc) + kvE_gate(0, Nc) + kvE_compact(tau), Nc = floor((n - W) / C).
 * aw is NULL unless the aggregator has an MLP. */
int kvE_refresh(kvE_store* st, int layer, const kvE_agg_weights* aw, const kvE_lstm_weights* lw, float tau, void* stream);

/* The gating-strategy variant the paper names for its ablations (Sec. 5): keep the k highest-scoring gated
 * chunks of every sequence instead of thresholding.  Equal scores: the older chunk ranks first, so the
 * list is unique.  Writes keep_idx / keep_cnt like kvE_compact (ascending ids; k <= 0 keeps nothing,
 * k >= gated chunks keeps all).  Work grows with the square of the gated chunks per sequence.  After it,
 * kvE_reclaim_pages(KVE_RECLAIM_DISCARDED) returns KVE_ERR_STATE (there is no threshold to judge by). */
int kvE_compact_topk(kvE_store* st, int layer, int k, void* stream);

/* Sec. 3.3 (n' = W + M, memory ratio n / (W + M)) and the KV-memory reduction of Sec. 4.2: hand the pages
 * of gated chunks back to the caller.  Chunks [chunk_begin, chunk_end) of every sequence of `layer` must
 * be covered by the keep list (kvE_compact; its tau decides "discarded").
 *   mode KVE_RECLAIM_DISCARDED: pages of chunks with s_t < tau (never attended to again);
 *   mode KVE_RECLAIM_GATED:     pages of all chunks in the range; needs cfg.attend == KVE_ATTEND_SUMMARY,
 *                               where a retained chunk is read through its one summary row.
 * free_list: DEVICE int32 [capacity], receives the page ids, sequences in order, chunks ascending;
 * free_count: DEVICE int32, receives how many.  The page_table entries handed back become -1 (the
 * library writes the caller's page table here); entries that are already -1 are skipped.  If the
 * list would not fit, nothing is handed back, *free_count is 0 and the status word gets
 * KVE_ERR_CAPACITY.  Afterwards the raw rows of those chunks are gone: summarising them again or
 * kvE_decode_attn_dense flags KVE_ERR_CAPACITY in the status word instead of reading them. */
enum { KVE_RECLAIM_DISCARDED = 0, KVE_RECLAIM_GATED = 1 };
int kvE_reclaim_pages(kvE_store* st, int layer, int chunk_begin, int chunk_end, int mode, int32_t* free_list,
                      int64_t capacity, int32_t* free_count, void* stream);

/* Sec. 3.3 + Eq. 1: out = softmax(q K'^T * scale) V' over [kept chunks ; raw tail] of `layer`.
 * q, out: DEVICE bf16 [S][d]; lse: DEVICE fp32 [S] or NULL (log-sum-exp of the scaled logits). */
int kvE_decode_attn(kvE_store* st, int layer, const void* q, void* out, float* lse, float scale,
                    void* stream);

/* One decode step of `layer` between two gate triggers in ONE launch: append the step's token to every sequence
 * (k_new, v_new: DEVICE bf16 [S][d]) and attend over [kept chunks ; raw tail] with it included (Sec. 3.2 "temporal
 * order" + Sec. 3.3 + Eq. 1).  Same result as kvE_append_next(n_new = 1) followed by kvE_decode_attn.  The token goes
 * to the position the DEVICE holds (seq_len), which the call advances by one, so the call can be captured in a CUDA
 * graph and every replay handles the next token (the buffers are read at replay time); n_reserve as in
 * kvE_append_next.  The handle's own length advances by one per call, not per replay: give it the true length with
 * kvE_set_len before the next summarise / gate.  A full cache sets KVE_ERR_CAPACITY in the status word and attends
 * over what is stored.  q, out: DEVICE bf16 [S][d]; lse: DEVICE fp32 [S] or NULL. */
int kvE_decode_step(kvE_store* st, int layer, const void* k_new, const void* v_new, const void* q, void* out, float* lse,
                    float scale, int n_reserve, void* stream);

/* Eq. 1 over all n stored tokens of `layer` (the full-cache baseline of Sec. 3.3). */
int kvE_decode_attn_dense(kvE_store* st, int layer, const void* q, void* out, float* lse,
                          float scale, void* stream);

/* Sec. 3.3 + Eq. 1 for a block of queries: n_query_tokens tokens decoded together (the action tokens of one
 * control step) on all Hq query heads, Hq / Hkv of which share each KV head (grouped-query attention, the
 * 32-head / 8-KV-head model of Sec. 4.1).  Every (token, head) pair is an independent query against the
 * retained set [kept chunks ; raw tail] of its KV head (dense != 0: against all n stored tokens).
 *   causal == 0: every query token sees the whole cache (tokens decoded in parallel, e.g. an action chunk);
 *   causal != 0: the block's tokens are the n_query_tokens NEWEST tokens of the cache (append them first) and
 *   query token t sees the cache up to and including its own position only (Eq. 1 for each of several
 *   tokens handled in one call), i.e. all but the last n_query_tokens - 1 - t rows.  Each retained K/V row is read once per KV head, and the
 * products run on the tensor cores.
 *   The softmax numerators enter the tensor core as bf16: against exact weights an output moves by at
 *   most 2^-8 * sum_i p_i |v_i| / sum_i p_i (accumulation in fp32, one bf16 rounding of the result).
 *   q, out: DEVICE bf16 [B][n_query_tokens][Hq][d]; lse: DEVICE fp32 [B][n_query_tokens][Hq] or NULL.
 *   KVE_ERR_STATE if cfg.max_query_tokens == 0, or if causal != 0 and the raw tail (all stored tokens when
 *   dense != 0) holds fewer rows than n_query_tokens; KVE_ERR_CAPACITY if n_query_tokens exceeds
 *   cfg.max_query_tokens. */
int kvE_decode_attn_block(kvE_store* st, int layer, const void* q, int n_query_tokens, int dense, int causal,
                          void* out, float* lse, float scale, void* stream);

/* kvE_decode_attn without any scratch from the caller.  (The paper has no counterpart: this is a
 * deployment aid.)  Some users of this library must not allocate device memory once they are
 * running: a robot-control loop that handed the whole GPU to its framework's memory pool at
 * start-up and may not stall on, or fail in, an allocation between two control ticks; a plug-in that
 * is given device pointers by a host application and has no right to allocate on that device.  For
 * them the partial results and tickets of the attention kernel live in a device array that
 * is part of the library image itself (KVE_STATIC_SCRATCH_BYTES, about 2.1 MiB, held by every GPU that
 * loads the library until the process exits) instead of the handle's workspace, and this call
 * performs no cudaMalloc / cudaFree and calls no allocating routine.
 *   - same arguments, result and errors as kvE_decode_attn (gated attention of `layer`, mode from
 *     cfg.attend); q, out: DEVICE bf16 [S][d]; lse: DEVICE fp32 [S] or NULL.
 *   - limits: S <= KVE_STATIC_MAX_SEQUENCES and S + CTAs <= KVE_STATIC_MAX_PARTIALS, where CTAs (at most two
 *     per SM: 296 on a B200) is the size of the launch the library picks for the layer's current state;
 *     beyond that the call returns KVE_ERR_CAPACITY without launching (text via kvE_last_cuda_error).
 *   - the first call on each device looks up the array's device address (that device must be
 *     current); make that first call outside any stream capture.
 *   - one array per device, shared by every handle and stream: the call clears the tickets it
 *     needs on `stream` before the kernel, but two calls that overlap on the GPU (different
 *     streams, or different handles) race on it.  Serialise them, or use kvE_decode_attn. */
#define KVE_STATIC_MAX_SEQUENCES 2048
#define KVE_STATIC_MAX_PARTIALS 4096
#define KVE_STATIC_SCRATCH_BYTES (KVE_STATIC_MAX_SEQUENCES * 4 + KVE_STATIC_MAX_PARTIALS * 132 * 4)
int kvE_decode_attn_static(kvE_store* st, int layer, const void* q, void* out, float* lse, float scale,
                           void* stream);

/* One whole decode step of `layer` from HOST memory: copies k_new, v_new, q (bf16 [S][d] each,
 * ideally pinned) to the device, appends the token, brings summaries, gate and keep list up to
 * date for every chunk that has left the window (from scratch, through kvE_refresh, if `from_scratch` != 0), runs
 * kvE_decode_attn and copies out (bf16 [S][d]) back to host memory.  Staging uses the tail of the
 * workspace.  Waits for the stream before returning. */
int kvE_decode_step_host(kvE_store* st, int layer, const void* k_new_host, const void* v_new_host,
                         const void* q_host, void* out_host, const kvE_agg_weights* aw,
                         const kvE_lstm_weights* lw, float tau, float scale, int from_scratch,
                         void* stream);

/* The same step without the final wait: everything (copies included) is only enqueued on `stream`.
 * The host buffers must be pinned and must stay untouched until the stream has passed this step
 * (out_host is valid from then on); the next step may be enqueued right away, its copies and kernels
 * queue up behind this one's. */
int kvE_decode_step_host_async(kvE_store* st, int layer, const void* k_new_host, const void* v_new_host,
                               const void* q_host, void* out_host, const kvE_agg_weights* aw,
                               const kvE_lstm_weights* lw, float tau, float scale, int from_scratch,
                               void* stream);

/* Reads *status_word (synchronises the device) into *device_status and clears it. */
int kvE_poll_status(kvE_store* st, int* device_status);

/* Host-side view of a layer: tokens stored, chunks summarised, gated and covered by the keep list. */
int kvE_layer_state(const kvE_store* st, int layer, int* n_tokens, int* n_summarised, int* n_gated,
                    int* n_compacted);

/* Per-kernel timing.  While enabled, every kernel launch of this handle is bracketed by a pair of CUDA
 * events on the launch stream (events are created on the first enable; no device memory).
 * kvE_profile_read synchronises the device and writes, per kernel id, the duration in microseconds
 * of that kernel's most recent launch, or -1 if it has not run since profiling was enabled. */
enum { KVE_K_APPEND = 0, KVE_K_CHUNK_MEAN, KVE_K_CHUNK_MLP, KVE_K_GATE_PROJ, KVE_K_GATE_RNN, KVE_K_COMPACT,
       KVE_K_ATTN, KVE_K_ATTN_DENSE, KVE_K_ATTN_BLOCK, KVE_K_COUNT };
int kvE_profile(kvE_store* st, int enable);
int kvE_profile_read(kvE_store* st, float* us /* [KVE_K_COUNT] */);

/* Text of the last CUDA runtime error seen by this handle's calls ("" if none). */
const char* kvE_last_cuda_error(const kvE_store* st);

/* ---- self-test (not part of the paper's path) ----------------------------------------------------------------------
 * Makes a bounded device-side wait run out on purpose, without a fault: a small kernel waits on a barrier that nothing
 * ever completes, with a limit of a few thousand polls (which == 0: the wait the copy pipelines and tensor-core
 * commits use) or two milliseconds (which == 1: the wait between the CTAs of a cluster in the gate recurrence).  The
 * kernel returns by itself, the status word reads KVE_ERR_TIMEOUT at the next kvE_poll_status, and the handle stays
 * usable.  A way to check, on the installed driver and GPU, that the failure path every kernel relies on works. */
int kvE_selftest_timeout(kvE_store* st, int which, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* KVE_H_ */

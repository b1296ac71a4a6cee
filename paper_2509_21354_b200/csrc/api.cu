// Host side of libkve: the C ABI of include/kve.h.  Validates arguments, tracks per-layer progress
// (tokens stored, chunks summarised / gated / compacted) and enqueues the kernels.  Allocates no
// device memory.
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "../../include/kve.h"
#include "kernels.h"

using namespace kve;

struct LayerState {
  int n_tokens = 0;      // tokens stored (every sequence of the layer), as far as the host knows
  int reserve_upper = 0; // kvE_append_next: replays may take the device-side length up to here; attention is sized for it
  int n_summarised = 0;  // chunks [0, n_summarised) have summaries
  int n_gated = 0;       // chunks [0, n_gated) have scores; LSTM state stands after chunk n_gated-1
  int n_compacted = 0;   // keep list covers chunks [0, n_compacted); attention reads raw rows from there on
  float tau = 0.f;       // threshold of the last kvE_compact
  bool by_topk = false;  // the keep list came from kvE_compact_topk (no threshold to tell "discarded" by)
};

struct kvE_store {
  kvE_config cfg;
  kvE_buffers buf;
  int gate_planes = 2;   // bf16 planes of h in the recurrent product (kvE_set_gate_planes)
  int device = -1;       // the device that was current at kvE_create: owner of every buffer; calls check it
  int S, max_chunks;
  // workspace carve-up (byte offsets)
  size_t off_P, off_H, off_partials, off_counters, off_stage, off_reclaim, off_ticket, off_block, off_kept_k, off_kept_v, off_listed, ws_needed;
  int attn_grid_max;     // most CTAs an attention launch uses (two per SM of the handle's device): sizes the partial records
  // block-of-queries attention: tensor maps over the page pools and the summary store (encoded at
  // create when cfg.max_query_tokens > 0), rows per page box, split cap the workspace was sized for
  alignas(64) unsigned char block_maps[4 * ATTN_BLOCK_MAP_BYTES];
  bool block_ready = false;
  int block_hp = 0, block_split_cap = 1;
  std::vector<LayerState> layers;
  std::string cuda_error;

  // optional per-kernel timing: one (start, stop) event pair per kernel id
  bool profiling = false;
  cudaEvent_t ev[2 * KVE_K_COUNT] = {};
  bool ev_made = false;
  bool ev_used[KVE_K_COUNT] = {};
};

// SM count of the current device, looked up once per device
int kve::sm_count() {
  static std::atomic<int> cached[MAX_DEVICES];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return 148;
  int n = cached[dev].load(std::memory_order_acquire);
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  cached[dev].store(n, std::memory_order_release);
  return n;
}

namespace {

constexpr int MAX_SPLITS = 32;            // block-of-queries attention: most splits per sequence
constexpr size_t ATTN_GRID_LIMIT = 1024;  // most CTAs of one kvE_decode_attn launch the workspace is sized for (>= 2 per SM)
constexpr size_t ALIGN = 256;
size_t align_up(size_t x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }
constexpr size_t align_const(size_t x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }

int check_config(const kvE_config* c) {
  if (!c) return KVE_ERR_ARG;
  if (c->B <= 0 || c->Hq <= 0 || c->Hkv <= 0 || c->C <= 0 || c->W < 0 || c->max_tokens <= 0 || c->n_layers <= 0)
    return KVE_ERR_ARG;
  if (c->agg != KVE_AGG_MEAN && c->agg != KVE_AGG_MLP && c->agg != KVE_AGG_IDENTITY && c->agg != KVE_AGG_MAX &&
      c->agg != KVE_AGG_TOKEN_MLP)
    return KVE_ERR_ARG;
  if (c->attend != KVE_ATTEND_SUMMARY && c->attend != KVE_ATTEND_RAW) return KVE_ERR_ARG;
  if (c->d != 128 || c->Hq % c->Hkv != 0 || c->C > 1024) return KVE_ERR_GEOMETRY;
  if (c->max_query_tokens < 0) return KVE_ERR_ARG;
  if (c->max_query_tokens > 0 &&
      ((long long)c->max_query_tokens * (c->Hq / c->Hkv) > ATTN_BLOCK_MAX_ROWS || attn_block_hp(c->C) < 8))
    return KVE_ERR_GEOMETRY;
  if (c->agg == KVE_AGG_IDENTITY && c->C != 1) return KVE_ERR_GEOMETRY;
  if (c->agg == KVE_AGG_MLP && (c->d_sum <= 0 || c->d_sum % 8 != 0 || c->d_sum > 1024)) return KVE_ERR_GEOMETRY;
  if (c->agg == KVE_AGG_TOKEN_MLP && !token_mlp_supported(c->C, c->d_sum)) return KVE_ERR_GEOMETRY;
  if (c->d_g != 64 && c->d_g != 128 && c->d_g != 256) return KVE_ERR_GEOMETRY;
  if ((long long)c->B * c->Hkv > 65535) return KVE_ERR_GEOMETRY;
  return KVE_OK;
}

struct Carve {
  size_t off_P, off_H, off_partials, off_counters, off_stage, off_reclaim, off_ticket, off_block, off_kept_k, off_kept_v, off_listed, total;
};
// most CTAs of one attention launch: two resident per SM (148 SMs assumed where no device can be asked)
int attn_grid_cap() {
  int dev = 0;
  return 2 * (cudaGetDevice(&dev) == cudaSuccess ? sm_count() : 148);
}
// most splits per sequence the block-of-queries attention uses: one CTA per SM, one wave
int block_split_cap(long long S) {
  long long c = sm_count() / S;
  return (int)(c < 1 ? 1 : (c > MAX_SPLITS ? MAX_SPLITS : c));
}
Carve carve(const kvE_config& c) {
  const size_t S = (size_t)c.B * c.Hkv;
  const size_t max_chunks = ((size_t)c.max_tokens + c.C - 1) / c.C;
  Carve k;
  size_t o = 0;
  // gate projection P [S max_chunks][4 d_g]; the per-token MLP aggregator, which runs before the gate, borrows it
  // for its pooled activations [2][S max_chunks][d_sum]
  size_t p_floats = S * max_chunks * 4 * (size_t)c.d_g;
  if (c.agg == KVE_AGG_TOKEN_MLP && 2 * S * max_chunks * (size_t)c.d_sum > p_floats) p_floats = 2 * S * max_chunks * (size_t)c.d_sum;
  k.off_P = o;        o = align_up(o + p_floats * sizeof(float));
  // h_t of every gated (sequence, chunk) of one kvE_gate call, [S max_chunks][d_g]: what the score head reads
  k.off_H = o;        o = align_up(o + S * max_chunks * (size_t)c.d_g * sizeof(float));
  // attention partial records: the one of (sequence s, CTA c) at s + c, at most ATTN_GRID_LIMIT CTAs
  k.off_partials = o; o = align_up(o + (S + ATTN_GRID_LIMIT) * ATTN_PARTIAL_FLOATS * sizeof(float));
  k.off_counters = o; o = align_up(o + S * sizeof(int32_t));
  k.off_stage = o;    o = align_up(o + 4 * S * 128 * 2);   // k_new, v_new, q, out of kvE_decode_step_host
  k.off_reclaim = o;  o = align_up(o + (2 * S + 1) * sizeof(int32_t));   // per-sequence counts and offsets of kvE_reclaim_pages
  k.off_ticket = o;   o = align_up(o + sizeof(int32_t));       // last-CTA ticket of kvE_append_next
  k.off_block = o;    // split records of kvE_decode_attn_block: [S][splits][query rows, padded to 16][132] fp32
  if (c.max_query_tokens > 0) {
    const size_t rows = ((size_t)c.max_query_tokens * (c.Hq / c.Hkv) + 15) / 16 * 16;
    o = align_up(o + S * block_split_cap((long long)S) * rows * ATTN_PARTIAL_FLOATS * sizeof(float));
  }
  // what kvE_compact leaves for attention: the kept summary rows, compacted per sequence
  const size_t sum_bytes = (size_t)c.n_layers * S * max_chunks * 128 * 2;
  k.off_kept_k = o;   o = align_up(o + sum_bytes);
  k.off_kept_v = o;   o = align_up(o + sum_bytes);
  k.off_listed = o;   o = align_up(o + (size_t)c.n_layers * 2 * sizeof(int32_t));  // per layer: chunks the keep list covers; behind them, per layer: arrival ticket of the gate-step kernel
  k.total = o;
  return k;
}

// brackets the launches issued during its lifetime with the kernel id's event pair
struct Prof {
  kvE_store* st;
  int id;
  cudaStream_t s;
  Prof(kvE_store* st_, int id_, cudaStream_t s_) : st(st_), id(id_), s(s_) {
    if (st->profiling) cudaEventRecord(st->ev[2 * id], s);
  }
  ~Prof() {
    if (st->profiling) {
      cudaEventRecord(st->ev[2 * id + 1], s);
      st->ev_used[id] = true;
    }
  }
};

int cuda_fail(kvE_store* st, cudaError_t e) {
  st->cuda_error = cudaGetErrorString(e);
  return KVE_ERR_CUDA;
}

LayerView view(const kvE_store* st, int layer) {
  const kvE_config& c = st->cfg;
  const kvE_buffers& b = st->buf;
  const size_t S = st->S, mc = st->max_chunks, L = (size_t)layer;
  LayerView v;
  v.k_pages = static_cast<uint16_t*>(b.k_pages);
  v.v_pages = static_cast<uint16_t*>(b.v_pages);
  v.n_pages = b.n_pages;
  v.page_table = b.page_table + L * S * mc;
  v.seq_len = b.seq_len + L * c.B;
  v.ksum_f32 = b.ksum_f32 + L * S * mc * 128;
  v.vsum_f32 = b.vsum_f32 + L * S * mc * 128;
  v.ksum_bf16 = static_cast<uint16_t*>(b.ksum_bf16) + L * S * mc * 128;
  v.vsum_bf16 = static_cast<uint16_t*>(b.vsum_bf16) + L * S * mc * 128;
  v.scores = b.scores + L * S * mc;
  v.keep_idx = b.keep_idx + L * S * mc;
  v.keep_cnt = b.keep_cnt + L * S;
  v.lstm_h = b.lstm_h + L * S * c.d_g;
  v.lstm_c = b.lstm_c + L * S * c.d_g;
  v.status = b.status_word;
  v.n_listed = reinterpret_cast<int32_t*>(static_cast<char*>(b.workspace) + st->off_listed) + layer;
  v.step_ticket = v.n_listed + st->cfg.n_layers;
  v.B = c.B; v.H = c.Hkv; v.S = st->S; v.C = c.C; v.max_chunks = st->max_chunks; v.max_tokens = c.max_tokens;
  return v;
}

int stale_chunks(const kvE_config& c, int n) { return n > c.W ? (n - c.W) / c.C : 0; }

bool bad_layer(const kvE_store* st, int layer) { return !st || layer < 0 || layer >= st->cfg.n_layers; }

// every launch goes to the current device: it must be the one the handle's buffers live on
bool wrong_device(const kvE_store* st) {
  int dev = -1;
  return cudaGetDevice(&dev) != cudaSuccess || dev != st->device;
}

// How an attention launch is cut up.  Every sequence is cut into k equal parts and CTA c of G takes the contiguous
// run of parts [c S k / G, (c + 1) S k / G), which it streams as one piece (no break between parts of one sequence).
// G is one resident wave at most (two CTAs per SM).  k is chosen by a small cost model in microseconds, fitted to
// measurements: a CTA takes about 1.4 us per 64-row tile whether it shares its SM or not (its eight consumer warps set
// that pace; two CTAs per SM are what saturates HBM), so the launch lasts as long as the busiest CTA's tiles, plus its
// end: about 0.5 us when every CTA owns whole sequences (k = 1), about 3.5 us and growing with the number of records
// when sequences are shared and the last ones go through global memory (record, fence, ticket, merge).
struct AttnCut { int k, grid; };
AttnCut attention_cut(const kvE_store* st, AttnMode mode, const LayerState& ls) {
  const long long n_upper = ls.reserve_upper > ls.n_tokens ? ls.reserve_upper : ls.n_tokens;
  long long tail, lead;
  if (mode == ATTN_DENSE) { tail = n_upper; lead = 0; }
  else {
    tail = n_upper - (long long)ls.n_compacted * st->cfg.C;
    lead = (long long)ls.n_compacted * (mode == ATTN_RAW ? st->cfg.C : 1) / 2;      // about half of the chunks are kept
  }
  long long tiles = (tail + ATTN_TILE_ROWS - 1) / ATTN_TILE_ROWS + (lead + ATTN_TILE_ROWS - 1) / ATTN_TILE_ROWS;
  if (tiles < 1) tiles = 1;
  const long long G = st->attn_grid_max, S = st->S;
  const long long k_max = tiles < MAX_SPLITS ? tiles : MAX_SPLITS;
  auto cost_of = [&](long long k, long long* grid_out) {
    const long long parts = S * k, grid = parts < G ? parts : G;
    const long long rounds = (parts + grid - 1) / grid;                 // parts of the busiest CTA
    if (grid_out) *grid_out = grid;
    return (double)rounds * (double)tiles / (double)k * 1.4 + (k > 1 ? 4.5 + 0.06 * (double)k : 0.5);
  };
  // the kernel cuts the parts up in 32-bit arithmetic: S k (G + 1) must stay below 2^32
  double best = 1e30;
  for (long long k = 1; k <= k_max && S * k * (G + 1) < (1LL << 32); ++k)
    if (cost_of(k, nullptr) < best) best = cost_of(k, nullptr);
  long long k_pick = 1;      // whole sequences only when that is the cheapest; else near-ties go to the finer cut (evener bytes per CTA)
  for (long long k = 2; k <= k_max && S * k * (G + 1) < (1LL << 32); ++k)
    if (cost_of(k, nullptr) <= best + 0.3 && cost_of(1, nullptr) > best + 1e-9) k_pick = k;
  long long grid = 1;
  cost_of(k_pick, &grid);
  return AttnCut{(int)k_pick, (int)grid};
}

struct KeptRows { void *k, *v; };      // kept summary rows of a layer, compacted by kvE_compact
KeptRows kept_rows(const kvE_store* st, int layer) {
  char* ws = static_cast<char*>(st->buf.workspace);
  const size_t rows = (size_t)layer * st->S * st->max_chunks;
  return KeptRows{ws + st->off_kept_k + rows * 256, ws + st->off_kept_v + rows * 256};
}

int run_attention(kvE_store* st, int layer, AttnMode mode, const void* q, void* out, float* lse, float scale,
                  float* partials, int32_t* counters, cudaStream_t stream, const void* k_new = nullptr, const void* v_new = nullptr) {
  const LayerState& ls = st->layers[layer];
  const KeptRows kr = kept_rows(st, layer);
  const AttnCut cut = attention_cut(st, mode, ls);
  int32_t* ticket = reinterpret_cast<int32_t*>(static_cast<char*>(st->buf.workspace) + st->off_ticket);
  Prof prof(st, mode == ATTN_DENSE ? KVE_K_ATTN_DENSE : KVE_K_ATTN, stream);
  cudaError_t e = launch_attn(view(st, layer), mode, ls.n_compacted, cut.k, cut.grid, q, out, lse, scale, kr.k, kr.v, partials,
                              counters, k_new, v_new, ticket, stream);
  return e == cudaSuccess ? KVE_OK : cuda_fail(st, e);
}

int run_attention(kvE_store* st, int layer, AttnMode mode, const void* q, void* out, float* lse, float scale,
                  cudaStream_t stream) {
  char* ws = static_cast<char*>(st->buf.workspace);
  return run_attention(st, layer, mode, q, out, lse, scale, reinterpret_cast<float*>(ws + st->off_partials),
                       reinterpret_cast<int32_t*>(ws + st->off_counters), stream);
}

void release_host_objects(kvE_store* st) {
  if (st->ev_made)
    for (cudaEvent_t e : st->ev) cudaEventDestroy(e);
}

// the keep list no longer covers chunks from `value` on (their summaries or scores changed): host count and device count
int lower_listed(kvE_store* st, int layer, int value, cudaStream_t stream) {
  LayerState& ls = st->layers[layer];
  if (ls.n_compacted <= value) return KVE_OK;
  ls.n_compacted = value;
  cudaError_t e = launch_set_listed(view(st, layer), value, stream);
  return e == cudaSuccess ? KVE_OK : cuda_fail(st, e);
}

}  // namespace

extern "C" {

size_t kvE_workspace_bytes(const kvE_config* cfg) {
  if (check_config(cfg) != KVE_OK) return 0;
  return carve(*cfg).total;
}

int kvE_create(const kvE_config* cfg, const kvE_buffers* buf, kvE_store** out) {
  if (!out) return KVE_ERR_ARG;
  *out = nullptr;
  int rc = check_config(cfg);
  if (rc != KVE_OK) return rc;
  if (!buf || !buf->k_pages || !buf->v_pages || !buf->page_table || !buf->seq_len || !buf->ksum_f32 ||
      !buf->vsum_f32 || !buf->ksum_bf16 || !buf->vsum_bf16 || !buf->scores || !buf->keep_idx || !buf->keep_cnt ||
      !buf->lstm_h || !buf->lstm_c || !buf->workspace || !buf->status_word || buf->n_pages <= 0)
    return KVE_ERR_ARG;
  const Carve k = carve(*cfg);
  if (buf->workspace_bytes < k.total) return KVE_ERR_CAPACITY;
  if (reinterpret_cast<uintptr_t>(buf->workspace) % ALIGN != 0) return KVE_ERR_ARG;
  kvE_store* st = new (std::nothrow) kvE_store();
  if (!st) return KVE_ERR_ARG;
  st->cfg = *cfg;
  st->buf = *buf;
  if (cudaGetDevice(&st->device) != cudaSuccess) {
    delete st;
    return KVE_ERR_CUDA;
  }
  st->S = cfg->B * cfg->Hkv;
  st->max_chunks = (cfg->max_tokens + cfg->C - 1) / cfg->C;
  st->off_P = k.off_P; st->off_H = k.off_H; st->off_partials = k.off_partials; st->off_counters = k.off_counters;
  st->off_stage = k.off_stage; st->off_reclaim = k.off_reclaim; st->off_ticket = k.off_ticket; st->off_block = k.off_block;
  st->off_kept_k = k.off_kept_k; st->off_kept_v = k.off_kept_v; st->off_listed = k.off_listed; st->ws_needed = k.total;
  st->attn_grid_max = attn_grid_cap();
  if ((size_t)st->attn_grid_max > ATTN_GRID_LIMIT) st->attn_grid_max = (int)ATTN_GRID_LIMIT;
  if (cfg->max_query_tokens > 0) {
    st->block_hp = attn_block_hp(cfg->C);
    st->block_split_cap = block_split_cap(st->S);
    // maps over the page pools and over the compacted kept summary rows (all layers) in the workspace
    char* ws0 = static_cast<char*>(buf->workspace);
    const cudaError_t em = encode_attn_block_maps(st->block_maps, buf->k_pages, buf->v_pages, (long long)buf->n_pages * cfg->C,
                                                  st->block_hp, ws0 + k.off_kept_k, ws0 + k.off_kept_v,
                                                  (long long)cfg->n_layers * st->S * st->max_chunks);
    if (em != cudaSuccess) {
      delete st;
      return KVE_ERR_CUDA;
    }
    st->block_ready = true;
  }
  st->layers.assign(cfg->n_layers, LayerState());
  // partial records, tickets ... and the kept-row buffers (a box of the query-block kernel may reach past a sequence's
  // kept count: what it finds there must be finite)
  cudaError_t e = cudaMemset(static_cast<char*>(buf->workspace) + k.off_partials, 0, k.total - k.off_partials);
  if (e == cudaSuccess) e = cudaMemset(buf->status_word, 0, sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMemset(buf->seq_len, 0, sizeof(int32_t) * (size_t)cfg->n_layers * cfg->B);
  if (e == cudaSuccess) e = cudaMemset(buf->keep_cnt, 0, sizeof(int32_t) * (size_t)cfg->n_layers * st->S);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    release_host_objects(st);
    delete st;
    return KVE_ERR_CUDA;
  }
  *out = st;
  return KVE_OK;
}

int kvE_destroy(kvE_store* st) {
  if (st) release_host_objects(st);
  delete st;
  return KVE_OK;
}

int kvE_append(kvE_store* st, int layer, const void* k_new, const void* v_new, int n_new, int* n_ready, void* stream) {
  if (bad_layer(st, layer) || !k_new || !v_new || n_new < 0) return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  LayerState& ls = st->layers[layer];
  if ((long long)ls.n_tokens + n_new > st->cfg.max_tokens) return KVE_ERR_CAPACITY;
  if (n_new > 0) {
    Prof prof(st, KVE_K_APPEND, static_cast<cudaStream_t>(stream));
    cudaError_t e = launch_append(view(st, layer), k_new, v_new, n_new, ls.n_tokens, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(st, e);
    ls.n_tokens += n_new;
    ls.reserve_upper = 0;
  }
  if (n_ready) *n_ready = stale_chunks(st->cfg, ls.n_tokens) - ls.n_gated;
  return KVE_OK;
}

int kvE_append_next(kvE_store* st, int layer, const void* k_new, const void* v_new, int n_new, int n_reserve, void* stream) {
  if (bad_layer(st, layer) || !k_new || !v_new || n_new <= 0 || n_reserve < 0) return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  LayerState& ls = st->layers[layer];
  if ((long long)ls.n_tokens + n_new > st->cfg.max_tokens) return KVE_ERR_CAPACITY;
  Prof prof(st, KVE_K_APPEND, static_cast<cudaStream_t>(stream));
  int32_t* ticket = reinterpret_cast<int32_t*>(static_cast<char*>(st->buf.workspace) + st->off_ticket);
  cudaError_t e = launch_append_next(view(st, layer), k_new, v_new, n_new, ticket, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(st, e);
  long long upper = (long long)ls.n_tokens + n_new + n_reserve;
  if (upper > st->cfg.max_tokens) upper = st->cfg.max_tokens;
  if (upper > ls.reserve_upper) ls.reserve_upper = (int)upper;
  ls.n_tokens += n_new;
  return KVE_OK;
}

int kvE_set_len(kvE_store* st, int layer, int n, void* stream) {
  if (bad_layer(st, layer) || n < 0) return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  if (n > st->cfg.max_tokens) return KVE_ERR_CAPACITY;
  LayerState& ls = st->layers[layer];
  const int nc = stale_chunks(st->cfg, n);
  // a keep list that reaches past the new stale range is dropped, on the device too (-1: leave the device's count alone)
  cudaError_t e = launch_set_len(view(st, layer), n, ls.n_compacted > nc ? 0 : -1, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(st, e);
  ls.n_tokens = n;
  ls.reserve_upper = 0;
  if (ls.n_summarised > nc) ls.n_summarised = nc;
  if (ls.n_gated > nc) ls.n_gated = 0;          // the carried LSTM state is past the cut: gate again from chunk 0
  if (ls.n_compacted > nc) {
    // the keep list on the device may name chunks that are raw tail again: drop it; attention reads
    // every stored row until the next kvE_compact / kvE_compact_topk, which is exact
    ls.n_compacted = 0;
    ls.by_topk = false;
  }
  return KVE_OK;
}

int kvE_set_attend(kvE_store* st, int attend) {
  if (!st || (attend != KVE_ATTEND_SUMMARY && attend != KVE_ATTEND_RAW)) return KVE_ERR_ARG;
  st->cfg.attend = attend;
  return KVE_OK;
}

int kvE_set_gate_planes(kvE_store* st, int planes) {
  if (!st || (planes != 2 && planes != 3)) return KVE_ERR_ARG;
  st->gate_planes = planes;
  return KVE_OK;
}

int kvE_summarize_chunks(kvE_store* st, int layer, int chunk_begin, int chunk_end, const kvE_agg_weights* w,
                         void* stream) {
  if (bad_layer(st, layer) || chunk_begin < 0 || chunk_end < chunk_begin) return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  LayerState& ls = st->layers[layer];
  if (chunk_end > stale_chunks(st->cfg, ls.n_tokens)) return KVE_ERR_STATE;   // the window is never summarised
  const bool token_mlp = st->cfg.agg == KVE_AGG_TOKEN_MLP;
  const bool mlp = st->cfg.agg == KVE_AGG_MLP;
  if ((mlp || token_mlp) && (!w || !w->W1K || !w->W2K || !w->W1V || !w->W2V || !w->b1K || !w->b2K || !w->b1V || !w->b2V))
    return KVE_ERR_ARG;
  if (chunk_end == chunk_begin) return KVE_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const LayerView v = view(st, layer);
  cudaError_t e = cudaSuccess;
  if (!token_mlp) {
    Prof prof(st, KVE_K_CHUNK_MEAN, s);
    e = launch_chunk_mean(v, chunk_begin, chunk_end, !mlp, st->cfg.agg == KVE_AGG_MAX, s, -1);
  } else {
    Prof prof(st, KVE_K_CHUNK_MLP, s);
    MlpWeights mw;
    mw.W1K = static_cast<const uint16_t*>(w->W1K); mw.W2K = static_cast<const uint16_t*>(w->W2K);
    mw.W1V = static_cast<const uint16_t*>(w->W1V); mw.W2V = static_cast<const uint16_t*>(w->W2V);
    mw.b1K = w->b1K; mw.b2K = w->b2K; mw.b1V = w->b1V; mw.b2V = w->b2V;
    e = launch_chunk_token_mlp(v, chunk_begin, chunk_end, mw, st->cfg.d_sum,
                               reinterpret_cast<float*>(static_cast<char*>(st->buf.workspace) + st->off_P), s);
  }
  if (e == cudaSuccess && mlp) {
    Prof prof(st, KVE_K_CHUNK_MLP, s);
    MlpWeights mw;
    mw.W1K = static_cast<const uint16_t*>(w->W1K); mw.W2K = static_cast<const uint16_t*>(w->W2K);
    mw.W1V = static_cast<const uint16_t*>(w->W1V); mw.W2V = static_cast<const uint16_t*>(w->W2V);
    mw.b1K = w->b1K; mw.b2K = w->b2K; mw.b1V = w->b1V; mw.b2V = w->b2V;
    e = launch_chunk_mlp(v, chunk_begin, chunk_end, mw, st->cfg.d_sum, s, -1);
  }
  if (e != cudaSuccess) return cuda_fail(st, e);
  if (chunk_begin <= ls.n_summarised && chunk_end > ls.n_summarised) ls.n_summarised = chunk_end;
  return lower_listed(st, layer, chunk_begin, s);                   // the compacted copies of these summaries are stale
}

int kvE_gate(kvE_store* st, int layer, int chunk_begin, int chunk_end, const kvE_lstm_weights* w, void* stream) {
  if (bad_layer(st, layer) || chunk_begin < 0 || chunk_end < chunk_begin) return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  if (!w || !w->W_ih || !w->W_hh || !w->b_ih || !w->b_hh || !w->w_s) return KVE_ERR_ARG;
  LayerState& ls = st->layers[layer];
  if (chunk_end > ls.n_summarised) return KVE_ERR_STATE;
  if (chunk_begin != 0 && chunk_begin != ls.n_gated) return KVE_ERR_STATE;
  if (chunk_end == chunk_begin) {
    if (chunk_begin == 0) ls.n_gated = 0;
    return KVE_OK;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const LayerView v = view(st, layer);
  float* P = reinterpret_cast<float*>(static_cast<char*>(st->buf.workspace) + st->off_P);
  cudaError_t e;
  {
    Prof prof(st, KVE_K_GATE_PROJ, s);
    e = launch_gate_proj(v, chunk_begin, chunk_end, static_cast<const uint16_t*>(w->W_ih), w->b_ih, w->b_hh,
                         st->cfg.d_g, P, s);
  }
  if (e == cudaSuccess) {
    Prof prof(st, KVE_K_GATE_RNN, s);
    e = launch_gate_rnn(v, chunk_begin, chunk_end, static_cast<const uint16_t*>(w->W_hh), w->w_s, w->b_s, st->cfg.d_g,
                        P, reinterpret_cast<float*>(static_cast<char*>(st->buf.workspace) + st->off_H), chunk_begin == 0,
                        st->gate_planes, s);
  }
  if (e != cudaSuccess) return cuda_fail(st, e);
  ls.n_gated = chunk_end;
  return lower_listed(st, layer, chunk_begin, s);                   // scores changed under the keep list
}

int kvE_compact(kvE_store* st, int layer, float tau, void* stream) {
  if (bad_layer(st, layer)) return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  LayerState& ls = st->layers[layer];
  Prof prof(st, KVE_K_COMPACT, static_cast<cudaStream_t>(stream));
  const KeptRows kr = kept_rows(st, layer);
  cudaError_t e = launch_compact(view(st, layer), ls.n_gated, tau, kr.k, kr.v, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(st, e);
  ls.n_compacted = ls.n_gated;
  ls.tau = tau;
  ls.by_topk = false;
  return KVE_OK;
}

int kvE_gate_next(kvE_store* st, int layer, const kvE_lstm_weights* w, float tau, void* stream) {
  if (bad_layer(st, layer)) return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  if (!w || !w->W_ih || !w->W_hh || !w->b_ih || !w->b_hh || !w->w_s) return KVE_ERR_ARG;
  LayerState& ls = st->layers[layer];
  const int t = ls.n_gated;
  if (t >= ls.n_summarised) return KVE_ERR_STATE;
  if (t == 0 || ls.n_compacted != t || ls.by_topk || ls.tau != tau) {      // no list to append to: the general path
    const int rc = kvE_gate(st, layer, t, t + 1, w, stream);
    return rc != KVE_OK ? rc : kvE_compact(st, layer, tau, stream);
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const KeptRows kr = kept_rows(st, layer);
  cudaError_t e;
  {
    Prof prof(st, KVE_K_GATE_RNN, s);
    e = launch_gate_step(view(st, layer), t, static_cast<const uint16_t*>(w->W_ih), static_cast<const uint16_t*>(w->W_hh),
                         w->b_ih, w->b_hh, w->w_s, w->b_s, tau, st->cfg.d_g, st->gate_planes,
                         static_cast<uint16_t*>(kr.k), static_cast<uint16_t*>(kr.v), -1, s);
  }
  if (e != cudaSuccess) return cuda_fail(st, e);
  ls.n_gated = ls.n_compacted = t + 1;
  return KVE_OK;
}

int kvE_refresh_next(kvE_store* st, int layer, const kvE_agg_weights* aw, const kvE_lstm_weights* lw, float tau, void* stream) {
  if (bad_layer(st, layer)) return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  if (!lw || !lw->W_ih || !lw->W_hh || !lw->b_ih || !lw->b_hh || !lw->w_s) return KVE_ERR_ARG;
  if (st->cfg.agg == KVE_AGG_TOKEN_MLP) return KVE_ERR_GEOMETRY;      // its kernels take their position from the launch only
  const bool mlp = st->cfg.agg == KVE_AGG_MLP;
  if (mlp && (!aw || !aw->W1K || !aw->W2K || !aw->W1V || !aw->W2V || !aw->b1K || !aw->b2K || !aw->b1V || !aw->b2V)) return KVE_ERR_ARG;
  LayerState& ls = st->layers[layer];
  // a keep list under this tau that covers everything gated, and nothing summarised ahead of it: the device appends to it
  if (ls.n_compacted < 1 || ls.n_compacted != ls.n_gated || ls.n_summarised != ls.n_gated || ls.by_topk || ls.tau != tau)
    return KVE_ERR_STATE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const LayerView v = view(st, layer);
  const int W = st->cfg.W;
  cudaError_t e;
  {
    Prof prof(st, KVE_K_CHUNK_MEAN, s);
    e = launch_chunk_mean(v, 0, 1, !mlp, st->cfg.agg == KVE_AGG_MAX, s, W);
  }
  if (e == cudaSuccess && mlp) {
    Prof prof(st, KVE_K_CHUNK_MLP, s);
    MlpWeights mw;
    mw.W1K = static_cast<const uint16_t*>(aw->W1K); mw.W2K = static_cast<const uint16_t*>(aw->W2K);
    mw.W1V = static_cast<const uint16_t*>(aw->W1V); mw.W2V = static_cast<const uint16_t*>(aw->W2V);
    mw.b1K = aw->b1K; mw.b2K = aw->b2K; mw.b1V = aw->b1V; mw.b2V = aw->b2V;
    e = launch_chunk_mlp(v, 0, 1, mw, st->cfg.d_sum, s, W);
  }
  if (e == cudaSuccess) {
    Prof prof(st, KVE_K_GATE_RNN, s);
    const KeptRows kr = kept_rows(st, layer);
    e = launch_gate_step(v, 0, static_cast<const uint16_t*>(lw->W_ih), static_cast<const uint16_t*>(lw->W_hh), lw->b_ih,
                         lw->b_hh, lw->w_s, lw->b_s, tau, st->cfg.d_g, st->gate_planes, static_cast<uint16_t*>(kr.k),
                         static_cast<uint16_t*>(kr.v), W, s);
  }
  if (e != cudaSuccess) return cuda_fail(st, e);
  // what this call does when it executes once on the state the host knows of
  if (stale_chunks(st->cfg, ls.n_tokens) > ls.n_gated && ls.n_gated < st->max_chunks)
    ls.n_summarised = ls.n_gated = ls.n_compacted = ls.n_gated + 1;
  return KVE_OK;
}

int kvE_adopt_device_state(kvE_store* st, int layer, void* stream) {
  if (bad_layer(st, layer)) return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  LayerState& ls = st->layers[layer];
  const LayerView v = view(st, layer);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t len = 0, listed = 0;
  cudaError_t e = cudaMemcpyAsync(&len, v.seq_len, sizeof(len), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(&listed, v.n_listed, sizeof(listed), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_fail(st, e);
  if (len < 0 || len > st->cfg.max_tokens || listed < 0 || listed > stale_chunks(st->cfg, len)) return KVE_ERR_STATE;
  ls.n_tokens = len;
  ls.reserve_upper = 0;
  if (ls.n_compacted > 0 && ls.n_compacted == ls.n_gated && ls.n_summarised == ls.n_gated && listed > 0)
    ls.n_summarised = ls.n_gated = ls.n_compacted = listed;      // triggers executed on the device move all three together
  return KVE_OK;
}

int kvE_refresh(kvE_store* st, int layer, const kvE_agg_weights* aw, const kvE_lstm_weights* lw, float tau, void* stream) {
  if (bad_layer(st, layer)) return KVE_ERR_ARG;
  const int nc = stale_chunks(st->cfg, st->layers[layer].n_tokens);
  int rc = kvE_summarize_chunks(st, layer, 0, nc, aw, stream);
  if (rc == KVE_OK) rc = kvE_gate(st, layer, 0, nc, lw, stream);
  if (rc == KVE_OK) rc = kvE_compact(st, layer, tau, stream);
  return rc;
}

int kvE_compact_topk(kvE_store* st, int layer, int k, void* stream) {
  if (bad_layer(st, layer)) return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  LayerState& ls = st->layers[layer];
  Prof prof(st, KVE_K_COMPACT, static_cast<cudaStream_t>(stream));
  const KeptRows kr = kept_rows(st, layer);
  cudaError_t e = launch_compact_topk(view(st, layer), ls.n_gated, k, kr.k, kr.v, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(st, e);
  ls.n_compacted = ls.n_gated;
  ls.by_topk = true;
  return KVE_OK;
}

int kvE_reclaim_pages(kvE_store* st, int layer, int chunk_begin, int chunk_end, int mode, int32_t* free_list,
                      int64_t capacity, int32_t* free_count, void* stream) {
  if (bad_layer(st, layer) || chunk_begin < 0 || chunk_end < chunk_begin || !free_list || !free_count || capacity < 0)
    return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  if (mode != KVE_RECLAIM_DISCARDED && mode != KVE_RECLAIM_GATED) return KVE_ERR_ARG;
  const LayerState& ls = st->layers[layer];
  if (chunk_end > ls.n_compacted) return KVE_ERR_STATE;                        // only chunks the retention rule has judged
  if (mode == KVE_RECLAIM_GATED && st->cfg.attend != KVE_ATTEND_SUMMARY) return KVE_ERR_STATE;   // RAW attention still reads kept pages
  if (mode == KVE_RECLAIM_DISCARDED && ls.by_topk) return KVE_ERR_STATE;       // "discarded" is defined by the threshold rule
  if (chunk_end == chunk_begin) {
    cudaError_t e = cudaMemsetAsync(free_count, 0, sizeof(int32_t), static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? KVE_OK : cuda_fail(st, e);
  }
  int32_t* scratch = reinterpret_cast<int32_t*>(static_cast<char*>(st->buf.workspace) + st->off_reclaim);
  cudaError_t e = launch_reclaim(view(st, layer), chunk_begin, chunk_end, ls.tau, mode, scratch, free_list, capacity, free_count,
                                 static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? KVE_OK : cuda_fail(st, e);
}

int kvE_decode_attn(kvE_store* st, int layer, const void* q, void* out, float* lse, float scale, void* stream) {
  if (bad_layer(st, layer) || !q || !out) return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  if (st->cfg.Hq != st->cfg.Hkv) return KVE_ERR_GEOMETRY;      // grouped query heads go through kvE_decode_attn_block
  const AttnMode mode = st->cfg.attend == KVE_ATTEND_RAW ? ATTN_RAW : ATTN_SUMMARY;
  return run_attention(st, layer, mode, q, out, lse, scale, static_cast<cudaStream_t>(stream));
}

int kvE_decode_step(kvE_store* st, int layer, const void* k_new, const void* v_new, const void* q, void* out, float* lse,
                    float scale, int n_reserve, void* stream) {
  if (bad_layer(st, layer) || !k_new || !v_new || !q || !out || n_reserve < 0) return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  if (st->cfg.Hq != st->cfg.Hkv) return KVE_ERR_GEOMETRY;
  LayerState& ls = st->layers[layer];
  if ((long long)ls.n_tokens + 1 > st->cfg.max_tokens) return KVE_ERR_CAPACITY;
  // the launch is sized for the cache with the new token (and the announced growth) in it
  long long upper = (long long)ls.n_tokens + 1 + n_reserve;
  if (upper > st->cfg.max_tokens) upper = st->cfg.max_tokens;
  if (upper > ls.reserve_upper) ls.reserve_upper = (int)upper;
  ls.n_tokens += 1;
  const AttnMode mode = st->cfg.attend == KVE_ATTEND_RAW ? ATTN_RAW : ATTN_SUMMARY;
  char* ws = static_cast<char*>(st->buf.workspace);
  return run_attention(st, layer, mode, q, out, lse, scale, reinterpret_cast<float*>(ws + st->off_partials),
                       reinterpret_cast<int32_t*>(ws + st->off_counters), static_cast<cudaStream_t>(stream), k_new, v_new);
}

int kvE_decode_attn_dense(kvE_store* st, int layer, const void* q, void* out, float* lse, float scale, void* stream) {
  if (bad_layer(st, layer) || !q || !out) return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  if (st->cfg.Hq != st->cfg.Hkv) return KVE_ERR_GEOMETRY;
  return run_attention(st, layer, ATTN_DENSE, q, out, lse, scale, static_cast<cudaStream_t>(stream));
}

int kvE_decode_attn_block(kvE_store* st, int layer, const void* q, int n_query_tokens, int dense, int causal, void* out,
                          float* lse, float scale, void* stream) {
  if (bad_layer(st, layer) || !q || !out || n_query_tokens <= 0) return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  if (!st->block_ready) return KVE_ERR_STATE;                  // cfg.max_query_tokens was 0
  if (n_query_tokens > st->cfg.max_query_tokens) return KVE_ERR_CAPACITY;
  const AttnMode mode = dense ? ATTN_DENSE : (st->cfg.attend == KVE_ATTEND_RAW ? ATTN_RAW : ATTN_SUMMARY);
  const LayerState& ls = st->layers[layer];
  // padded rows per sequence: the raw tail rounded up to whole tiles, then the kept rows
  long long tail, lead;
  const long long n_upper = ls.reserve_upper > ls.n_tokens ? ls.reserve_upper : ls.n_tokens;
  if (mode == ATTN_DENSE) { tail = n_upper; lead = 0; }
  else {
    tail = n_upper - (long long)ls.n_compacted * st->cfg.C;
    lead = (long long)ls.n_compacted * (mode == ATTN_RAW ? st->cfg.C : 1);
  }
  // causal: the block's tokens are the newest rows of the raw tail; a tail shorter than the block would
  // leave the first tokens without a defined position
  if (causal && (long long)ls.n_tokens - (mode == ATTN_DENSE ? 0 : (long long)ls.n_compacted * st->cfg.C) < n_query_tokens)
    return KVE_ERR_STATE;
  const long long tiles = (tail + ATTN_TILE_ROWS - 1) / ATTN_TILE_ROWS + (lead + ATTN_TILE_ROWS - 1) / ATTN_TILE_ROWS;
  long long splits = st->block_split_cap;
  if (splits > tiles) splits = tiles;
  if (splits < 1) splits = 1;
  const long long tiles_per_split = tiles > 0 ? (tiles + splits - 1) / splits : 1;
  AttnPlan plan;
  plan.rows_per_split = (int)(tiles_per_split * ATTN_TILE_ROWS);
  plan.max_splits = (int)(tiles > 0 ? (tiles + tiles_per_split - 1) / tiles_per_split : 1);
  char* ws = static_cast<char*>(st->buf.workspace);
  Prof prof(st, KVE_K_ATTN_BLOCK, static_cast<cudaStream_t>(stream));
  cudaError_t e = launch_attn_block(view(st, layer), st->block_maps, mode, ls.n_compacted, plan, n_query_tokens,
                                    st->cfg.Hq / st->cfg.Hkv, causal ? 1 : 0, st->block_hp, (long long)layer * st->S * st->max_chunks, q, out,
                                    lse, scale, reinterpret_cast<float*>(ws + st->off_block),
                                    reinterpret_cast<int32_t*>(ws + st->off_counters), static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? KVE_OK : cuda_fail(st, e);
}

static int decode_step_host(kvE_store* st, int layer, const void* k_new_host, const void* v_new_host, const void* q_host,
                            void* out_host, const kvE_agg_weights* aw, const kvE_lstm_weights* lw, float tau, float scale,
                            int from_scratch, void* stream, bool wait) {
  if (bad_layer(st, layer) || !k_new_host || !v_new_host || !q_host || !out_host || !lw) return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  if (st->cfg.Hq != st->cfg.Hkv) return KVE_ERR_GEOMETRY;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t row_bytes = (size_t)st->S * 128 * 2;
  char* stage = static_cast<char*>(st->buf.workspace) + st->off_stage;
  char *dk = stage, *dv = stage + row_bytes, *dq = stage + 2 * row_bytes, *dout = stage + 3 * row_bytes;
  cudaError_t e = cudaMemcpyAsync(dk, k_new_host, row_bytes, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(dv, v_new_host, row_bytes, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(dq, q_host, row_bytes, cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return cuda_fail(st, e);
  int rc = kvE_append(st, layer, dk, dv, 1, nullptr, stream);
  if (rc != KVE_OK) return rc;
  LayerState& ls = st->layers[layer];
  const int nc = stale_chunks(st->cfg, ls.n_tokens);
  if (from_scratch) {
    rc = kvE_refresh(st, layer, aw, lw, tau, stream);
    if (rc != KVE_OK) return rc;
  }
  const int s0 = ls.n_summarised;
  if (nc > s0) {
    rc = kvE_summarize_chunks(st, layer, s0, nc, aw, stream);
    if (rc != KVE_OK) return rc;
  }
  const int g0 = ls.n_gated;
  if (nc == g0 + 1) {      // the usual trigger: one chunk has left the window
    rc = kvE_gate_next(st, layer, lw, tau, stream);
    if (rc != KVE_OK) return rc;
  } else if (nc > g0) {
    rc = kvE_gate(st, layer, g0, nc, lw, stream);
    if (rc != KVE_OK) return rc;
  }
  if (ls.n_compacted != ls.n_gated) {
    rc = kvE_compact(st, layer, tau, stream);
    if (rc != KVE_OK) return rc;
  }
  rc = kvE_decode_attn(st, layer, dq, dout, nullptr, scale, stream);
  if (rc != KVE_OK) return rc;
  e = cudaMemcpyAsync(out_host, dout, row_bytes, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess && wait) e = cudaStreamSynchronize(s);
  return e == cudaSuccess ? KVE_OK : cuda_fail(st, e);
}

int kvE_decode_step_host(kvE_store* st, int layer, const void* k_new_host, const void* v_new_host, const void* q_host,
                         void* out_host, const kvE_agg_weights* aw, const kvE_lstm_weights* lw, float tau, float scale,
                         int from_scratch, void* stream) {
  return decode_step_host(st, layer, k_new_host, v_new_host, q_host, out_host, aw, lw, tau, scale, from_scratch, stream, true);
}

int kvE_decode_step_host_async(kvE_store* st, int layer, const void* k_new_host, const void* v_new_host, const void* q_host,
                               void* out_host, const kvE_agg_weights* aw, const kvE_lstm_weights* lw, float tau, float scale,
                               int from_scratch, void* stream) {
  return decode_step_host(st, layer, k_new_host, v_new_host, q_host, out_host, aw, lw, tau, scale, from_scratch, stream, false);
}

int kvE_poll_status(kvE_store* st, int* device_status) {
  if (!st || !device_status) return KVE_ERR_ARG;
  cudaError_t e = cudaDeviceSynchronize();
  int32_t word = 0;
  if (e == cudaSuccess) e = cudaMemcpy(&word, st->buf.status_word, sizeof(word), cudaMemcpyDeviceToHost);
  if (e == cudaSuccess && word != 0) e = cudaMemset(st->buf.status_word, 0, sizeof(word));
  if (e != cudaSuccess) return cuda_fail(st, e);
  *device_status = word;
  return KVE_OK;
}

int kvE_layer_state(const kvE_store* st, int layer, int* n_tokens, int* n_summarised, int* n_gated, int* n_compacted) {
  if (bad_layer(st, layer)) return KVE_ERR_ARG;
  const LayerState& ls = st->layers[layer];
  if (n_tokens) *n_tokens = ls.n_tokens;
  if (n_summarised) *n_summarised = ls.n_summarised;
  if (n_gated) *n_gated = ls.n_gated;
  if (n_compacted) *n_compacted = ls.n_compacted;
  return KVE_OK;
}

int kvE_profile(kvE_store* st, int enable) {
  if (!st) return KVE_ERR_ARG;
  if (enable && !st->ev_made) {
    for (cudaEvent_t& e : st->ev) {
      cudaError_t rc = cudaEventCreate(&e);
      if (rc != cudaSuccess) return cuda_fail(st, rc);
    }
    st->ev_made = true;
  }
  st->profiling = enable != 0;
  for (bool& u : st->ev_used) u = false;
  return KVE_OK;
}

int kvE_profile_read(kvE_store* st, float* us) {
  if (!st || !us) return KVE_ERR_ARG;
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(st, e);
  for (int k = 0; k < KVE_K_COUNT; ++k) {
    us[k] = -1.f;
    if (st->ev_made && st->ev_used[k]) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, st->ev[2 * k], st->ev[2 * k + 1]) == cudaSuccess) us[k] = ms * 1000.f;
    }
  }
  return KVE_OK;
}

const char* kvE_last_cuda_error(const kvE_store* st) { return st ? st->cuda_error.c_str() : ""; }

int kvE_selftest_timeout(kvE_store* st, int which, void* stream) {
  if (!st || (which != 0 && which != 1)) return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  cudaError_t e = launch_selftest_timeout(which, st->buf.status_word, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? KVE_OK : cuda_fail(st, e);
}

}  // extern "C"

// ---- kvE_decode_attn_static: gated attention whose split-K scratch lives inside the library ----------
// The scratch is a file-scope device array: every GPU that loads the library carries it until the
// process exits.  In host code `g_static_scratch` is only a stand-in for the symbol, not a device
// address, so the address the kernel gets is looked up once per device with cudaGetSymbolAddress.
namespace {

constexpr int STATIC_MAX_SEQ = KVE_STATIC_MAX_SEQUENCES;
constexpr int STATIC_MAX_REC = KVE_STATIC_MAX_PARTIALS;
constexpr size_t STATIC_COUNTER_BYTES = align_const(STATIC_MAX_SEQ * sizeof(int32_t));
constexpr size_t STATIC_BYTES = STATIC_COUNTER_BYTES + (size_t)STATIC_MAX_REC * ATTN_PARTIAL_FLOATS * sizeof(float);

static __device__ __align__(256) unsigned char g_static_scratch[STATIC_BYTES];

constexpr int MAX_DEVICES = 64;
std::mutex g_static_mutex;
unsigned char* g_static_ptr[MAX_DEVICES] = {};

// device address of the scratch on the CURRENT device (looked up on the first call per device)
cudaError_t static_scratch(unsigned char** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_static_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_static_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" int kvE_decode_attn_static(kvE_store* st, int layer, const void* q, void* out, float* lse, float scale,
                                      void* stream) {
  if (bad_layer(st, layer) || !q || !out) return KVE_ERR_ARG;
  if (wrong_device(st)) return KVE_ERR_STATE;
  if (st->cfg.Hq != st->cfg.Hkv) return KVE_ERR_GEOMETRY;
  const AttnMode mode = st->cfg.attend == KVE_ATTEND_RAW ? ATTN_RAW : ATTN_SUMMARY;
  const LayerState& ls = st->layers[layer];
  // the kernel needs S + G partial records for a launch of G CTAs
  const int grid = attention_cut(st, mode, ls).grid;
  const long long records = (long long)st->S + grid;
  if (st->S > STATIC_MAX_SEQ || records > STATIC_MAX_REC) {
    st->cuda_error = "kvE_decode_attn_static: " + std::to_string(st->S) + " sequences on " + std::to_string(grid) +
                     " CTAs exceed the built-in scratch (" + std::to_string(STATIC_MAX_SEQ) + " sequences, " +
                     std::to_string(STATIC_MAX_REC) + " partial records); use kvE_decode_attn";
    return KVE_ERR_CAPACITY;
  }
  unsigned char* scratch = nullptr;
  cudaError_t e = static_scratch(&scratch);
  if (e != cudaSuccess) return cuda_fail(st, e);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t* counters = reinterpret_cast<int32_t*>(scratch);
  float* partials = reinterpret_cast<float*>(scratch + STATIC_COUNTER_BYTES);
  // the array keeps whatever the last call left: the tickets must start at zero
  e = cudaMemsetAsync(counters, 0, sizeof(int32_t) * (size_t)st->S, s);
  if (e != cudaSuccess) return cuda_fail(st, e);
  return run_attention(st, layer, mode, q, out, lse, scale, partials, counters, s);
}

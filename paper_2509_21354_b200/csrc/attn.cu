// Flash-decode over the retained set (Sec. 3.3, softmax of Eq. 1):
//   out = softmax(q K'^T * scale) V',  rows of K', V' = [raw tail] ++ [kept chunks, oldest first]
// and, with mode = DENSE, Eq. 1 over every stored token (the full-cache baseline).
//
// HBM-bound: every retained K and V row (256 bytes each) is read exactly once, so the kernel is built
// to keep every SM streaming from its first microsecond to its last:
//  * A sequence's rows form 64-row tiles (raw tail first, kept chunks after it).  The host picks k,
//    the number of equal parts every sequence is cut into, so that the S k parts divide evenly over
//    the CTAs of one resident wave (two per SM); CTA c takes parts [c S k / G, (c + 1) S k / G): a
//    contiguous run that may span several sequences.  Its pipeline runs across sequence boundaries
//    without draining, every CTA moves nearly the same number of bytes whatever S is, and where a
//    part begins follows from the launch arguments, the stored length and one keep count, so the
//    first copies leave two dependent loads after the kernel starts.
//  * Warp 8 (producer) turns tiles into addresses (page table; kept summary rows sit compacted in
//    one contiguous run per sequence), merges rows that are contiguous in memory into runs with a
//    ballot, and issues one bulk copy (TMA engine, global -> shared, mbarrier byte counting) per run
//    into a 3-stage ring of 64-row K and V tiles.  The query row of a sequence travels with the
//    first tile of that sequence.
//  * Warps 0-7 (consumers) each take 8 rows of a tile: q.k partial sums per lane (4 head dims per
//    lane), a butterfly transpose-reduce that leaves one row's logit per group of four lanes, online
//    softmax with warp shuffles, then p.V with each lane owning 4 output dims.  When a CTA's run
//    leaves a sequence, the consumers drop their (m, l, acc) into a double-buffered exchange area
//    and carry on with the next sequence.
//  * Warp 9 (merger) folds the eight consumer states of a finished sequence (or part of one), and
//    either writes the output (this CTA had the whole sequence) or a partial record plus an atomic
//    ticket; the CTA that draws a sequence's last ticket merges its records by log-sum-exp.  Nobody
//    spins on another CTA.
//  * Fused append (kvE_decode_step): the step's new token need not be in its page yet.  Its row is streamed from the
//    caller's buffer as the last row of the raw tail, the CTA that streams it also stores it in the page, and the last
//    CTA to finish advances the stored length: one launch per decode step and layer instead of two.
// Every mbarrier wait is bounded; on give-up the status word gets KVE_ERR_TIMEOUT.
#include "common.cuh"
#include "kernels.h"

namespace kve {

// Optional per-CTA time stamps (build with -DKVE_ATTN_STAMPS, see attn_stamps.py): where a launch's time goes.
// Slots: 0 kernel entry, 1 after the wait for the predecessor, 2 first copy issued, 3 first tile landed,
// 4 last tile consumed, 5 merger warp done, 6 producer warp done.  Compiled out of the product library.
#ifdef KVE_ATTN_STAMPS
constexpr int STAMP_CTAS = 2048, STAMP_SLOTS = 8;
__device__ unsigned long long g_attn_stamps[STAMP_CTAS * STAMP_SLOTS];
__device__ __forceinline__ void stamp(int slot) {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  if (blockIdx.x < STAMP_CTAS) g_attn_stamps[blockIdx.x * STAMP_SLOTS + slot] = t;
}
#define KVE_STAMP(cond, slot) do { if (cond) stamp(slot); } while (0)
#else
#define KVE_STAMP(cond, slot) do { } while (0)
#endif

constexpr int AT_TILE = ATTN_TILE_ROWS;       // rows per stage
constexpr int AT_STAGES = 3;
constexpr int AT_CWARPS = 8;                  // consumer warps
constexpr int AT_SUB = AT_TILE / AT_CWARPS;   // 8 rows per consumer warp per tile
constexpr int AT_PRODUCER = AT_CWARPS;        // warp ids
constexpr int AT_THREADS = (AT_CWARPS + 2) * 32;
constexpr int AT_STAGE_ELEMS = AT_TILE * D;   // bf16 elements of one K (or V) tile
static_assert(AT_SUB == 8, "the transpose-reduce below is written for 8 rows per warp");

// shared-memory carve-up (bytes)
constexpr int AT_OFF_K = 0;
constexpr int AT_OFF_V = AT_OFF_K + AT_STAGES * AT_STAGE_ELEMS * 2;
constexpr int AT_OFF_Q = AT_OFF_V + AT_STAGES * AT_STAGE_ELEMS * 2;                 // [stages][128] bf16
constexpr int AT_OFF_COMB = AT_OFF_Q + AT_STAGES * ROW_BYTES;                       // [2][consumer warps][132] fp32
constexpr int AT_OFF_INFO = AT_OFF_COMB + 2 * AT_CWARPS * ATTN_PARTIAL_FLOATS * 4;  // [stages] int4
constexpr int AT_OFF_FINFO = AT_OFF_INFO + AT_STAGES * 16;                          // [2] int4
constexpr int AT_OFF_BAR = AT_OFF_FINFO + 2 * 16;                                   // full[3], empty[3], ffull[2], fempty[2]
constexpr int AT_SMEM_BYTES = AT_OFF_BAR + (2 * AT_STAGES + 4) * 8;
static_assert(AT_OFF_COMB % 16 == 0 && AT_OFF_INFO % 16 == 0 && AT_OFF_BAR % 8 == 0, "alignment of the carve-up");

int attn_smem_bytes() { return AT_SMEM_BYTES; }

// tile flags handed from the producer to the consumers
constexpr int TF_NEW = 1;      // first tile of a (sequence, list) in this CTA: fresh softmax state, query row in the stage
constexpr int TF_FLUSH = 2;    // last tile of a (sequence, list) in this CTA: hand the state to the merger afterwards
constexpr int TF_END = 4;      // no tile: the CTA's work is done

struct AttnArgs {
  LayerView v;
  int mode;
  int n_chunks;                // the host's count of chunks under the keep list: a prefetch hint; the kernel reads the device's
  int k;                       // parts per sequence
  const uint16_t* q;
  uint16_t* out;
  float* lse;
  float scale;
  const uint16_t* kkept;       // [S][max_chunks][128] kept summary rows, compacted (SUMMARY mode)
  const uint16_t* vkept;
  float* partials;             // [S + G][132]: the record of (sequence s, CTA c) sits at s + c
  int32_t* counters;           // [S], zero between launches
  // fused append (kvE_decode_step): one new token per sequence, placed at the length the device holds
  const uint16_t* k_new;       // [S][128] or null
  const uint16_t* v_new;
  int32_t* ticket;             // last CTA to finish publishes the new length
};

// what every role derives from the launch arguments and the stored length
struct AttnGeo {
  int n_tail, raw0, TT, per;   // tail rows / tiles per sequence; rows a kept chunk contributes
  int n;                       // tokens attended to (the new one included when one is being appended)
  int n_chunks;                // chunks the keep list covers (0 for full-cache attention)
  bool appending;              // the last tail row of every sequence is the new token, taken from k_new / v_new
  uint32_t I, P;               // parts in the launch (S k); CTAs that get any (min(G, I): none of them is empty)
};

// CTA c of P takes parts [c I / P, (c + 1) I / P); CTAs c >= P take none.  32-bit arithmetic (64-bit division
// would sit on the path to the first copy): the host keeps I * G below 2^32.
__device__ __forceinline__ uint32_t piece_begin(uint32_t c, uint32_t I, uint32_t P) { return c >= P ? I : (c * I) / P; }
// the CTA that holds part x
__device__ __forceinline__ uint32_t piece_of(uint32_t x, uint32_t I, uint32_t P) { return ((x + 1u) * P - 1u) / I; }

__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// Pulls what the producer will look up for sequence s into L2 (fire and forget: the keep count, the page ids
// of the raw tail, the head of the kept-chunk list), so that the dependent look-ups that follow cost an L2 hit each.
__device__ __forceinline__ void prefetch_sequence_metadata(const AttnArgs& a, int s, int lane) {
  const LayerView& v = a.v;
  if (s < 0 || s >= v.S) return;
  const long long sb = (long long)s * v.max_chunks;
  const int first_tail_chunk = (a.mode == ATTN_DENSE) ? 0 : a.n_chunks;
  if (lane == 0) prefetch_l2(v.keep_cnt + s);
  // page ids of the tail: 32 entries per 128-byte line; up to 8 lines (256 chunks) ahead
  if (lane < 8 && first_tail_chunk + lane * 32 < v.max_chunks) prefetch_l2(v.page_table + sb + first_tail_chunk + lane * 32);
  if (a.mode == ATTN_RAW && lane == 8) prefetch_l2(v.keep_idx + sb);
}

// rows the kept chunks of sequence s contribute
__device__ __forceinline__ int lead_rows_from(const AttnArgs& a, const AttnGeo& g, int keep_cnt) {
  if (a.mode == ATTN_DENSE || g.n_chunks <= 0) return 0;
  return min(max(keep_cnt, 0), g.n_chunks) * g.per;
}
__device__ __forceinline__ int lead_rows_of(const AttnArgs& a, const AttnGeo& g, int s) {
  if (a.mode == ATTN_DENSE || g.n_chunks <= 0) return 0;
  return lead_rows_from(a, g, a.v.keep_cnt[s]);
}

#define KVE_TR_ROUND(OFF, CNT)                                                        \
  {                                                                                   \
    const bool upper = (lane & (OFF)) != 0;                                           \
    _Pragma("unroll") for (int j = 0; j < (CNT); ++j) {                               \
      const float send = upper ? part[j] : part[j + (CNT)];                           \
      const float keep = upper ? part[j + (CNT)] : part[j];                           \
      part[j] = keep + __shfl_xor_sync(0xffffffffu, send, (OFF));                     \
    }                                                                                 \
  }

// one tile of the CTA's work as the producer sees it
struct TileDesc {
  int s, list, j, rows, flags;      // list 0: raw tail, 1: kept chunks; j: tile index inside the sequence's list
};

__global__ void __launch_bounds__(AT_THREADS, 2) kve_decode_attn_kernel(AttnArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  uint16_t* Ks = reinterpret_cast<uint16_t*>(smem + AT_OFF_K);
  uint16_t* Vs = reinterpret_cast<uint16_t*>(smem + AT_OFF_V);
  uint16_t* Qs = reinterpret_cast<uint16_t*>(smem + AT_OFF_Q);
  float* comb = reinterpret_cast<float*>(smem + AT_OFF_COMB);
  int4* info = reinterpret_cast<int4*>(smem + AT_OFF_INFO);
  int4* finfo = reinterpret_cast<int4*>(smem + AT_OFF_FINFO);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + AT_OFF_BAR);
  uint64_t* empty = full + AT_STAGES;
  uint64_t* ffull = empty + AT_STAGES;
  uint64_t* fempty = ffull + 2;

  pdl_launch_dependents();
  const LayerView& v = a.v;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  KVE_STAMP(threadIdx.x == 0, 0);
  if (warp == AT_PRODUCER) {
    // where this CTA starts follows from the launch arguments alone: warm L2 with what the first look-ups need
    // while the barriers are set up and the predecessor drains (prefetches return nothing, so they may run early)
    const uint32_t I = (uint32_t)v.S * (uint32_t)a.k, P = min(gridDim.x, I);
    if (blockIdx.x < P) prefetch_sequence_metadata(a, (int)(piece_begin(blockIdx.x, I, P) / (uint32_t)a.k), lane);
    if (lane == 31) prefetch_l2(v.seq_len);
    if (lane == 30) prefetch_l2(v.n_listed);
  }
  if (threadIdx.x == 0) {
    for (int i = 0; i < AT_STAGES; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], AT_CWARPS);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&ffull[i], AT_CWARPS);
      mbar_init(&fempty[i], 1);
    }
    mbar_fence_init();
  }
  __syncthreads();
  pdl_wait();      // lengths, keep lists, summaries and the new token come from earlier kernels
  KVE_STAMP(threadIdx.x == 0, 1);

  // this CTA's parts follow from the launch arguments; the producer asks for its first sequence's keep count at once,
  // together with the length and the coverage below: three look-ups in flight instead of one after the other
  const uint32_t c = blockIdx.x, uk = (uint32_t)a.k;
  const uint32_t n_items = (uint32_t)v.S * uk, n_pieces = min(gridDim.x, n_items);
  const uint32_t i0 = piece_begin(c, n_items, n_pieces), i1 = piece_begin(c + 1, n_items, n_pieces);
  int keep_cnt_first = 0;
  if (warp == AT_PRODUCER && i0 < i1 && a.mode != ATTN_DENSE) keep_cnt_first = v.keep_cnt[i0 / uk];

  // ---- geometry (every thread) ---------------------------------------------------------------------------
  AttnGeo g;
  {
    int n = v.seq_len[0];
    // chunks the keep list covers: the device's own count, so that a launch replayed from a CUDA graph follows the
    // gate triggers that happened since it was captured (the launch argument is only the host's view at capture time).
    // Requested together with the length: nothing that could alias stands between the two loads.
    const int listed = (a.mode == ATTN_DENSE) ? 0 : *v.n_listed;
    n = min(max(n, 0), v.max_tokens);
    g.appending = a.k_new != nullptr && n < v.max_tokens;
    if (a.k_new != nullptr && !g.appending && blockIdx.x == 0 && threadIdx.x == 0) set_status(v.status, ERR_CAPACITY);   // cache full
    if (g.appending) n += 1;
    g.n = n;
    g.n_chunks = min(max(listed, 0), v.max_chunks);
    g.raw0 = g.n_chunks * v.C;
    g.n_tail = max(0, n - g.raw0);
    g.TT = (g.n_tail + AT_TILE - 1) / AT_TILE;
    g.per = (a.mode == ATTN_RAW) ? v.C : 1;
    g.I = n_items;
    g.P = n_pieces;
  }

  if (warp == AT_PRODUCER) {
    // ================= producer warp =================
    // walks the CTA's parts in order, sequence by sequence; within a sequence the tiles [j_lo, j_hi) that
    // its parts in this CTA cover (part p of a sequence with T tiles: tiles [p T / k, (p + 1) T / k))
    const int s_first = (int)(i0 / uk), s_last = (int)((i1 - 1u) / uk);      // meaningful when i0 < i1
    int s = s_first, j = 0, j_hi = 0, lt_rows = 0, tiles = 0;
    bool fresh = true;                      // the next tile is the first one of sequence s in this CTA
    auto enter_sequence = [&]() {
      if (s < s_last) prefetch_sequence_metadata(a, s + 1, lane);      // the next one's look-ups will hit L2
      lt_rows = (s == s_first) ? lead_rows_from(a, g, keep_cnt_first) : lead_rows_of(a, g, s);
      tiles = g.TT + (lt_rows + AT_TILE - 1) / AT_TILE;
      // part p of the sequence's tiles: [p tiles / k, (p + 1) tiles / k); p <= 32 and tiles < 2^20, so 32 bits do
      const uint32_t p_lo = (s == s_first) ? i0 - (uint32_t)s * uk : 0u;
      const uint32_t p_hi = (s == s_last) ? i1 - (uint32_t)s * uk : uk;
      j = (int)((p_lo * (uint32_t)tiles) / uk);
      j_hi = (int)((p_hi * (uint32_t)tiles) / uk);
      fresh = true;
    };
    bool done = i0 >= i1;
    if (!done) enter_sequence();
    auto next_tile = [&](TileDesc& t) {
      if (done) {
        t.s = -1; t.list = 0; t.j = 0; t.rows = 0; t.flags = TF_END;
        return;
      }
      t.s = s;
      if (j >= j_hi) {
        // parts without a tile (fewer tiles than parts, or a sequence without a retained row): an empty tile keeps
        // the bookkeeping uniform - the merger still gets this CTA's (empty) share of the sequence
        t.list = 0; t.j = 0; t.rows = 0;
        t.flags = TF_NEW | TF_FLUSH;
      } else {
        t.list = j >= g.TT ? 1 : 0;
        t.j = t.list ? j - g.TT : j;
        t.rows = min(AT_TILE, (t.list ? lt_rows : g.n_tail) - t.j * AT_TILE);
        t.flags = (fresh ? TF_NEW : 0) | (j + 1 >= j_hi ? TF_FLUSH : 0);
        fresh = false;
        ++j;
      }
      if (t.flags & TF_FLUSH) {
        if (s == s_last) done = true;
        else { ++s; enter_sequence(); }
      }
    };
    // addresses of the tile's rows: lane l resolves rows l and l + 32
    struct TileAddr { const uint16_t *k[AT_TILE / 32], *v[AT_TILE / 32]; };
    auto resolve = [&](const TileDesc& t, TileAddr& ta) {
#pragma unroll
      for (int half = 0; half < AT_TILE / 32; ++half) ta.k[half] = ta.v[half] = nullptr;
      if (t.flags & TF_END) return;
      const long long sb = (long long)t.s * v.max_chunks;
#pragma unroll
      for (int half = 0; half < AT_TILE / 32; ++half) {
        const int rl = half * 32 + lane;
        if (rl >= t.rows) continue;
        const int L = t.j * AT_TILE + rl;              // row inside the sequence's list
        int chunk, r;
        if (t.list == 0) {
          if (g.appending && L == g.n_tail - 1) {      // the token being appended: straight from the caller's buffers
            ta.k[half] = a.k_new + (long long)t.s * D;
            ta.v[half] = a.v_new + (long long)t.s * D;
            continue;
          }
          const int p = g.raw0 + L;
          chunk = p / v.C;
          r = p - chunk * v.C;
        } else if (a.mode == ATTN_SUMMARY) {
          ta.k[half] = a.kkept + (sb + L) * D;
          ta.v[half] = a.vkept + (sb + L) * D;
          continue;
        } else {                                       // RAW: row r of the (L / C)-th kept chunk
          const int ci = L / v.C;
          r = L - ci * v.C;
          chunk = v.keep_idx[sb + ci];
          if (chunk < 0 || chunk >= g.n_chunks) { set_status(v.status, ERR_CAPACITY); chunk = 0; }
        }
        long long page = v.page_table[sb + chunk];
        if (page < 0 || page >= v.n_pages) { set_status(v.status, ERR_CAPACITY); page = 0; }
        const long long off = (page * v.C + r) * D;
        ta.k[half] = v.k_pages + off;
        ta.v[half] = v.v_pages + off;
      }
    };
    // waits for the stage, publishes the tile's description, issues its copies; false on a timed-out wait
    auto issue = [&](int i, const TileDesc& t, const TileAddr& ta) -> bool {
      const int stage = i % AT_STAGES, round = i / AT_STAGES;
      if (round > 0 && !mbar_wait_bounded(&empty[stage], (round - 1) & 1)) {
        if (lane == 0) set_status(v.status, ERR_TIMEOUT);
        return false;
      }
      if (lane == 0) {
        info[stage] = make_int4(t.s, t.rows, t.flags, t.list);
        const bool with_q = (t.flags & TF_NEW) != 0;
        const uint32_t bytes = (uint32_t)t.rows * 2u * ROW_BYTES + (with_q ? (uint32_t)ROW_BYTES : 0u);
        mbar_arrive_expect_tx(&full[stage], bytes);      // release: the description is visible to whoever sees the phase
        if (with_q) bulk_g2s(Qs + stage * D, a.q + (long long)t.s * D, ROW_BYTES, &full[stage]);
      }
      __syncwarp();
#pragma unroll
      for (int half = 0; half < AT_TILE / 32; ++half) {
        const int rl = half * 32 + lane;
        const bool valid = rl < t.rows;
        const uint16_t *kp = ta.k[half], *vp = ta.v[half];
        const unsigned long long ka = (unsigned long long)kp, va = (unsigned long long)vp;
        const unsigned long long kprev = __shfl_up_sync(0xffffffffu, ka, 1);
        const unsigned long long vprev = __shfl_up_sync(0xffffffffu, va, 1);
        const bool contiguous = valid && lane > 0 && ka == kprev + ROW_BYTES && va == vprev + ROW_BYTES;
        const bool head = valid && !contiguous;
        const unsigned headmask = __ballot_sync(0xffffffffu, head);
        const unsigned validmask = __ballot_sync(0xffffffffu, valid);
        if (head) {
          const unsigned above = (lane == 31) ? 0u : (headmask & ~((2u << lane) - 1u));
          const int run_end = above ? (__ffs(above) - 1) : __popc(validmask);   // valid lanes form a prefix
          const uint32_t bytes = (uint32_t)(run_end - lane) * ROW_BYTES;
          bulk_g2s(Ks + stage * AT_STAGE_ELEMS + rl * D, kp, bytes, &full[stage]);
          bulk_g2s(Vs + stage * AT_STAGE_ELEMS + rl * D, vp, bytes, &full[stage]);
        }
      }
      return true;
    };
    // The first tiles go out as soon as each is resolved; from then on the addresses of tile i + 1 are
    // looked up before the wait for its stage, i.e. while the consumers still work on the tiles in flight.
    // The END description takes a stage of its own (no copies): that is how the consumers learn that they are done.
    // fused append: whoever streams a sequence's last tail tile also stores the new token's row in its page
    // (lanes 0-15 the K row, 16-31 the V row, 16 bytes each)
    auto store_new_token = [&](const TileDesc& td) {
      if (!g.appending || (td.flags & TF_END) || td.list != 0 || td.rows == 0 || td.j * AT_TILE + td.rows != g.n_tail) return;
      const int pos = g.n - 1, chunk = pos / v.C, r = pos - chunk * v.C;
      const long long page = v.page_table[(long long)td.s * v.max_chunks + chunk];
      if (page < 0 || page >= v.n_pages) {
        if (lane == 0) set_status(v.status, ERR_CAPACITY);
        return;
      }
      const int is_v = lane >> 4, l16 = lane & 15;
      const uint4* src = reinterpret_cast<const uint4*>((is_v ? a.v_new : a.k_new) + (long long)td.s * D) + l16;
      uint4* dst = reinterpret_cast<uint4*>((is_v ? v.v_pages : v.k_pages) + (page * v.C + r) * D) + l16;
      *dst = __ldg(src);
    };
    TileDesc d;
    TileAddr t;
    for (int i = 0;; ++i) {
      next_tile(d);
      resolve(d, t);
      store_new_token(d);
      if (!issue(i, d, t) || (d.flags & TF_END)) break;
      KVE_STAMP(i == 0 && lane == 0, 2);
    }
    KVE_STAMP(lane == 0, 6);
  } else if (warp < AT_CWARPS) {
    // ================= consumer warps =================
    const float sl2 = a.scale * 1.44269504088896340736f;   // logits kept in log2 units
    float qf[4] = {0.f, 0.f, 0.f, 0.f};
    float m = -INFINITY, l = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
    int n_flush = 0;
    for (int i = 0;; ++i) {
      const int stage = i % AT_STAGES, round = i / AT_STAGES;
      if (!mbar_wait_bounded(&full[stage], round & 1)) {
        if (lane == 0) set_status(v.status, ERR_TIMEOUT);
        break;
      }
      const int4 ti = info[stage];                 // (sequence, rows, flags, list)
      KVE_STAMP(i == 0 && warp == 0 && lane == 0, 3);
      if (ti.z & TF_END) {
        KVE_STAMP(warp == 0 && lane == 0, 4);
        // tell the merger that nothing more comes
        const int fb = n_flush & 1;
        if (n_flush >= 2 && !mbar_wait_bounded(&fempty[fb], ((n_flush >> 1) - 1) & 1)) {
          if (lane == 0) set_status(v.status, ERR_TIMEOUT);
          break;
        }
        if (warp == 0 && lane == 0) finfo[fb] = make_int4(-1, 0, 0, 0);
        __syncwarp();
        if (lane == 0) mbar_arrive(&ffull[fb]);
        break;
      }
      if (ti.z & TF_NEW) {
        const uint2 qw = *reinterpret_cast<const uint2*>(Qs + stage * D + lane * 4);
        qf[0] = bf16lo(qw.x); qf[1] = bf16hi(qw.x); qf[2] = bf16lo(qw.y); qf[3] = bf16hi(qw.y);
        m = -INFINITY; l = 0.f;
        acc[0] = acc[1] = acc[2] = acc[3] = 0.f;
      }
      const int nvalid = min(max(ti.y - warp * AT_SUB, 0), AT_SUB);
      if (nvalid > 0) {
        const uint16_t* kt = Ks + stage * AT_STAGE_ELEMS + (warp * AT_SUB) * D + lane * 4;
        const uint16_t* vt = Vs + stage * AT_STAGE_ELEMS + (warp * AT_SUB) * D + lane * 4;
        float part[AT_SUB];
#pragma unroll
        for (int r = 0; r < AT_SUB; ++r) {
          const uint2 w = *reinterpret_cast<const uint2*>(kt + r * D);
          part[r] = qf[0] * bf16lo(w.x);
          part[r] = fmaf(qf[1], bf16hi(w.x), part[r]);
          part[r] = fmaf(qf[2], bf16lo(w.y), part[r]);
          part[r] = fmaf(qf[3], bf16hi(w.y), part[r]);
        }
        KVE_TR_ROUND(16, 4)
        KVE_TR_ROUND(8, 2)
        KVE_TR_ROUND(4, 1)
        float dot = part[0] + __shfl_xor_sync(0xffffffffu, part[0], 2);
        dot += __shfl_xor_sync(0xffffffffu, dot, 1);                             // row (lane >> 2), full sum
        const float logit = ((lane >> 2) < nvalid) ? dot * sl2 : -INFINITY;
        const float m_new = fmaxf(m, warp_max(logit));
        const float p = ex2_fast(logit - m_new);
        const float alpha = ex2_fast(m - m_new);
        l = fmaf(l, alpha, 0.25f * warp_sum(p));    // every row sits on four lanes
        m = m_new;
#pragma unroll
        for (int x = 0; x < 4; ++x) acc[x] *= alpha;
#pragma unroll
        for (int r = 0; r < AT_SUB; ++r) {
          const float pr = __shfl_sync(0xffffffffu, p, 4 * r);
          if (r < nvalid) {
            const uint2 w = *reinterpret_cast<const uint2*>(vt + r * D);
            acc[0] = fmaf(pr, bf16lo(w.x), acc[0]);
            acc[1] = fmaf(pr, bf16hi(w.x), acc[1]);
            acc[2] = fmaf(pr, bf16lo(w.y), acc[2]);
            acc[3] = fmaf(pr, bf16hi(w.y), acc[3]);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[stage]);
      if (ti.z & TF_FLUSH) {
        // hand (m, l, acc) of this (sequence, list) to the merger; the exchange area is double-buffered
        const int fb = n_flush & 1;
        if (n_flush >= 2 && !mbar_wait_bounded(&fempty[fb], ((n_flush >> 1) - 1) & 1)) {
          if (lane == 0) set_status(v.status, ERR_TIMEOUT);
          break;
        }
        float* cw = comb + (fb * AT_CWARPS + warp) * ATTN_PARTIAL_FLOATS;
        *reinterpret_cast<float4*>(cw + lane * 4) = make_float4(acc[0], acc[1], acc[2], acc[3]);
        if (lane == 0) { cw[128] = m; cw[129] = l; }
        if (warp == 0 && lane == 0) finfo[fb] = make_int4(ti.x, ti.w, 0, 0);
        __syncwarp();
        if (lane == 0) mbar_arrive(&ffull[fb]);      // release
        ++n_flush;
      }
    }
  } else {
    // ================= merger warp =================
    for (int f = 0;; ++f) {
      const int fb = f & 1;
      if (!mbar_wait_bounded(&ffull[fb], (f >> 1) & 1)) {
        if (lane == 0) set_status(v.status, ERR_TIMEOUT);
        break;
      }
      const int4 fi = finfo[fb];                   // (sequence, -, -, -); sequence < 0: no more work
      const int s = fi.x;
      if (s < 0) break;
      // ---- the eight consumer states -> one ----
      const float* cb = comb + fb * AT_CWARPS * ATTN_PARTIAL_FLOATS;
      float mC = -INFINITY;
#pragma unroll
      for (int w = 0; w < AT_CWARPS; ++w) mC = fmaxf(mC, cb[w * ATTN_PARTIAL_FLOATS + 128]);
      float lC = 0.f, accC[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int w = 0; w < AT_CWARPS; ++w) {
        const float mw = cb[w * ATTN_PARTIAL_FLOATS + 128];
        const float sc = (mw == -INFINITY) ? 0.f : exp2f(mw - mC);
        lC = fmaf(cb[w * ATTN_PARTIAL_FLOATS + 129], sc, lC);
        const float4 av = *reinterpret_cast<const float4*>(cb + w * ATTN_PARTIAL_FLOATS + lane * 4);
        accC[0] = fmaf(av.x, sc, accC[0]); accC[1] = fmaf(av.y, sc, accC[1]);
        accC[2] = fmaf(av.z, sc, accC[2]); accC[3] = fmaf(av.w, sc, accC[3]);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&fempty[fb]);     // the exchange buffer may be refilled

      // ---- which CTAs hold parts of sequence s ----
      const uint32_t c0 = piece_of((uint32_t)s * uk, g.I, g.P), c1 = piece_of((uint32_t)(s + 1) * uk - 1u, g.I, g.P);
      const int n_parts = (int)(c1 - c0 + 1u);
      if (n_parts > 1) {
        float* mine = a.partials + (long long)(s + c) * ATTN_PARTIAL_FLOATS;
        *reinterpret_cast<float4*>(mine + lane * 4) = make_float4(accC[0], accC[1], accC[2], accC[3]);
        if (lane == 0) { mine[128] = mC; mine[129] = lC; }
        // The ticket is an acquire-release atomic at device scope: taken by lane 0 after the warp has synchronised, it
        // publishes the whole warp's record (release is cumulative over what the barrier ordered before it) and, for the
        // last arriver, makes the other CTAs' records visible to the warp once it has synchronised again - one round
        // trip to L2 instead of fence, atomic, fence.
        __syncwarp();
        int ticket = 0;
        if (lane == 0)
          asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(ticket) : "l"(a.counters + s) : "memory");
        ticket = __shfl_sync(0xffffffffu, ticket, 0);
        if (ticket != n_parts - 1) continue;       // somebody else finishes later and merges
        __syncwarp();
        // records of sequence s: CTAs c0 .. c1, at s + c0 .. s + c1; lanes fetch the (m, l) pairs side by side
        const float* base = a.partials + (long long)(s + c0) * ATTN_PARTIAL_FLOATS;
        mC = -INFINITY;
        for (int p = lane; p < n_parts; p += 32) mC = fmaxf(mC, __ldcg(base + (long long)p * ATTN_PARTIAL_FLOATS + 128));
        mC = warp_max(mC);
        lC = 0.f;
        for (int p = lane; p < n_parts; p += 32) {
          const float mw = __ldcg(base + (long long)p * ATTN_PARTIAL_FLOATS + 128);
          const float sc = (mw == -INFINITY) ? 0.f : exp2f(mw - mC);
          lC = fmaf(__ldcg(base + (long long)p * ATTN_PARTIAL_FLOATS + 129), sc, lC);
        }
        lC = warp_sum(lC);
        accC[0] = accC[1] = accC[2] = accC[3] = 0.f;
#pragma unroll 4
        for (int p = 0; p < n_parts; ++p) {
          const float* ps = base + (long long)p * ATTN_PARTIAL_FLOATS;
          const float mw = __ldcg(ps + 128);
          const float4 av = __ldcg(reinterpret_cast<const float4*>(ps + lane * 4));
          const float sc = (mw == -INFINITY) ? 0.f : exp2f(mw - mC);
          accC[0] = fmaf(av.x, sc, accC[0]); accC[1] = fmaf(av.y, sc, accC[1]);
          accC[2] = fmaf(av.z, sc, accC[2]); accC[3] = fmaf(av.w, sc, accC[3]);
        }
        if (lane == 0) a.counters[s] = 0;          // leave the ticket counter clean for the next launch
      }
      const float inv = (lC > 0.f) ? (1.f / lC) : 0.f;
      uint2 o;
      o.x = pack_bf16x2(accC[0] * inv, accC[1] * inv);
      o.y = pack_bf16x2(accC[2] * inv, accC[3] * inv);
      *reinterpret_cast<uint2*>(a.out + (long long)s * D + lane * 4) = o;
      if (a.lse && lane == 0) a.lse[s] = (lC > 0.f) ? (mC + log2f(lC)) * 0.69314718055994530942f : -INFINITY;
    }
    // fused append: every CTA read the old length when it started; the last one to get here publishes the new one
    if (g.appending) {
      __syncwarp();
      int last = 0;
      if (lane == 0) {
        int arrived;
        asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(arrived) : "l"(a.ticket) : "memory");
        last = arrived == (int)gridDim.x - 1;
      }
      last = __shfl_sync(0xffffffffu, last, 0);
      if (last) {
        for (int b = lane; b < v.B; b += 32) v.seq_len[b] = g.n;
        if (lane == 0) *a.ticket = 0;      // clean for the next launch
      }
    }
    KVE_STAMP(lane == 0, 5);
  }
}

cudaError_t launch_attn(const LayerView& v, AttnMode mode, int n_chunks, int parts_per_seq, int grid, const void* q, void* out,
                        float* lse, float scale, const void* kkept, const void* vkept, float* partials, int32_t* counters,
                        const void* k_new, const void* v_new, int32_t* ticket, cudaStream_t st) {
  if (v.S <= 0) return cudaSuccess;
  static DeviceFlags opted;
  {
    cudaError_t e = smem_opt_in(opted, kve_decode_attn_kernel, AT_SMEM_BYTES);
    if (e != cudaSuccess) return e;
  }
  AttnArgs a;
  a.v = v; a.mode = (int)mode; a.n_chunks = n_chunks; a.k = parts_per_seq < 1 ? 1 : parts_per_seq;
  a.q = static_cast<const uint16_t*>(q); a.out = static_cast<uint16_t*>(out); a.lse = lse; a.scale = scale;
  a.kkept = static_cast<const uint16_t*>(kkept); a.vkept = static_cast<const uint16_t*>(vkept);
  a.partials = partials; a.counters = counters;
  a.k_new = static_cast<const uint16_t*>(k_new); a.v_new = static_cast<const uint16_t*>(v_new); a.ticket = ticket;
  return launch_pdl(kve_decode_attn_kernel, dim3((unsigned)(grid < 1 ? 1 : grid)), dim3(AT_THREADS), AT_SMEM_BYTES, st, a);
}

}  // namespace kve

#ifdef KVE_ATTN_STAMPS
// instrumented build only: copy the stamps of the last launch to the host / clear them
extern "C" int kve_attn_stamps_read(unsigned long long* host, int n) {
  return (int)cudaMemcpyFromSymbol(host, kve::g_attn_stamps, sizeof(unsigned long long) * n);
}
extern "C" int kve_attn_stamps_clear() {
  void* p = nullptr;
  cudaError_t e = cudaGetSymbolAddress(&p, kve::g_attn_stamps);
  if (e == cudaSuccess) e = cudaMemset(p, 0, sizeof(kve::g_attn_stamps));
  return (int)e;
}
#endif

// Split-K flash-decode over the retained set (Sec. 3.3, softmax of Eq. 1):
//   out = softmax(q K'^T * scale) V',  rows of K', V' = [kept chunks, oldest first] ++ [raw tail]
// and, with mode = DENSE, Eq. 1 over every stored token (the full-cache baseline).
//
// HBM-bound: every retained K and V row (256 bytes each) is read exactly once.
//  * grid = (splits, sequences); a CTA owns a contiguous range of a sequence's logical rows
//    (raw tail first, kept chunks after it).
//  * one producer warp turns logical rows into addresses (summary store / page table), merges
//    rows that are contiguous in memory into runs with a ballot, and issues one bulk copy
//    (TMA engine, global -> shared, mbarrier byte counting) per run into a 3-stage ring of
//    64-row K and V tiles.
//  * eight consumer warps each take 8 rows of a tile: q.k partial sums per lane (4 head dims per
//    lane), a butterfly transpose-reduce that leaves one row's logit per group of four lanes, online softmax
//    with warp shuffles, then p.V with each lane owning 4 output dims.
//  * per-CTA (m, l, acc) partials go to the workspace; the last CTA of a sequence to finish (atomic
//    ticket, nobody spins) merges them by log-sum-exp and writes the bf16 output.
// Every mbarrier wait is bounded; on give-up the status word gets KVE_ERR_TIMEOUT.
#include "common.cuh"
#include "kernels.h"

namespace kve {

constexpr int AT_TILE = ATTN_TILE_ROWS;       // rows per stage
constexpr int AT_STAGES = 3;
constexpr int AT_CWARPS = 8;                  // consumer warps
constexpr int AT_SUB = AT_TILE / AT_CWARPS;   // 8 rows per consumer warp per tile
constexpr int AT_THREADS = (AT_CWARPS + 1) * 32;
constexpr int AT_STAGE_ELEMS = AT_TILE * D;   // bf16 elements of one K (or V) tile
constexpr int AT_SMEM_BYTES = 2 * AT_STAGES * AT_STAGE_ELEMS * 2 + AT_CWARPS * ATTN_PARTIAL_FLOATS * 4 + 2 * AT_STAGES * 8 + 16;
static_assert(AT_SUB == 8, "the transpose-reduce below is written for 8 rows per warp");

int attn_smem_bytes() { return AT_SMEM_BYTES; }

struct AttnArgs {
  LayerView v;
  int mode, n_chunks, rows_per_split, max_splits;
  const uint16_t* q;
  uint16_t* out;
  float* lse;
  float scale;
  float* partials;     // [S][max_splits][132]
  int32_t* counters;   // [S], zero between launches
};

// address of logical row L of sequence s (K and V); falls back to a safe row and flags the status
// word when an index is out of range
// The CTA walks a sequence's rows in the order [raw tail ; kept chunks]: the raw tail's addresses need
// only the page table, so the first tiles can be requested while the keep list is still on its way
// (softmax does not care about the order of its rows).
__device__ __forceinline__ void row_address(const AttnArgs& a, int s, int L, int n_tail, int raw0,
                                            const uint16_t*& kp, const uint16_t*& vp) {
  const LayerView& v = a.v;
  const long long sb = (long long)s * v.max_chunks;
  int chunk, r;
  if (L < n_tail) {
    const int p = raw0 + L;
    chunk = p / v.C;
    r = p - chunk * v.C;
  } else if (a.mode == ATTN_SUMMARY) {
    int t = v.keep_idx[sb + (L - n_tail)];
    if (t < 0 || t >= a.n_chunks) { set_status(v.status, ERR_CAPACITY); t = 0; }
    kp = v.ksum_bf16 + (sb + t) * D;
    vp = v.vsum_bf16 + (sb + t) * D;
    return;
  } else {            // RAW: row r of the ((L - n_tail) / C)-th kept chunk
    const int ci = (L - n_tail) / v.C;
    r = (L - n_tail) - ci * v.C;
    chunk = v.keep_idx[sb + ci];
    if (chunk < 0 || chunk >= a.n_chunks) { set_status(v.status, ERR_CAPACITY); chunk = 0; }
  }
  long long page = v.page_table[sb + chunk];
  if (page < 0 || page >= v.n_pages) { set_status(v.status, ERR_CAPACITY); page = 0; }
  const long long off = (page * v.C + r) * D;
  kp = v.k_pages + off;
  vp = v.v_pages + off;
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

__global__ void __launch_bounds__(AT_THREADS, 2) kve_decode_attn_kernel(AttnArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  uint16_t* Ks = reinterpret_cast<uint16_t*>(smem);
  uint16_t* Vs = Ks + AT_STAGES * AT_STAGE_ELEMS;
  float* comb = reinterpret_cast<float*>(Vs + AT_STAGES * AT_STAGE_ELEMS);          // [AT_CWARPS][132]
  uint64_t* full = reinterpret_cast<uint64_t*>(comb + AT_CWARPS * ATTN_PARTIAL_FLOATS);   // 16-byte aligned
  uint64_t* empty = full + AT_STAGES;

  pdl_launch_dependents();
  const LayerView& v = a.v;
  const int s = blockIdx.y, split = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_wait();      // lengths, keep lists and summaries come from earlier kernels

  int n = v.seq_len[s / v.H];
  n = min(max(n, 0), v.max_tokens);
  const int M = (a.mode == ATTN_DENSE) ? 0 : min(max(v.keep_cnt[s], 0), a.n_chunks);
  const int raw0 = (a.mode == ATTN_DENSE) ? 0 : a.n_chunks * v.C;
  const int n_lead = (a.mode == ATTN_RAW) ? M * v.C : M;
  const int n_tail = max(0, n - raw0);
  const int n_rows = n_tail + n_lead;
  int n_splits = max(1, (n_rows + a.rows_per_split - 1) / a.rows_per_split);
  // the sequence has outgrown what this launch was sized for (a replayed launch): rows beyond the grid
  // are dropped, which the status word reports; the splits that exist still merge, so the ticket
  // counter returns to zero and a later, correctly sized launch starts clean
  if (n_splits > (int)gridDim.x) {
    if (split == 0 && threadIdx.x == 0) set_status(v.status, ERR_CAPACITY);
    n_splits = (int)gridDim.x;
  }
  if (split >= n_splits) return;
  const int r_begin = split * a.rows_per_split;
  const int r_end = min(n_rows, r_begin + a.rows_per_split);
  const int n_tiles = (max(r_end - r_begin, 0) + AT_TILE - 1) / AT_TILE;

  if (threadIdx.x == 0) {
    for (int i = 0; i < AT_STAGES; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], AT_CWARPS);
    }
    mbar_fence_init();
  }
  __syncthreads();

  if (warp == AT_CWARPS) {
    // ================= producer warp =================
    // Row addresses need up to two dependent global loads (keep list, page table).  They are resolved
    // AT_STAGES tiles ahead of the copies, each tile in a slot of its own, so the look-ups of several
    // tiles are in flight together and never sit between a freed stage and its refill.
    struct TileAddr { const uint16_t *k[AT_TILE / 32], *v[AT_TILE / 32]; };
    auto resolve = [&](int i, TileAddr& t) {
      const int row0 = r_begin + i * AT_TILE;
      const int rows_in_tile = (i < n_tiles) ? min(AT_TILE, r_end - row0) : 0;
#pragma unroll
      for (int half = 0; half < AT_TILE / 32; ++half) {
        const int rl = half * 32 + lane;
        t.k[half] = t.v[half] = nullptr;
        if (rl < rows_in_tile) row_address(a, s, row0 + rl, n_tail, raw0, t.k[half], t.v[half]);
      }
    };
    // waits for the stage, issues the copies of tile i from its resolved addresses; false on a timed-out wait
    auto issue = [&](int i, const TileAddr& t) -> bool {
      const int stage = i % AT_STAGES, round = i / AT_STAGES;
      if (round > 0 && !mbar_wait_bounded(&empty[stage], (round - 1) & 1)) {
        if (lane == 0) set_status(v.status, ERR_TIMEOUT);
        return false;
      }
      const int row0 = r_begin + i * AT_TILE;
      const int rows_in_tile = min(AT_TILE, r_end - row0);
      if (lane == 0) mbar_arrive_expect_tx(&full[stage], (uint32_t)rows_in_tile * 2u * ROW_BYTES);
      __syncwarp();
#pragma unroll
      for (int half = 0; half < AT_TILE / 32; ++half) {
        const int rl = half * 32 + lane;
        const bool valid = rl < rows_in_tile;
        const uint16_t *kp = t.k[half], *vp = t.v[half];
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
    static_assert(AT_STAGES == 3, "three slots of look-ahead");
    TileAddr t0, t1, t2;
    resolve(0, t0);
    resolve(1, t1);
    resolve(2, t2);
    for (int i = 0; i < n_tiles; i += AT_STAGES) {
      if (!issue(i, t0)) break;
      resolve(i + 3, t0);
      if (i + 1 < n_tiles) { if (!issue(i + 1, t1)) break; resolve(i + 4, t1); }
      if (i + 2 < n_tiles) { if (!issue(i + 2, t2)) break; resolve(i + 5, t2); }
    }
  } else {
    // ================= consumer warps =================
    float qf[4];
    {
      const uint2 qw = *reinterpret_cast<const uint2*>(a.q + (long long)s * D + lane * 4);
      qf[0] = bf16lo(qw.x); qf[1] = bf16hi(qw.x); qf[2] = bf16lo(qw.y); qf[3] = bf16hi(qw.y);
    }
    const float sl2 = a.scale * 1.44269504088896340736f;   // logits kept in log2 units
    float m = -INFINITY, l = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int i = 0; i < n_tiles; ++i) {
      const int stage = i % AT_STAGES, round = i / AT_STAGES;
      if (!mbar_wait_bounded(&full[stage], round & 1)) {
        if (lane == 0) set_status(v.status, ERR_TIMEOUT);
        break;
      }
      const int rows_in_tile = min(AT_TILE, r_end - (r_begin + i * AT_TILE));
      const int nvalid = min(max(rows_in_tile - warp * AT_SUB, 0), AT_SUB);
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
    }
    float* cw = comb + warp * ATTN_PARTIAL_FLOATS;
    *reinterpret_cast<float4*>(cw + lane * 4) = make_float4(acc[0], acc[1], acc[2], acc[3]);
    if (lane == 0) { cw[128] = m; cw[129] = l; }
  }
  __syncthreads();
  if (warp != 0) return;

  // ---- warp 0: merge the consumer warps of this CTA ------------------------------------------------
  float mC = -INFINITY;
#pragma unroll
  for (int w = 0; w < AT_CWARPS; ++w) mC = fmaxf(mC, comb[w * ATTN_PARTIAL_FLOATS + 128]);
  float lC = 0.f, accC[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int w = 0; w < AT_CWARPS; ++w) {
    const float mw = comb[w * ATTN_PARTIAL_FLOATS + 128];
    const float sc = (mw == -INFINITY) ? 0.f : exp2f(mw - mC);
    lC = fmaf(comb[w * ATTN_PARTIAL_FLOATS + 129], sc, lC);
    const float4 av = *reinterpret_cast<const float4*>(comb + w * ATTN_PARTIAL_FLOATS + lane * 4);
    accC[0] = fmaf(av.x, sc, accC[0]); accC[1] = fmaf(av.y, sc, accC[1]);
    accC[2] = fmaf(av.z, sc, accC[2]); accC[3] = fmaf(av.w, sc, accC[3]);
  }

  if (n_splits > 1) {
    float* mine = a.partials + ((long long)s * a.max_splits + split) * ATTN_PARTIAL_FLOATS;
    *reinterpret_cast<float4*>(mine + lane * 4) = make_float4(accC[0], accC[1], accC[2], accC[3]);
    if (lane == 0) { mine[128] = mC; mine[129] = lC; }
    __threadfence();
    __syncwarp();
    int ticket = 0;
    if (lane == 0) ticket = atomicAdd(a.counters + s, 1);
    ticket = __shfl_sync(0xffffffffu, ticket, 0);
    if (ticket != n_splits - 1) return;      // somebody else finishes later and merges
    __threadfence();
    const float* base = a.partials + (long long)s * a.max_splits * ATTN_PARTIAL_FLOATS;
    mC = -INFINITY;
    for (int sp = 0; sp < n_splits; ++sp) mC = fmaxf(mC, __ldcg(base + sp * ATTN_PARTIAL_FLOATS + 128));
    lC = 0.f;
    accC[0] = accC[1] = accC[2] = accC[3] = 0.f;
    for (int sp = 0; sp < n_splits; ++sp) {
      const float* ps = base + sp * ATTN_PARTIAL_FLOATS;
      const float mw = __ldcg(ps + 128);
      const float sc = (mw == -INFINITY) ? 0.f : exp2f(mw - mC);
      lC = fmaf(__ldcg(ps + 129), sc, lC);
      const float4 av = __ldcg(reinterpret_cast<const float4*>(ps + lane * 4));
      accC[0] = fmaf(av.x, sc, accC[0]); accC[1] = fmaf(av.y, sc, accC[1]);
      accC[2] = fmaf(av.z, sc, accC[2]); accC[3] = fmaf(av.w, sc, accC[3]);
    }
    if (lane == 0) a.counters[s] = 0;        // leave the ticket counter clean for the next launch
  }

  const float inv = (lC > 0.f) ? (1.f / lC) : 0.f;
  uint2 o;
  o.x = pack_bf16x2(accC[0] * inv, accC[1] * inv);
  o.y = pack_bf16x2(accC[2] * inv, accC[3] * inv);
  *reinterpret_cast<uint2*>(a.out + (long long)s * D + lane * 4) = o;
  if (a.lse && lane == 0) a.lse[s] = (lC > 0.f) ? (mC + log2f(lC)) * 0.69314718055994530942f : -INFINITY;
}

cudaError_t launch_attn(const LayerView& v, AttnMode mode, int n_chunks, int n_tokens_upper, AttnPlan plan,
                        const void* q, void* out, float* lse, float scale, float* partials, int32_t* counters,
                        cudaStream_t st) {
  (void)n_tokens_upper;
  if (v.S <= 0) return cudaSuccess;
  static DeviceFlags opted;
  {
    cudaError_t e = smem_opt_in(opted, kve_decode_attn_kernel, AT_SMEM_BYTES);
    if (e != cudaSuccess) return e;
  }
  AttnArgs a;
  a.v = v; a.mode = (int)mode; a.n_chunks = n_chunks;
  a.rows_per_split = plan.rows_per_split; a.max_splits = plan.max_splits;
  a.q = static_cast<const uint16_t*>(q); a.out = static_cast<uint16_t*>(out); a.lse = lse; a.scale = scale;
  a.partials = partials; a.counters = counters;
  dim3 grid((unsigned)plan.max_splits, (unsigned)v.S);
  return launch_pdl(kve_decode_attn_kernel, grid, dim3(AT_THREADS), AT_SMEM_BYTES, st, a);
}

}  // namespace kve

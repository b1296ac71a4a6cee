// Attention of a BLOCK of queries over the retained set (Sec. 3.3, softmax of Eq. 1): the T query
// tokens that are decoded together (the action tokens) times the G = Hq / Hkv query heads that share
// one KV head (grouped-query attention, Sec. 4.1) form R = T * G query rows per KV sequence, and
//   out[r] = softmax(q[r] K'^T * scale) V',   rows of K', V' = [raw tail] ++ [kept chunks]
// (or every stored token with mode = DENSE).  The rows of a block do not attend to each other.
//
// With R rows per K/V row read, Q K^T and P V are real contractions (2 * 2 * 128 * R flop per 512
// bytes), so they run on the tensor cores; the kernel is still bound by the K/V stream from HBM,
// every retained row being read once per KV sequence instead of once per query row.
//  * grid = (splits, KV sequences), one CTA per SM; a CTA owns a contiguous range of the sequence's
//    64-row tiles.  The raw tail is padded to a whole number of tiles, so a tile is either all
//    tail or all kept rows.
//  * one producer warp resolves page ids three tiles ahead and fetches tiles with 2-D tensor
//    copies (TMA, mbarrier byte counts) into a 6-stage ring.  The tensor maps describe the page
//    pools and the summary store as [rows][128] bf16 with boxes of 64 columns and the 128-byte
//    swizzle, so a tile lands as two K-blocks [64 rows][128 bytes] in which ldmatrix is free of bank
//    conflicts: page rows in boxes of `hp` rows (hp = largest power of two <= 64 dividing C),
//    summary rows one box per row.
//  * MB * KVW consumer warps: warp (mb, kw) owns query rows 16 mb .. +15 and tile rows
//    (64 / KVW) kw .. ; S = Q K^T with mma.sync m16n8k16 (Q fragments live in registers), online
//    softmax on the accumulator fragments (fp32, log2 domain), P split into two bf16 planes
//    (hi + lo, error 2^-17) so that P V loses nothing against an fp32 product, V fragments by
//    ldmatrix.trans.
//  * warps of one query-row block merge through shared memory (the ring is free by then); splits
//    leave (m, l, acc) records in the workspace and the last CTA of a sequence to finish (atomic
//    ticket, nobody spins) merges them and writes bf16 rows.
// Every mbarrier wait is bounded; on give-up the status word gets KVE_ERR_TIMEOUT.
#include <cuda.h>

#include "common.cuh"
#include "kernels.h"

namespace kve {

constexpr int BK_TILE = ATTN_TILE_ROWS;         // 64 rows per stage
constexpr int BK_STAGES = 6;
constexpr int BK_KBLOCK_BYTES = BK_TILE * 128;  // one K-block: 64 rows x 64 bf16
constexpr int BK_TILE_BYTES = 2 * BK_KBLOCK_BYTES;        // K (or V) tile, 16 KB
constexpr int BK_STAGE_BYTES = 2 * BK_TILE_BYTES;         // K tile then V tile
constexpr int BK_SMEM_BYTES = BK_STAGES * BK_STAGE_BYTES + 2 * BK_STAGES * 8 + 64 + 1024;   // + slack for the 1024-byte alignment
constexpr int BK_REC = ATTN_PARTIAL_FLOATS;     // floats per (row) record: acc[128], m, l, pad

struct BlockArgs {
  LayerView v;
  int mode, n_chunks, rows_per_split, max_splits;
  int T, G, R;              // query tokens, query heads per KV head, T * G
  int hp;                   // rows per page box
  long long sum_row0;       // first row of this layer in the summary tensor maps
  const uint16_t* q;        // [B][T][Hq][128]
  uint16_t* out;            // [B][T][Hq][128]
  float* lse;               // [B][T][Hq] or null
  float scale;
  float* partials;          // [S][max_splits][16 MB][BK_REC]
  int32_t* counters;        // [S], zero between launches
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst_smem, const CUtensorMap* tm, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
          dst_smem),
      "l"(tm), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}
// byte offset of the 16-byte piece p16 (0..15 along the 128 head dims) of tile row `row`
__device__ __forceinline__ uint32_t tile_piece(int row, int p16) {
  return (uint32_t)((p16 >> 3) * BK_KBLOCK_BYTES + row * 128 + (((p16 & 7) ^ (row & 7)) << 4));
}

// element offset of query / output row r of KV sequence s in the [B][T][Hq][128] layout
__device__ __forceinline__ long long q_row_offset(const BlockArgs& a, int s, int r) {
  const int b = s / a.v.H, h = s - b * a.v.H;
  const int t = r / a.G, g = r - t * a.G;
  return ((((long long)b * a.T + t) * (a.G * a.v.H)) + h * a.G + g) * D;
}

template <int MB, int KVW>
__global__ void __launch_bounds__((MB * KVW + 1) * 32, 1)
kve_decode_attn_block_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                             const __grid_constant__ CUtensorMap tmKs, const __grid_constant__ CUtensorMap tmVs,
                             BlockArgs a) {
  constexpr int NCW = MB * KVW;            // consumer warps
  constexpr int RW = BK_TILE / KVW;        // tile rows per consumer warp
  constexpr int NB = RW / 8;               // 8-row blocks of S per warp
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + BK_STAGES * BK_STAGE_BYTES);
  uint64_t* empty = full + BK_STAGES;
  int* flag = reinterpret_cast<int*>(empty + BK_STAGES);

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
  const int tail_pad = (n_tail + BK_TILE - 1) / BK_TILE * BK_TILE;
  const int n_rows = tail_pad + n_lead;                     // padded logical rows
  const int n_splits = max(1, (n_rows + a.rows_per_split - 1) / a.rows_per_split);
  if (split >= n_splits) return;
  const int r_begin = split * a.rows_per_split;
  const int r_end = min(n_rows, r_begin + a.rows_per_split);
  const int n_tiles = (max(r_end - r_begin, 0) + BK_TILE - 1) / BK_TILE;
  // valid rows of the tile that starts at padded row `row0`
  auto rows_valid = [&](int row0) { return row0 < tail_pad ? min(BK_TILE, n_tail - row0) : min(BK_TILE, n_rows - row0); };

  if (threadIdx.x == 0) {
    for (int i = 0; i < BK_STAGES; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], NCW);
    }
    mbar_fence_init();
  }
  __syncthreads();

  // per-thread softmax state of the consumer warps (rows g and g + 8 of the warp's 16 query rows)
  float o[16][4];
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
#pragma unroll
  for (int i = 0; i < 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;

  if (warp == NCW) {
    // ================= producer warp =================
    // What a lane fetches for a tile: up to two boxes (K and V each, both 64-column halves):
    //   page tiles:    lane j < granules: hp rows from global row src[0] to tile row j * hp
    //   summary tiles: lane j: row j (src[0]) and row j + 32 (src[1]), one row each
    struct TileSrc { int src[2]; };
    const long long sb = (long long)s * v.max_chunks;
    auto page_row = [&](int chunk, int r) -> int {
      long long page = v.page_table[sb + chunk];
      if (page < 0 || page >= v.n_pages) { set_status(v.status, ERR_CAPACITY); page = 0; }
      return (int)(page * v.C + r);
    };
    auto resolve = [&](int i, TileSrc& t) {
      t.src[0] = t.src[1] = -1;
      if (i >= n_tiles) return;
      const int row0 = r_begin + i * BK_TILE;
      const int valid = rows_valid(row0);
      if (row0 < tail_pad) {
        if (lane * a.hp < valid) {
          const int p = raw0 + row0 + lane * a.hp;
          const int chunk = p / v.C;
          t.src[0] = page_row(chunk, p - chunk * v.C);
        }
      } else if (a.mode == ATTN_RAW) {
        if (lane * a.hp < valid) {
          const int ll = row0 - tail_pad + lane * a.hp;
          const int ci = ll / v.C;
          int chunk = v.keep_idx[sb + ci];
          if (chunk < 0 || chunk >= a.n_chunks) { set_status(v.status, ERR_CAPACITY); chunk = 0; }
          t.src[0] = page_row(chunk, ll - ci * v.C);
        }
      } else {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int l = lane + 32 * h;
          if (l < valid) {
            int c = v.keep_idx[sb + (row0 - tail_pad) + l];
            if (c < 0 || c >= a.n_chunks) { set_status(v.status, ERR_CAPACITY); c = 0; }
            t.src[h] = (int)(a.sum_row0 + sb + c);
          }
        }
      }
    };
    auto issue = [&](int i, const TileSrc& t) -> bool {
      const int stage = i % BK_STAGES, round = i / BK_STAGES;
      if (round > 0 && !mbar_wait_bounded(&empty[stage], (round - 1) & 1)) {
        if (lane == 0) set_status(v.status, ERR_TIMEOUT);
        return false;
      }
      const int row0 = r_begin + i * BK_TILE;
      const int valid = rows_valid(row0);
      const bool pages = row0 < tail_pad || a.mode == ATTN_RAW;
      const uint32_t bytes = pages ? (uint32_t)((valid + a.hp - 1) / a.hp) * a.hp * 2u * ROW_BYTES
                                   : (uint32_t)valid * 2u * ROW_BYTES;
      if (lane == 0) mbar_arrive_expect_tx(&full[stage], bytes);
      __syncwarp();
      const uint32_t kdst = smem_u32(smem + stage * BK_STAGE_BYTES), vdst = kdst + BK_TILE_BYTES;
      if (pages) {
        if (t.src[0] >= 0) {
          const uint32_t off = (uint32_t)(lane * a.hp) * 128u;
          tma_load_2d(kdst + off, &tmK, 0, t.src[0], &full[stage]);
          tma_load_2d(kdst + BK_KBLOCK_BYTES + off, &tmK, 64, t.src[0], &full[stage]);
          tma_load_2d(vdst + off, &tmV, 0, t.src[0], &full[stage]);
          tma_load_2d(vdst + BK_KBLOCK_BYTES + off, &tmV, 64, t.src[0], &full[stage]);
        }
      } else {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (t.src[h] >= 0) {
            const uint32_t off = (uint32_t)(lane + 32 * h) * 128u;
            tma_load_2d(kdst + off, &tmKs, 0, t.src[h], &full[stage]);
            tma_load_2d(kdst + BK_KBLOCK_BYTES + off, &tmKs, 64, t.src[h], &full[stage]);
            tma_load_2d(vdst + off, &tmVs, 0, t.src[h], &full[stage]);
            tma_load_2d(vdst + BK_KBLOCK_BYTES + off, &tmVs, 64, t.src[h], &full[stage]);
          }
        }
      }
      return true;
    };
    TileSrc t0, t1, t2;
    resolve(0, t0);
    resolve(1, t1);
    resolve(2, t2);
    for (int i = 0; i < n_tiles; i += 3) {
      if (!issue(i, t0)) break;
      resolve(i + 3, t0);
      if (i + 1 < n_tiles) { if (!issue(i + 1, t1)) break; resolve(i + 4, t1); }
      if (i + 2 < n_tiles) { if (!issue(i + 2, t2)) break; resolve(i + 5, t2); }
    }
  } else {
    // ================= consumer warps =================
    const int mb = warp / KVW, kw = warp - mb * KVW;
    const int g = lane >> 2, tq = lane & 3;
    // Q fragments (A operand, rows = query rows, k = head dims), zero beyond R
    uint32_t qa[8][4];
    {
      const int r_lo = mb * 16 + g, r_hi = r_lo + 8;
      const uint16_t* q_lo = a.q + q_row_offset(a, s, min(r_lo, a.R - 1));
      const uint16_t* q_hi = a.q + q_row_offset(a, s, min(r_hi, a.R - 1));
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const int c = ks * 16 + 2 * tq;
        qa[ks][0] = (r_lo < a.R) ? *reinterpret_cast<const uint32_t*>(q_lo + c) : 0u;
        qa[ks][1] = (r_hi < a.R) ? *reinterpret_cast<const uint32_t*>(q_hi + c) : 0u;
        qa[ks][2] = (r_lo < a.R) ? *reinterpret_cast<const uint32_t*>(q_lo + c + 8) : 0u;
        qa[ks][3] = (r_hi < a.R) ? *reinterpret_cast<const uint32_t*>(q_hi + c + 8) : 0u;
      }
    }
    const float sl2 = a.scale * 1.44269504088896340736f;   // logits kept in log2 units
    const int mi = lane >> 3, rr = lane & 7;               // ldmatrix: this lane addresses row rr of matrix mi
    for (int i = 0; i < n_tiles; ++i) {
      const int stage = i % BK_STAGES, round = i / BK_STAGES;
      if (!mbar_wait_bounded(&full[stage], round & 1)) {
        if (lane == 0) set_status(v.status, ERR_TIMEOUT);
        break;
      }
      const int valid = rows_valid(r_begin + i * BK_TILE);
      const int rw0 = kw * RW;
      if (rw0 < valid) {
        const uint32_t kbase = smem_u32(smem + stage * BK_STAGE_BYTES), vbase = kbase + BK_TILE_BYTES;
        // ---- S = Q K^T for this warp's RW tile rows ----
        float sc[NB][4];
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
          sc[nb][0] = sc[nb][1] = sc[nb][2] = sc[nb][3] = 0.f;
          const int row = rw0 + nb * 8 + rr;
#pragma unroll
          for (int kp = 0; kp < 4; ++kp) {
            uint32_t b[4];      // matrices: (k-step 2kp, k 0..7), (2kp, 8..15), (2kp+1, 0..7), (2kp+1, 8..15)
            ldsm_x4(b, kbase + tile_piece(row, kp * 4 + mi));
            mma_bf16_16816(sc[nb], qa[2 * kp], b[0], b[1]);
            mma_bf16_16816(sc[nb], qa[2 * kp + 1], b[2], b[3]);
          }
        }
        // ---- online softmax (rows g: elements 0, 1; rows g + 8: elements 2, 3) ----
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int col = rw0 + nb * 8 + 2 * tq + (e & 1);
            sc[nb][e] = (col < valid) ? sc[nb][e] * sl2 : -INFINITY;
            mx[e >> 1] = fmaxf(mx[e >> 1], sc[nb][e]);
          }
        float alpha[2], m_use[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
          mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
          const float m_new = fmaxf(m_run[h], mx[h]);        // finite: the warp has at least one valid column
          alpha[h] = exp2f(m_run[h] - m_new);
          m_run[h] = m_new;
          m_use[h] = m_new;
          l_run[h] *= alpha[h];
        }
#pragma unroll
        for (int nbd = 0; nbd < 16; ++nbd) {
          o[nbd][0] *= alpha[0]; o[nbd][1] *= alpha[0];
          o[nbd][2] *= alpha[1]; o[nbd][3] *= alpha[1];
        }
        // ---- O += P V, 16 tile rows per step; P = hi + lo bf16 planes ----
        const bool ragged = valid < rw0 + RW;
#pragma unroll
        for (int kk = 0; kk < RW / 16; ++kk) {
          uint32_t phi[4], plo[4];
#pragma unroll
          for (int x = 0; x < 4; ++x) {     // A fragment: x = 0: (row g, k 0..7), 1: (g + 8, k 0..7), 2: (g, k 8..15), 3: (g + 8, k 8..15)
            const int nb = 2 * kk + (x >> 1), h = x & 1;
            const float p0 = exp2f(sc[nb][2 * h] - m_use[h]), p1 = exp2f(sc[nb][2 * h + 1] - m_use[h]);
            l_run[h] += p0 + p1;
            phi[x] = pack_bf16x2(p0, p1);
            plo[x] = pack_bf16x2(p0 - bf16lo(phi[x]), p1 - bf16hi(phi[x]));
          }
          // rows whose copy was cut short (beyond `valid`) hold stale bytes: P is 0 there, but 0 * NaN is
          // not, so those V elements are cleared
          uint32_t keep0 = 0xffffffffu, keep1 = 0xffffffffu;
          if (ragged) {
            const int k0 = rw0 + kk * 16 + 2 * tq;
            keep0 = (k0 < valid ? 0xffffu : 0u) | (k0 + 1 < valid ? 0xffff0000u : 0u);
            keep1 = (k0 + 8 < valid ? 0xffffu : 0u) | (k0 + 9 < valid ? 0xffff0000u : 0u);
          }
          const int row = rw0 + kk * 16 + (mi & 1) * 8 + rr;
#pragma unroll
          for (int nbp = 0; nbp < 8; ++nbp) {
            uint32_t b[4];      // matrices: (k 0..7, dims 16 nbp ..+7), (k 8..15, same), (k 0..7, dims +8..+15), (k 8..15, same)
            ldsm_x4_trans(b, vbase + tile_piece(row, nbp * 2 + (mi >> 1)));
            b[0] &= keep0; b[1] &= keep1; b[2] &= keep0; b[3] &= keep1;
            mma_bf16_16816(o[2 * nbp], phi, b[0], b[1]);
            mma_bf16_16816(o[2 * nbp], plo, b[0], b[1]);
            mma_bf16_16816(o[2 * nbp + 1], phi, b[2], b[3]);
            mma_bf16_16816(o[2 * nbp + 1], plo, b[2], b[3]);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[stage]);
    }
  }
  __syncthreads();      // every tile has been consumed: the ring is free and becomes the merge area

  // ---- per-warp results into shared memory: [warp][16 rows][acc 128, m, l, pad] ---------------------
  constexpr int NT = (NCW + 1) * 32;
  constexpr int ROWS = MB * 16;
  float* comb = reinterpret_cast<float*>(smem);
  if (warp < NCW) {
    const int g = lane >> 2, tq = lane & 3;
    float* mine = comb + (size_t)warp * 16 * BK_REC;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float l = l_run[h];
      l += __shfl_xor_sync(0xffffffffu, l, 1);
      l += __shfl_xor_sync(0xffffffffu, l, 2);
      float* row = mine + (g + 8 * h) * BK_REC;
#pragma unroll
      for (int nbd = 0; nbd < 16; ++nbd)
        *reinterpret_cast<float2*>(row + nbd * 8 + 2 * tq) = make_float2(o[nbd][2 * h], o[nbd][2 * h + 1]);
      if (tq == 0) { row[128] = m_run[h]; row[129] = l; }
    }
  }
  __syncthreads();

  // merges `cnt` records (stride `stride` floats apart, read through `ld`) of one query row
  auto merge = [&](auto ld4, auto ld1, const float* rec, int cnt, long long stride, int c4, float4& acc, float& mC, float& lC) {
    mC = -INFINITY;
    for (int k = 0; k < cnt; ++k) mC = fmaxf(mC, ld1(rec + k * stride + 128));
    lC = 0.f;
    acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k = 0; k < cnt; ++k) {
      const float mw = ld1(rec + k * stride + 128);
      const float scl = (mw == -INFINITY) ? 0.f : exp2f(mw - mC);
      lC = fmaf(ld1(rec + k * stride + 129), scl, lC);
      const float4 av = ld4(reinterpret_cast<const float4*>(rec + k * stride + c4 * 4));
      acc.x = fmaf(av.x, scl, acc.x); acc.y = fmaf(av.y, scl, acc.y);
      acc.z = fmaf(av.z, scl, acc.z); acc.w = fmaf(av.w, scl, acc.w);
    }
  };
  auto write_out = [&](int row, int c4, const float4& acc, float mC, float lC) {
    if (row >= a.R) return;
    const float inv = (lC > 0.f) ? (1.f / lC) : 0.f;
    const long long off = q_row_offset(a, s, row);
    uint2 w;
    w.x = pack_bf16x2(acc.x * inv, acc.y * inv);
    w.y = pack_bf16x2(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(a.out + off + c4 * 4) = w;
    if (a.lse && c4 == 0) a.lse[off / D] = (lC > 0.f) ? (mC + log2f(lC)) * 0.69314718055994530942f : -INFINITY;
  };
  auto lds4 = [](const float4* p) { return *p; };
  auto lds1 = [](const float* p) { return *p; };
  auto ldg4 = [](const float4* p) { return __ldcg(p); };
  auto ldg1 = [](const float* p) { return __ldcg(p); };

  float* my_rec = a.partials + ((long long)s * a.max_splits + split) * ROWS * BK_REC;
  for (int it = threadIdx.x; it < ROWS * 32; it += NT) {
    const int row = it >> 5, c4 = it & 31;
    float4 acc;
    float mC, lC;
    merge(lds4, lds1, comb + ((size_t)(row >> 4) * KVW * 16 + (row & 15)) * BK_REC, KVW, 16 * BK_REC, c4, acc, mC, lC);
    if (n_splits == 1) {
      write_out(row, c4, acc, mC, lC);
    } else {
      *reinterpret_cast<float4*>(my_rec + row * BK_REC + c4 * 4) = acc;
      if (c4 == 0) *reinterpret_cast<float2*>(my_rec + row * BK_REC + 128) = make_float2(mC, lC);
    }
  }
  if (n_splits == 1) return;

  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) *flag = (atomicAdd(a.counters + s, 1) == n_splits - 1) ? 1 : 0;
  __syncthreads();
  if (*flag == 0) return;        // somebody else finishes later and merges
  __threadfence();
  const float* base = a.partials + (long long)s * a.max_splits * ROWS * BK_REC;
  for (int it = threadIdx.x; it < ROWS * 32; it += NT) {
    const int row = it >> 5, c4 = it & 31;
    float4 acc;
    float mC, lC;
    merge(ldg4, ldg1, base + row * BK_REC, n_splits, (long long)ROWS * BK_REC, c4, acc, mC, lC);
    write_out(row, c4, acc, mC, lC);
  }
  if (threadIdx.x == 0) a.counters[s] = 0;      // leave the ticket counter clean for the next launch
}

// ---- host side ------------------------------------------------------------------------------------
int attn_block_hp(int C) {
  int hp = 64;
  while (hp > 1 && C % hp != 0) hp >>= 1;
  return hp;
}

// [rows][128] bf16, boxes of 64 columns x box_rows rows, 128-byte swizzle
static cudaError_t encode_rows_map(CUtensorMap* tm, const void* base, unsigned long long rows, unsigned box_rows) {
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                               const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static EncodeFn encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    encode = reinterpret_cast<EncodeFn>(fn);
  }
  if (rows == 0 || rows >= (1ULL << 31)) return cudaErrorInvalidValue;
  const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ROW_BYTES};
  const cuuint32_t box[2] = {64u, box_rows};
  const cuuint32_t estr[2] = {1u, 1u};
  const CUresult r = encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

static_assert(sizeof(CUtensorMap) == ATTN_BLOCK_MAP_BYTES, "tensor map size");

cudaError_t encode_attn_block_maps(void* maps, const void* k_pages, const void* v_pages, long long page_rows, int hp,
                                   const void* ksum, const void* vsum, long long sum_rows) {
  CUtensorMap* tm = static_cast<CUtensorMap*>(maps);
  cudaError_t e = encode_rows_map(tm + 0, k_pages, (unsigned long long)page_rows, (unsigned)hp);
  if (e == cudaSuccess) e = encode_rows_map(tm + 1, v_pages, (unsigned long long)page_rows, (unsigned)hp);
  if (e == cudaSuccess) e = encode_rows_map(tm + 2, ksum, (unsigned long long)sum_rows, 1u);
  if (e == cudaSuccess) e = encode_rows_map(tm + 3, vsum, (unsigned long long)sum_rows, 1u);
  return e;
}

template <int MB, int KVW>
static cudaError_t launch_block_t(const CUtensorMap* tm, const BlockArgs& a, dim3 grid, cudaStream_t st) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(kve_decode_attn_block_kernel<MB, KVW>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         BK_SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  return launch_pdl(kve_decode_attn_block_kernel<MB, KVW>, grid, dim3((MB * KVW + 1) * 32), BK_SMEM_BYTES, st, tm[0], tm[1],
                    tm[2], tm[3], a);
}

cudaError_t launch_attn_block(const LayerView& v, const void* maps, AttnMode mode, int n_chunks, AttnPlan plan, int T, int G,
                              int hp, long long sum_row0, const void* q, void* out, float* lse, float scale, float* partials,
                              int32_t* counters, cudaStream_t st) {
  if (v.S <= 0 || T <= 0) return cudaSuccess;
  const int R = T * G;
  if (R > ATTN_BLOCK_MAX_ROWS || hp < 8) return cudaErrorInvalidValue;
  BlockArgs a;
  a.v = v; a.mode = (int)mode; a.n_chunks = n_chunks;
  a.rows_per_split = plan.rows_per_split; a.max_splits = plan.max_splits;
  a.T = T; a.G = G; a.R = R; a.hp = hp; a.sum_row0 = sum_row0;
  a.q = static_cast<const uint16_t*>(q); a.out = static_cast<uint16_t*>(out); a.lse = lse; a.scale = scale;
  a.partials = partials; a.counters = counters;
  const CUtensorMap* tm = static_cast<const CUtensorMap*>(maps);
  dim3 grid((unsigned)plan.max_splits, (unsigned)v.S);
  switch ((R + 15) / 16) {
    case 1: return launch_block_t<1, 4>(tm, a, grid, st);
    case 2: return launch_block_t<2, 4>(tm, a, grid, st);
    case 3: return launch_block_t<3, 2>(tm, a, grid, st);
    default: return launch_block_t<4, 2>(tm, a, grid, st);
  }
}

}  // namespace kve

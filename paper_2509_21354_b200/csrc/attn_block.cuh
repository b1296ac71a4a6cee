// Pieces shared by the block-of-queries attention kernels: launch arguments, the geometry of a
// sequence's padded logical rows, the TMA producer warp and the merge of split records.
//
// Logical rows of a sequence: the raw tail (padded up to whole 64-row tiles), then the kept rows
// (summary rows, or the raw rows of kept chunks), so a tile is either all tail or all kept rows.  A
// tile lands in shared memory as K tile then V tile, each two K-blocks [64 rows][64 bf16] with the
// 128-byte swizzle (what a tensor copy with that swizzle mode writes): the 16-byte piece c of row r
// of a K-block sits at r * 128 + ((c ^ (r & 7)) << 4).
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "kernels.h"

namespace kve {

constexpr int BK_TILE = ATTN_TILE_ROWS;         // 64 rows per stage
constexpr int BK_KBLOCK_BYTES = BK_TILE * 128;  // one K-block: 64 rows x 64 bf16
constexpr int BK_TILE_BYTES = 2 * BK_KBLOCK_BYTES;        // K (or V) tile, 16 KB
constexpr int BK_STAGE_BYTES = 2 * BK_TILE_BYTES;         // K tile then V tile
constexpr int BK_SUM_BOX = ATTN_BLOCK_SUM_BOX;   // rows per tensor-copy box over the compacted kept summary rows
constexpr int BK_REC = ATTN_PARTIAL_FLOATS;     // floats per (query row) record: acc[128], m, l, pad

struct BlockArgs {
  LayerView v;
  int mode, n_chunks, rows_per_split, max_splits;
  int T, G, R;              // query tokens, query heads per KV head, T * G
  int rec_rows;             // query-row records per (sequence, split) in `partials`
  int causal;               // query token t sees the cache up to its own position only
  int hp;                   // rows per page box
  long long sum_row0;       // first row of this layer in the tensor maps over the compacted kept summary rows
  const uint16_t* q;        // [B][T][Hq][128]
  uint16_t* out;            // [B][T][Hq][128]
  float* lse;               // [B][T][Hq] or null
  float scale;
  float* partials;          // [S][max_splits][rec_rows][BK_REC]
  int32_t* counters;        // [S], zero between launches
};

struct BlockGeom {
  int raw0, n_tail, tail_pad, n_rows, n_splits, r_begin, r_end, n_tiles;
  bool outgrown;      // the sequence needs more splits than the launch has: rows beyond the grid are dropped (flagged)
  // valid rows of the tile that starts at padded row `row0`
  __device__ __forceinline__ int rows_valid(int row0) const {
    return row0 < tail_pad ? min(BK_TILE, n_tail - row0) : min(BK_TILE, n_rows - row0);
  }
};

__device__ __forceinline__ BlockGeom block_geometry(const BlockArgs& a, int s, int split) {
  const LayerView& v = a.v;
  BlockGeom g;
  int n = v.seq_len[s / v.H];
  n = min(max(n, 0), v.max_tokens);
  const int M = (a.mode == ATTN_DENSE) ? 0 : min(max(v.keep_cnt[s], 0), a.n_chunks);
  g.raw0 = (a.mode == ATTN_DENSE) ? 0 : a.n_chunks * v.C;
  const int n_lead = (a.mode == ATTN_RAW) ? M * v.C : M;
  g.n_tail = max(0, n - g.raw0);
  g.tail_pad = (g.n_tail + BK_TILE - 1) / BK_TILE * BK_TILE;
  g.n_rows = g.tail_pad + n_lead;
  g.n_splits = max(1, (g.n_rows + a.rows_per_split - 1) / a.rows_per_split);
  // a replayed launch the sequence has outgrown: the splits that exist still merge and the ticket
  // counter still returns to zero; the caller learns about the dropped rows from the status word
  g.outgrown = g.n_splits > (int)gridDim.x;
  g.n_splits = min(g.n_splits, (int)gridDim.x);
  g.r_begin = split * a.rows_per_split;
  g.r_end = min(g.n_rows, g.r_begin + a.rows_per_split);
  g.n_tiles = (max(g.r_end - g.r_begin, 0) + BK_TILE - 1) / BK_TILE;
  return g;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst_smem, const CUtensorMap* tm, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
          dst_smem),
      "l"(tm), "r"(smem_u32(bar)), "r"(x), "r"(y)
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

// Producer warp: resolves page ids three tiles ahead and fetches the CTA's tiles with 2-D tensor
// copies into the ring `ring` (STAGES stages), arming full[stage] with the byte count and waiting
// (bounded) on empty[stage] before a stage is reused.
// What a lane fetches for a tile: up to two boxes (K and V each, both 64-column halves):
//   page tiles:    lane j < granules: hp rows from global row src[0] to tile row j * hp
//   summary tiles: lane j < ceil(valid / 16): 16 kept summary rows (compacted by kvE_compact) from global row src[0]
template <int STAGES>
__device__ __forceinline__ void block_producer(const BlockArgs& a, const BlockGeom& gm, int s, int lane,
                                               const CUtensorMap* tmK, const CUtensorMap* tmV, const CUtensorMap* tmKs,
                                               const CUtensorMap* tmVs, unsigned char* ring, uint64_t* full,
                                               uint64_t* empty) {
  const LayerView& v = a.v;
  struct TileSrc { int src[2]; };
  const long long sb = (long long)s * v.max_chunks;
  auto page_row = [&](int chunk, int r) -> int {
    long long page = v.page_table[sb + chunk];
    if (page < 0 || page >= v.n_pages) { set_status(v.status, ERR_CAPACITY); page = 0; }
    return (int)(page * v.C + r);
  };
  auto resolve = [&](int i, TileSrc& t) {
    t.src[0] = t.src[1] = -1;
    if (i >= gm.n_tiles) return;
    const int row0 = gm.r_begin + i * BK_TILE;
    const int valid = gm.rows_valid(row0);
    if (row0 < gm.tail_pad) {
      if (lane * a.hp < valid) {
        const int p = gm.raw0 + row0 + lane * a.hp;
        const int chunk = p / v.C;
        t.src[0] = page_row(chunk, p - chunk * v.C);
      }
    } else if (a.mode == ATTN_RAW) {
      if (lane * a.hp < valid) {
        const int ll = row0 - gm.tail_pad + lane * a.hp;
        const int ci = ll / v.C;
        int chunk = v.keep_idx[sb + ci];
        if (chunk < 0 || chunk >= a.n_chunks) { set_status(v.status, ERR_CAPACITY); chunk = 0; }
        t.src[0] = page_row(chunk, ll - ci * v.C);
      }
    } else {
      // kept summary rows sit compacted, one contiguous run per sequence: boxes of BK_SUM_BOX rows, lane j the j-th
      if (lane * BK_SUM_BOX < valid) t.src[0] = (int)(a.sum_row0 + sb + (row0 - gm.tail_pad) + lane * BK_SUM_BOX);
    }
  };
  auto issue = [&](int i, const TileSrc& t) -> bool {
    const int stage = i % STAGES, round = i / STAGES;
    if (round > 0 && !mbar_wait_bounded(&empty[stage], (round - 1) & 1)) {
      if (lane == 0) set_status(v.status, ERR_TIMEOUT);
      return false;
    }
    const int row0 = gm.r_begin + i * BK_TILE;
    const int valid = gm.rows_valid(row0);
    const bool pages = row0 < gm.tail_pad || a.mode == ATTN_RAW;
    const uint32_t bytes = pages ? (uint32_t)((valid + a.hp - 1) / a.hp) * a.hp * 2u * ROW_BYTES
                                 : (uint32_t)((valid + BK_SUM_BOX - 1) / BK_SUM_BOX) * BK_SUM_BOX * 2u * ROW_BYTES;
    if (lane == 0) mbar_arrive_expect_tx(&full[stage], bytes);
    __syncwarp();
    const uint32_t kdst = smem_u32(ring + stage * BK_STAGE_BYTES), vdst = kdst + BK_TILE_BYTES;
    if (pages) {
      if (t.src[0] >= 0) {
        const uint32_t off = (uint32_t)(lane * a.hp) * 128u;
        tma_load_2d(kdst + off, tmK, 0, t.src[0], &full[stage]);
        tma_load_2d(kdst + BK_KBLOCK_BYTES + off, tmK, 64, t.src[0], &full[stage]);
        tma_load_2d(vdst + off, tmV, 0, t.src[0], &full[stage]);
        tma_load_2d(vdst + BK_KBLOCK_BYTES + off, tmV, 64, t.src[0], &full[stage]);
      }
    } else if (t.src[0] >= 0) {
      // rows beyond the kept count inside the last box are older kept rows or zeros (finite), masked by the row count
      const uint32_t off = (uint32_t)(lane * BK_SUM_BOX) * 128u;
      tma_load_2d(kdst + off, tmKs, 0, t.src[0], &full[stage]);
      tma_load_2d(kdst + BK_KBLOCK_BYTES + off, tmKs, 64, t.src[0], &full[stage]);
      tma_load_2d(vdst + off, tmVs, 0, t.src[0], &full[stage]);
      tma_load_2d(vdst + BK_KBLOCK_BYTES + off, tmVs, 64, t.src[0], &full[stage]);
    }
    return true;
  };
  TileSrc t0, t1, t2;
  resolve(0, t0);
  resolve(1, t1);
  resolve(2, t2);
  for (int i = 0; i < gm.n_tiles; i += 3) {
    if (!issue(i, t0)) break;
    resolve(i + 3, t0);
    if (i + 1 < gm.n_tiles) { if (!issue(i + 1, t1)) break; resolve(i + 4, t1); }
    if (i + 2 < gm.n_tiles) { if (!issue(i + 2, t2)) break; resolve(i + 5, t2); }
  }
}

// merges `cnt` records of one query row (`stride` floats apart; read through ld4 / ld1) for output
// columns 4 c4 .. 4 c4 + 3
template <typename L4, typename L1>
__device__ __forceinline__ void merge_records(L4 ld4, L1 ld1, const float* rec, int cnt, long long stride, int c4,
                                              float4& acc, float& mC, float& lC) {
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
}

// normalises one query row's columns 4 c4 .. +3 and writes them (bf16) and, from c4 == 0, the row's lse
__device__ __forceinline__ void write_block_out(const BlockArgs& a, int s, int row, int c4, const float4& acc, float mC,
                                                float lC) {
  if (row >= a.R) return;
  const float inv = (lC > 0.f) ? (1.f / lC) : 0.f;
  const long long off = q_row_offset(a, s, row);
  uint2 w;
  w.x = pack_bf16x2(acc.x * inv, acc.y * inv);
  w.y = pack_bf16x2(acc.z * inv, acc.w * inv);
  *reinterpret_cast<uint2*>(a.out + off + c4 * 4) = w;
  if (a.lse && c4 == 0) a.lse[off / D] = (lC > 0.f) ? (mC + log2f(lC)) * 0.69314718055994530942f : -INFINITY;
}

// After every thread of the CTA has written its part of this split's records: takes a ticket; the
// last CTA of the sequence merges all splits' records and writes the output.  `flag`: an int in
// shared memory.  Called by all NT threads of the CTA.
__device__ __forceinline__ void block_merge_splits(const BlockArgs& a, int s, int n_splits, int rows, int* flag, int NT) {
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) *flag = (atomicAdd(a.counters + s, 1) == n_splits - 1) ? 1 : 0;
  __syncthreads();
  if (*flag == 0) return;        // somebody else finishes later and merges
  __threadfence();
  const float* base = a.partials + (long long)s * a.max_splits * a.rec_rows * BK_REC;
  auto ldg4 = [](const float4* p) { return __ldcg(p); };
  auto ldg1 = [](const float* p) { return __ldcg(p); };
  for (int it = threadIdx.x; it < rows * 32; it += NT) {
    const int row = it >> 5, c4 = it & 31;
    float4 acc;
    float mC, lC;
    merge_records(ldg4, ldg1, base + row * BK_REC, n_splits, (long long)a.rec_rows * BK_REC, c4, acc, mC, lC);
    write_block_out(a, s, row, c4, acc, mC, lC);
  }
  if (threadIdx.x == 0) a.counters[s] = 0;      // leave the ticket counter clean for the next launch
}

}  // namespace kve

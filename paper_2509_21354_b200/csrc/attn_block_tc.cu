// Attention of a block of queries over the retained set (Sec. 3.3, softmax of Eq. 1) on the 5th-generation
// tensor cores: the T query tokens decoded together times the G = Hq / Hkv query heads sharing a KV
// head form R = T * G <= 128 query rows per KV sequence; out[r] = softmax(q[r] K'^T * scale) V'.
//
// Every retained K/V row is fetched once per KV sequence (HBM-bound), both products run as
// tcgen05.mma with accumulators in tensor memory:
//  * grid = (splits, KV sequences), one CTA per SM, ten warps:
//      warp 0   producer: 2-D tensor copies (TMA, 128-byte swizzle) of 64-row K/V tiles into a ring;
//               a tile arrives as two K-blocks [64 rows][64 bf16], which is at once the K-major B
//               operand of S = Q K^T and the MN-major B operand of O += P V;
//      warp 1   one thread issues the MMAs: S(i) = Q K_i^T (M 128, N 64, K 128) into the S buffer of
//               tile parity i & 1, and O_{i&1} += P_i V_i (M 128, N 128, K 64 per bf16 plane of P),
//               whichever has its inputs ready; commits signal the softmax warps, free the ring stage
//               and the P buffer;
//      warps 2-5, 6-9  two softmax groups, even and odd tiles, each with its own running (m_ref, l)
//               and its own accumulator O in tensor memory (merged at the end), so two tiles are in
//               softmax at any time.  Thread = query row = tensor-memory lane.  Reads its 64 logits of the tile,
//               p = exp2(s * scale * log2 e - m_ref) by the special-function unit, writes P as bf16 into
//               the swizzled A-operand layout (rounding p moves an output by at most
//               2^-8 sum p |v| / sum p (bf16 keeps 8 significant bits: half a step is 2^-8 relative); TC_PLANES = 2 adds a second plane p - bf16(p) and removes that
//               error at the price of a ring stage).  m_ref follows the running maximum lazily: only
//               when a row's maximum has grown by more than 8 (log2 units) does the warp rescale its
//               rows of O in tensor memory, so p stays below 2^8 and the usual per-tile rescale of O
//               disappears.
//  * with R <= 32 (<= 64) query rows the block is laid out four times (twice) down the 128 rows of the
//    A operand, and each copy's warp takes a quarter (half) of a tile's 64 columns: the softmax of
//    a tile then runs on all four warps of a group, one per scheduler, instead of on one.
//  * Q sits in shared memory as the K-major A operand for the whole CTA.
//  * tile rows beyond the valid ones (ragged tail, partial tiles of kept rows) hold stale bytes:
//    their logits are masked and their V rows are zeroed before P V (0 * NaN would poison O).
//  * splits leave (m_ref, l, O) records in the workspace; the last CTA of a sequence to finish (atomic
//    ticket, nobody spins) merges them and writes bf16 rows.
// Every mbarrier wait is bounded; on give-up the status word gets KVE_ERR_TIMEOUT, the CTA skips the
// rest of its work and still frees its tensor memory.
#include "attn_block.cuh"
#include "umma.cuh"

namespace kve {

constexpr int TC_STAGES = 5;
constexpr int TC_PLANES = 1;                       // bf16 planes of P (2: hi + lo, P exact to 2^-16, at the price of a ring stage)
constexpr int TC_Q_BYTES = 2 * 128 * 128;          // two K-blocks [128 rows][128 bytes]
constexpr int TC_P_BYTES = 128 * 128;              // one plane of one P buffer: [128 rows][64 bf16]
constexpr int TC_OFF_Q = 0;
constexpr int TC_OFF_P = TC_OFF_Q + TC_Q_BYTES;
constexpr int TC_OFF_RING = TC_OFF_P + 2 * TC_PLANES * TC_P_BYTES;
constexpr int TC_OFF_BAR = TC_OFF_RING + TC_STAGES * BK_STAGE_BYTES;
constexpr int TC_N_BARS = 2 * TC_STAGES + 10;
constexpr int TC_OFF_MISC = TC_OFF_BAR + TC_N_BARS * 8;            // tensor-memory base, ticket flag
constexpr int TC_OFF_MX = TC_OFF_MISC + 16;                        // [2 tile parities][2 groups][128 lanes] column maxima
constexpr int TC_SMEM_BYTES = TC_OFF_MX + 4 * 128 * 4;             // 226.2 KB: everything an SM has, so no alignment slack;
                                                                   // the kernel checks that the base is 1024-byte aligned
constexpr int TC_OFF_L = 128 * BK_REC * 4;                         // [2 groups][128 lanes] partial row sums, behind the exchange
                                                                   // area of the final merge (both valid once the ring is free)
static_assert(TC_SMEM_BYTES <= 227 * 1024, "shared memory of one CTA");
constexpr int TC_THREADS = 320;
constexpr int TC_TMEM_COLS = 512;                  // O of the two groups: 2 x 128 columns, then S: two buffers of 64
constexpr float TC_RESCALE_STEP = 8.f;             // log2 units a row maximum may run ahead of m_ref

// bounded wait with one outcome for the whole warp
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity) {
  return __all_sync(0xffffffffu, mbar_wait_bounded(bar, parity));
}

template <int REP>
__global__ void __launch_bounds__(TC_THREADS, 1)
kve_decode_attn_block_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                                const __grid_constant__ CUtensorMap tmKs, const __grid_constant__ CUtensorMap tmVs,
                                BlockArgs a) {
  extern __shared__ __align__(1024) unsigned char smem[];
  if ((smem_u32(smem) & 1023u) != 0u) {      // the swizzled operand tiles need it; never seen otherwise
    if (threadIdx.x == 0) set_status(a.v.status, ERR_CAPACITY);
    return;
  }
  unsigned char* Qs = smem + TC_OFF_Q;
  unsigned char* Ps = smem + TC_OFF_P;
  unsigned char* ring = smem + TC_OFF_RING;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + TC_OFF_BAR);
  uint64_t* empty = full + TC_STAGES;
  uint64_t* s_full = empty + TC_STAGES;     // [2] S buffer written (MMA commit)
  uint64_t* s_free = s_full + 2;            // [2] S buffer read by the four warps of its softmax group
  uint64_t* p_full = s_free + 2;            // [2] P buffer written by the four warps of its softmax group
  uint64_t* pv_done = p_full + 2;           // [2] O += P V of the buffer's tile complete (MMA commit)
  uint64_t* mx_full = pv_done + 2;          // [2] the group's four warps have posted their column maxima
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + TC_OFF_MISC);
  int* flag = reinterpret_cast<int*>(tmem_slot + 1);
  float* mx_x = reinterpret_cast<float*>(smem + TC_OFF_MX);
  float* l_x = reinterpret_cast<float*>(smem + TC_OFF_L);      // valid only after the tile loops

  pdl_launch_dependents();
  const LayerView& v = a.v;
  const int s = blockIdx.y, split = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // ---- set-up that needs nothing from earlier kernels: barriers, tensor memory, P cleared -----------------
  if (threadIdx.x == 0) {
    for (int i = 0; i < TC_STAGES; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s_full[i], 1);
      mbar_init(&s_free[i], 4);       // one arrival per warp of the group (an arrival per thread would
      mbar_init(&p_full[i], 4);       // serialise 128 updates of one shared-memory word)
      mbar_init(&pv_done[i], 1);
      mbar_init(&mx_full[i], 4);
    }
    mbar_fence_init();
  }
  if (warp == 1) umma::tmem_alloc(tmem_slot, TC_TMEM_COLS);
  for (int idx = threadIdx.x; idx < 2 * TC_PLANES * TC_P_BYTES / 16; idx += TC_THREADS)
    *reinterpret_cast<uint4*>(Ps + idx * 16) = make_uint4(0u, 0u, 0u, 0u);
  umma::fence_smem_to_async();
  umma::fence_before_sync();
  __syncthreads();
  umma::fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_o = tmem_base, tmem_s = tmem_base + 256;

  pdl_wait();      // lengths, keep lists, summaries and the queries come from earlier kernels

  const BlockGeom gm = block_geometry(a, s, split);
  // the sequence has outgrown what this launch was sized for (a replayed launch): rows would be dropped
  if (gm.outgrown && split == 0 && threadIdx.x == 0) set_status(v.status, ERR_CAPACITY);
  if (split >= gm.n_splits) {      // nothing for this CTA
    if (warp == 1) umma::tmem_dealloc(tmem_base, TC_TMEM_COLS);
    return;
  }
  const int n_tiles = gm.n_tiles;

  // ---- Q as the A operand: staged by everybody but the producer warp, which is already fetching tiles ----------------
  if (warp != 0) {
    for (int idx = threadIdx.x - 32; idx < 128 * 16; idx += TC_THREADS - 32) {
      const int arow = idx >> 4, p16 = idx & 15;      // row of the A operand = tensor-memory lane of S
      const int qrow = arow % (128 / REP);             // the query block repeats REP times down the lanes
      uint4 val = make_uint4(0u, 0u, 0u, 0u);
      if (qrow < a.R) val = *reinterpret_cast<const uint4*>(a.q + q_row_offset(a, s, qrow) + p16 * 8);
      *reinterpret_cast<uint4*>(Qs + (p16 >> 3) * (128 * 128) + arow * 128 + (((p16 & 7) ^ (arow & 7)) << 4)) = val;
    }
    umma::fence_smem_to_async();
    asm volatile("bar.sync 2, %0;" ::"n"(TC_THREADS - 32) : "memory");
  }

  if (warp == 0) {
    // ================= producer warp =================
    block_producer<TC_STAGES>(a, gm, s, lane, &tmK, &tmV, &tmKs, &tmVs, ring, full, empty);
  } else if (warp == 1) {
    // ================= MMA issue (one thread) =================
    if (lane == 0) {
      constexpr uint32_t idesc_s = umma::instr_desc_bf16(128, 64);
      constexpr uint32_t idesc_pv = umma::instr_desc_bf16_b_mn(128, 128);
      const uint32_t q_base = smem_u32(Qs), p_base = smem_u32(Ps), ring_base = smem_u32(ring);
      // S(i) = Q K_i^T into S buffer i & 1
      auto issue_s = [&](int i) {
        const int stage = i % TC_STAGES;
        umma::fence_after_sync();
        const uint32_t kbase = ring_base + stage * BK_STAGE_BYTES;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint64_t da = umma::smem_desc(q_base + (ks >> 2) * (128 * 128) + (ks & 3) * 32);
          const uint64_t db = umma::smem_desc(kbase + (ks >> 2) * BK_KBLOCK_BYTES + (ks & 3) * 32);
          umma::mma_bf16(tmem_s + (i & 1) * 64, da, db, idesc_s, ks != 0);
        }
        umma::commit(&s_full[i & 1]);
      };
      // O_{i & 1} += P_i V_i, then the ring stage and the P buffer are free
      auto issue_pv = [&](int i) {
        umma::fence_after_sync();
        const int stage = i % TC_STAGES;
        const uint32_t vbase = ring_base + stage * BK_STAGE_BYTES + BK_TILE_BYTES;
#pragma unroll
        for (int pl = 0; pl < TC_PLANES; ++pl) {
#pragma unroll
          for (int k = 0; k < 4; ++k) {      // 16 tile rows per MMA
            const uint64_t da = umma::smem_desc(p_base + ((i & 1) * TC_PLANES + pl) * TC_P_BYTES + k * 32);
            const uint64_t db = umma::smem_desc_mn_major(vbase + k * 16 * 128, BK_KBLOCK_BYTES);
            umma::mma_bf16(tmem_o + (i & 1) * 128, da, db, idesc_pv, i >= 2 || (pl | k) != 0);
          }
        }
        umma::commit(&empty[stage]);
        umma::commit(&pv_done[i & 1]);
      };
      // Issue whatever is ready, S in tile order and P V in tile order; S(i) needs tile i in the ring and
      // S(i-2) read by its softmax group, P V(i) needs P_i.  Gives up after a bounded number of idle polls.
      int next_s = 0, next_pv = 0;
      uint32_t idle = 0;
      while (next_pv < n_tiles) {
        bool progress = false;
        if (next_s < n_tiles && next_s < next_pv + TC_STAGES) {
          const int i = next_s;
          if (mbar_test_wait(&full[i % TC_STAGES], (i / TC_STAGES) & 1) &&
              (i < 2 || mbar_test_wait(&s_free[i & 1], ((i >> 1) + 1) & 1))) {
            issue_s(i);
            ++next_s;
            progress = true;
          }
        }
        if (next_pv < next_s && mbar_test_wait(&p_full[next_pv & 1], (next_pv >> 1) & 1)) {
          issue_pv(next_pv);
          ++next_pv;
          progress = true;
        }
        if (progress) idle = 0;
        else if (++idle > (1u << 24)) { set_status(v.status, ERR_TIMEOUT); break; }
        else if (idle > 4096) __nanosleep(64);
      }
    }
  } else {
    // ================= softmax warps =================
    // Tensor-memory lane L carries query row L % RB, RB = 128 / REP: with few query rows the block is
    // replicated REP times down the 128 lanes (the tensor core computes all 128 rows of S anyway) and
    // replica L / RB works on its own CW = 64 / REP columns of every tile, so a tile's softmax is spread
    // over all four warps of the group (one per scheduler) instead of sitting on one.  The replicas
    // of a row exchange their column maxima through shared memory once per tile, keep identical
    // m_ref, write their columns of P into the row of replica 0, and add up their sums at the end.
    constexpr int RB = 128 / REP, CW = 64 / REP;
    const int group = (warp - 2) >> 2;                  // 0: even tiles, 1: odd tiles
    const int quarter = warp & 3;                       // the lanes a warp may touch follow from its index
    const int L = quarter * 32 + lane;
    const int row = L % RB, rep = L / RB;
    const bool warp_active = (quarter * 32) % RB < a.R; // some lane of this warp carries a real query row
    const bool owns_o = warp_active && rep == 0;        // rows of O live in the lanes of replica 0
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const uint32_t my_o = tmem_o + lane_addr + group * 128, my_s = tmem_s + lane_addr + group * 64 + rep * CW;
    const float sl2 = a.scale * 1.44269504088896340736f;   // logits in log2 units
    const int tok = min(row, a.R - 1) / a.G;                // query token of this lane's row
    float m_ref = -INFINITY, l_run = 0.f;
    bool alive = true;
    int last_tile = -1;
    for (int i = group; alive && i < n_tiles; i += 2) {
      const int b = group, stage = i % TC_STAGES, j = i >> 1;      // j: how many tiles this group has done
      if (!warp_wait(&s_full[b], j & 1)) { alive = false; break; }
      umma::fence_after_sync();
      float sv[CW];
      if (warp_active) {
        if (CW == 16) {
          umma::tmem_ld16(my_s, reinterpret_cast<float(&)[16]>(sv));
        } else {
#pragma unroll
          for (int c = 0; c < CW / 32; ++c) umma::tmem_ld32(my_s + c * 32, reinterpret_cast<float(&)[32]>(sv[c * 32 % CW]));
        }
      }
      umma::fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_free[b]);
      const int row0 = gm.r_begin + i * BK_TILE;
      const int valid = gm.rows_valid(row0);
      // causal blocks: query token t sees the cache up to its own position, i.e. all but the last
      // T - 1 - t rows of the raw tail (the block's own tokens are the newest rows of the tail)
      const bool edge = a.causal && row0 < gm.tail_pad && row0 + BK_TILE > gm.n_tail - (a.T - 1);
      const int visible = edge ? min(valid, gm.n_tail - (a.T - 1 - tok) - row0) : valid;      // columns of this tile the row may use
      const bool plain = valid == BK_TILE && sl2 > 0.f && !edge;      // no masking, and max(s * sl2) = max(s) * sl2

      float mx = -INFINITY;
      if (warp_active) {
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        if (plain) {
#pragma unroll
          for (int x = 0; x < CW; ++x) mx4[x & 3] = fmaxf(mx4[x & 3], sv[x]);
        } else {
#pragma unroll
          for (int x = 0; x < CW; ++x) {
            sv[x] = (rep * CW + x < visible) ? sv[x] * sl2 : -INFINITY;
            mx4[x & 3] = fmaxf(mx4[x & 3], sv[x]);
          }
        }
        mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        if (plain) mx *= sl2;
      }
      if (REP > 1) {
        // the row's maximum over all replicas' columns (buffers alternate, one barrier phase per tile)
        float* slot = mx_x + ((j & 1) * 2 + group) * 128;
        slot[L] = mx;
        __syncwarp();
        if (lane == 0) mbar_arrive(&mx_full[group]);
        if (!warp_wait(&mx_full[group], j & 1)) { alive = false; break; }
#pragma unroll
        for (int r2 = 0; r2 < REP; ++r2) mx = fmaxf(mx, slot[row + r2 * RB]);
      }
      if (warp_active) {
        if (__any_sync(0xffffffffu, mx > m_ref + TC_RESCALE_STEP)) {      // m_ref = -inf on the group's first tile
          const float m_new = fmaxf(m_ref, mx);
          if (j > 0) {
            const float f = (m_ref == -INFINITY) ? 0.f : ex2_fast(m_ref - m_new);      // nothing accumulated yet: O row is 0
            if (owns_o) {
              // O holds this group's earlier tiles once their last product is complete; rescale this warp's rows
              if (!warp_wait(&pv_done[b], (j + 1) & 1)) { alive = false; break; }
              umma::fence_after_sync();
#pragma unroll 1
              for (int c = 0; c < 4; ++c) {
                float o[32];
                umma::tmem_ld32(my_o + c * 32, o);
#pragma unroll
                for (int x = 0; x < 32; ++x) o[x] *= f;
                umma::tmem_st32(my_o + c * 32, o);
              }
              umma::fence_before_sync();
            }
            l_run *= f;
          }
          m_ref = m_new;
        }
      }
      if (valid < BK_TILE) {
        // stale V rows of a partial tile: cleared by the group's threads before P V may start
        mbar_wait_bounded(&full[stage], (i / TC_STAGES) & 1);      // complete already: orders this thread after the copies
        unsigned char* vt = ring + stage * BK_STAGE_BYTES + BK_TILE_BYTES;
        const int n_pieces = (BK_TILE - valid) * 16;
        for (int idx = (warp - 2 - 4 * group) * 32 + lane; idx < n_pieces; idx += 128) {
          const int r = valid + (idx >> 4), p16 = idx & 15;
          *reinterpret_cast<uint4*>(vt + tile_piece(r, p16)) = make_uint4(0u, 0u, 0u, 0u);
        }
      }
      if (j > 0 && !warp_wait(&pv_done[b], (j + 1) & 1)) { alive = false; break; }   // P buffer b is free
      if (warp_active) {
        unsigned char* prow = Ps + (b * TC_PLANES) * TC_P_BYTES + row * 128;
        float l4[4] = {0.f, 0.f, 0.f, 0.f};
        // (a row that has not seen a single column yet has m_ref = -inf: its p are 0, not exp2(-inf + inf))
        const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref, mul = plain ? sl2 : 1.f;      // the masked path has stored s * sl2 already
#pragma unroll
        for (int c = 0; c < CW / 8; ++c) {
          float p[8];
#pragma unroll
          for (int x = 0; x < 8; ++x) {
            p[x] = ex2_fast(fmaf(sv[c * 8 + x], mul, neg_m));
            l4[x & 3] += p[x];
          }
          uint4 hi, lo;
          hi.x = pack_bf16x2(p[0], p[1]); hi.y = pack_bf16x2(p[2], p[3]);
          hi.z = pack_bf16x2(p[4], p[5]); hi.w = pack_bf16x2(p[6], p[7]);
          lo.x = pack_bf16x2(p[0] - bf16lo(hi.x), p[1] - bf16hi(hi.x));
          lo.y = pack_bf16x2(p[2] - bf16lo(hi.y), p[3] - bf16hi(hi.y));
          lo.z = pack_bf16x2(p[4] - bf16lo(hi.z), p[5] - bf16hi(hi.z));
          lo.w = pack_bf16x2(p[6] - bf16lo(hi.w), p[7] - bf16hi(hi.w));
          const int off = ((rep * (CW / 8) + c) ^ (row & 7)) << 4;
          *reinterpret_cast<uint4*>(prow + off) = hi;
          if (TC_PLANES == 2) *reinterpret_cast<uint4*>(prow + TC_P_BYTES + off) = lo;
        }
        l_run += (l4[0] + l4[1]) + (l4[2] + l4[3]);
      }
      umma::fence_smem_to_async();      // P rows and cleared V rows -> visible to the tensor core
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[b]);
      last_tile = i;
    }

    // ---- the group's result (m_ref, l, O); the odd group hands its rows over through shared memory ----
    if (alive && last_tile >= 0) alive = warp_wait(&pv_done[group], (last_tile >> 1) & 1);
    umma::fence_after_sync();
    // every product of BOTH groups has completed after this barrier (or the CTA has given up): Q, P and the
    // ring are free.  Exchange areas: [128 rows][BK_REC] fp32 from the start of shared memory, the
    // replicas' partial row sums behind it
    float* xch = reinterpret_cast<float*>(smem);
    static_assert(TC_OFF_L + 2 * 128 * 4 <= TC_OFF_BAR, "exchange areas lie in the Q / P / ring region");
    asm volatile("bar.sync 1, 256;" ::: "memory");
    l_x[group * 128 + L] = l_run;
    asm volatile("bar.sync 1, 256;" ::: "memory");
    float l_tot = 0.f;
#pragma unroll
    for (int r2 = 0; r2 < REP; ++r2) l_tot += l_x[group * 128 + row + r2 * RB];
    if (group == 1 && owns_o) {
      float* mine = xch + row * BK_REC;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        float o[32];
        if (last_tile >= 0 && alive) umma::tmem_ld32(my_o + c * 32, o);
        else {
#pragma unroll
          for (int x = 0; x < 32; ++x) o[x] = 0.f;
        }
#pragma unroll
        for (int x = 0; x < 32; x += 4)
          *reinterpret_cast<float4*>(mine + c * 32 + x) = make_float4(o[x], o[x + 1], o[x + 2], o[x + 3]);
      }
      mine[128] = (last_tile >= 0 && alive) ? m_ref : -INFINITY;
      mine[129] = l_tot;
    }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (group == 0 && owns_o && alive) {
      const float* other = xch + row * BK_REC;
      const float m1 = other[128], l1 = other[129];
      const float m0 = (last_tile >= 0) ? m_ref : -INFINITY;
      const float mC = fmaxf(m0, m1);
      const float f0 = (m0 == -INFINITY) ? 0.f : exp2f(m0 - mC), f1 = (m1 == -INFINITY) ? 0.f : exp2f(m1 - mC);
      const float lC = l_tot * f0 + l1 * f1;
      const bool direct = gm.n_splits == 1;
      const float inv = (lC > 0.f) ? 1.f / lC : 0.f;
      float* rec = a.partials + (((long long)s * a.max_splits + split) * a.rec_rows + row) * BK_REC;
      const long long off = q_row_offset(a, s, min(row, a.R - 1));
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        float o[32];
        if (last_tile >= 0) umma::tmem_ld32(my_o + c * 32, o);
#pragma unroll
        for (int x = 0; x < 32; ++x) {
          const float o0 = (last_tile >= 0) ? o[x] * f0 : 0.f;
          o[x] = (f1 != 0.f) ? fmaf(other[c * 32 + x], f1, o0) : o0;
        }
        if (row < a.R) {
          if (direct) {
#pragma unroll
            for (int x = 0; x < 32; x += 8) {
              uint4 w;
              w.x = pack_bf16x2(o[x] * inv, o[x + 1] * inv); w.y = pack_bf16x2(o[x + 2] * inv, o[x + 3] * inv);
              w.z = pack_bf16x2(o[x + 4] * inv, o[x + 5] * inv); w.w = pack_bf16x2(o[x + 6] * inv, o[x + 7] * inv);
              *reinterpret_cast<uint4*>(a.out + off + c * 32 + x) = w;
            }
          } else {
#pragma unroll
            for (int x = 0; x < 32; x += 4)
              *reinterpret_cast<float4*>(rec + c * 32 + x) = make_float4(o[x], o[x + 1], o[x + 2], o[x + 3]);
          }
        }
      }
      if (row < a.R) {
        if (direct) {
          if (a.lse) a.lse[off / D] = (lC > 0.f) ? (mC + log2f(lC)) * 0.69314718055994530942f : -INFINITY;
        } else {
          *reinterpret_cast<float2*>(rec + 128) = make_float2(mC, lC);
        }
      }
    }
    umma::fence_before_sync();
  }

  if (gm.n_splits > 1) block_merge_splits(a, s, gm.n_splits, a.R, flag, TC_THREADS);
  umma::fence_before_sync();
  __syncthreads();
  if (warp == 1) umma::tmem_dealloc(tmem_base, TC_TMEM_COLS);
}

template <int REP>
static cudaError_t launch_tc(const CUtensorMap* tm, const BlockArgs& a, dim3 grid, cudaStream_t st) {
  static DeviceFlags opted;
  {
    cudaError_t e = smem_opt_in(opted, kve_decode_attn_block_tc_kernel<REP>, TC_SMEM_BYTES);
    if (e != cudaSuccess) return e;
  }
  return launch_pdl(kve_decode_attn_block_tc_kernel<REP>, grid, dim3(TC_THREADS), TC_SMEM_BYTES, st, tm[0], tm[1], tm[2], tm[3], a);
}

cudaError_t launch_attn_block_tc(const CUtensorMap* tm, const BlockArgs& a, dim3 grid, cudaStream_t st) {
  if (a.R <= 32) return launch_tc<4>(tm, a, grid, st);
  if (a.R <= 64) return launch_tc<2>(tm, a, grid, st);
  return launch_tc<1>(tm, a, grid, st);
}

}  // namespace kve

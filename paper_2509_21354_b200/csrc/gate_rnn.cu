// LSTM recurrence + score head of the gate (Eq. 3): for every sequence, chunks oldest first,
//   pre_t = P_t + W_hh h_{t-1};  i,f,o = sigmoid, g = tanh;  c_t = f c_{t-1} + i g;  h_t = o tanh(c_t)
//   s_t   = sigmoid(w_s . h_t + b_s)
// P_t (= W_ih x_t + b_ih + b_hh) comes from the projection GEMM.
//
// The chain over t is strictly sequential, so the kernel is built for latency per step:
//  * A thread-block cluster of CL CTAs owns NG groups of 8 sequences for all steps (NG = 2 when one
//    group per cluster would not fit the GPU in one wave: the groups are independent pipelines, and a
//    warp handles them one after the other, so one group's exchange overlaps the other's arithmetic).  Each CTA owns
//    HU = d_g / CL hidden units, i.e. 4*HU rows of W_hh, and keeps them in REGISTERS as mma A
//    fragments for the whole kernel (128 registers per thread at d_g = 256, CL = 4).
//  * Per step the CTA computes its rows of W_hh h for all its sequences with warp-level tensor-core
//    MMAs (m16n8k16, bf16 x bf16 -> fp32).  W_hh is bf16 by definition; the fp32 state h enters as
//    PL = 2 bf16 planes by default (h = hi + lo up to 2^-17 |h|: 16 of its 24 significant bits; a third
//    plane makes the products exact, moves the scores by 1e-7 - far below what the fast
//    exponentials of the cell update contribute, 5e-5 - and costs a third more MMAs: 119 vs 99 us
//    on 256 sequences x 56 chunks).  Each plane has its own accumulators (as many independent MMA
//    chains), added smallest plane first at the end.
//  * MMA rows are ordered so that one thread ends up holding the i, f, g, o pre-activations of the
//    same (hidden unit, sequence): the cell update is thread-local, c lives in registers.
//  * Exchange of h_t: a warp gathers the planes of its 8 hidden units in a small staging area of
//    its own, then 16-byte st.async stores (one per plane, sequence and destination CTA) put them
//    into the double-buffered h planes of every other CTA of the cluster (the own copy is a plain
//    store followed by a local arrive).  Each remote store counts its bytes on an mbarrier of the
//    receiving CTA, so a step costs one one-way transfer and no
//    cluster-wide barrier.  A CTA can only be sent step t+1 data after it has itself sent step t
//    data, i.e. after all its warps have finished reading the buffer that is being overwritten.
//  * The score head is not part of the chain: h_t is stored as row (s, t) of a buffer of its own, and a
//    second, fully parallel kernel computes s_t = sigmoid(w_s . h_t + b_s) for all (s, t) afterwards, with
//    a fixed summation order.
//  * P_{t+1} is fetched into registers while step t computes: the projection kernel stores the four
//    pre-activations of a hidden unit side by side, so a thread takes them with one 16-byte load.
// Every mbarrier wait is bounded (one second); on give-up the status word gets KVE_ERR_TIMEOUT and
// the CTA stops sending, which lets its peers run into their own limits and leave as well.
#include "gate_rnn.cuh"

namespace kve {

// Optional cycle budget of one recurrence step (build with -DKVE_RNN_STAMPS, see rnn_stamps.py): warp 0 of CTA 0 adds
// up, over all steps and groups, the clock64 cycles between five points of a step - 0: waiting for the peers' h,
// 1: fragment loads + MMA chain, 2: prefetch of the next step's P, 3: cell update and plane split, 4: sending h,
// 6: from the end of one round to the start of the next (the loaded P moves into place, barrier bookkeeping) - and
// slot 5 counts the (step, group) rounds.  The marks are contiguous: the slots add up to the whole step loop.  Compiled out of the product library.
#ifdef KVE_RNN_STAMPS
__device__ unsigned long long g_rnn_cycles[8];
#define KVE_RNN_MARK(slot)                                                                   \
  do {                                                                                       \
    if (blockIdx.x == 0 && warp == 0 && lane == 0) {                                         \
      const long long now_ = clock64();                                                      \
      atomicAdd(&g_rnn_cycles[slot], (unsigned long long)(now_ - mark_));                    \
      mark_ = now_;                                                                          \
    }                                                                                        \
  } while (0)
#define KVE_RNN_MARK_BEGIN() long long mark_ = clock64()
__device__ unsigned long long g_rnn_once[8];
#define KVE_RNN_ONCE(slot)                                                                   \
  do {                                                                                       \
    if (blockIdx.x == 0 && threadIdx.x == 0) {                                               \
      unsigned long long t_;                                                                 \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                                 \
      g_rnn_once[slot] = t_;                                                                 \
    }                                                                                        \
  } while (0)
#else
#define KVE_RNN_MARK(slot) do { } while (0)
#define KVE_RNN_MARK_BEGIN() do { } while (0)
#define KVE_RNN_ONCE(slot) do { } while (0)
#endif

// NG independent groups of 8 sequences per cluster.  A group is one pipeline (own h buffers, barriers,
// staging and cell state); a warp works through the groups one after the other within a step, so
// while group A's new h is on its way between the CTAs the warp is busy with group B.
template <int DG, int CL, int NG, int PL>
__global__ void __cluster_dims__(CL, 1, 1) __launch_bounds__(RNN_THREADS, 1) kve_gate_rnn_kernel(RnnArgs a) {
  constexpr int HU = DG / CL;            // hidden units owned by this CTA
  constexpr int UW = HU / RNN_WARPS;     // hidden units per warp
  constexpr int MP = UW / 8;             // pairs of m16 tiles per warp (a pair = 8 units x 4 gates)
  constexpr int KT = DG / 16;            // k tiles
  constexpr int NS = 8;                  // sequences per group: the n of the m16n8k16 MMA
  constexpr int KBLK = PL * NS * 8;                     // bf16 elements of one k-block: [plane][sequence][8 units]
  constexpr int HS_BUF = (DG / 8) * KBLK;                       // bf16 elements per h buffer: [k-block][plane][sequence][8]
  constexpr int STG_WARP = MP * KBLK;                           // bf16 elements of one warp's staging area (its k-blocks)
  constexpr uint32_t H_BYTES = PL * NS * (DG - HU) * 2; // bytes of h planes a CTA receives from its peers per step and group
  constexpr int OFF_STAGE = NG * 2 * HS_BUF * 2;
  constexpr int OFF_BARS = OFF_STAGE + NG * RNN_WARPS * STG_WARP * 2;
  static_assert(UW % 8 == 0 && MP >= 1, "8 warps x 8k hidden units per CTA");
  static_assert(OFF_STAGE % 16 == 0 && OFF_BARS % 16 == 0, "16-byte pieces");

  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint16_t* hs = reinterpret_cast<uint16_t*>(smem_raw);                          // [NG][2][DG / 8][PLANES][NS][8]
  uint16_t* stage = reinterpret_cast<uint16_t*>(smem_raw + OFF_STAGE);           // [NG][warps][MP][PLANES][NS][8]
  uint64_t* hbar = reinterpret_cast<uint64_t*>(smem_raw + OFF_BARS);             // [NG][2] h planes landed

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, tig = lane & 3;
  const uint32_t rank = cluster_rank();
  const int cid = blockIdx.x / CL;
  const int seq0 = cid * NS * NG;        // group gi owns sequences seq0 + 8 gi .. + 7

  pdl_launch_dependents();
  KVE_RNN_ONCE(0);
  if (tid == 0) {
    for (int i = 0; i < 2 * NG; ++i) mbar_init(&hbar[i], 1 + RNN_WARPS);
    mbar_fence_init();
  }

  // ---- W_hh rows of this CTA as A fragments, resident in registers --------------------------------
  // Register j of the fragment of k tile kt holds the two bf16 at k = 16 kt + 8 (j >> 1) + 2 tig of row (j & 1): word
  // 8 kt + 4 (j >> 1) + tig of the row.  The four lanes of a group (equal g) fetch 16 consecutive words of the row with one
  // 16-byte load each (lane tig: words 4 tig ..) and turn the 4 x 4 block among themselves with shuffles, so that lane tig
  // ends up with words tig, 4 + tig, 8 + tig, 12 + tig: a quarter of the load instructions of word-by-word fetches (5 -> 2 us).
  // With two groups per cluster the kernel sits at the register limit and that order of definition cost 10 % in the step
  // loop (measured), so there the words are fetched one by one.
  uint32_t A[2 * MP][KT][4];
  static_assert(KT % 2 == 0, "k tiles are fetched in pairs");
  if constexpr (NG == 1) {
#pragma unroll
    for (int mt = 0; mt < 2 * MP; ++mt) {
      const int ug = (int)rank * HU + warp * UW + (mt >> 1) * 8 + g;
#pragma unroll
      for (int rs = 0; rs < 2; ++rs) {
        const int gate = (mt & 1) * 2 + rs;
        const uint4* wrow = reinterpret_cast<const uint4*>(a.W_hh + ((long long)gate * DG + ug) * DG) + tig;
#pragma unroll
        for (int kp = 0; kp < KT / 2; ++kp) {
          const uint4 w = __ldg(wrow + kp * 4);
          const bool hi = (tig & 2) != 0, lo = (tig & 1) != 0;
          // lanes t and t ^ 2 swap halves: afterwards y0, y1 come from lane (t & 1), y2, y3 from lane (t & 1) + 2, words 2 hi, 2 hi + 1
          const uint32_t r0 = __shfl_xor_sync(0xffffffffu, hi ? w.x : w.z, 2), r1 = __shfl_xor_sync(0xffffffffu, hi ? w.y : w.w, 2);
          const uint32_t y0 = hi ? r0 : w.x, y1 = hi ? r1 : w.y, y2 = hi ? w.z : r0, y3 = hi ? w.w : r1;
          // lanes t and t ^ 1 swap the word the other one wants
          const uint32_t u0 = __shfl_xor_sync(0xffffffffu, lo ? y0 : y1, 1), u1 = __shfl_xor_sync(0xffffffffu, lo ? y2 : y3, 1);
          const uint32_t k0 = lo ? y1 : y0, k1 = lo ? y3 : y2;
          A[mt][2 * kp][rs] = lo ? u0 : k0;              // word tig of the lane group's 16
          A[mt][2 * kp][rs + 2] = lo ? k0 : u0;          // word 4 + tig
          A[mt][2 * kp + 1][rs] = lo ? u1 : k1;          // word 8 + tig
          A[mt][2 * kp + 1][rs + 2] = lo ? k1 : u1;      // word 12 + tig
        }
      }
    }
  } else {
#pragma unroll
    for (int mt = 0; mt < 2 * MP; ++mt) {
      const int ug = (int)rank * HU + warp * UW + (mt >> 1) * 8 + g;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int gate = (mt & 1) * 2 + (j & 1);
        const uint32_t* wrow = reinterpret_cast<const uint32_t*>(a.W_hh + ((long long)gate * DG + ug) * DG);
#pragma unroll
        for (int kt = 0; kt < KT; ++kt) A[mt][kt][j] = __ldg(wrow + kt * 8 + (j >> 1) * 4 + tig);
      }
    }
  }

  KVE_RNN_ONCE(1);
  pdl_wait();      // W_hh is in registers; the carried state and P come from earlier kernels
  KVE_RNN_ONCE(2);
  // ---- initial state: every CTA needs the full h of its sequences as planes in buffer 0 of each group -------------
  for (int i = tid; i < NG * NS * (DG / 2); i += RNN_THREADS) {
    const int js = i / (DG / 2), k2 = i % (DG / 2);      // js: sequence of the cluster, 0 .. 8 NG - 1
    const int gi = js / NS, j = js % NS;
    const int s = seq0 + js;
    float h0 = 0.f, h1 = 0.f;
    if (!a.reset && s < a.S) {
      const float2 hv = *reinterpret_cast<const float2*>(a.lstm_h + (long long)s * DG + k2 * 2);
      h0 = hv.x; h1 = hv.y;
    }
    uint32_t p0[3], p1[3];      // the leading PL pieces are used
    split3(h0, p0);
    split3(h1, p1);
#pragma unroll
    for (int pl = 0; pl < PL; ++pl)
      *reinterpret_cast<uint32_t*>(hs + gi * 2 * HS_BUF + (k2 >> 2) * KBLK + (pl * NS + j) * 8 + (k2 & 3) * 2) = p0[pl] | (p1[pl] << 16);
  }
  float c[NG][MP][2], hlast[NG][MP][2];
  float pin[NG][MP][4][2];     // P of the current step
  const int n_cols = 4 * DG;
#pragma unroll
  for (int gi = 0; gi < NG; ++gi)
#pragma unroll
    for (int p = 0; p < MP; ++p)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int s = seq0 + gi * NS + tig * 2 + e;
        const int ug = (int)rank * HU + warp * UW + p * 8 + g;
        const bool live = !a.reset && s < a.S;
        c[gi][p][e] = live ? a.lstm_c[(long long)s * DG + ug] : 0.f;
        hlast[gi][p][e] = live ? a.lstm_h[(long long)s * DG + ug] : 0.f;
        // the four pre-activations of a unit lie side by side in P: one 16-byte load
        const float4 pv = (s < a.S) ? __ldcs(reinterpret_cast<const float4*>(a.P + ((long long)s * a.n_range) * n_cols) + ug)
                                    : make_float4(0.f, 0.f, 0.f, 0.f);
        pin[gi][p][0][e] = pv.x; pin[gi][p][1][e] = pv.y; pin[gi][p][2][e] = pv.z; pin[gi][p][3][e] = pv.w;
      }

  // lane r < CL feeds peer r: that CTA's h buffers and barriers, as addresses in the cluster window
  const uint32_t peer_hs = map_to_rank(smem_u32(hs), lane < CL ? lane : 0);
  const uint32_t peer_bar = map_to_rank(smem_u32(&hbar[0]), lane < CL ? lane : 0);

  // barriers initialised and buffer 0 filled in every CTA before anyone sends
  KVE_RNN_ONCE(3);
  cluster_sync_all();
  KVE_RNN_ONCE(4);

  bool alive = true;
  KVE_RNN_MARK_BEGIN();
  for (int step = 0; step < a.n_range && alive; ++step) {
    const int buf = step & 1;
    const bool send_h = step + 1 < a.n_range;
    // this step's sends of the cluster land in buffer buf^1 of each group: announce the bytes
    if (tid == 0 && send_h) {
#pragma unroll
      for (int gi = 0; gi < NG; ++gi) mbar_arrive_expect_tx(&hbar[2 * gi + (buf ^ 1)], H_BYTES);
    }
#pragma unroll
    for (int gi = 0; gi < NG; ++gi) {
      uint16_t* hs_g = hs + gi * 2 * HS_BUF;
      uint16_t* my_stage = stage + (gi * RNN_WARPS + warp) * STG_WARP;
      uint64_t* hbar_g = hbar + 2 * gi;
      const int seq_g = seq0 + gi * NS;
      KVE_RNN_MARK(6);
      if (step > 0) {
        // h_{t-1} of this group from every CTA of the cluster (each buffer completes once per two steps)
        if (!mbar_wait_cluster_bounded(&hbar_g[buf], ((step - 1) >> 1) & 1)) {
          if (lane == 0) set_status(a.status, ERR_TIMEOUT);
          alive = false;
        }
        if (!__all_sync(0xffffffffu, alive)) alive = false;
        if (!alive) break;
      }

      KVE_RNN_MARK(0);
      // ---- W_hh h_{t-1} on the tensor cores: one accumulator set per plane ---------------------------
      float acc[PL][2 * MP][4];
#pragma unroll
      for (int pl = 0; pl < PL; ++pl)
#pragma unroll
        for (int mt = 0; mt < 2 * MP; ++mt)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[pl][mt][e] = 0.f;
      // B fragments: one ldmatrix.x4 brings the 8 sequences x 32 k-values of a plane (two k tiles);
      // lane l addresses row (l & 7) of the 8 x 8 block (l >> 3).  Loaded one k-tile pair ahead.
      const uint32_t hb_lane = smem_u32(hs_g + buf * HS_BUF + (lane >> 3) * KBLK + (lane & 7) * 8);
      uint32_t bf[2][PL][4];
#pragma unroll
      for (int pl = 0; pl < PL; ++pl) ldmatrix_x4(bf[0][pl], hb_lane + (uint32_t)(pl * NS * 8 * 2));
#pragma unroll
      for (int kp = 0; kp < KT / 2; ++kp) {
        const int cur = kp & 1;
        if (kp + 1 < KT / 2) {
#pragma unroll
          for (int pl = 0; pl < PL; ++pl)
            ldmatrix_x4(bf[cur ^ 1][pl], hb_lane + (uint32_t)(((kp + 1) * 4 * KBLK + pl * NS * 8) * 2));
        }
#pragma unroll
        for (int half = 0; half < 2; ++half)
#pragma unroll
          for (int pl = 0; pl < PL; ++pl)
#pragma unroll
            for (int mt = 0; mt < 2 * MP; ++mt)
              mma_bf16_16816(acc[pl][mt], A[mt][2 * kp + half], bf[cur][pl][2 * half], bf[cur][pl][2 * half + 1]);
      }

      KVE_RNN_MARK(1);
      // ---- P_{t+1} into registers while the MMAs drain ----------------------------------------------------
      float pnext[MP][4][2];
#pragma unroll
      for (int p = 0; p < MP; ++p)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int s = seq_g + tig * 2 + e;
          const int ug = (int)rank * HU + warp * UW + p * 8 + g;
          const bool live = s < a.S && send_h;
          const float4* prow = reinterpret_cast<const float4*>(a.P + ((long long)s * a.n_range + step + 1) * n_cols) + ug;
          const float4 pv = live ? __ldcs(prow) : make_float4(0.f, 0.f, 0.f, 0.f);
          pnext[p][0][e] = pv.x; pnext[p][1][e] = pv.y; pnext[p][2][e] = pv.z; pnext[p][3][e] = pv.w;
          // the 8 lanes of a group cover one 128-byte line of the row after it: one of them asks L2 for it
          if (s < a.S && step + 2 < a.n_range && g == 0) asm volatile("prefetch.global.L2 [%0];" ::"l"(prow + n_cols / 4));
        }

      KVE_RNN_MARK(2);
      // ---- cell update (thread-local), planes of h_t into the warp's staging area ---------------------
      asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
      __syncwarp();      // earlier copies have read the staging areas
#pragma unroll
      for (int p = 0; p < MP; ++p) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          float pre[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {   // q: 0 = i, 1 = f (tile 2p, rows g / g+8), 2 = g, 3 = o (tile 2p+1)
            const int mt = 2 * p + (q >> 1), ai = (q & 1) * 2 + e;
            float sum = acc[PL - 1][mt][ai];      // smallest plane first
#pragma unroll
            for (int pl = PL - 2; pl >= 0; --pl) sum += acc[pl][mt][ai];
            pre[q] = sum + pin[gi][p][q][e];
          }
          const float ig = fast_sigmoid(pre[0]);
          const float fg = fast_sigmoid(pre[1]);
          const float gg = fast_tanh(pre[2]);
          const float og = fast_sigmoid(pre[3]);
          const float cn = fmaf(fg, c[gi][p][e], ig * gg);
          c[gi][p][e] = cn;
          const float hv = og * fast_tanh(cn);
          hlast[gi][p][e] = hv;
          {
            // h_t for the score kernel
            const int sq = seq_g + tig * 2 + e;
            if (sq < a.S) a.H[((long long)sq * a.n_range + step) * DG + (int)rank * HU + warp * UW + p * 8 + g] = hv;
          }
          if (send_h) {
            uint32_t pl3[3];
            split3(hv, pl3);
            const int j = tig * 2 + e;
#pragma unroll
            for (int pl = 0; pl < PL; ++pl) my_stage[p * KBLK + (pl * NS + j) * 8 + g] = (uint16_t)pl3[pl];
          }
        }
      }
      KVE_RNN_MARK(3);
      // ---- the warp's k-blocks (8 units each: [plane][sequence][8], contiguous) to every CTA of the cluster ----
      if (send_h) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // staging writes -> visible to the bulk copies
        __syncwarp();
#pragma unroll
        for (int p = 0; p < MP; ++p) {
          const uint32_t off = (uint32_t)(((gi * 2 + (buf ^ 1)) * HS_BUF + ((int)rank * (HU / 8) + warp * MP + p) * KBLK) * 2);
          // peers: one bulk copy per k-block and peer, its bytes counted on the receiver's barrier
          if (lane < CL && lane != (int)rank)
            bulk_s2cluster(peer_hs + off, smem_u32(my_stage + p * KBLK), KBLK * 2, peer_bar + (2 * gi + (buf ^ 1)) * 8);
          // own CTA: plain 16-byte stores (ordered by this warp's arrive below)
          for (int idx = lane; idx < KBLK / 8; idx += 32)
            *reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(hs) + off + idx * 16) =
                *reinterpret_cast<const uint4*>(my_stage + p * KBLK + idx * 8);
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&hbar_g[buf ^ 1]);     // release: this warp's local pieces are in place
      }

      KVE_RNN_MARK(4);
#ifdef KVE_RNN_STAMPS
      if (blockIdx.x == 0 && warp == 0 && lane == 0) atomicAdd(&g_rnn_cycles[5], 1ull);
#endif
#pragma unroll
      for (int p = 0; p < MP; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q)
#pragma unroll
          for (int e = 0; e < 2; ++e) pin[gi][p][q][e] = pnext[p][q][e];
    }
  }

  KVE_RNN_ONCE(5);
  // ---- carried state out ---------------------------------------------------------------------------
#pragma unroll
  for (int gi = 0; gi < NG; ++gi)
#pragma unroll
    for (int p = 0; p < MP; ++p)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int s = seq0 + gi * NS + tig * 2 + e;
        const int ug = (int)rank * HU + warp * UW + p * 8 + g;
        if (s < a.S && alive) {
          a.lstm_c[(long long)s * DG + ug] = c[gi][p][e];
          a.lstm_h[(long long)s * DG + ug] = hlast[gi][p][e];
        }
      }
  // nobody leaves while a peer may still be sending into its shared memory
  cluster_sync_all();
  KVE_RNN_ONCE(6);
}

// ---- score head: s_t = sigmoid(w_s . h_t + b_s), one warp per SCORE_ROWS (sequence, chunk) rows --------------------
// h_t is row (s, t) of H.  Lane l sums elements l*4 .. l*4+3 (+128 per round) in
// order, then a butterfly over the lanes: the same order for every launch.  A warp has the loads of all its rows in
// flight before it starts to add.
constexpr int SCORE_ROWS = 4;
constexpr int SCORE_WARPS = 8;

template <int DG>
__global__ void __launch_bounds__(SCORE_WARPS * 32) kve_gate_score_kernel(const float* __restrict__ H, const float* __restrict__ w_s,
                                                                         float b_s, float* __restrict__ scores, long long n_rows,
                                                                         int n_range, int t0, int max_chunks) {
  constexpr int ROUNDS = (DG / 4 + 31) / 32;      // 16-byte pieces per lane and row
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const long long row0 = ((long long)blockIdx.x * SCORE_WARPS + (threadIdx.x >> 5)) * SCORE_ROWS;
  if (row0 >= n_rows) return;
  const float4* w = reinterpret_cast<const float4*>(w_s);
  float4 hv[SCORE_ROWS][ROUNDS];
#pragma unroll
  for (int r = 0; r < SCORE_ROWS; ++r) {
    const float4* h = reinterpret_cast<const float4*>(H + (row0 + r) * DG);
#pragma unroll
    for (int i = 0; i < ROUNDS; ++i)
      hv[r][i] = (row0 + r < n_rows && lane + 32 * i < DG / 4) ? __ldcs(h + lane + 32 * i) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  float4 wv[ROUNDS];
#pragma unroll
  for (int i = 0; i < ROUNDS; ++i) wv[i] = (lane + 32 * i < DG / 4) ? __ldg(w + lane + 32 * i) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
  for (int r = 0; r < SCORE_ROWS; ++r) {
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < ROUNDS; ++i) {
      if (lane + 32 * i < DG / 4) {
        acc = fmaf(hv[r][i].x, wv[i].x, acc); acc = fmaf(hv[r][i].y, wv[i].y, acc);
        acc = fmaf(hv[r][i].z, wv[i].z, acc); acc = fmaf(hv[r][i].w, wv[i].w, acc);
      }
    }
    acc = warp_sum(acc);
    const long long row = row0 + r;
    if (lane == 0 && row < n_rows) {
      const int s = (int)(row / n_range);
      const int t = t0 + (int)(row - (long long)s * n_range);
      scores[(long long)s * max_chunks + t] = 1.f / (1.f + expf(-(acc + b_s)));
    }
  }
}

static cudaError_t launch_score(const float* H, const float* w_s, float b_s, float* scores, long long n_rows, int n_range, int t0,
                                int max_chunks, int d_g, cudaStream_t st) {
  const dim3 grid((unsigned)((n_rows + SCORE_WARPS * SCORE_ROWS - 1) / (SCORE_WARPS * SCORE_ROWS))), block(SCORE_WARPS * 32);
  switch (d_g) {
    case 256: return launch_pdl(kve_gate_score_kernel<256>, grid, block, 0, st, H, w_s, b_s, scores, n_rows, n_range, t0, max_chunks);
    case 128: return launch_pdl(kve_gate_score_kernel<128>, grid, block, 0, st, H, w_s, b_s, scores, n_rows, n_range, t0, max_chunks);
    case 64:  return launch_pdl(kve_gate_score_kernel<64>, grid, block, 0, st, H, w_s, b_s, scores, n_rows, n_range, t0, max_chunks);
    default:  return cudaErrorInvalidValue;
  }
}

template <int DG, int CL, int NG, int PL>
static cudaError_t launch_rnn_t(const RnnArgs& a, cudaStream_t st) {
  constexpr int NS = 8 * NG;      // sequences per cluster
  constexpr int smem = 2 * PL * NS * DG * 2 + PL * NS * (DG / CL) * 2 + NG * 2 * 8;
  static DeviceFlags opted;
  {
    cudaError_t e = smem_opt_in(opted, kve_gate_rnn_kernel<DG, CL, NG, PL>, smem);
    if (e != cudaSuccess) return e;
  }
  const int clusters = (a.S + NS - 1) / NS;
  return launch_pdl(kve_gate_rnn_kernel<DG, CL, NG, PL>, dim3(clusters * CL), dim3(RNN_THREADS), smem, st, a);
}

template <int PL>
static cudaError_t launch_rnn_planes(const RnnArgs& a, int d_g, cudaStream_t st) {
  // two 8-sequence groups per cluster once one group per cluster would need more than one wave of clusters
  switch (d_g) {
    case 256: return (a.S > 8 * (sm_count() / 4)) ? launch_rnn_t<256, 4, 2, PL>(a, st) : launch_rnn_t<256, 4, 1, PL>(a, st);
    case 128: return launch_rnn_t<128, 1, 1, PL>(a, st);
    case 64:  return (a.S > 8 * sm_count()) ? launch_rnn_t<64, 1, 2, PL>(a, st) : launch_rnn_t<64, 1, 1, PL>(a, st);
    default:  return cudaErrorInvalidValue;
  }
}

cudaError_t launch_gate_rnn(const LayerView& v, int t0, int t1, const uint16_t* W_hh, const float* w_s, float b_s,
                            int d_g, const float* P, float* H, bool reset_state, int planes, cudaStream_t st) {
  if (t1 <= t0 || v.S <= 0) return cudaSuccess;
  RnnArgs a;
  a.P = P; a.H = H; a.W_hh = W_hh; a.w_s = w_s; a.b_s = b_s;
  a.scores = v.scores; a.lstm_h = v.lstm_h; a.lstm_c = v.lstm_c; a.status = v.status;
  a.S = v.S; a.max_chunks = v.max_chunks; a.t0 = t0; a.n_range = t1 - t0; a.reset = reset_state ? 1 : 0;
  const cudaError_t e = planes == 3 ? launch_rnn_planes<3>(a, d_g, st) : launch_rnn_planes<2>(a, d_g, st);
  if (e != cudaSuccess) return e;
  const long long n_rows = (long long)v.S * a.n_range;
  return launch_score(H, w_s, b_s, v.scores, n_rows, a.n_range, t0, v.max_chunks, d_g, st);
}

}  // namespace kve

#ifdef KVE_RNN_STAMPS
// instrumented build only: read and clear the cycle sums
extern "C" int kve_rnn_once_read(unsigned long long* host) {
  return (int)cudaMemcpyFromSymbol(host, kve::g_rnn_once, sizeof(kve::g_rnn_once));
}
extern "C" int kve_rnn_cycles_read(unsigned long long* host) {
  cudaError_t e = cudaMemcpyFromSymbol(host, kve::g_rnn_cycles, sizeof(kve::g_rnn_cycles));
  void* p = nullptr;
  if (e == cudaSuccess) e = cudaGetSymbolAddress(&p, kve::g_rnn_cycles);
  if (e == cudaSuccess) e = cudaMemset(p, 0, sizeof(kve::g_rnn_cycles));
  return (int)e;
}
#endif

// The gate's work at a trigger (Sec. 3.3: "whenever the KV cache grows to a certain size, we trigger an
// aggregation-and-gating step") when ONE chunk per sequence has left the window: a single LSTM step (Eq. 3) on the
// new summary with the carried state, its score, and the retention decision (Sec. 3.2) appended to the keep list -
// one launch instead of projection GEMM + recurrence + score head + compaction + kept-row gather.
//
//   pre = W_ih [Kbar_t ; Vbar_t] + b_ih + b_hh + W_hh h_{t-1};  i,f,o = sigmoid, g = tanh;
//   c_t = f c_{t-1} + i g;  h_t = o tanh(c_t);  s_t = sigmoid(w_s . h_t + b_s);  keep t iff s_t >= tau
//
//  * A cluster of CL CTAs owns NG groups of 8 sequences; CTA r owns hidden units [r HU, (r + 1) HU), i.e. 4 HU rows
//    of W_ih and W_hh.  The step is a skinny product (8 columns per group): warp-level m16n8k16 MMAs, bf16 x bf16 ->
//    fp32.  The weight rows stream from L2 straight into A fragments, each loaded once and used for all NG groups;
//    the B operands - the bf16 summary rows and the PL bf16 planes of h_{t-1} - wait in shared memory.
//  * Both operands are fetched 16 bytes at a time: lane (g, tig) takes the 8 consecutive k of its row that start at
//    8 tig, which feed the k positions of TWO MMAs.  That permutes k inside a block of 32 in the same way for A and B,
//    which a contraction does not notice.
//  * MMA rows are ordered as in the recurrence kernel, so one thread holds i, f, g, o of a (unit, sequence) pair:
//    the cell update is thread-local.  Every CTA reads all of h_{t-1} and writes its slice of h_t: a split cluster
//    barrier (arrive after the reads, wait before the writes) keeps the two apart.
//  * Score: per-CTA partial dot products in a fixed order, sent to CTA 0 of the cluster through distributed
//    shared memory, summed there in rank order.  CTA 0 appends the kept chunks to keep_idx / keep_cnt and copies
//    their summary rows behind the sequence's compacted run; the coverage count on the device advances.
// No wait in this kernel can run out: the only synchronisation is the cluster barrier, which every thread reaches.
#include "gate_rnn.cuh"

namespace kve {

struct GateStepArgs {
  const uint16_t* W_ih;      // bf16 [4 d_g][256]
  const uint16_t* W_hh;      // bf16 [4 d_g][d_g]
  const float *b_ih, *b_hh, *w_s;
  float b_s, tau;
  const uint16_t *ksum, *vsum;      // bf16 [S][max_chunks][128]
  float *scores, *lstm_h, *lstm_c;
  int32_t *keep_idx, *keep_cnt, *n_listed, *ticket;
  const int32_t* seq_len;
  uint16_t *kept_k, *kept_v;        // bf16 [S][max_chunks][128]
  int S, max_chunks, t;
  int C, dev_window;      // dev_window >= 0: t comes from the device (the chunk behind the keep list, if it has left the window)
};

constexpr int STEP_MAX_SEQ = 32;      // sequences per cluster at most (NG = 4)

template <int DG, int CL, int NG, int PL>
__global__ void __cluster_dims__(CL, 1, 1) __launch_bounds__(RNN_THREADS, 1) kve_gate_step_kernel(GateStepArgs a) {
  constexpr int HU = DG / CL;            // hidden units owned by this CTA
  constexpr int NSEQ = 8 * NG;           // sequences per cluster
  constexpr int XSTR = 2 * D * 2 + 64;   // bytes per summary row in shared memory; 64 mod 128: 16-byte reads of 8 rows x 64 B do not collide
  constexpr int HSTR = DG * 2 + 64;      // bytes per row of a plane of h
  static_assert(HU == 8 * RNN_WARPS, "one m16 tile pair (8 units x 4 gates) per warp");
  static_assert(NSEQ <= STEP_MAX_SEQ, "shared arrays below");

  extern __shared__ __align__(16) unsigned char step_smem[];
  unsigned char* xs = step_smem;                         // [NSEQ][XSTR]: [Kbar ; Vbar] bf16
  unsigned char* hsm = step_smem + NSEQ * XSTR;          // [PL][NSEQ][HSTR]: planes of h_{t-1}
  __shared__ float part[RNN_WARPS][STEP_MAX_SEQ];        // per-warp partial dot products w_s . h_t
  __shared__ float cpart[CL][STEP_MAX_SEQ];              // CTA 0 of the cluster: the CTAs' partial sums
  __shared__ int kept_slot[STEP_MAX_SEQ];                // CTA 0: position of chunk t in the sequence's keep list, or -1

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, tig = lane & 3;
  const uint32_t rank = cluster_rank();
  const int seq0 = (blockIdx.x / CL) * NSEQ;

  pdl_launch_dependents();
  pdl_wait();
  if (a.dev_window >= 0) {
    // every CTA reads the same count: it only moves when the last cluster of this launch has arrived at the end
    const NextChunk nx = next_chunk(a.n_listed, a.seq_len, a.C, a.dev_window, a.max_chunks);
    if (!nx.due) return;
    a.t = nx.t;
  }

  // ---- B operands into shared memory -----------------------------------------------------------------------------------
  for (int i = tid; i < NSEQ * 32; i += RNN_THREADS) {      // 16-byte pieces of the summary rows: 16 of Kbar, 16 of Vbar
    const int j = i >> 5, p = i & 31, s = seq0 + j;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (s < a.S) v = __ldg(reinterpret_cast<const uint4*>((p < 16 ? a.ksum : a.vsum) + ((long long)s * a.max_chunks + a.t) * D) + (p & 15));
    *reinterpret_cast<uint4*>(xs + j * XSTR + p * 16) = v;
  }
  for (int i = tid; i < NSEQ * (DG / 8); i += RNN_THREADS) {      // 8 consecutive units of h: one 16-byte piece per plane
    const int j = i / (DG / 8), p = i % (DG / 8), s = seq0 + j;
    float h[8];
    if (s < a.S) {
      const float4* src = reinterpret_cast<const float4*>(a.lstm_h + (long long)s * DG + p * 8);
      const float4 lo = src[0], hi = src[1];
      h[0] = lo.x; h[1] = lo.y; h[2] = lo.z; h[3] = lo.w; h[4] = hi.x; h[5] = hi.y; h[6] = hi.z; h[7] = hi.w;
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) h[e] = 0.f;
    }
    uint32_t pk[3][4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      uint32_t p0[3], p1[3];      // the leading PL pieces are used
      split3(h[2 * e], p0);
      split3(h[2 * e + 1], p1);
#pragma unroll
      for (int pl = 0; pl < 3; ++pl) pk[pl][e] = p0[pl] | (p1[pl] << 16);
    }
#pragma unroll
    for (int pl = 0; pl < PL; ++pl)
      *reinterpret_cast<uint4*>(hsm + (pl * NSEQ + j) * HSTR + p * 16) = make_uint4(pk[pl][0], pk[pl][1], pk[pl][2], pk[pl][3]);
  }
  __syncthreads();
  // every CTA of the cluster has read h_{t-1} before any of them stores h_t
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");

  // ---- pre-activations: weight rows stream through the A fragments -------------------------------------------------
  float acc[NG][PL + 1][2][4];      // per group: [0] W_ih x, [1 + pl] W_hh (plane pl of h); two m16 tiles: i | f and g | o
#pragma unroll
  for (int gi = 0; gi < NG; ++gi)
#pragma unroll
    for (int i = 0; i < PL + 1; ++i)
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[gi][i][mt][e] = 0.f;
  const int ug = (int)rank * HU + warp * 8 + g;      // this thread's hidden unit
#pragma unroll
  for (int mt = 0; mt < 2; ++mt) {
    // rows g of the tile: gate 2 mt, rows g + 8: gate 2 mt + 1; this lane's 8 consecutive k start at 8 tig
    const uint4* wxa = reinterpret_cast<const uint4*>(a.W_ih + ((long long)(2 * mt) * DG + ug) * (2 * D)) + tig;
    const uint4* wxb = reinterpret_cast<const uint4*>(a.W_ih + ((long long)(2 * mt + 1) * DG + ug) * (2 * D)) + tig;
    const uint4* wha = reinterpret_cast<const uint4*>(a.W_hh + ((long long)(2 * mt) * DG + ug) * DG) + tig;
    const uint4* whb = reinterpret_cast<const uint4*>(a.W_hh + ((long long)(2 * mt + 1) * DG + ug) * DG) + tig;
#pragma unroll
    for (int kk = 0; kk < (2 * D) / 32; ++kk) {      // 32 k per round: two MMAs per group
      const uint4 ra = __ldg(wxa + kk * 4), rb = __ldg(wxb + kk * 4);
      const uint32_t A0[4] = {ra.x, rb.x, ra.y, rb.y}, A1[4] = {ra.z, rb.z, ra.w, rb.w};
#pragma unroll
      for (int gi = 0; gi < NG; ++gi) {
        const uint4 bb = *reinterpret_cast<const uint4*>(xs + (gi * 8 + g) * XSTR + kk * 64 + tig * 16);
        mma_bf16_16816(acc[gi][0][mt], A0, bb.x, bb.y);
        mma_bf16_16816(acc[gi][0][mt], A1, bb.z, bb.w);
      }
    }
    if (a.t > 0) {      // chunk 0 starts from h = 0
#pragma unroll
      for (int kk = 0; kk < DG / 32; ++kk) {
        const uint4 ra = __ldg(wha + kk * 4), rb = __ldg(whb + kk * 4);
        const uint32_t A0[4] = {ra.x, rb.x, ra.y, rb.y}, A1[4] = {ra.z, rb.z, ra.w, rb.w};
#pragma unroll
        for (int gi = 0; gi < NG; ++gi)
#pragma unroll
          for (int pl = 0; pl < PL; ++pl) {
            const uint4 bb = *reinterpret_cast<const uint4*>(hsm + (pl * NSEQ + gi * 8 + g) * HSTR + kk * 64 + tig * 16);
            mma_bf16_16816(acc[gi][1 + pl][mt], A0, bb.x, bb.y);
            mma_bf16_16816(acc[gi][1 + pl][mt], A1, bb.z, bb.w);
          }
      }
    }
  }

  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");

  // ---- cell update (thread-local), partial score ------------------------------------------------------------------------
  float bias[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) bias[q] = __ldg(a.b_ih + q * DG + ug) + __ldg(a.b_hh + q * DG + ug);
  const float ws = __ldg(a.w_s + ug);
#pragma unroll
  for (int gi = 0; gi < NG; ++gi) {
    float dot[2];      // this thread's part of w_s . h_t for sequences 2 tig, 2 tig + 1 of the group
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int s = seq0 + gi * 8 + tig * 2 + e;
      float pre[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {   // q: 0 = i, 1 = f (tile 0, rows g / g+8), 2 = g, 3 = o (tile 1)
        const int mt = q >> 1, ai = (q & 1) * 2 + e;
        float sum = acc[gi][PL][mt][ai];      // smallest plane first
#pragma unroll
        for (int pl = PL - 2; pl >= 0; --pl) sum += acc[gi][1 + pl][mt][ai];
        pre[q] = (acc[gi][0][mt][ai] + bias[q]) + sum;      // P_t as the projection kernel forms it, then the recurrent term
      }
      const float c_prev = (a.t > 0 && s < a.S) ? a.lstm_c[(long long)s * DG + ug] : 0.f;
      const float ig = fast_sigmoid(pre[0]);
      const float fg = fast_sigmoid(pre[1]);
      const float gg = fast_tanh(pre[2]);
      const float og = fast_sigmoid(pre[3]);
      const float cn = fmaf(fg, c_prev, ig * gg);
      const float hv = og * fast_tanh(cn);
      if (s < a.S) {
        a.lstm_c[(long long)s * DG + ug] = cn;
        a.lstm_h[(long long)s * DG + ug] = hv;
      }
      // over the 8 units a lane group holds (lanes with equal tig), fixed order
      float d = ws * hv;
      d += __shfl_xor_sync(0xffffffffu, d, 4);
      d += __shfl_xor_sync(0xffffffffu, d, 8);
      d += __shfl_xor_sync(0xffffffffu, d, 16);
      dot[e] = d;
    }
    if (g == 0) {
      part[warp][gi * 8 + tig * 2 + 0] = dot[0];
      part[warp][gi * 8 + tig * 2 + 1] = dot[1];
    }
  }
  __syncthreads();
  if (tid < NSEQ) {
    float sum = 0.f;
#pragma unroll
    for (int w = 0; w < RNN_WARPS; ++w) sum += part[w][tid];
    // to CTA 0 of the cluster
    const uint32_t dst = map_to_rank(smem_u32(&cpart[rank][tid]), 0);
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(dst), "f"(sum) : "memory");
  }
  cluster_sync_all();
  if (rank != 0) return;

  // ---- CTA 0: score, retention decision, keep list ---------------------------------------------------------------------
  if (tid < NSEQ) {
    const int s = seq0 + tid;
    int slot = -1;
    if (s < a.S) {
      float sum = 0.f;
#pragma unroll
      for (int r = 0; r < CL; ++r) sum += cpart[r][tid];
      const float score = 1.f / (1.f + expf(-(sum + a.b_s)));
      a.scores[(long long)s * a.max_chunks + a.t] = score;
      if (score >= a.tau) {
        slot = a.keep_cnt[s];
        a.keep_idx[(long long)s * a.max_chunks + slot] = a.t;
        a.keep_cnt[s] = slot + 1;
      }
    }
    kept_slot[tid] = slot;
  }
  if (a.dev_window < 0 && blockIdx.x == 0 && tid == 0) *a.n_listed = a.t + 1;
  __syncthreads();
  // a warp copies a kept sequence's summary rows (K and V: 2 x 256 bytes) behind its compacted run
  for (int j = warp; j < NSEQ; j += RNN_WARPS) {
    if (kept_slot[j] < 0) continue;
    const int s = seq0 + j;
    const long long src = ((long long)s * a.max_chunks + a.t) * D, dst = ((long long)s * a.max_chunks + kept_slot[j]) * D;
    if (lane < 16) reinterpret_cast<uint4*>(a.kept_k + dst)[lane] = reinterpret_cast<const uint4*>(a.ksum + src)[lane];
    else reinterpret_cast<uint4*>(a.kept_v + dst)[lane - 16] = reinterpret_cast<const uint4*>(a.vsum + src)[lane - 16];
  }
  if (a.dev_window >= 0) {
    // the coverage count moves when the last cluster is through: until then every CTA of the launch finds the same t
    __syncthreads();
    if (tid == 0) {
      __threadfence();
      const int clusters = gridDim.x / CL;
      if (atomicAdd(a.ticket, 1) == clusters - 1) {
        *a.ticket = 0;
        *a.n_listed = a.t + 1;
      }
    }
  }
}

template <int DG, int CL, int NG, int PL>
static cudaError_t launch_step_t(const GateStepArgs& a, cudaStream_t st) {
  constexpr int smem = 8 * NG * ((2 * D * 2 + 64) + PL * (DG * 2 + 64));
  static DeviceFlags opted;
  {
    cudaError_t e = smem_opt_in(opted, kve_gate_step_kernel<DG, CL, NG, PL>, smem);
    if (e != cudaSuccess) return e;
  }
  const int clusters = (a.S + 8 * NG - 1) / (8 * NG);
  return launch_pdl(kve_gate_step_kernel<DG, CL, NG, PL>, dim3(clusters * CL), dim3(RNN_THREADS), smem, st, a);
}

// groups of 8 sequences per cluster: as few as keep the clusters within one wave, so the weights cross L2 -> SM as
// rarely as possible without leaving SMs idle
template <int DG, int CL, int PL>
static cudaError_t launch_step_groups(const GateStepArgs& a, cudaStream_t st) {
  const int groups = (a.S + 7) / 8, wave = sm_count() / CL;
  if (groups <= wave) return launch_step_t<DG, CL, 1, PL>(a, st);
  if (groups <= 2 * wave || PL == 3) return launch_step_t<DG, CL, 2, PL>(a, st);
  return launch_step_t<DG, CL, (PL == 3 ? 2 : 4), PL>(a, st);
}

template <int PL>
static cudaError_t launch_step_planes(const GateStepArgs& a, int d_g, cudaStream_t st) {
  switch (d_g) {
    case 256: return launch_step_groups<256, 4, PL>(a, st);
    case 128: return launch_step_groups<128, 2, PL>(a, st);
    case 64:  return launch_step_groups<64, 1, PL>(a, st);
    default:  return cudaErrorInvalidValue;
  }
}

cudaError_t launch_gate_step(const LayerView& v, int t, const uint16_t* W_ih, const uint16_t* W_hh, const float* b_ih,
                             const float* b_hh, const float* w_s, float b_s, float tau, int d_g, int planes,
                             uint16_t* kept_k, uint16_t* kept_v, int dev_window, cudaStream_t st) {
  if (v.S <= 0) return cudaSuccess;
  GateStepArgs a;
  a.W_ih = W_ih; a.W_hh = W_hh; a.b_ih = b_ih; a.b_hh = b_hh; a.w_s = w_s; a.b_s = b_s; a.tau = tau;
  a.ksum = v.ksum_bf16; a.vsum = v.vsum_bf16; a.scores = v.scores; a.lstm_h = v.lstm_h; a.lstm_c = v.lstm_c;
  a.keep_idx = v.keep_idx; a.keep_cnt = v.keep_cnt; a.n_listed = v.n_listed; a.kept_k = kept_k; a.kept_v = kept_v;
  a.S = v.S; a.max_chunks = v.max_chunks; a.t = t;
  a.ticket = v.step_ticket; a.seq_len = v.seq_len; a.C = v.C; a.dev_window = dev_window;
  return planes == 3 ? launch_step_planes<3>(a, d_g, st) : launch_step_planes<2>(a, d_g, st);
}

}  // namespace kve

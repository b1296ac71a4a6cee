// LSTM recurrence + score head of the gate (Eq. 3): for every sequence, chunks oldest first,
//   pre_t = P_t + W_hh h_{t-1};  i,f,o = sigmoid, g = tanh;  c_t = f c_{t-1} + i g;  h_t = o tanh(c_t)
//   s_t   = sigmoid(w_s . h_t + b_s)
// P_t (= W_ih x_t + b_ih + b_hh) comes from the projection GEMM.
//
// The chain over t is strictly sequential, so the kernel is built for latency per step:
//  * A thread-block cluster of CL CTAs owns NS = 8*NT sequences for all steps.  Each CTA owns
//    HU = d_g / CL hidden units, i.e. 4*HU rows of W_hh, and keeps them in REGISTERS as mma A
//    fragments for the whole kernel (128 registers per thread at d_g = 256, CL = 4).
//  * Per step the CTA computes its rows of W_hh h for all its sequences with warp-level tensor-core
//    MMAs (m16n8k16, bf16 x bf16 -> fp32).  W_hh is bf16 by definition; the fp32 state h is split
//    exactly into three bf16 planes (h = hi + mid + lo), so the products are exact and only the
//    accumulation order differs from a plain fp32 loop.
//  * MMA rows are ordered so that one thread ends up holding the i, f, g, o pre-activations of the
//    same (hidden unit, sequence): the cell update is thread-local, c lives in registers.
//  * New h values are split into planes and stored into the shared memory of every CTA of the
//    cluster (distributed shared memory, double-buffered), one cluster barrier per step.
//  * Per-warp partial dot products of the score head go to CTA 0 of the cluster, which adds them in a
//    fixed order (deterministic) and writes s_t.
#include "common.cuh"
#include "kernels.h"

namespace kve {

constexpr int RNN_WARPS = 8;
constexpr int RNN_THREADS = RNN_WARPS * 32;
constexpr int RNN_PLANES = 3;

struct RnnArgs {
  const float* P;          // [S * n_range][4 d_g]
  const uint16_t* W_hh;    // bf16 [4 d_g][d_g]
  const float* w_s;        // [d_g]
  float b_s;
  float* scores;           // [S][max_chunks]
  float* lstm_h;           // [S][d_g]
  float* lstm_c;
  int S, max_chunks, t0, n_range, reset;
};

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_cluster_u32(uint32_t addr, uint32_t val) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(val) : "memory");
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float val) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(val) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ float fast_sigmoid(float x) { return __fdividef(1.f, 1.f + __expf(-x)); }
__device__ __forceinline__ float fast_tanh(float x) { return 2.f * fast_sigmoid(2.f * x) - 1.f; }

// exact 3-way split of an fp32 value into bf16 pieces: x = p0 + p1 + p2
__device__ __forceinline__ void split3(float x, uint32_t (&p)[3]) {
  p[0] = f32_to_bf16_bits(x);
  const float r1 = x - __uint_as_float(p[0] << 16);
  p[1] = f32_to_bf16_bits(r1);
  const float r2 = r1 - __uint_as_float(p[1] << 16);
  p[2] = f32_to_bf16_bits(r2);
}

template <int DG, int CL, int NT>
__global__ void __cluster_dims__(CL, 1, 1) __launch_bounds__(RNN_THREADS, 1) kve_gate_rnn_kernel(RnnArgs a) {
  constexpr int HU = DG / CL;            // hidden units owned by this CTA
  constexpr int UW = HU / RNN_WARPS;     // hidden units per warp
  constexpr int MP = UW / 8;             // pairs of m16 tiles per warp (a pair = 8 units x 4 gates)
  constexpr int KT = DG / 16;            // k tiles
  constexpr int NS = 8 * NT;             // sequences per cluster
  constexpr int LDH = DG + 8;            // padded plane row (bf16 elements): conflict-free B fragments
  static_assert(UW % 8 == 0 && MP >= 1, "8 warps x 8k hidden units per CTA");
  static_assert(CL * RNN_WARPS <= 32, "score partials fit one warp");

  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint16_t* hs = reinterpret_cast<uint16_t*>(smem_raw);                                   // [2][PLANES][NS][LDH]
  float* spart = reinterpret_cast<float*>(smem_raw + 2 * RNN_PLANES * NS * LDH * 2);      // [2][NS][32]
  constexpr int HS_BUF = RNN_PLANES * NS * LDH;   // elements per buffer

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, tig = lane & 3;
  const uint32_t rank = cluster_rank();
  const int cid = blockIdx.x / CL;
  const int seq0 = cid * NS;

  // ---- W_hh rows of this CTA as A fragments, resident in registers --------------------------------
  uint32_t A[2 * MP][KT][4];
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
  float wsu[MP];
#pragma unroll
  for (int p = 0; p < MP; ++p) wsu[p] = a.w_s[(int)rank * HU + warp * UW + p * 8 + g];

  // ---- initial state ---------------------------------------------------------------------------
  // every CTA needs the full h of its sequences (all d_g units) as planes in buffer 0
  for (int i = tid; i < NS * (DG / 2); i += RNN_THREADS) {
    const int j = i / (DG / 2), k2 = i % (DG / 2);
    const int s = seq0 + j;
    float h0 = 0.f, h1 = 0.f;
    if (!a.reset && s < a.S) {
      const float2 hv = *reinterpret_cast<const float2*>(a.lstm_h + (long long)s * DG + k2 * 2);
      h0 = hv.x; h1 = hv.y;
    }
    uint32_t p0[3], p1[3];
    split3(h0, p0);
    split3(h1, p1);
#pragma unroll
    for (int pl = 0; pl < RNN_PLANES; ++pl)
      *reinterpret_cast<uint32_t*>(hs + (pl * NS + j) * LDH + k2 * 2) = p0[pl] | (p1[pl] << 16);
  }
  float c[MP][NT][2], hlast[MP][NT][2];
#pragma unroll
  for (int p = 0; p < MP; ++p)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int s = seq0 + nt * 8 + tig * 2 + e;
        const int ug = (int)rank * HU + warp * UW + p * 8 + g;
        const bool live = !a.reset && s < a.S;
        c[p][nt][e] = live ? a.lstm_c[(long long)s * DG + ug] : 0.f;
        hlast[p][nt][e] = live ? a.lstm_h[(long long)s * DG + ug] : 0.f;
      }
  // all CTAs of the cluster are running and have filled buffer 0 before anyone writes remotely
  cluster_sync_all();

  const int n_cols = 4 * DG;
  for (int step = 0; step < a.n_range; ++step) {
    const int buf = step & 1;
    // ---- P_t for this thread's (unit, gate, sequence) entries; prefetch P_{t+1} into L2 ----------
    float pin[MP][NT][4][2];
#pragma unroll
    for (int p = 0; p < MP; ++p)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int s = seq0 + nt * 8 + tig * 2 + e;
          const int ug = (int)rank * HU + warp * UW + p * 8 + g;
          const float* prow = a.P + ((long long)s * a.n_range + step) * n_cols + ug;
#pragma unroll
          for (int gate = 0; gate < 4; ++gate) pin[p][nt][gate][e] = (s < a.S) ? __ldcs(prow + gate * DG) : 0.f;
          if (s < a.S && step + 1 < a.n_range) {
#pragma unroll
            for (int gate = 0; gate < 4; ++gate)
              asm volatile("prefetch.global.L2 [%0];" ::"l"(prow + n_cols + gate * DG));
          }
        }

    // ---- W_hh h_{t-1} on the tensor cores ---------------------------------------------------------
    float acc[2 * MP][NT][4];
#pragma unroll
    for (int mt = 0; mt < 2 * MP; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0.f;
    const uint16_t* hb = hs + buf * HS_BUF;
#pragma unroll
    for (int kt = 0; kt < KT; ++kt) {
#pragma unroll
      for (int pl = RNN_PLANES - 1; pl >= 0; --pl) {     // smallest plane first
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const uint32_t* brow = reinterpret_cast<const uint32_t*>(hb + (pl * NS + nt * 8 + g) * LDH + kt * 16);
          const uint32_t b0 = brow[tig], b1 = brow[4 + tig];
#pragma unroll
          for (int mt = 0; mt < 2 * MP; ++mt) mma_bf16_16816(acc[mt][nt], A[mt][kt], b0, b1);
        }
      }
    }

    // ---- cell update (thread-local), h exchange, score partials ----------------------------------
    float spv[NT][2];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) spv[nt][0] = spv[nt][1] = 0.f;
    uint16_t* hn = hs + (buf ^ 1) * HS_BUF;
#pragma unroll
    for (int p = 0; p < MP; ++p) {
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        float hv[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const float ig = fast_sigmoid(acc[2 * p][nt][e] + pin[p][nt][0][e]);
          const float fg = fast_sigmoid(acc[2 * p][nt][2 + e] + pin[p][nt][1][e]);
          const float gg = fast_tanh(acc[2 * p + 1][nt][e] + pin[p][nt][2][e]);
          const float og = fast_sigmoid(acc[2 * p + 1][nt][2 + e] + pin[p][nt][3][e]);
          const float cn = fmaf(fg, c[p][nt][e], ig * gg);
          c[p][nt][e] = cn;
          hv[e] = og * fast_tanh(cn);
          hlast[p][nt][e] = hv[e];
          spv[nt][e] = fmaf(wsu[p], hv[e], spv[nt][e]);
        }
        // pair up neighbouring units (g even / odd) so each thread stores 2 units of one sequence
        const bool odd = g & 1;
        const float other = __shfl_xor_sync(0xffffffffu, odd ? hv[0] : hv[1], 4);
        const float lo_unit = odd ? other : hv[0];
        const float hi_unit = odd ? hv[1] : other;
        const int j = nt * 8 + tig * 2 + (odd ? 1 : 0);
        const int k = (int)rank * HU + warp * UW + p * 8 + (g & ~1);
        uint32_t pl0[3], pl1[3];
        split3(lo_unit, pl0);
        split3(hi_unit, pl1);
#pragma unroll
        for (int pl = 0; pl < RNN_PLANES; ++pl) {
          const uint32_t word = pl0[pl] | (pl1[pl] << 16);
          const uint32_t local = smem_u32(hn + (pl * NS + j) * LDH + k);
#pragma unroll
          for (int r = 0; r < CL; ++r) st_cluster_u32(map_to_rank(local, r), word);
        }
      }
    }
    // reduce score partials over the 8 units of the warp's lane groups (lanes differ in g)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        float vsum = spv[nt][e];
        vsum += __shfl_xor_sync(0xffffffffu, vsum, 4);
        vsum += __shfl_xor_sync(0xffffffffu, vsum, 8);
        vsum += __shfl_xor_sync(0xffffffffu, vsum, 16);
        if (g == 0) {
          const int j = nt * 8 + tig * 2 + e;
          const uint32_t local = smem_u32(spart + (buf * NS + j) * 32 + (int)rank * RNN_WARPS + warp);
          st_cluster_f32(map_to_rank(local, 0), vsum);
        }
      }

    cluster_sync_all();   // h_t planes and score partials are visible everywhere

    if (rank == 0) {
      for (int j = warp; j < NS; j += RNN_WARPS) {
        float vsum = (lane < CL * RNN_WARPS) ? spart[(buf * NS + j) * 32 + lane] : 0.f;
        vsum = warp_sum(vsum);
        const int s = seq0 + j;
        if (lane == 0 && s < a.S) {
          const float z = vsum + a.b_s;
          a.scores[(long long)s * a.max_chunks + a.t0 + step] = 1.f / (1.f + expf(-z));
        }
      }
    }
  }

  // ---- carried state out ---------------------------------------------------------------------------
#pragma unroll
  for (int p = 0; p < MP; ++p)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int s = seq0 + nt * 8 + tig * 2 + e;
        const int ug = (int)rank * HU + warp * UW + p * 8 + g;
        if (s < a.S) {
          a.lstm_c[(long long)s * DG + ug] = c[p][nt][e];
          a.lstm_h[(long long)s * DG + ug] = hlast[p][nt][e];
        }
      }
}

template <int DG, int CL, int NT>
static cudaError_t launch_rnn_t(const RnnArgs& a, cudaStream_t st) {
  constexpr int NS = 8 * NT;
  constexpr int smem = 2 * RNN_PLANES * NS * (DG + 8) * 2 + 2 * NS * 32 * 4;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(kve_gate_rnn_kernel<DG, CL, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const int clusters = (a.S + NS - 1) / NS;
  kve_gate_rnn_kernel<DG, CL, NT><<<clusters * CL, RNN_THREADS, smem, st>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_gate_rnn(const LayerView& v, int t0, int t1, const uint16_t* W_hh, const float* w_s, float b_s,
                            int d_g, const float* P, bool reset_state, cudaStream_t st) {
  if (t1 <= t0 || v.S <= 0) return cudaSuccess;
  RnnArgs a;
  a.P = P; a.W_hh = W_hh; a.w_s = w_s; a.b_s = b_s;
  a.scores = v.scores; a.lstm_h = v.lstm_h; a.lstm_c = v.lstm_c;
  a.S = v.S; a.max_chunks = v.max_chunks; a.t0 = t0; a.n_range = t1 - t0; a.reset = reset_state ? 1 : 0;
  // 16 sequences per cluster once 8 per cluster would need more than one wave of clusters
  switch (d_g) {
    case 256: return (v.S > 8 * (148 / 4)) ? launch_rnn_t<256, 4, 2>(a, st) : launch_rnn_t<256, 4, 1>(a, st);
    case 128: return launch_rnn_t<128, 1, 1>(a, st);
    case 64:  return (v.S > 8 * 148) ? launch_rnn_t<64, 1, 2>(a, st) : launch_rnn_t<64, 1, 1>(a, st);
    default:  return cudaErrorInvalidValue;
  }
}

}  // namespace kve

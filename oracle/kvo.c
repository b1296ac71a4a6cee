/*
 * kvo — the ORACLE for the RNN-gated chunked KV cache (test infrastructure, not product code).
 *
 * A plain, slow, one-loop-per-sum CPU statement of what the method computes, written from the
 * paper's prose and equations (its pseudocode figure is not available).  It shares no code with
 * the CUDA library: only tests, the smoke check and the benchmark's cpu_baseline leg may call it.
 *
 * Arithmetic type: `real`, chosen at compile time (-DKVO_REAL=float or double).  The double build
 * is the mathematical reference; the float build takes every floating-point decision (bf16
 * rounding of summaries, score >= tau) in the precision the GPU kernels use.
 *
 * Data layout is the paper's plain one: the cache of a sequence s (one (batch, head) pair) is a
 * dense [n][d] matrix in temporal order, no paging.  K, V, q and the rounded summaries are bf16
 * bit patterns (uint16_t), the precision the paper states for the model; weights arrive as float
 * arrays whose values the caller has already made bf16-representable where that matters.
 *
 * Steps (names follow the paper):
 *   kvo_summarize   Sec. 3.2, Eq. 2 (aggregator; mean / mean->2-layer MLP / identity)
 *   kvo_gate        Sec. 3.2, Eq. 3 (LSTM over chunk summaries, score s_t in [0,1])
 *   kvo_compact     Sec. 3.2 retention rule "s_t >= tau"
 *   kvo_compact_topk  the top-k gating variant (Sec. 5 names gating strategies as an ablation)
 *   kvo_reclaim     Sec. 3.3 memory reduction: pages of gated chunks handed back
 *   kvo_attn        Sec. 3.3 attention over window + retained chunks, with Eq. 1 as the softmax
 *   kvo_attn_dense  Eq. 1 over the full cache (the baseline of Sec. 3.3)
 *
 * Every open choice of the paper (aggregator form, activation, score head, threshold sense,
 * window handling, rounding points) is listed with its reading in oracle/README.md.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifndef KVO_REAL
#define KVO_REAL double
#endif
typedef KVO_REAL real;

#define KVO_AGG_MEAN 0
#define KVO_AGG_MLP 1
#define KVO_AGG_IDENTITY 2
#define KVO_AGG_MAX 3
#define KVO_AGG_TOKEN_MLP 4
#define KVO_ATTEND_SUMMARY 0
#define KVO_ATTEND_RAW 1

int kvo_real_bytes(void) { return (int)sizeof(real); }

/* ---- bf16 <-> real ------------------------------------------------------------------------ */

/* widen a bf16 bit pattern: exact */
static real bf16_to_real(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, 4);
  return (real)f;
}

/* round-to-nearest-even to bf16 (8 significant bits, float's exponent range), straight from the
 * wide value so the double build never rounds twice */
static uint16_t real_to_bf16(real xr) {
  double x = (double)xr;
  uint16_t sign = (uint16_t)(signbit(x) ? 0x8000u : 0u);
  if (isnan(x)) return 0x7fc0u;
  if (isinf(x)) return (uint16_t)(sign | 0x7f80u);
  double a = fabs(x);
  if (a == 0.0) return sign;
  int e;
  (void)frexp(a, &e);                 /* a = m * 2^e, m in [0.5, 1) */
  int qexp = e - 8;                   /* spacing of 8-significant-bit numbers around a */
  if (qexp < -133) qexp = -133;       /* bf16 subnormal spacing 2^-133 */
  double q = nearbyint(ldexp(a, -qexp));   /* default rounding mode = ties to even */
  double r = ldexp(q, qexp);
  if (r >= ldexp(1.0, 128)) return (uint16_t)(sign | 0x7f80u);
  float f = (float)r;                 /* exact: r has at most 8 significant bits */
  uint32_t u;
  memcpy(&u, &f, 4);
  return (uint16_t)(sign | (uint16_t)(u >> 16));
}

uint16_t kvo_bf16_rne(double x) { return real_to_bf16((real)x); }
double kvo_bf16_widen(uint16_t b) { return (double)bf16_to_real(b); }

/* ---- small pieces ------------------------------------------------------------------------- */

static real sigmoid_r(real x) { return (real)1 / ((real)1 + (real)exp((double)-x)); }

/* exact (erf) form of GELU: x * Phi(x) */
static real gelu_erf(real x) {
  return (real)0.5 * x * ((real)1 + (real)erf((double)x * 0.70710678118654752440));
}

/* y = W2 * gelu(W1 * m + b1) + b2 ; W1 [d_sum][d], W2 [d][d_sum], row-major */
static void mlp2(const real* m, int d, int d_sum, const float* W1, const float* b1,
                 const float* W2, const float* b2, real* hid, real* y) {
  for (int u = 0; u < d_sum; ++u) {
    real acc = 0;
    for (int x = 0; x < d; ++x) acc += (real)W1[(size_t)u * d + x] * m[x];
    hid[u] = gelu_erf(acc + (real)b1[u]);
  }
  for (int x = 0; x < d; ++x) {
    real acc = 0;
    for (int u = 0; u < d_sum; ++u) acc += (real)W2[(size_t)x * d_sum + u] * hid[u];
    y[x] = acc + (real)b2[x];
  }
}

/* ---- Eq. 2: one representative (Kbar_t, Vbar_t) per chunk --------------------------------- */
/*
 * K, V        [S][n][d] bf16
 * chunks      t in [t0, t1), chunk t = tokens [t*C, (t+1)*C); caller guarantees t1*C <= n
 * agg         MEAN: Kbar = (1/C) sum_j k_j
 *             MLP : Kbar = MLP_K(mean), Vbar = MLP_V(mean)  (2 layers, hidden d_sum, erf-GELU)
 *             IDENTITY (C == 1 only): Kbar = k
 *             MAX : Kbar = element-wise maximum of the chunk's keys ("pooling", Sec. 3.1), Vbar likewise
 *             TOKEN_MLP: Eq. 2 taken literally, the MLP acting on every element of the set {k_j}:
 *                   y_j = MLP_K(k_j) for each of the C tokens, Kbar = (1/C) sum_j y_j  (mean-pool of the outputs)
 * outputs     ksum, vsum [S][stride][d] real at row t; *_b16 the same values rounded to bf16
 * returns 0, or -1 on a bad argument
 */
int kvo_summarize(const uint16_t* K, const uint16_t* V, int S, int n, int d, int C, int t0, int t1,
                  int agg, int d_sum,
                  const float* W1K, const float* b1K, const float* W2K, const float* b2K,
                  const float* W1V, const float* b1V, const float* W2V, const float* b2V,
                  int stride, real* ksum, real* vsum, uint16_t* ksum_b16, uint16_t* vsum_b16) {
  if (S < 0 || n < 0 || d <= 0 || C <= 0 || t0 < 0 || t1 < t0 || (long)t1 * C > n || t1 > stride)
    return -1;
  if (agg == KVO_AGG_IDENTITY && C != 1) return -1;
  if ((agg == KVO_AGG_MLP || agg == KVO_AGG_TOKEN_MLP) &&
      (d_sum <= 0 || !W1K || !b1K || !W2K || !b2K || !W1V || !b1V || !W2V || !b2V))
    return -1;
  if (agg != KVO_AGG_MEAN && agg != KVO_AGG_MLP && agg != KVO_AGG_IDENTITY && agg != KVO_AGG_MAX &&
      agg != KVO_AGG_TOKEN_MLP)
    return -1;
#pragma omp parallel for schedule(static)
  for (int s = 0; s < S; ++s) {
    real* mk = (real*)malloc(sizeof(real) * (size_t)d);
    real* mv = (real*)malloc(sizeof(real) * (size_t)d);
    real* yk = (real*)malloc(sizeof(real) * (size_t)d);
    real* yv = (real*)malloc(sizeof(real) * (size_t)d);
    real* tk = (real*)malloc(sizeof(real) * (size_t)d);
    real* tv = (real*)malloc(sizeof(real) * (size_t)d);
    real* hid = (real*)malloc(sizeof(real) * (size_t)(d_sum > 0 ? d_sum : 1));
    for (int t = t0; t < t1; ++t) {
      for (int x = 0; x < d; ++x) {
        real sk = 0, sv = 0;
        for (int j = 0; j < C; ++j) {
          size_t row = ((size_t)s * n + (size_t)t * C + j) * d;
          sk += bf16_to_real(K[row + x]);
          sv += bf16_to_real(V[row + x]);
        }
        mk[x] = sk / (real)C;
        mv[x] = sv / (real)C;
        if (agg == KVO_AGG_MAX) {          /* max-pool: the largest entry of the chunk in each dimension (exact) */
          size_t row0 = ((size_t)s * n + (size_t)t * C) * d;
          real bk = bf16_to_real(K[row0 + x]), bv = bf16_to_real(V[row0 + x]);
          for (int j = 1; j < C; ++j) {
            real a = bf16_to_real(K[row0 + (size_t)j * d + x]), b = bf16_to_real(V[row0 + (size_t)j * d + x]);
            if (a > bk) bk = a;
            if (b > bv) bv = b;
          }
          mk[x] = bk;
          mv[x] = bv;
        }
      }
      const real *ok = mk, *ov = mv;
      if (agg == KVO_AGG_MLP) {
        mlp2(mk, d, d_sum, W1K, b1K, W2K, b2K, hid, yk);
        mlp2(mv, d, d_sum, W1V, b1V, W2V, b2V, hid, yv);
        ok = yk;
        ov = yv;
      }
      if (agg == KVO_AGG_TOKEN_MLP) {      /* the MLP on each token, then the mean of the C outputs */
        for (int x = 0; x < d; ++x) yk[x] = yv[x] = 0;
        for (int j = 0; j < C; ++j) {
          size_t row = ((size_t)s * n + (size_t)t * C + j) * d;
          for (int x = 0; x < d; ++x) {      /* the token itself (mk, mv reused as the MLP input) */
            mk[x] = bf16_to_real(K[row + x]);
            mv[x] = bf16_to_real(V[row + x]);
          }
          mlp2(mk, d, d_sum, W1K, b1K, W2K, b2K, hid, tk);
          mlp2(mv, d, d_sum, W1V, b1V, W2V, b2V, hid, tv);
          for (int x = 0; x < d; ++x) {
            yk[x] += tk[x];
            yv[x] += tv[x];
          }
        }
        for (int x = 0; x < d; ++x) {
          yk[x] = yk[x] / (real)C;
          yv[x] = yv[x] / (real)C;
        }
        ok = yk;
        ov = yv;
      }
      size_t o = ((size_t)s * stride + t) * d;
      for (int x = 0; x < d; ++x) {
        ksum[o + x] = ok[x];
        vsum[o + x] = ov[x];
        ksum_b16[o + x] = real_to_bf16(ok[x]);
        vsum_b16[o + x] = real_to_bf16(ov[x]);
      }
    }
    free(mk); free(mv); free(yk); free(yv); free(tk); free(tv); free(hid);
  }
  return 0;
}

/* ---- Eq. 3: h_t, s_t = LSTM([Kbar_t, Vbar_t], h_{t-1}) ------------------------------------ */
/*
 * One standard LSTM layer, gate rows ordered i, f, g, o; input x_t = [Kbar_t ; Vbar_t] taken from
 * the bf16-rounded summaries (2d values); score s_t = sigmoid(w_s . h_t + b_s).
 * Chunks are fed oldest first, every chunk passes through whether it is later kept or not.
 * h, c [S][d_g]: carried state, read at entry and left at the value after chunk t1-1
 * (the caller zeroes them before the first chunk).  scores [S][stride] written at t0..t1-1.
 */
int kvo_gate(const uint16_t* ksum_b16, const uint16_t* vsum_b16, int S, int stride, int d,
             int t0, int t1, int d_g,
             const float* W_ih, const float* W_hh, const float* b_ih, const float* b_hh,
             const float* w_s, float b_s, real* h, real* c, real* scores) {
  if (S < 0 || d <= 0 || d_g <= 0 || t0 < 0 || t1 < t0 || t1 > stride) return -1;
  const int in = 2 * d;
#pragma omp parallel for schedule(static)
  for (int s = 0; s < S; ++s) {
    real* x = (real*)malloc(sizeof(real) * (size_t)in);
    real* pre = (real*)malloc(sizeof(real) * (size_t)(4 * d_g));
    real* hs = h + (size_t)s * d_g;
    real* cs = c + (size_t)s * d_g;
    for (int t = t0; t < t1; ++t) {
      size_t o = ((size_t)s * stride + t) * d;
      for (int k = 0; k < d; ++k) {
        x[k] = bf16_to_real(ksum_b16[o + k]);
        x[d + k] = bf16_to_real(vsum_b16[o + k]);
      }
      for (int r = 0; r < 4 * d_g; ++r) {
        real ax = 0, ah = 0;
        for (int k = 0; k < in; ++k) ax += (real)W_ih[(size_t)r * in + k] * x[k];
        for (int k = 0; k < d_g; ++k) ah += (real)W_hh[(size_t)r * d_g + k] * hs[k];
        pre[r] = (ax + (real)b_ih[r]) + (ah + (real)b_hh[r]);
      }
      real dot = 0;
      for (int u = 0; u < d_g; ++u) {
        real ig = sigmoid_r(pre[u]);
        real fg = sigmoid_r(pre[d_g + u]);
        real gg = (real)tanh((double)pre[2 * d_g + u]);
        real og = sigmoid_r(pre[3 * d_g + u]);
        cs[u] = fg * cs[u] + ig * gg;
        hs[u] = og * (real)tanh((double)cs[u]);
      }
      for (int u = 0; u < d_g; ++u) dot += (real)w_s[u] * hs[u];
      scores[(size_t)s * stride + t] = sigmoid_r(dot + (real)b_s);
    }
    free(x); free(pre);
  }
  return 0;
}

/* ---- retention rule: keep chunk t iff s_t >= tau (inclusive) ------------------------------ */
/* keep_idx [S][stride]: ascending kept chunk ids, first keep_cnt[s] entries valid, rest -1 */
int kvo_compact(const real* scores, int S, int stride, int n_chunks, double tau,
                int32_t* keep_idx, int32_t* keep_cnt) {
  if (S < 0 || n_chunks < 0 || n_chunks > stride) return -1;
  const real tr = (real)tau;
  for (int s = 0; s < S; ++s) {
    int m = 0;
    for (int t = 0; t < n_chunks; ++t)
      if (scores[(size_t)s * stride + t] >= tr) keep_idx[(size_t)s * stride + m++] = t;
    keep_cnt[s] = m;
    for (int t = m; t < stride; ++t) keep_idx[(size_t)s * stride + t] = -1;
  }
  return 0;
}

/* ---- gating-strategy variant (Sec. 5, planned ablation): keep the k best chunks instead of thresholding ---- */
/*
 * keep chunk t iff fewer than k chunks rank before it, where u ranks before t when s_u > s_t, or
 * s_u == s_t and u < t (equal scores: the older chunk first, which makes the result unique).
 * Output as kvo_compact: ascending ids, count, -1 padding.  k <= 0 keeps nothing, k >= n_chunks all.
 */
int kvo_compact_topk(const real* scores, int S, int stride, int n_chunks, int k,
                     int32_t* keep_idx, int32_t* keep_cnt) {
  if (S < 0 || n_chunks < 0 || n_chunks > stride) return -1;
  for (int s = 0; s < S; ++s) {
    const real* sc = scores + (size_t)s * stride;
    int m = 0;
    for (int t = 0; t < n_chunks; ++t) {
      int before = 0;
      for (int u = 0; u < n_chunks; ++u)
        if (sc[u] > sc[t] || (sc[u] == sc[t] && u < t)) ++before;
      if (before < k) keep_idx[(size_t)s * stride + m++] = t;
    }
    keep_cnt[s] = m;
    for (int t = m; t < stride; ++t) keep_idx[(size_t)s * stride + t] = -1;
  }
  return 0;
}

/* ---- Sec. 3.3 / Sec. 4.2: the memory side of the method --------------------------------------- */
/*
 * Once a chunk has been summarised and gated, its raw tokens are no longer needed: a discarded
 * chunk is never attended to again, and a retained chunk is attended to through its one summary
 * row (n' = W + M rows instead of n, the memory ratio n / (W + M) of Sec. 3.3).  This returns the
 * pages of such chunks to the caller.
 *
 * page_table  [S][stride] page id of chunk t of sequence s; entries handed back become -1
 * scores      [S][stride]; chunk t is discarded iff scores < tau (the complement of kvo_compact)
 * chunks      t in [t0, t1)
 * mode        0: only discarded chunks give their page back (valid whatever attention reads)
 *             1: every chunk in the range does (valid when retained chunks are read as summaries)
 * free_list   receives the page ids, sequences in order, chunks ascending within a sequence;
 *             entries already -1 are skipped.  Returns the number written, or -1 on a bad argument.
 */
long kvo_reclaim(int32_t* page_table, const real* scores, int S, int stride, int t0, int t1,
                 double tau, int mode, int32_t* free_list) {
  if (S < 0 || t0 < 0 || t1 < t0 || t1 > stride || (mode != 0 && mode != 1)) return -1;
  const real tr = (real)tau;
  long m = 0;
  for (int s = 0; s < S; ++s)
    for (int t = t0; t < t1; ++t) {
      const size_t i = (size_t)s * stride + t;
      const int discarded = !(scores[i] >= tr);
      if ((mode == 1 || discarded) && page_table[i] >= 0) {
        free_list[m++] = page_table[i];
        page_table[i] = -1;
      }
    }
  return m;
}

/* ---- Eq. 1 over an explicit row list ------------------------------------------------------ */
/* two-pass softmax, max-subtracted; rows given as n_rows pointers to bf16 vectors of length d */
static void softmax_attend(const uint16_t* q, const uint16_t* const* krows, const uint16_t* const* vrows,
                           long n_rows, int d, real scale, real* out, uint16_t* out_b16, real* lse,
                           real* logit /* scratch [n_rows] */) {
  if (n_rows == 0) {
    for (int x = 0; x < d; ++x) { out[x] = 0; out_b16[x] = 0; }
    if (lse) *lse = (real)-INFINITY;
    return;
  }
  real mx = (real)-INFINITY;
  for (long r = 0; r < n_rows; ++r) {
    real acc = 0;
    for (int x = 0; x < d; ++x) acc += bf16_to_real(q[x]) * bf16_to_real(krows[r][x]);
    logit[r] = acc * scale;
    if (logit[r] > mx) mx = logit[r];
  }
  real den = 0;
  for (long r = 0; r < n_rows; ++r) {
    logit[r] = (real)exp((double)(logit[r] - mx));
    den += logit[r];
  }
  for (int x = 0; x < d; ++x) {
    real acc = 0;
    for (long r = 0; r < n_rows; ++r) acc += logit[r] * bf16_to_real(vrows[r][x]);
    out[x] = acc / den;
    out_b16[x] = real_to_bf16(out[x]);
  }
  if (lse) *lse = mx + (real)log((double)den);
}

/*
 * Attention of Sec. 3.3: rows = retained chunks (oldest first) followed by the raw tail.
 *   n_chunks   chunks [0, n_chunks) have been gated; tokens [n_chunks*C, n) are raw (window +
 *              trailing partial chunk) and are never transformed
 *   SUMMARY    a kept chunk t contributes ONE row (ksum_b16[t], vsum_b16[t])      n' = R + M
 *   RAW        a kept chunk t contributes its C raw rows                           n' = R + M*C
 * q [S][d] bf16; out [S][d] real, out_b16 rounded; lse [S] (nullable); n_eff [S] = n' (nullable)
 */
int kvo_attn(const uint16_t* q, const uint16_t* K, const uint16_t* V, int S, int n, int d, int C,
             int n_chunks, const int32_t* keep_idx, const int32_t* keep_cnt,
             const uint16_t* ksum_b16, const uint16_t* vsum_b16, int stride, int attend,
             double scale, real* out, uint16_t* out_b16, real* lse, int64_t* n_eff) {
  if (S < 0 || n < 0 || d <= 0 || C <= 0 || n_chunks < 0 || (long)n_chunks * C > n || n_chunks > stride)
    return -1;
  if (attend != KVO_ATTEND_SUMMARY && attend != KVO_ATTEND_RAW) return -1;
  int bad = 0;
#pragma omp parallel for schedule(static)
  for (int s = 0; s < S; ++s) {
    const int m = keep_cnt[s];
    const long raw0 = (long)n_chunks * C;
    const long per = (attend == KVO_ATTEND_RAW) ? C : 1;
    const long n_rows = (long)m * per + (n - raw0);
    const uint16_t** kr = (const uint16_t**)malloc(sizeof(void*) * (size_t)(n_rows > 0 ? n_rows : 1));
    const uint16_t** vr = (const uint16_t**)malloc(sizeof(void*) * (size_t)(n_rows > 0 ? n_rows : 1));
    real* logit = (real*)malloc(sizeof(real) * (size_t)(n_rows > 0 ? n_rows : 1));
    long r = 0;
    for (int i = 0; i < m; ++i) {
      int t = keep_idx[(size_t)s * stride + i];
      if (t < 0 || t >= n_chunks) { bad = 1; t = 0; }
      if (attend == KVO_ATTEND_RAW) {
        for (int j = 0; j < C; ++j, ++r) {
          kr[r] = K + ((size_t)s * n + (size_t)t * C + j) * d;
          vr[r] = V + ((size_t)s * n + (size_t)t * C + j) * d;
        }
      } else {
        kr[r] = ksum_b16 + ((size_t)s * stride + t) * d;
        vr[r] = vsum_b16 + ((size_t)s * stride + t) * d;
        ++r;
      }
    }
    for (long p = raw0; p < n; ++p, ++r) {
      kr[r] = K + ((size_t)s * n + p) * d;
      vr[r] = V + ((size_t)s * n + p) * d;
    }
    softmax_attend(q + (size_t)s * d, kr, vr, n_rows, d, (real)scale, out + (size_t)s * d,
                   out_b16 + (size_t)s * d, lse ? lse + s : NULL, logit);
    if (n_eff) n_eff[s] = n_rows;
    free(kr); free(vr); free(logit);
  }
  return bad ? -2 : 0;
}

/* Eq. 1 over all n cached positions */
int kvo_attn_dense(const uint16_t* q, const uint16_t* K, const uint16_t* V, int S, int n, int d,
                   double scale, real* out, uint16_t* out_b16, real* lse) {
  if (S < 0 || n < 0 || d <= 0) return -1;
#pragma omp parallel for schedule(static)
  for (int s = 0; s < S; ++s) {
    const uint16_t** kr = (const uint16_t**)malloc(sizeof(void*) * (size_t)(n > 0 ? n : 1));
    const uint16_t** vr = (const uint16_t**)malloc(sizeof(void*) * (size_t)(n > 0 ? n : 1));
    real* logit = (real*)malloc(sizeof(real) * (size_t)(n > 0 ? n : 1));
    for (long p = 0; p < n; ++p) {
      kr[p] = K + ((size_t)s * n + p) * d;
      vr[p] = V + ((size_t)s * n + p) * d;
    }
    softmax_attend(q + (size_t)s * d, kr, vr, n, d, (real)scale, out + (size_t)s * d,
                   out_b16 + (size_t)s * d, lse ? lse + s : NULL, logit);
    free(kr); free(vr); free(logit);
  }
  return 0;
}

/*
 * rocs_ref.c -- CPU oracle for the ROCS request-candidate layers.
 *
 * TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only tests, the smoke check and the
 * benchmark's cpu_baseline / reference legs may load this library.  It shares no
 * code with the CUDA path and is deliberately plain and slow: every operator is
 * evaluated in its MATERIALISED-BROADCAST form (the request tensors are
 * replicated into a per-candidate buffer, exactly what the paper's "dense
 * implementation" does, Section 4 first paragraph) and all arithmetic is fp64
 * in index order.  Inputs are read in their storage type (bf16 bits, fp32 or
 * fp64; widening to fp64 is exact) and every result is written as fp64.
 *
 * Parity pins (tests/test_oracle_*.py): numpy / torch library routines on the
 * special cases that reduce to them, closed forms, the GLM invariant (Eq. 1),
 * the sharing identity (Eq. 11), decomposed form == materialised form (Eq. 14,
 * Section 4.1) and pure-Python brute force on tiny inputs.  The paper prints no
 * numeric worked example of any operator, so parity against printed values is
 * "parity unpinned"; the definitions and invariants above are the pins.
 *
 * The *_decomposed / *_shared functions evaluate the request-once forms of
 * Section 4.1; they exist only so the tests can check that both forms agree.
 *
 * Threads: OpenMP over candidates (they are independent, Eq. 1), nothing else.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { REF_BF16 = 0, REF_F32 = 1, REF_F64 = 2 };

static double load_as_f64(const void *p, int dtype, int64_t idx) {
  if (dtype == REF_BF16) {
    uint32_t bits = ((uint32_t)((const uint16_t *)p)[idx]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
  }
  if (dtype == REF_F32) return (double)((const float *)p)[idx];
  return ((const double *)p)[idx];
}

int rocs_ref_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* The index map m of Section 4.1: m[i] = request of candidate i, for candidates
 * stored consecutively per request (cand_offsets[r] .. cand_offsets[r+1]-1). */
static int32_t *materialise_index_map(int32_t R, int64_t N, const int32_t *cand_offsets) {
  int32_t *m = (int32_t *)malloc(sizeof(int32_t) * (size_t)(N > 0 ? N : 1));
  if (!m) return NULL;
  for (int32_t r = 0; r < R; ++r)
    for (int64_t i = cand_offsets[r]; i < cand_offsets[r + 1]; ++i) m[i] = r;
  return m;
}

static int64_t pick(const int64_t *sample, int64_t s) { return sample ? sample[s] : s; }

/* ------------------------------------------------------------------------- *
 * GLM linear, two groups (Eq. 4):  y^C = W_CR x^R + W_CC x^C + b, then the
 * pointwise activation (Eq. 8).  Materialised form: u = [x^R[m_i] ; x^C[i]] is
 * built per candidate and multiplied by the block row [W_CR | W_CC].
 * W is [d_out, d_req + d_cand] row-major.  Y is [n_out_rows, d_out] fp64 where
 * row s is candidate sample[s] (or s when sample == NULL).
 * act: 0 none, 1 ReLU.  bias may be NULL.
 * ------------------------------------------------------------------------- */
int rocs_ref_ikbo_linear(int dtype, int32_t R, int64_t N, const int32_t *cand_offsets,
                         int32_t d_req, int32_t d_cand, int32_t d_out, const void *XR,
                         const void *XC, const void *W, const double *bias, int act,
                         const int64_t *sample, int64_t n_sample, double *Y) {
  int32_t *m = materialise_index_map(R, N, cand_offsets);
  if (!m) return -1;
  const int64_t rows = sample ? n_sample : N;
  const int32_t d_in = d_req + d_cand;
#pragma omp parallel
  {
    double *u = (double *)malloc(sizeof(double) * (size_t)(d_in > 0 ? d_in : 1));
#pragma omp for schedule(dynamic, 16)
    for (int64_t s = 0; s < rows; ++s) {
      const int64_t i = pick(sample, s);
      const int32_t r = m[i];
      for (int32_t k = 0; k < d_req; ++k) u[k] = load_as_f64(XR, dtype, (int64_t)r * d_req + k);
      for (int32_t k = 0; k < d_cand; ++k) u[d_req + k] = load_as_f64(XC, dtype, i * d_cand + k);
      for (int32_t o = 0; o < d_out; ++o) {
        double acc = 0.0;
        for (int32_t k = 0; k < d_in; ++k) acc += load_as_f64(W, dtype, (int64_t)o * d_in + k) * u[k];
        if (bias) acc += bias[o];
        if (act == 1 && acc < 0.0) acc = 0.0;
        Y[s * d_out + o] = acc;
      }
    }
    free(u);
  }
  free(m);
  return 0;
}

/* Request-once form (Section 4.1): Z = W_CR X^R at batch size R, then
 * Y_i = Z[m_i] + W_CC X^C_i (Eq. 14).  Z (fp64 [R, d_out], includes the bias) is
 * returned as well.  Used by tests to check Eq. 14 against the form above. */
int rocs_ref_ikbo_linear_decomposed(int dtype, int32_t R, int64_t N, const int32_t *cand_offsets,
                                    int32_t d_req, int32_t d_cand, int32_t d_out, const void *XR,
                                    const void *XC, const void *W, const double *bias, int act,
                                    double *Z, double *Y) {
  const int32_t d_in = d_req + d_cand;
  for (int32_t r = 0; r < R; ++r)
    for (int32_t o = 0; o < d_out; ++o) {
      double acc = 0.0;
      for (int32_t k = 0; k < d_req; ++k)
        acc += load_as_f64(W, dtype, (int64_t)o * d_in + k) * load_as_f64(XR, dtype, (int64_t)r * d_req + k);
      if (bias) acc += bias[o];
      Z[(int64_t)r * d_out + o] = acc;
    }
  for (int32_t r = 0; r < R; ++r)
    for (int64_t i = cand_offsets[r]; i < cand_offsets[r + 1]; ++i)
      for (int32_t o = 0; o < d_out; ++o) {
        double acc = 0.0;
        for (int32_t k = 0; k < d_cand; ++k)
          acc += load_as_f64(W, dtype, (int64_t)o * d_in + d_req + k) * load_as_f64(XC, dtype, i * d_cand + k);
        acc += Z[(int64_t)r * d_out + o];
        if (act == 1 && acc < 0.0) acc = 0.0;
        Y[i * d_out + o] = acc;
      }
  return 0;
}

/* ------------------------------------------------------------------------- *
 * Group-wise cross attention, candidate side (Eq. 13):
 *   A^C = Attn(Q^C, K, V) with K = S W_K, V = S W_V of the candidate's request.
 * Attn is scaled dot-product attention with a softmax over the request's
 * sequence positions, per head.  Materialised form: the request's K and V are
 * copied into candidate-batched buffers K_i, V_i first (Section 4.3, second
 * paragraph), then plain attention runs on the copies.
 * Q [N, n_q, H, dh]; K, V [T, H, dh] packed, request r owns sequence rows
 * seq_offsets[r] .. seq_offsets[r+1]-1.  O [rows, n_q, H, dh] fp64.
 * A request with an empty sequence yields zeros.
 * ------------------------------------------------------------------------- */
int rocs_ref_dca_attention(int dtype, int32_t R, int64_t N, const int32_t *cand_offsets,
                           const int32_t *seq_offsets, int32_t n_q, int32_t H, int32_t dh,
                           double scale, const void *Q, const void *K, const void *V,
                           const int64_t *sample, int64_t n_sample, double *O) {
  int32_t *m = materialise_index_map(R, N, cand_offsets);
  if (!m) return -1;
  const int64_t rows = sample ? n_sample : N;
  const int64_t hd = (int64_t)H * dh;
  int failed = 0;
#pragma omp parallel
  {
#pragma omp for schedule(dynamic, 1)
    for (int64_t s = 0; s < rows; ++s) {
      const int64_t i = pick(sample, s);
      const int32_t r = m[i];
      const int64_t t0 = seq_offsets[r];
      const int32_t L = seq_offsets[r + 1] - seq_offsets[r];
      /* candidate-batched copies of the request's K and V */
      double *Ki = (double *)malloc(sizeof(double) * (size_t)(L > 0 ? L * hd : 1));
      double *Vi = (double *)malloc(sizeof(double) * (size_t)(L > 0 ? L * hd : 1));
      double *p = (double *)malloc(sizeof(double) * (size_t)(L > 0 ? L : 1));
      if (!Ki || !Vi || !p) {
        failed = 1;
      } else {
        for (int64_t e = 0; e < (int64_t)L * hd; ++e) {
          Ki[e] = load_as_f64(K, dtype, t0 * hd + e);
          Vi[e] = load_as_f64(V, dtype, t0 * hd + e);
        }
        for (int32_t t = 0; t < n_q; ++t)
          for (int32_t h = 0; h < H; ++h) {
            double *o = O + ((s * n_q + t) * H + h) * dh;
            for (int32_t e = 0; e < dh; ++e) o[e] = 0.0;
            if (L == 0) continue;
            const int64_t qbase = ((i * n_q + t) * H + h) * dh;
            double smax = -INFINITY;
            for (int32_t j = 0; j < L; ++j) {
              double dot = 0.0;
              for (int32_t e = 0; e < dh; ++e)
                dot += load_as_f64(Q, dtype, qbase + e) * Ki[(int64_t)j * hd + (int64_t)h * dh + e];
              p[j] = scale * dot;
              if (p[j] > smax) smax = p[j];
            }
            double denom = 0.0;
            for (int32_t j = 0; j < L; ++j) {
              p[j] = exp(p[j] - smax);
              denom += p[j];
            }
            for (int32_t j = 0; j < L; ++j) {
              const double w = p[j] / denom;
              for (int32_t e = 0; e < dh; ++e) o[e] += w * Vi[(int64_t)j * hd + (int64_t)h * dh + e];
            }
          }
      }
      free(Ki);
      free(Vi);
      free(p);
    }
  }
  free(m);
  return failed ? -1 : 0;
}

/* Shared form (Section 4.3.1): candidates index the request's K/V in place
 * through m_i; nothing is copied.  Only for the both-forms-agree test. */
int rocs_ref_dca_attention_shared(int dtype, int32_t R, int64_t N, const int32_t *cand_offsets,
                                  const int32_t *seq_offsets, int32_t n_q, int32_t H, int32_t dh,
                                  double scale, const void *Q, const void *K, const void *V,
                                  double *O) {
  const int64_t hd = (int64_t)H * dh;
  for (int32_t r = 0; r < R; ++r) {
    const int64_t t0 = seq_offsets[r];
    const int32_t L = seq_offsets[r + 1] - seq_offsets[r];
    double *p = (double *)malloc(sizeof(double) * (size_t)(L > 0 ? L : 1));
    if (!p) return -1;
    for (int64_t i = cand_offsets[r]; i < cand_offsets[r + 1]; ++i)
      for (int32_t t = 0; t < n_q; ++t)
        for (int32_t h = 0; h < H; ++h) {
          double *o = O + ((i * n_q + t) * H + h) * dh;
          for (int32_t e = 0; e < dh; ++e) o[e] = 0.0;
          if (L == 0) continue;
          const int64_t qbase = ((i * n_q + t) * H + h) * dh;
          double smax = -INFINITY;
          for (int32_t j = 0; j < L; ++j) {
            double dot = 0.0;
            for (int32_t e = 0; e < dh; ++e)
              dot += load_as_f64(Q, dtype, qbase + e) * load_as_f64(K, dtype, (t0 + j) * hd + (int64_t)h * dh + e);
            p[j] = scale * dot;
            if (p[j] > smax) smax = p[j];
          }
          double denom = 0.0;
          for (int32_t j = 0; j < L; ++j) {
            p[j] = exp(p[j] - smax);
            denom += p[j];
          }
          for (int32_t j = 0; j < L; ++j)
            for (int32_t e = 0; e < dh; ++e)
              o[e] += p[j] / denom * load_as_f64(V, dtype, (t0 + j) * hd + (int64_t)h * dh + e);
        }
    free(p);
  }
  return 0;
}

/* ------------------------------------------------------------------------- *
 * GLM factorization machine, two groups (Eq. 9-10), followed by the optional
 * ROCSified linear compression on the row axis (Eq. 5-6).
 * Materialised form: X = [X^R[m_i] ; X^C[i]] in R^{n x d}, n = n_r + n_c, is
 * built per candidate; G = X X^T; the block mask (Eq. 3) zeroes G[0:n_r, n_r:].
 * G_out [rows, n, n] fp64 receives the whole masked matrix: its first n_r rows
 * are the request-side output Y^R, the last n_c rows the candidate-side Y^C.
 * If W != NULL it is [n_ro + n_co, n]; the masked weight W~ has
 * W~[0:n_ro, n_r:] = 0 and O = W~ G; O_out [rows, n_ro + n_co, n] fp64
 * (first n_ro rows = request-side O^R, remaining n_co rows = candidate-side O^C).
 * ------------------------------------------------------------------------- */
int rocs_ref_glm_interaction(int dtype, int32_t R, int64_t N, const int32_t *cand_offsets,
                             int32_t n_r, int32_t n_c, int32_t d, const void *XR, const void *XC,
                             const void *W, int32_t n_ro, int32_t n_co, const int64_t *sample,
                             int64_t n_sample, double *G_out, double *O_out) {
  int32_t *m = materialise_index_map(R, N, cand_offsets);
  if (!m) return -1;
  const int64_t rows = sample ? n_sample : N;
  const int32_t n = n_r + n_c;
  const int32_t n_o = n_ro + n_co;
#pragma omp parallel
  {
    double *X = (double *)malloc(sizeof(double) * (size_t)n * d);
    double *G = (double *)malloc(sizeof(double) * (size_t)n * n);
#pragma omp for schedule(dynamic, 16)
    for (int64_t s = 0; s < rows; ++s) {
      const int64_t i = pick(sample, s);
      const int32_t r = m[i];
      for (int32_t a = 0; a < n_r; ++a)
        for (int32_t e = 0; e < d; ++e) X[a * d + e] = load_as_f64(XR, dtype, ((int64_t)r * n_r + a) * d + e);
      for (int32_t a = 0; a < n_c; ++a)
        for (int32_t e = 0; e < d; ++e) X[(n_r + a) * d + e] = load_as_f64(XC, dtype, (i * n_c + a) * d + e);
      for (int32_t a = 0; a < n; ++a)
        for (int32_t b = 0; b < n; ++b) {
          double acc = 0.0;
          for (int32_t e = 0; e < d; ++e) acc += X[a * d + e] * X[b * d + e];
          G[a * n + b] = acc;
        }
      for (int32_t a = 0; a < n_r; ++a)
        for (int32_t b = n_r; b < n; ++b) G[a * n + b] = 0.0;
      if (G_out) memcpy(G_out + s * n * n, G, sizeof(double) * (size_t)n * n);
      if (W && O_out)
        for (int32_t o = 0; o < n_o; ++o)
          for (int32_t b = 0; b < n; ++b) {
            double acc = 0.0;
            for (int32_t a = 0; a < n; ++a) {
              double w = load_as_f64(W, dtype, (int64_t)o * n + a);
              if (o < n_ro && a >= n_r) w = 0.0; /* W~ = W (.) block mask */
              acc += w * G[a * n + b];
            }
            O_out[(s * n_o + o) * n + b] = acc;
          }
    }
    free(X);
    free(G);
  }
  free(m);
  return 0;
}

/* Request-once form of the same operator (Section 4.1 applied to Eq. 6 / 10):
 *   YR[r]  = [X^R X^R^T , 0]                      [R, n_r, n]
 *   YC[i]  = [X^C_i X^R_{m_i}^T , X^C_i X^C_i^T]  [N, n_c, n]
 *   OR[r]  = W_RR YR[r]                            [R, n_ro, n]
 *   OC[i]  = W_CR YR[m_i] + W_CC YC[i]             [N, n_co, n]
 * Any output pointer may be NULL.  Only for the both-forms-agree test. */
int rocs_ref_glm_interaction_decomposed(int dtype, int32_t R, int64_t N, const int32_t *cand_offsets,
                                        int32_t n_r, int32_t n_c, int32_t d, const void *XR,
                                        const void *XC, const void *W, int32_t n_ro, int32_t n_co,
                                        double *YR, double *YC, double *OR_, double *OC) {
  const int32_t n = n_r + n_c;
  double *yr = (double *)malloc(sizeof(double) * (size_t)(n_r > 0 ? n_r : 1) * n);
  double *yc = (double *)malloc(sizeof(double) * (size_t)(n_c > 0 ? n_c : 1) * n);
  double *zr = (double *)malloc(sizeof(double) * (size_t)(n_co > 0 ? n_co : 1) * n);
  if (!yr || !yc || !zr) return -1;
  for (int32_t r = 0; r < R; ++r) {
    for (int32_t a = 0; a < n_r; ++a)
      for (int32_t b = 0; b < n; ++b) {
        double acc = 0.0;
        if (b < n_r)
          for (int32_t e = 0; e < d; ++e)
            acc += load_as_f64(XR, dtype, ((int64_t)r * n_r + a) * d + e) *
                   load_as_f64(XR, dtype, ((int64_t)r * n_r + b) * d + e);
        yr[a * n + b] = acc;
      }
    if (YR) memcpy(YR + (int64_t)r * n_r * n, yr, sizeof(double) * (size_t)n_r * n);
    if (W) {
      for (int32_t o = 0; o < n_ro; ++o)
        for (int32_t b = 0; b < n; ++b) {
          double acc = 0.0;
          for (int32_t a = 0; a < n_r; ++a) acc += load_as_f64(W, dtype, (int64_t)o * n + a) * yr[a * n + b];
          if (OR_) OR_[((int64_t)r * n_ro + o) * n + b] = acc;
        }
      for (int32_t o = 0; o < n_co; ++o)
        for (int32_t b = 0; b < n; ++b) {
          double acc = 0.0;
          for (int32_t a = 0; a < n_r; ++a)
            acc += load_as_f64(W, dtype, (int64_t)(n_ro + o) * n + a) * yr[a * n + b];
          zr[o * n + b] = acc;
        }
    }
    for (int64_t i = cand_offsets[r]; i < cand_offsets[r + 1]; ++i) {
      for (int32_t a = 0; a < n_c; ++a)
        for (int32_t b = 0; b < n; ++b) {
          double acc = 0.0;
          for (int32_t e = 0; e < d; ++e) {
            const double xa = load_as_f64(XC, dtype, (i * n_c + a) * d + e);
            const double xb = b < n_r ? load_as_f64(XR, dtype, ((int64_t)r * n_r + b) * d + e)
                                      : load_as_f64(XC, dtype, (i * n_c + (b - n_r)) * d + e);
            acc += xa * xb;
          }
          yc[a * n + b] = acc;
        }
      if (YC) memcpy(YC + i * n_c * n, yc, sizeof(double) * (size_t)n_c * n);
      if (W && OC)
        for (int32_t o = 0; o < n_co; ++o)
          for (int32_t b = 0; b < n; ++b) {
            double acc = zr[o * n + b];
            for (int32_t a = 0; a < n_c; ++a)
              acc += load_as_f64(W, dtype, (int64_t)(n_ro + o) * n + n_r + a) * yc[a * n + b];
            OC[(i * n_co + o) * n + b] = acc;
          }
    }
  }
  free(yr);
  free(yc);
  free(zr);
  return 0;
}

/* ------------------------------------------------------------------------- *
 * GLM factorization machine followed by a projection of its column axis
 * (Eq. 9-10, then the k-column compression an FM block applies to its
 * n x n interaction matrix; k is the "compression dimension" of the Wukong
 * row of the hyper-parameter table in the appendix).  The paper prints no
 * formula for the projection; the reading taken here is  F = G P  with a
 * learned P in R^{n x k}, G the masked interaction matrix of Eq. 9-10.
 * Materialised form: X = [X^R[m_i] ; X^C[i]] per candidate, G = X X^T with
 * G[0:n_r, n_r:] = 0, F = G P.  F_out [rows, n, k] fp64: first n_r rows are
 * the request side, the last n_c rows the candidate side.
 * ------------------------------------------------------------------------- */
int rocs_ref_glm_fm_projection(int dtype, int32_t R, int64_t N, const int32_t *cand_offsets,
                               int32_t n_r, int32_t n_c, int32_t d, int32_t k, const void *XR,
                               const void *XC, const void *P, const int64_t *sample, int64_t n_sample,
                               double *F_out) {
  int32_t *m = materialise_index_map(R, N, cand_offsets);
  if (!m) return -1;
  const int64_t rows = sample ? n_sample : N;
  const int32_t n = n_r + n_c;
#pragma omp parallel
  {
    double *X = (double *)malloc(sizeof(double) * (size_t)n * d);
    double *G = (double *)malloc(sizeof(double) * (size_t)n * n);
#pragma omp for schedule(dynamic, 16)
    for (int64_t s = 0; s < rows; ++s) {
      const int64_t i = pick(sample, s);
      const int32_t r = m[i];
      for (int32_t a = 0; a < n_r; ++a)
        for (int32_t e = 0; e < d; ++e) X[a * d + e] = load_as_f64(XR, dtype, ((int64_t)r * n_r + a) * d + e);
      for (int32_t a = 0; a < n_c; ++a)
        for (int32_t e = 0; e < d; ++e) X[(n_r + a) * d + e] = load_as_f64(XC, dtype, (i * n_c + a) * d + e);
      for (int32_t a = 0; a < n; ++a)
        for (int32_t b = 0; b < n; ++b) {
          double acc = 0.0;
          for (int32_t e = 0; e < d; ++e) acc += X[a * d + e] * X[b * d + e];
          G[a * n + b] = acc;
        }
      for (int32_t a = 0; a < n_r; ++a)
        for (int32_t b = n_r; b < n; ++b) G[a * n + b] = 0.0;
      for (int32_t a = 0; a < n; ++a)
        for (int32_t c = 0; c < k; ++c) {
          double acc = 0.0;
          for (int32_t b = 0; b < n; ++b) acc += G[a * n + b] * load_as_f64(P, dtype, (int64_t)b * k + c);
          F_out[(s * n + a) * k + c] = acc;
        }
    }
    free(X);
    free(G);
  }
  free(m);
  return 0;
}

/* Request-once form of the same operator (Section 4.1 applied to F = G P):
 *   T[r]  = X^R_r^T P_R                 [R, d, k]     (P_R = P[0:n_r], P_C = P[n_r:])
 *   FR[r] = X^R_r T[r]                  [R, n_r, k]
 *   FC[i] = X^C_i (T[m_i] + X^C_i^T P_C)   [N, n_c, k]
 * Only for the both-forms-agree test. */
int rocs_ref_glm_fm_projection_decomposed(int dtype, int32_t R, int64_t N, const int32_t *cand_offsets,
                                          int32_t n_r, int32_t n_c, int32_t d, int32_t k, const void *XR,
                                          const void *XC, const void *P, double *FR, double *FC) {
  (void)N;
  double *T = (double *)malloc(sizeof(double) * (size_t)d * k);
  double *H = (double *)malloc(sizeof(double) * (size_t)d * k);
  if (!T || !H) return -1;
  for (int32_t r = 0; r < R; ++r) {
    for (int32_t e = 0; e < d; ++e)
      for (int32_t c = 0; c < k; ++c) {
        double acc = 0.0;
        for (int32_t a = 0; a < n_r; ++a)
          acc += load_as_f64(XR, dtype, ((int64_t)r * n_r + a) * d + e) * load_as_f64(P, dtype, (int64_t)a * k + c);
        T[e * k + c] = acc;
      }
    if (FR)
      for (int32_t a = 0; a < n_r; ++a)
        for (int32_t c = 0; c < k; ++c) {
          double acc = 0.0;
          for (int32_t e = 0; e < d; ++e) acc += load_as_f64(XR, dtype, ((int64_t)r * n_r + a) * d + e) * T[e * k + c];
          FR[((int64_t)r * n_r + a) * k + c] = acc;
        }
    for (int64_t i = cand_offsets[r]; i < cand_offsets[r + 1]; ++i) {
      for (int32_t e = 0; e < d; ++e)
        for (int32_t c = 0; c < k; ++c) {
          double acc = T[e * k + c];
          for (int32_t a = 0; a < n_c; ++a)
            acc += load_as_f64(XC, dtype, (i * n_c + a) * d + e) * load_as_f64(P, dtype, (int64_t)(n_r + a) * k + c);
          H[e * k + c] = acc;
        }
      if (FC)
        for (int32_t a = 0; a < n_c; ++a)
          for (int32_t c = 0; c < k; ++c) {
            double acc = 0.0;
            for (int32_t e = 0; e < d; ++e) acc += load_as_f64(XC, dtype, (i * n_c + a) * d + e) * H[e * k + c];
            FC[(i * n_c + a) * k + c] = acc;
          }
    }
  }
  free(T);
  free(H);
  return 0;
}

/* ------------------------------------------------------------------------- *
 * Group-local normalisation (Eq. 7): y^(i) = Norm_i(x^(i)), one group's tensor
 * at a time, so no statistic ever spans two groups.  X [M, d]; every row is
 * normalised over its d coordinates.
 *   kind 0  LayerNorm:  y = (x - mean) / sqrt(var + eps) * gamma + beta   (biased variance)
 *   kind 1  RMSNorm:    y = x / sqrt(mean(x^2) + eps) * gamma             (beta ignored)
 * gamma / beta may be NULL (1 / 0).  Y_out [M, d] fp64.
 * ------------------------------------------------------------------------- */
int rocs_ref_group_norm(int dtype, int64_t M, int32_t d, const void *X, const void *gamma, const void *beta,
                        double eps, int kind, double *Y_out) {
  if (kind != 0 && kind != 1) return -1;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < M; ++i) {
    double mean = 0.0, sq = 0.0;
    for (int32_t e = 0; e < d; ++e) mean += load_as_f64(X, dtype, i * d + e);
    mean /= d;
    if (kind == 0) {
      for (int32_t e = 0; e < d; ++e) {
        const double c = load_as_f64(X, dtype, i * d + e) - mean;
        sq += c * c;
      }
    } else {
      for (int32_t e = 0; e < d; ++e) {
        const double v = load_as_f64(X, dtype, i * d + e);
        sq += v * v;
      }
    }
    const double inv = 1.0 / sqrt(sq / d + eps);
    for (int32_t e = 0; e < d; ++e) {
      const double g = gamma ? load_as_f64(gamma, dtype, e) : 1.0;
      const double b = (beta && kind == 0) ? load_as_f64(beta, dtype, e) : 0.0;
      const double v = load_as_f64(X, dtype, i * d + e);
      Y_out[i * d + e] = (kind == 0 ? (v - mean) : v) * inv * g + b;
    }
  }
  return 0;
}

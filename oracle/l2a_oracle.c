/*
 * L2A conditional attention layer -- fp64 CPU oracle.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, obviously-correct restatement of what the layer computes.  It shares no code with
 * the CUDA library and must never be called from the product path; only the tests, the smoke check
 * and the benchmark's CPU-baseline leg use it.
 *
 * What is computed (paper Section 3.1, Eq. 2-5, with the masks of Section 2):
 *   local  neighbourhood of a query at position p :  max(0, p-W) <= j <= p   (self + W predecessors)
 *   global neighbourhood                          :  0 <= j <= p
 *   s_t = softmax-average of V over the local  neighbourhood           (Eq. 2, sliding-window mask)
 *   d_t = 1[z_t >= thr]  on the router logit (thr = 0 <=> sigmoid >= 0.5)           (Eq. 3)
 *   a_t = softmax-average of V over the global neighbourhood if d_t = 1, else 0     (Eq. 4)
 *   o_t = s_t + d_t * a_t                                                           (Eq. 5)
 *   Q_idx = ascending positions with d_t = 1, n_c their count (Section 3.2 / Algorithm 1 step 1)
 *   exported log-sum-exp  L = m + log(l), natural log          (Algorithm 1, finalisation lines)
 * The method is exact attention on a subset of queries, so the oracle is the definition written
 * out: a two-pass (max, then sum) softmax in fp64, no tiling, no online rescaling.
 *
 * Backward: the paper gives no algorithm (Section 3.2 says only that gradients are computed for
 * active queries).  It is the vector-Jacobian product of the forward above with the routing mask
 * held fixed.  For each of the two attentions X with output out_i and upstream gradient dout_i
 * (dout = dO for local, d_t*dO for global):
 *   Delta_i = dout_i . out_i ;  dP_ij = dout_i . v_j ;  dS_ij = P_ij (dP_ij - Delta_i)
 *   dV_j += P_ij dout_i ;  dQ_i += scale * dS_ij k_j ;  dK_j += scale * dS_ij q_i
 * K/V gradients of a KV head sum over the query heads of its group (GQA).
 *
 * Layouts: Q [B,Lq,Hq,D], K/V [B,Lk,Hkv,D], dO like Q, all contiguous, bf16 bit patterns (uint16)
 * upcast exactly to fp64.  Query row t sits at position p = t + q_pos_offset.
 *
 * Pins (see tests): brute-force masked attention on tiny inputs, K==0 closed forms, V==const,
 * reductions d==0 / d==1 / W>=L-1 / W==0 to textbook attention, an independent transcription of
 * Algorithm 1, finite-difference gradients, dS row-sum and dV column-sum identities.
 * Parity unpinned beyond those: the paper prints no numerical worked example of the layer.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
  int32_t B, Lq, Lk, Hq, Hkv, D;
  int32_t window;        /* W: keys j with 0 <= p - j <= W */
  int32_t q_pos_offset;  /* p = t + q_pos_offset */
  double scale;          /* softmax scale, normally 1/sqrt(D) */
} l2a_oracle_shape;

/* Input element type.  The default build reads bf16 bit patterns; building with
 * -DL2A_ORACLE_F64_INPUT reads fp64 inputs instead (same code otherwise), which is what the
 * finite-difference gradient check perturbs. */
#ifdef L2A_ORACLE_F64_INPUT
typedef double in_t;
static inline double LD(in_t x) { return x; }
#else
typedef uint16_t in_t;
static inline double LD(in_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}
#endif

int l2a_oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Eq. 3 on the logit: d = (z >= thr) evaluated in fp32; NaN compares false. */
void l2a_oracle_route(const float *z, int64_t n, float thr, uint8_t *d) {
  for (int64_t i = 0; i < n; ++i) d[i] = (z[i] >= thr) ? 1 : 0;
}

/* Section 3.2: ascending list of routed positions per batch row, its length, and the exclusive
 * prefix count.  q_idx is [B,L] with the tail filled with -1; prefix is [B,L+1]. */
void l2a_oracle_compact(const uint8_t *d, int32_t B, int32_t L, int32_t *q_idx, int32_t *n_routed,
                        int32_t *prefix) {
  for (int32_t b = 0; b < B; ++b) {
    int32_t c = 0;
    for (int32_t t = 0; t < L; ++t) {
      prefix[(int64_t)b * (L + 1) + t] = c;
      if (d[(int64_t)b * L + t]) q_idx[(int64_t)b * L + c++] = t;
    }
    prefix[(int64_t)b * (L + 1) + L] = c;
    n_routed[b] = c;
    for (int32_t t = c; t < L; ++t) q_idx[(int64_t)b * L + t] = -1;
  }
}

static inline const in_t *q_row(const l2a_oracle_shape *s, const in_t *Q, int b, int t, int h) {
  return Q + (((int64_t)b * s->Lq + t) * s->Hq + h) * s->D;
}
static inline const in_t *kv_row(const l2a_oracle_shape *s, const in_t *K, int b, int j, int g) {
  return K + (((int64_t)b * s->Lk + j) * s->Hkv + g) * s->D;
}

/* One attention row over keys lo..hi (inclusive) of KV head g:
 * score_j = scale * q.k_j ; lse = log sum exp ; out = sum_j exp(score_j - lse) v_j.
 * p (length hi-lo+1) receives the probabilities when non-NULL. */
static void attn_row(const l2a_oracle_shape *s, const in_t *q, const in_t *K, const in_t *V,
                     int b, int g, int lo, int hi, double *out, double *lse, double *p) {
  const int D = s->D;
  const int n = hi - lo + 1;
  double *sc = p ? p : (double *)malloc(sizeof(double) * (size_t)n);
  double m = -INFINITY;
  for (int j = lo; j <= hi; ++j) {
    const in_t *k = kv_row(s, K, b, j, g);
    double acc = 0.0;
    for (int e = 0; e < D; ++e) acc += LD(q[e]) * LD(k[e]);
    acc *= s->scale;
    sc[j - lo] = acc;
    if (acc > m) m = acc;
  }
  double l = 0.0;
  for (int j = 0; j < n; ++j) l += exp(sc[j] - m);
  *lse = m + log(l);
  for (int e = 0; e < D; ++e) out[e] = 0.0;
  for (int j = lo; j <= hi; ++j) {
    const double pj = exp(sc[j - lo] - *lse);
    sc[j - lo] = pj;
    const in_t *v = kv_row(s, V, b, j, g);
    for (int e = 0; e < D; ++e) out[e] += pj * LD(v[e]);
  }
  if (!p) free(sc);
}

static inline int local_lo(const l2a_oracle_shape *s, int p) { return p - s->window > 0 ? p - s->window : 0; }

/* Forward for a list of (b, h, t) rows.  Outputs are [nrows, D] (s, a, o) and [nrows] (lse).
 * For a non-routed row a = 0 and lse_glb = NaN (undefined). */
void l2a_oracle_forward_rows(const l2a_oracle_shape *s, const in_t *Q, const in_t *K,
                             const in_t *V, const uint8_t *d, int64_t nrows, const int32_t *rb,
                             const int32_t *rh, const int32_t *rt, double *s_out, double *a_out,
                             double *o_out, double *lse_loc, double *lse_glb) {
  const int D = s->D, G = s->Hq / s->Hkv;
#pragma omp parallel for schedule(dynamic, 4)
  for (int64_t r = 0; r < nrows; ++r) {
    const int b = rb[r], h = rh[r], t = rt[r], g = h / G;
    const int p = t + s->q_pos_offset;
    const in_t *q = q_row(s, Q, b, t, h);
    double *so = s_out + r * D, *ao = a_out + r * D, *oo = o_out + r * D;
    attn_row(s, q, K, V, b, g, local_lo(s, p), p, so, &lse_loc[r], NULL);
    if (d[(int64_t)b * s->Lq + t]) {
      attn_row(s, q, K, V, b, g, 0, p, ao, &lse_glb[r], NULL);
    } else {
      for (int e = 0; e < D; ++e) ao[e] = 0.0;
      lse_glb[r] = NAN;
    }
    for (int e = 0; e < D; ++e) oo[e] = so[e] + ao[e];
  }
}

/* VJP of one attention row: adds this row's contribution into dq (length D) and, where the
 * pointers are non-NULL, into dK/dV rows (full [B,Lk,Hkv,D] fp64 arrays).  keep[j-lo] (optional)
 * restricts the dK/dV accumulation to flagged keys. */
static void attn_row_bwd(const l2a_oracle_shape *s, const in_t *q, const in_t *K, const in_t *V,
                         const double *dout, int b, int g, int lo, int hi, double *dq, double *dK,
                         double *dV, const uint8_t *keep_abs) {
  const int D = s->D;
  const int n = hi - lo + 1;
  double *p = (double *)malloc(sizeof(double) * (size_t)n);
  double *out = (double *)malloc(sizeof(double) * (size_t)D);
  double lse;
  attn_row(s, q, K, V, b, g, lo, hi, out, &lse, p);
  double delta = 0.0;
  for (int e = 0; e < D; ++e) delta += dout[e] * out[e];
  for (int j = lo; j <= hi; ++j) {
    const in_t *k = kv_row(s, K, b, j, g);
    const in_t *v = kv_row(s, V, b, j, g);
    double dp = 0.0;
    for (int e = 0; e < D; ++e) dp += dout[e] * LD(v[e]);
    const double pj = p[j - lo];
    const double ds = pj * (dp - delta);
    if (dq)
      for (int e = 0; e < D; ++e) dq[e] += s->scale * ds * LD(k[e]);
    if (dK && (!keep_abs || keep_abs[j])) {
      double *dk = dK + (((int64_t)b * s->Lk + j) * s->Hkv + g) * D;
      double *dv = dV + (((int64_t)b * s->Lk + j) * s->Hkv + g) * D;
      for (int e = 0; e < D; ++e) {
        dk[e] += s->scale * ds * LD(q[e]);
        dv[e] += pj * dout[e];
      }
    }
  }
  free(p);
  free(out);
}

/* Full backward: dQ [B,Lq,Hq,D], dK, dV [B,Lk,Hkv,D] in fp64 (overwritten).  Parallel over
 * (b, KV head) so that no two threads add into the same dK/dV row. */
void l2a_oracle_backward_full(const l2a_oracle_shape *s, const in_t *Q, const in_t *K,
                              const in_t *V, const uint8_t *d, const in_t *dO, double *dQ,
                              double *dK, double *dV) {
  const int D = s->D, G = s->Hq / s->Hkv;
  memset(dQ, 0, sizeof(double) * (size_t)s->B * s->Lq * s->Hq * D);
  memset(dK, 0, sizeof(double) * (size_t)s->B * s->Lk * s->Hkv * D);
  memset(dV, 0, sizeof(double) * (size_t)s->B * s->Lk * s->Hkv * D);
#pragma omp parallel for schedule(dynamic, 1) collapse(2)
  for (int b = 0; b < s->B; ++b) {
    for (int g = 0; g < s->Hkv; ++g) {
      double *dout = (double *)malloc(sizeof(double) * (size_t)D);
      for (int h = g * G; h < (g + 1) * G; ++h) {
        for (int t = 0; t < s->Lq; ++t) {
          const int p = t + s->q_pos_offset;
          const in_t *q = q_row(s, Q, b, t, h);
          const in_t *go = q_row(s, dO, b, t, h);
          double *dq = dQ + (((int64_t)b * s->Lq + t) * s->Hq + h) * D;
          for (int e = 0; e < D; ++e) dout[e] = LD(go[e]);
          attn_row_bwd(s, q, K, V, dout, b, g, local_lo(s, p), p, dq, dK, dV, NULL);
          if (d[(int64_t)b * s->Lq + t]) attn_row_bwd(s, q, K, V, dout, b, g, 0, p, dq, dK, dV, NULL);
        }
      }
      free(dout);
    }
  }
}

/* dQ for a list of (b, h, t) rows; out [nrows, D]. */
void l2a_oracle_dq_rows(const l2a_oracle_shape *s, const in_t *Q, const in_t *K, const in_t *V,
                        const uint8_t *d, const in_t *dO, int64_t nrows, const int32_t *rb,
                        const int32_t *rh, const int32_t *rt, double *dq_out) {
  const int D = s->D, G = s->Hq / s->Hkv;
#pragma omp parallel for schedule(dynamic, 4)
  for (int64_t r = 0; r < nrows; ++r) {
    const int b = rb[r], h = rh[r], t = rt[r], g = h / G;
    const int p = t + s->q_pos_offset;
    const in_t *q = q_row(s, Q, b, t, h);
    const in_t *go = q_row(s, dO, b, t, h);
    double *dout = (double *)malloc(sizeof(double) * (size_t)D);
    double *dq = dq_out + r * D;
    for (int e = 0; e < D; ++e) { dout[e] = LD(go[e]); dq[e] = 0.0; }
    attn_row_bwd(s, q, K, V, dout, b, g, local_lo(s, p), p, dq, NULL, NULL, NULL);
    if (d[(int64_t)b * s->Lq + t]) attn_row_bwd(s, q, K, V, dout, b, g, 0, p, dq, NULL, NULL, NULL);
    free(dout);
  }
}

/* dK, dV for the listed key positions js[0..nj) of one (b, KV head g); out [nj, D] each.
 * Every query row that can see one of those keys is visited, for every query head of the group. */
void l2a_oracle_dkv_cols(const l2a_oracle_shape *s, const in_t *Q, const in_t *K, const in_t *V,
                         const uint8_t *d, const in_t *dO, int32_t b, int32_t g, int32_t nj,
                         const int32_t *js, double *dk_out, double *dv_out) {
  const int D = s->D, G = s->Hq / s->Hkv;
  uint8_t *keep = (uint8_t *)calloc((size_t)s->Lk, 1);
  int jmin = s->Lk;
  for (int i = 0; i < nj; ++i) { keep[js[i]] = 1; if (js[i] < jmin) jmin = js[i]; }
  const int t_first = jmin - s->q_pos_offset > 0 ? jmin - s->q_pos_offset : 0;
  const int nthr = l2a_oracle_num_threads();
  /* per-thread private full-size accumulators would be huge; use per-thread [nj, D] slabs */
  int32_t *slot = (int32_t *)malloc(sizeof(int32_t) * (size_t)s->Lk);
  for (int j = 0; j < s->Lk; ++j) slot[j] = -1;
  for (int i = 0; i < nj; ++i) slot[js[i]] = i;
  double *acc_k = (double *)calloc((size_t)nthr * nj * D, sizeof(double));
  double *acc_v = (double *)calloc((size_t)nthr * nj * D, sizeof(double));
#pragma omp parallel
  {
#ifdef _OPENMP
    const int tid = omp_get_thread_num();
#else
    const int tid = 0;
#endif
    double *ak = acc_k + (size_t)tid * nj * D, *av = acc_v + (size_t)tid * nj * D;
    double *dout = (double *)malloc(sizeof(double) * (size_t)D);
    double *out = (double *)malloc(sizeof(double) * (size_t)D);
    double *p = (double *)malloc(sizeof(double) * (size_t)s->Lk);
#pragma omp for schedule(dynamic, 1) collapse(2)
    for (int h = g * G; h < (g + 1) * G; ++h) {
      for (int t = t_first; t < s->Lq; ++t) {
        const int pos = t + s->q_pos_offset;
        const in_t *q = q_row(s, Q, b, t, h);
        const in_t *go = q_row(s, dO, b, t, h);
        for (int e = 0; e < D; ++e) dout[e] = LD(go[e]);
        for (int pass = 0; pass < 2; ++pass) {
          if (pass == 1 && !d[(int64_t)b * s->Lq + t]) continue;
          const int lo = pass == 0 ? local_lo(s, pos) : 0;
          int any = 0;
          for (int i = 0; i < nj && !any; ++i) any = (js[i] >= lo && js[i] <= pos);
          if (!any) continue;
          double lse;
          attn_row(s, q, K, V, b, g, lo, pos, out, &lse, p);
          double delta = 0.0;
          for (int e = 0; e < D; ++e) delta += dout[e] * out[e];
          for (int i = 0; i < nj; ++i) {
            const int j = js[i];
            if (j < lo || j > pos || slot[j] != i) continue; /* duplicates in js count once */
            const in_t *v = kv_row(s, V, b, j, g);
            double dp = 0.0;
            for (int e = 0; e < D; ++e) dp += dout[e] * LD(v[e]);
            const double pj = p[j - lo];
            const double ds = pj * (dp - delta);
            for (int e = 0; e < D; ++e) {
              ak[(size_t)i * D + e] += s->scale * ds * LD(q[e]);
              av[(size_t)i * D + e] += pj * dout[e];
            }
          }
        }
      }
    }
    free(dout); free(out); free(p);
  }
  for (int64_t i = 0; i < (int64_t)nj * D; ++i) { dk_out[i] = 0.0; dv_out[i] = 0.0; }
  for (int th = 0; th < nthr; ++th)
    for (int64_t i = 0; i < (int64_t)nj * D; ++i) {
      dk_out[i] += acc_k[(size_t)th * nj * D + i];
      dv_out[i] += acc_v[(size_t)th * nj * D + i];
    }
  /* duplicate entries of js receive the value of their canonical slot */
  for (int i = 0; i < nj; ++i) {
    const int c = slot[js[i]];
    if (c != i)
      for (int e = 0; e < D; ++e) {
        dk_out[(size_t)i * D + e] = dk_out[(size_t)c * D + e];
        dv_out[(size_t)i * D + e] = dv_out[(size_t)c * D + e];
      }
  }
  free(keep); free(slot); free(acc_k); free(acc_v);
}

/* Straight-through gate gradient by-product (Eq. 7, first term): dgate_t = sum_h dO_{t,h} . a_{t,h}
 * with a the global-attention output of EVERY row (as when global attention is forced for all
 * tokens); rows listed by (b, t); out [nrows]. */
void l2a_oracle_dgate_rows(const l2a_oracle_shape *s, const in_t *Q, const in_t *K, const in_t *V,
                           const in_t *dO, int64_t nrows, const int32_t *rb, const int32_t *rt,
                           double *dgate) {
  const int D = s->D, G = s->Hq / s->Hkv;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t r = 0; r < nrows; ++r) {
    const int b = rb[r], t = rt[r], p = t + s->q_pos_offset;
    double *a = (double *)malloc(sizeof(double) * (size_t)D);
    double acc = 0.0, lse;
    for (int h = 0; h < s->Hq; ++h) {
      attn_row(s, q_row(s, Q, b, t, h), K, V, b, h / G, 0, p, a, &lse, NULL);
      const in_t *go = q_row(s, dO, b, t, h);
      for (int e = 0; e < D; ++e) acc += LD(go[e]) * a[e];
    }
    dgate[r] = acc;
    free(a);
  }
}

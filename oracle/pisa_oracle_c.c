/*
 * Compiled CPU oracle for the PISA forward path.  TEST INFRASTRUCTURE ONLY.
 *
 * The same definitions as oracle/pisa_oracle.py, written a second time in plain C (fp64 arithmetic,
 * one query at a time, no blocking or fusion), with OpenMP over the queries so that thousands of
 * sampled rows of a long sequence finish in seconds.  It is called only by the tests, the smoke
 * check and the benchmark's CPU-baseline leg; the CUDA library never calls it and shares no code
 * with it.  It was written independently of the NumPy oracle (no generated tables, no shared
 * helpers) and the two are compared with each other in tests/test_oracle_c_pins.py.
 *
 * Every function works on ONE (batch, KV head) unit, everything in fp64, everything 0-based:
 *   k, v      [N, d]      raw keys / values of the unit (stored values widened to fp64)
 *   levels    levels 1..L of the unit's pyramid back to back, level l = [M_l, d]
 *   q         [S, G, d]   the group's G query vectors of S sampled positions pos[0..S)
 *
 * What follows which passage of the paper:
 *   oc_hierarchy      Sec. 3.2 "Fine-to-coarse block aggregation": M_1 = ceil(N/C), M_{l+1} = ceil(M_l/g)
 *   oc_pyramid        Eq. "mean pyramid": unweighted mean of the valid children, each level rounded to
 *                     the storage dtype and pooled from the stored level below
 *   block_score       Eq. "direct child LSE"; Sec. 4.3 / App. A.2 for the mean and mean + var/2 scores
 *   oc_route          Sec. 3.2 "Coarse-to-fine block selection", Eq. "grouped score", App. B "Causal
 *                     masking": eligibility, forced first / previous / current nodes (inside the
 *                     budget, never scored), keep-all when at most K remain, ties to the smaller index
 *   oc_attend         Eq. "selected sparse attention" with the causal mask inside selected blocks
 *   oc_flat_mean      Sec. 3.1 flat selection with the per-head softmax of App. C before the head sum
 *   oc_backward_rows  App. B: softmax-attention gradients over the selected, visible keys with the
 *                     indices held fixed
 *
 * Pins: tests/test_oracle_c_pins.py (closed forms, torch's logsumexp / topk / dense causal attention /
 * autograd, the hand-derived pruned example, and the NumPy oracle as a second, independent witness
 * on shapes with fan-in 4, several heads per group and ragged hierarchies).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define OC_MAX_LEVELS 40
enum { OC_BF16 = 0, OC_FP32 = 1 };
enum { OC_LSE = 0, OC_MEAN = 1, OC_MEAN_VAR = 2 };

/* ------------------------------------------------------------------ storage rounding */

/* fp64 -> nearest bf16 value (ties to even), one rounding, returned as fp64 */
static double round_bf16(double x) {
  if (x == 0.0 || isnan(x) || isinf(x)) return x;
  int e;
  frexp(x, &e);                      /* |x| = f * 2^e, f in [0.5, 1) */
  int exp2 = e - 1;                  /* |x| in [2^exp2, 2^(exp2+1)) */
  if (exp2 < -126) exp2 = -126;      /* subnormal range of bf16: fixed spacing */
  const double ulp = ldexp(1.0, exp2 - 7);   /* 8 significant bits */
  return nearbyint(x / ulp) * ulp;   /* default rounding mode: to nearest, ties to even; exact scaling */
}

static double round_storage(double x, int dtype) {
  if (dtype == OC_BF16) return round_bf16(x);
  return (double)(float)x;
}

double oc_round_storage(double x, int dtype) { return round_storage(x, dtype); }
void oc_round_storage_array(double* x, int64_t n, int dtype) {
  for (int64_t i = 0; i < n; ++i) x[i] = round_storage(x[i], dtype);
}

/* ------------------------------------------------------------------ hierarchy and pyramid */

/* M[0] = N, M[1] = ceil(N/C), M[l+1] = ceil(M[l]/g) down to one node; returns L */
int oc_hierarchy(int N, int C, int g, int32_t* M) {
  M[0] = N;
  M[1] = (N + C - 1) / C;
  int L = 1;
  while (M[L] > 1) {
    M[L + 1] = (M[L] + g - 1) / g;
    ++L;
  }
  return L;
}

static void level_offsets(const int32_t* M, int L, int d, int64_t* off) {
  int64_t o = 0;
  for (int l = 1; l <= L; ++l) {
    off[l] = o;
    o += (int64_t)M[l] * d;
  }
  off[0] = 0;
  off[L + 1] = o;
}

/* elements of `levels` for these sizes */
int64_t oc_pyramid_elems(int N, int d, int C, int g) {
  int32_t M[OC_MAX_LEVELS];
  int64_t off[OC_MAX_LEVELS + 2];
  const int L = oc_hierarchy(N, C, g, M);
  level_offsets(M, L, d, off);
  return off[L + 1];
}

void oc_pyramid(const double* k, int N, int d, int C, int g, int dtype, double* levels) {
  int32_t M[OC_MAX_LEVELS];
  int64_t off[OC_MAX_LEVELS + 2];
  const int L = oc_hierarchy(N, C, g, M);
  level_offsets(M, L, d, off);
  for (int l = 1; l <= L; ++l) {
    const int fan = (l == 1) ? C : g;
    const double* below = (l == 1) ? k : levels + off[l - 1];
    const int nbelow = M[l - 1];
    double* cur = levels + off[l];
#pragma omp parallel for schedule(static)
    for (int i = 0; i < M[l]; ++i) {
      const int lo = i * fan;
      const int hi = (lo + fan < nbelow) ? lo + fan : nbelow;
      for (int e = 0; e < d; ++e) {
        double s = 0.0;
        for (int r = lo; r < hi; ++r) s += below[(int64_t)r * d + e];
        cur[(int64_t)i * d + e] = round_storage(s / (double)(hi - lo), dtype);
      }
    }
  }
}

/* ------------------------------------------------------------------ scores */

static double dot(const double* a, const double* b, int d) {
  double s = 0.0;
  for (int e = 0; e < d; ++e) s += a[e] * b[e];
  return s;
}

/* score of one head's logits z[0..m) */
static double block_score(const double* z, int m, int mode) {
  if (mode == OC_LSE) {
    double mx = z[0];
    for (int i = 1; i < m; ++i)
      if (z[i] > mx) mx = z[i];
    double s = 0.0;
    for (int i = 0; i < m; ++i) s += exp(z[i] - mx);
    return mx + log(s);
  }
  double mean = 0.0;
  for (int i = 0; i < m; ++i) mean += z[i];
  mean /= (double)m;
  if (mode == OC_MEAN) return mean;
  double var = 0.0;
  for (int i = 0; i < m; ++i) var += (z[i] - mean) * (z[i] - mean);
  return mean + 0.5 * var / (double)m;
}

/* grouped score of one candidate: sum over the G heads of the block score of q_h . x_r * scale */
static double grouped_score(const double* qg, int G, int d, const double* x, int m, double scale, int mode,
                            double* zbuf) {
  double u = 0.0;
  for (int h = 0; h < G; ++h) {
    for (int r = 0; r < m; ++r) zbuf[r] = dot(qg + (int64_t)h * d, x + (int64_t)r * d, d) * scale;
    u += block_score(zbuf, m, mode);
  }
  return u;
}

/* ------------------------------------------------------------------ Select_K */

static int is_in(const int* a, int n, int x) {
  for (int i = 0; i < n; ++i)
    if (a[i] == x) return 1;
  return 0;
}

/* forced nodes of a level: ancestors of the first, previous and current leaf, deduplicated */
static int forced_nodes(int c, int64_t span, int* F) {
  int n = 0;
  const int cand[3] = {0, (int)((c >= 1 ? c - 1 : 0) / span), (int)(c / span)};
  for (int i = 0; i < 3; ++i)
    if (!is_in(F, n, cand[i])) F[n++] = cand[i];
  return n;
}

/* V[0..nV): valid candidates; F: forced; score[i] for the non-forced ones.  Keeps the forced ones plus
 * the best K - nF of the rest (score descending, ties to the smaller node index); writes the kept set
 * ascending to I and returns its size; *gap = relative gap at the cut (infinity if nothing was cut). */
static int select_k(const int* V, int nV, const int* F, int nF, const double* score, int K, int* I, double* gap) {
  int* rest = (int*)malloc(sizeof(int) * (size_t)(nV > 0 ? nV : 1));
  double* rs = (double*)malloc(sizeof(double) * (size_t)(nV > 0 ? nV : 1));
  int nr = 0;
  for (int i = 0; i < nV; ++i)
    if (!is_in(F, nF, V[i])) { rest[nr] = V[i]; rs[nr] = score[i]; ++nr; }
  /* insertion sort: larger score first, equal scores by node index */
  for (int i = 1; i < nr; ++i) {
    const int ni = rest[i];
    const double si = rs[i];
    int j = i - 1;
    while (j >= 0 && (rs[j] < si || (rs[j] == si && rest[j] > ni))) {
      rest[j + 1] = rest[j];
      rs[j + 1] = rs[j];
      --j;
    }
    rest[j + 1] = ni;
    rs[j + 1] = si;
  }
  const int keep = K - nF;
  *gap = INFINITY;
  if (keep > 0 && keep < nr) {
    const double a = rs[keep - 1], b = rs[keep];
    *gap = (a - b) / (fabs(a) > 1.0 ? fabs(a) : 1.0);
  }
  int n = 0;
  for (int i = 0; i < nF; ++i) I[n++] = F[i];
  for (int i = 0; i < keep && i < nr; ++i) I[n++] = rest[i];
  for (int i = 1; i < n; ++i) {             /* ascending */
    const int x = I[i];
    int j = i - 1;
    while (j >= 0 && I[j] > x) { I[j + 1] = I[j]; --j; }
    I[j + 1] = x;
  }
  free(rest);
  free(rs);
  return n;
}

/* ------------------------------------------------------------------ routing */

static void route_one(const double* qg, int p, int G, const double* k, const double* levels, const int32_t* M,
                      const int64_t* off, int L, int N, int d, int C, int g, int K, double scale, int mode,
                      int32_t* idx_row, double* margin_out) {
  const int c = p / C;
  const int cap = g * K + 8;
  int* A = (int*)malloc(sizeof(int) * (size_t)cap);
  int* V = (int*)malloc(sizeof(int) * (size_t)cap);
  int* I = (int*)malloc(sizeof(int) * (size_t)cap);
  double* sc = (double*)malloc(sizeof(double) * (size_t)cap);
  double* zbuf = (double*)malloc(sizeof(double) * (size_t)(C > g ? C : g));
  int nA = 1, nI = 0;
  A[0] = 0;
  double margin = INFINITY;
  int64_t span = 1;
  for (int l = 1; l < L; ++l) span *= g;          /* g^(L-1) */
  for (int l = L; l >= 1; --l) {
    const int anc_c = (int)(c / span);
    int nV = 0;
    for (int i = 0; i < nA; ++i)
      if (A[i] < M[l] && A[i] <= anc_c) V[nV++] = A[i];
    int F[3];
    const int nF = forced_nodes(c, span, F);
    if (nV <= K) {
      nI = nV;
      memcpy(I, V, sizeof(int) * (size_t)nV);
    } else {
      const int fan = (l == 1) ? C : g;
      const double* below = (l == 1) ? k : levels + off[l - 1];
      for (int i = 0; i < nV; ++i) {
        sc[i] = 0.0;
        if (is_in(F, nF, V[i])) continue;
        const int lo = V[i] * fan;
        const int hi = (lo + fan < M[l - 1]) ? lo + fan : M[l - 1];
        sc[i] = grouped_score(qg, G, d, below + (int64_t)lo * d, hi - lo, scale, mode, zbuf);
      }
      double gap;
      nI = select_k(V, nV, F, nF, sc, K, I, &gap);
      if (gap < margin) margin = gap;
    }
    if (l > 1) {
      nA = 0;
      for (int i = 0; i < nI; ++i)
        for (int r = I[i] * g; r < (I[i] + 1) * g && r < M[l - 1]; ++r) A[nA++] = r;
      span /= g;
    }
  }
  for (int i = 1; i < nI; ++i) {                  /* ascending (kept-all levels keep A's order already) */
    const int x = I[i];
    int j = i - 1;
    while (j >= 0 && I[j] > x) { I[j + 1] = I[j]; --j; }
    I[j + 1] = x;
  }
  for (int s = 0; s < K; ++s) idx_row[s] = (s < nI) ? I[s] : -1;
  *margin_out = margin;
  free(A); free(V); free(I); free(sc); free(zbuf);
}

void oc_route(const double* q, const int32_t* pos, int S, int G, const double* k, const double* levels, int N,
              int d, int C, int g, int K, double scale, int mode, int32_t* idx, double* margin, int nthreads) {
  int32_t M[OC_MAX_LEVELS];
  int64_t off[OC_MAX_LEVELS + 2];
  const int L = oc_hierarchy(N, C, g, M);
  level_offsets(M, L, d, off);
  (void)nthreads;
#pragma omp parallel for schedule(dynamic, 4) num_threads(nthreads > 0 ? nthreads : 1)
  for (int s = 0; s < S; ++s)
    route_one(q + (int64_t)s * G * d, pos[s], G, k, levels, M, off, L, N, d, C, g, K, scale, mode,
              idx + (int64_t)s * K, margin + s);
}

/* ------------------------------------------------------------------ flat selection (Sec. 3.1, App. C) */

void oc_flat_mean(const double* q, const int32_t* pos, int S, int G, const double* level1, int d, int C, int K,
                  double scale, int32_t* idx, double* margin, int nthreads) {
  (void)nthreads;
#pragma omp parallel for schedule(dynamic, 4) num_threads(nthreads > 0 ? nthreads : 1)
  for (int s = 0; s < S; ++s) {
    const int c = pos[s] / C;
    const int n = c + 1;
    int32_t* row = idx + (int64_t)s * K;
    margin[s] = INFINITY;
    if (n <= K) {
      for (int j = 0; j < K; ++j) row[j] = (j < n) ? j : -1;
      continue;
    }
    double* u = (double*)calloc((size_t)n, sizeof(double));
    double* z = (double*)malloc(sizeof(double) * (size_t)n);
    int* V = (int*)malloc(sizeof(int) * (size_t)n);
    int* I = (int*)malloc(sizeof(int) * (size_t)(K + 3));
    for (int h = 0; h < G; ++h) {
      const double* qh = q + ((int64_t)s * G + h) * d;
      double mx = -INFINITY;
      for (int i = 0; i < n; ++i) {
        z[i] = dot(qh, level1 + (int64_t)i * d, d) * scale;
        if (z[i] > mx) mx = z[i];
      }
      double den = 0.0;
      for (int i = 0; i < n; ++i) { z[i] = exp(z[i] - mx); den += z[i]; }
      for (int i = 0; i < n; ++i) u[i] += z[i] / den;
    }
    for (int i = 0; i < n; ++i) V[i] = i;
    int F[3];
    const int nF = forced_nodes(c, 1, F);
    double gap;
    const int nI = select_k(V, n, F, nF, u, K, I, &gap);
    for (int j = 0; j < K; ++j) row[j] = (j < nI) ? I[j] : -1;
    margin[s] = gap;
    free(u); free(z); free(V); free(I);
  }
}

/* ------------------------------------------------------------------ attention */

/* visible tokens of the selected blocks of one row (ascending block order as given); returns count */
static int visible_tokens(const int32_t* blocks, int K, int p, int C, int N, int* toks) {
  int n = 0;
  for (int s = 0; s < K; ++s) {
    const int i = blocks[s];
    if (i < 0) continue;
    for (int j = i * C; j < (i + 1) * C && j < N; ++j)
      if (j <= p) toks[n++] = j;
  }
  return n;
}

/* out [S,G,d] before storage rounding, lse [S,G] natural log of the softmax denominator */
void oc_attend(const double* q, const int32_t* pos, int S, int G, const double* k, const double* v, int N, int d,
               int C, int K, double scale, const int32_t* idx, double* out, double* lse, int nthreads) {
  (void)nthreads;
#pragma omp parallel for schedule(dynamic, 4) num_threads(nthreads > 0 ? nthreads : 1)
  for (int s = 0; s < S; ++s) {
    int* toks = (int*)malloc(sizeof(int) * (size_t)K * C);
    double* z = (double*)malloc(sizeof(double) * (size_t)K * C);
    const int n = visible_tokens(idx + (int64_t)s * K, K, pos[s], C, N, toks);
    for (int h = 0; h < G; ++h) {
      const double* qh = q + ((int64_t)s * G + h) * d;
      double* o = out + ((int64_t)s * G + h) * d;
      double mx = -INFINITY;
      for (int j = 0; j < n; ++j) {
        z[j] = dot(qh, k + (int64_t)toks[j] * d, d) * scale;
        if (z[j] > mx) mx = z[j];
      }
      double den = 0.0;
      for (int j = 0; j < n; ++j) { z[j] = exp(z[j] - mx); den += z[j]; }
      for (int e = 0; e < d; ++e) o[e] = 0.0;
      for (int j = 0; j < n; ++j) {
        const double* vj = v + (int64_t)toks[j] * d;
        for (int e = 0; e < d; ++e) o[e] += z[j] * vj[e];
      }
      for (int e = 0; e < d; ++e) o[e] /= den;
      lse[(int64_t)s * G + h] = mx + log(den);
    }
    free(toks);
    free(z);
  }
}

/* ------------------------------------------------------------------ attention backward, frozen indices */

/* Per row with probabilities p_j over its visible selected keys and o = sum_j p_j v_j:
 *   dv_j += p_j do,  dp_j = do . v_j,  ds_j = p_j (dp_j - sum_i p_i dp_i),
 *   dq = scale sum_j ds_j k_j,  dk_j += scale ds_j q.
 * dq [S,G,d] is written; dk, dv [N,d] (nullable) are ACCUMULATED into, restricted to key rows in
 * [key_lo, key_hi) so that a caller can ask for a few key blocks only. */
void oc_backward_rows(const double* q, const double* dout, const int32_t* pos, int S, int G, const double* k,
                      const double* v, int N, int d, int C, int K, double scale, const int32_t* idx, double* dq,
                      double* dk, double* dv, int key_lo, int key_hi, int nthreads) {
  (void)nthreads;
#pragma omp parallel for schedule(dynamic, 4) num_threads(nthreads > 0 ? nthreads : 1)
  for (int s = 0; s < S; ++s) {
    int* toks = (int*)malloc(sizeof(int) * (size_t)K * C);
    double* pr = (double*)malloc(sizeof(double) * (size_t)K * C);
    double* dp = (double*)malloc(sizeof(double) * (size_t)K * C);
    const int n = visible_tokens(idx + (int64_t)s * K, K, pos[s], C, N, toks);
    for (int h = 0; h < G; ++h) {
      const double* qh = q + ((int64_t)s * G + h) * d;
      const double* doh = dout + ((int64_t)s * G + h) * d;
      double* dqh = dq + ((int64_t)s * G + h) * d;
      for (int e = 0; e < d; ++e) dqh[e] = 0.0;
      if (n == 0) continue;
      double mx = -INFINITY;
      for (int j = 0; j < n; ++j) {
        pr[j] = dot(qh, k + (int64_t)toks[j] * d, d) * scale;
        if (pr[j] > mx) mx = pr[j];
      }
      double den = 0.0;
      for (int j = 0; j < n; ++j) { pr[j] = exp(pr[j] - mx); den += pr[j]; }
      double delta = 0.0;
      for (int j = 0; j < n; ++j) {
        pr[j] /= den;
        dp[j] = dot(doh, v + (int64_t)toks[j] * d, d);
        delta += pr[j] * dp[j];
      }
      for (int j = 0; j < n; ++j) {
        const double ds = pr[j] * (dp[j] - delta);
        const double* kj = k + (int64_t)toks[j] * d;
        for (int e = 0; e < d; ++e) dqh[e] += scale * ds * kj[e];
        if (dk != NULL && toks[j] >= key_lo && toks[j] < key_hi) {
          double* dkj = dk + (int64_t)toks[j] * d;
          double* dvj = dv + (int64_t)toks[j] * d;
          for (int e = 0; e < d; ++e) {
            const double a = scale * ds * qh[e], b = pr[j] * doh[e];
#pragma omp atomic
            dkj[e] += a;
#pragma omp atomic
            dvj[e] += b;
          }
        }
      }
    }
    free(toks); free(pr); free(dp);
  }
}

int oc_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

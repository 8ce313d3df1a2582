/*
 * TSID template-recovery oracle: TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, single-threaded CPU statement of what one full-batch gradient
 * step of the masked low-rank (regularised matrix factorisation, RMF) objective
 * computes.  All sums are taken in double precision, looping over the COO
 * triples in input order.  No blocking, no fusion, no reordering.  It shares no
 * code with the CUDA library; only tests, the smoke check and the bench's CPU
 * baseline leg may call it.
 *
 * Passages followed (paper sections / equations):
 *   - objective: Sec. 3.2, Eq. (rmf-obj):
 *       L(P,Q) = sum_{(i,j) in Omega} (r_ij - p_i . q_j)^2 + lambda (|P|_F^2 + |Q|_F^2)
 *   - per-entry gradients: Sec. 5.1, Eqs. (update-p), (update-q):
 *       grad_p = -2 e q + 2 lambda p,   grad_q = -2 e p + 2 lambda q,  e = r - p.q
 *   - aggregated update and the 1/n normalisation: Sec. 5.1, Eq. 9
 *   - asymmetric clipping min(max(xi, -g), g): Sec. 5.3 (unnumbered equation)
 *
 * Readings taken where the paper is ambiguous:
 *   - the symbol added to the factors in Eq. 9 is the step DIRECTION
 *       D = -grad L = 2 G / s - 2 lambda x,   G_P = E Q,  G_Q = E^T P,
 *     E the sparse residual matrix; the update is x + eta * D;
 *   - the "n" in the 1/n factor is the number of observed entries that
 *     contribute to that factor row (norm = COUNT), s = max(1, count);
 *     norm = NONE gives s = 1 which is exactly -grad of Eq. (rmf-obj);
 *   - the regulariser enters once per factor row (-2 lambda x), not once per entry;
 *   - the clip acts on the aggregated, normalised, regularised direction;
 *     CLIP_ASYM_STEP: D <- min(max(xi,-D), D)   (caps increases at eta*xi);
 *     CLIP_ASYM_GRAD: the same formula applied to the loss gradient g = -D,
 *     then the step is -eta * clip(g);
 *   - both factor updates use the same residuals (Jacobi, simultaneous);
 *   - CLIP_ASYM_ENTRY is the equation of Sec. 5.3 taken literally, entry by entry: every
 *     observed (i,j) contributes its own clipped direction
 *         c_ij = min(max(xi, -d_ij), d_ij),  d_ij = 2 e_ij q_j - 2 lambda p_i   (for p_i),
 *     the contributions of a factor row are added and divided by s (Eq. 9's 1/n), and the
 *     row moves by eta times that.  Here the regulariser sits inside every entry's term, and a
 *     row without entries does not move.  The "gradient sums" returned in this mode are the
 *     sums of the c_ij.
 *
 * The emulation switch (argument bf16_emulate) has three levels: 0 reads the fp32 values; 1 rounds every factor
 * value read to bfloat16 (what the gather-reduce passes of a bf16 template read); 2 is what the tensor-core
 * variant forms (Sec. 5.1, half-precision multiplicands, fp32 accumulation): factors rounded to bfloat16, the
 * observed value r rounded to binary16, and the residual e rounded to bfloat16 before it multiplies a factor
 * row in the two gradient sums.  Level 2 acts on orc_residuals, orc_grad_sums and the aggregated modes of
 * orc_grad_step; the loss and the entry-wise clip treat it as level 1.
 *
 * Pins: every function below is pinned by tests marked "not gpu" (hand-worked
 * 3x2 and 8x6 examples stored as golden text, finite differences of the loss,
 * zero gradient at the true factors, the dense special case against numpy,
 * the trace identity, the single-entry case, monotone loss, closed form of the
 * clip, and the layout against numpy.lexsort).  The bf16 path has no exact pin
 * beyond the emulation switch (inputs rounded to bf16, round-to-nearest-even):
 * the rounding function itself is pinned against a table of hand-derived bit
 * patterns, and what the switch rounds is pinned in both branches: the aggregated
 * modes against the plain oracle on pre-rounded inputs (regulariser on the fp32
 * master), the entry-wise clip by a hand-worked value and the same identity
 * (there the regulariser sits inside each entry's term and reads the rounded value).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORC_CLIP_NONE = 0, ORC_CLIP_ASYM_STEP = 1, ORC_CLIP_ASYM_GRAD = 2, ORC_CLIP_ASYM_ENTRY = 3 };
enum { ORC_NORM_NONE = 0, ORC_NORM_COUNT = 1 };

/* Round a float to the nearest bfloat16 (ties to even) and return it as float.
 * bfloat16 keeps the top 16 bits of the IEEE-754 binary32 pattern. */
float orc_bf16_round(float x) {
  uint32_t u;
  memcpy(&u, &x, 4);
  if ((u & 0x7f800000u) == 0x7f800000u) { /* inf / nan: truncate, keep nan a nan */
    if (u & 0x007fffffu) u |= 0x00400000u;
    u &= 0xffff0000u;
  } else {
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    u &= 0xffff0000u;
  }
  float y;
  memcpy(&y, &u, 4);
  return y;
}

/* Round a float to the nearest IEEE-754 binary16 value (ties to even) and return it as float.  Values that
 * round beyond the largest half (65504) become infinity; below 2^-14 the half grid is k * 2^-24. */
float orc_fp16_round(float x) {
  uint32_t u;
  memcpy(&u, &x, 4);
  uint32_t a = u & 0x7fffffffu;
  if (a >= 0x7f800000u) return x;                       /* inf / nan */
  if (a < 0x38800000u) {                                /* |x| < 2^-14: subnormal halves */
    double q = rint((double)x * 16777216.0);            /* nearest even multiple of 2^-24 (default rounding mode) */
    return (float)(q / 16777216.0);
  }
  uint32_t lsb = (u >> 13) & 1u;
  u += 0x0fffu + lsb;
  u &= 0xffffe000u;
  if ((u & 0x7fffffffu) >= 0x47800000u) u = (u & 0x80000000u) | 0x7f800000u;   /* 65520 and beyond: infinity */
  float y;
  memcpy(&y, &u, 4);
  return y;
}

/* Sec. 5.3: the nested clip, written exactly as printed. */
double orc_clip_nested(double g, double xi) {
  double a = (xi > -g) ? xi : -g;   /* max(xi, -g) */
  return (a < g) ? a : g;           /* min(.., g)  */
}

static double read_factor(const float *X, int64_t idx, int bf16_emulate) {
  float v = X[idx];
  if (bf16_emulate) v = orc_bf16_round(v);
  return (double)v;
}

/* e_t = r_t - sum_l P[i_t,l] Q[j_t,l], t in input order (Eqs. update-p/q: the
 * factor (R_ji - p_j q_i^T)). */
void orc_residuals(int32_t m, int32_t n, int32_t k, int64_t nnz,
                   const int32_t *rows, const int32_t *cols, const float *vals,
                   const float *P, const float *Q, int bf16_emulate, double *e_out) {
  (void)m; (void)n;
  for (int64_t t = 0; t < nnz; ++t) {
    int64_t i = rows[t], j = cols[t];
    double dot = 0.0;
    for (int32_t l = 0; l < k; ++l)
      dot += read_factor(P, i * k + l, bf16_emulate) * read_factor(Q, j * k + l, bf16_emulate);
    if (bf16_emulate == 2) e_out[t] = (double)orc_bf16_round((float)((double)orc_fp16_round(vals[t]) - dot));
    else e_out[t] = (double)vals[t] - dot;
  }
}

/* Raw gradient sums G_P = E Q (m x k), G_Q = E^T P (n x k) and the per-row /
 * per-column observation counts.  Outputs are overwritten. */
void orc_grad_sums(int32_t m, int32_t n, int32_t k, int64_t nnz,
                   const int32_t *rows, const int32_t *cols, const float *vals,
                   const float *P, const float *Q, int bf16_emulate,
                   double *GP, double *GQ, int64_t *cntP, int64_t *cntQ) {
  memset(GP, 0, sizeof(double) * (size_t)m * k);
  memset(GQ, 0, sizeof(double) * (size_t)n * k);
  memset(cntP, 0, sizeof(int64_t) * (size_t)m);
  memset(cntQ, 0, sizeof(int64_t) * (size_t)n);
  for (int64_t t = 0; t < nnz; ++t) {
    int64_t i = rows[t], j = cols[t];
    double dot = 0.0;
    for (int32_t l = 0; l < k; ++l)
      dot += read_factor(P, i * k + l, bf16_emulate) * read_factor(Q, j * k + l, bf16_emulate);
    double e = (double)vals[t] - dot;
    if (bf16_emulate == 2) e = (double)orc_bf16_round((float)((double)orc_fp16_round(vals[t]) - dot));
    for (int32_t l = 0; l < k; ++l) {
      GP[i * k + l] += e * read_factor(Q, j * k + l, bf16_emulate);
      GQ[j * k + l] += e * read_factor(P, i * k + l, bf16_emulate);
    }
    cntP[i] += 1;
    cntQ[j] += 1;
  }
}

/* Direction for one factor matrix: D = 2 G / s - 2 lambda X, then the clip.
 * X is the fp32 master value (never the bf16-rounded one). */
static void direction(int64_t nrow, int32_t k, const double *G, const int64_t *cnt,
                      const float *X, double lambda, double xi, int clip, int norm,
                      double *D) {
  for (int64_t r = 0; r < nrow; ++r) {
    double s = 1.0;
    if (norm == ORC_NORM_COUNT) s = (cnt[r] > 1) ? (double)cnt[r] : 1.0;
    for (int32_t l = 0; l < k; ++l) {
      double d = 2.0 * G[r * k + l] / s - 2.0 * lambda * (double)X[r * k + l];
      if (clip == ORC_CLIP_ASYM_STEP) {
        d = orc_clip_nested(d, xi);
      } else if (clip == ORC_CLIP_ASYM_GRAD) {
        d = -orc_clip_nested(-d, xi);
      }
      D[r * k + l] = d;
    }
  }
}

/* One full-batch step.  P, Q are read; P_new, Q_new (fp32, may alias nothing)
 * receive x + eta D rounded once to fp32.  GP, GQ (double, m*k / n*k) receive
 * the raw sums; DP, DQ (double) the clipped directions.  Any of GP/GQ/DP/DQ
 * must be valid buffers (the caller allocates). */
void orc_grad_step(int32_t m, int32_t n, int32_t k, int64_t nnz,
                   const int32_t *rows, const int32_t *cols, const float *vals,
                   const float *P, const float *Q,
                   double eta, double lambda, double xi,
                   int clip, int norm_p, int norm_q, int bf16_emulate,
                   double *GP, double *GQ, double *DP, double *DQ,
                   float *P_new, float *Q_new) {
  int64_t *cntP = (int64_t *)malloc(sizeof(int64_t) * (size_t)(m > 0 ? m : 1));
  int64_t *cntQ = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n > 0 ? n : 1));
  if (clip == ORC_CLIP_ASYM_ENTRY) {
    memset(GP, 0, sizeof(double) * (size_t)m * k);
    memset(GQ, 0, sizeof(double) * (size_t)n * k);
    memset(cntP, 0, sizeof(int64_t) * (size_t)(m > 0 ? m : 1));
    memset(cntQ, 0, sizeof(int64_t) * (size_t)(n > 0 ? n : 1));
    for (int64_t t = 0; t < nnz; ++t) {
      int64_t i = rows[t], j = cols[t];
      double dot = 0.0;
      for (int32_t l = 0; l < k; ++l)
        dot += read_factor(P, i * k + l, bf16_emulate) * read_factor(Q, j * k + l, bf16_emulate);
      double e = (double)vals[t] - dot;
      for (int32_t l = 0; l < k; ++l) {
        double pv = read_factor(P, i * k + l, bf16_emulate), qv = read_factor(Q, j * k + l, bf16_emulate);
        GP[i * k + l] += orc_clip_nested(2.0 * e * qv - 2.0 * lambda * pv, xi);
        GQ[j * k + l] += orc_clip_nested(2.0 * e * pv - 2.0 * lambda * qv, xi);
      }
      cntP[i] += 1;
      cntQ[j] += 1;
    }
    for (int64_t r = 0; r < m; ++r) {
      double sc = (norm_p == ORC_NORM_COUNT && cntP[r] > 1) ? (double)cntP[r] : 1.0;
      for (int32_t l = 0; l < k; ++l) DP[r * k + l] = GP[r * k + l] / sc;
    }
    for (int64_t r = 0; r < n; ++r) {
      double sc = (norm_q == ORC_NORM_COUNT && cntQ[r] > 1) ? (double)cntQ[r] : 1.0;
      for (int32_t l = 0; l < k; ++l) DQ[r * k + l] = GQ[r * k + l] / sc;
    }
  } else {
    orc_grad_sums(m, n, k, nnz, rows, cols, vals, P, Q, bf16_emulate, GP, GQ, cntP, cntQ);
    direction(m, k, GP, cntP, P, lambda, xi, clip, norm_p, DP);
    direction(n, k, GQ, cntQ, Q, lambda, xi, clip, norm_q, DQ);
  }
  for (int64_t a = 0; a < (int64_t)m * k; ++a) P_new[a] = (float)((double)P[a] + eta * DP[a]);
  for (int64_t a = 0; a < (int64_t)n * k; ++a) Q_new[a] = (float)((double)Q[a] + eta * DQ[a]);
  free(cntP);
  free(cntQ);
}

/* SSE = sum e^2 and obj = SSE + lambda (|P|_F^2 + |Q|_F^2), Eq. (rmf-obj). */
void orc_loss(int32_t m, int32_t n, int32_t k, int64_t nnz,
              const int32_t *rows, const int32_t *cols, const float *vals,
              const float *P, const float *Q, double lambda, int bf16_emulate,
              double *sse_out, double *obj_out) {
  double sse = 0.0;
  for (int64_t t = 0; t < nnz; ++t) {
    int64_t i = rows[t], j = cols[t];
    double dot = 0.0;
    for (int32_t l = 0; l < k; ++l)
      dot += read_factor(P, i * k + l, bf16_emulate) * read_factor(Q, j * k + l, bf16_emulate);
    double e = (double)vals[t] - dot;
    sse += e * e;
  }
  double reg = 0.0;
  for (int64_t a = 0; a < (int64_t)m * k; ++a) reg += (double)P[a] * (double)P[a];
  for (int64_t a = 0; a < (int64_t)n * k; ++a) reg += (double)Q[a] * (double)Q[a];
  *sse_out = sse;
  *obj_out = sse + lambda * reg;
}

/* `epochs` steps in place on P, Q.  If sse_hist is non-null it receives
 * epochs+1 values: the SSE before the first step and after every step. */
void orc_fit(int32_t m, int32_t n, int32_t k, int64_t nnz,
             const int32_t *rows, const int32_t *cols, const float *vals,
             float *P, float *Q, int32_t epochs,
             double eta, double lambda, double xi,
             int clip, int norm_p, int norm_q, int bf16_emulate, double *sse_hist) {
  size_t mk = (size_t)m * k, nk = (size_t)n * k;
  double *GP = (double *)malloc(sizeof(double) * (mk ? mk : 1));
  double *GQ = (double *)malloc(sizeof(double) * (nk ? nk : 1));
  double *DP = (double *)malloc(sizeof(double) * (mk ? mk : 1));
  double *DQ = (double *)malloc(sizeof(double) * (nk ? nk : 1));
  float *Pn = (float *)malloc(sizeof(float) * (mk ? mk : 1));
  float *Qn = (float *)malloc(sizeof(float) * (nk ? nk : 1));
  double obj;
  if (sse_hist) orc_loss(m, n, k, nnz, rows, cols, vals, P, Q, lambda, bf16_emulate, &sse_hist[0], &obj);
  for (int32_t ep = 0; ep < epochs; ++ep) {
    orc_grad_step(m, n, k, nnz, rows, cols, vals, P, Q, eta, lambda, xi, clip, norm_p, norm_q,
                  bf16_emulate, GP, GQ, DP, DQ, Pn, Qn);
    memcpy(P, Pn, sizeof(float) * mk);
    memcpy(Q, Qn, sizeof(float) * nk);
    if (sse_hist)
      orc_loss(m, n, k, nnz, rows, cols, vals, P, Q, lambda, bf16_emulate, &sse_hist[ep + 1], &obj);
  }
  free(GP); free(GQ); free(DP); free(DQ); free(Pn); free(Qn);
}

/* Layout: order entry ids by (row, col, input position) -> CSR and by
 * (col, row, input position) -> CSC; perm[t] = CSR position of CSC entry t.
 * The order is unique when Omega is a set; ties (duplicates) break by input
 * position. */
typedef struct { int32_t a, b; int64_t id; } orc_key_t;

static int key_cmp(const void *x, const void *y) {
  const orc_key_t *u = (const orc_key_t *)x, *v = (const orc_key_t *)y;
  if (u->a != v->a) return (u->a < v->a) ? -1 : 1;
  if (u->b != v->b) return (u->b < v->b) ? -1 : 1;
  if (u->id != v->id) return (u->id < v->id) ? -1 : 1;
  return 0;
}

void orc_layout(int32_t m, int32_t n, int64_t nnz,
                const int32_t *rows, const int32_t *cols, const float *vals,
                int64_t *row_ptr, int32_t *col_idx, float *val_csr,
                int64_t *col_ptr, int32_t *row_idx, float *val_csc, uint32_t *perm) {
  orc_key_t *keys = (orc_key_t *)malloc(sizeof(orc_key_t) * (size_t)(nnz > 0 ? nnz : 1));
  int64_t *csr_pos = (int64_t *)malloc(sizeof(int64_t) * (size_t)(nnz > 0 ? nnz : 1));
  /* CSR */
  for (int64_t t = 0; t < nnz; ++t) { keys[t].a = rows[t]; keys[t].b = cols[t]; keys[t].id = t; }
  qsort(keys, (size_t)nnz, sizeof(orc_key_t), key_cmp);
  for (int64_t i = 0; i <= m; ++i) row_ptr[i] = 0;
  for (int64_t p = 0; p < nnz; ++p) {
    int64_t t = keys[p].id;
    col_idx[p] = cols[t];
    val_csr[p] = vals[t];
    csr_pos[t] = p;
    row_ptr[(int64_t)rows[t] + 1] += 1;
  }
  for (int64_t i = 0; i < m; ++i) row_ptr[i + 1] += row_ptr[i];
  /* CSC */
  for (int64_t t = 0; t < nnz; ++t) { keys[t].a = cols[t]; keys[t].b = rows[t]; keys[t].id = t; }
  qsort(keys, (size_t)nnz, sizeof(orc_key_t), key_cmp);
  for (int64_t j = 0; j <= n; ++j) col_ptr[j] = 0;
  for (int64_t p = 0; p < nnz; ++p) {
    int64_t t = keys[p].id;
    row_idx[p] = rows[t];
    val_csc[p] = vals[t];
    perm[p] = (uint32_t)csr_pos[t];
    col_ptr[(int64_t)cols[t] + 1] += 1;
  }
  for (int64_t j = 0; j < n; ++j) col_ptr[j + 1] += col_ptr[j];
  free(keys);
  free(csr_pos);
}

/* ---- template sampling (Sec. 5.1, "Sampling the TSID Template Submatrix") ---------------------
 * C = d = ceil(alpha n) columns drawn uniformly at random without replacement; the template keeps
 * the observed entries whose column is in C.  Readings: the draw is made reproducible by giving
 * column j the key SplitMix64(seed + (j+1) * 0x9E3779B97F4A7C15), i.e. the (j+1)-th output of the
 * SplitMix64 generator seeded with `seed`, and taking the d columns with the smallest (key, j)
 * (a uniformly random d-subset); the chosen columns are re-indexed 0..d-1 in ascending order of
 * their original index; rows are unchanged; kept entries stay in input order.
 * Pins: published SplitMix64 outputs; |C| = d; brute-force membership; inclusion frequency. */
uint64_t orc_splitmix64_at(uint64_t seed, uint64_t index1) {
  uint64_t z = seed + index1 * 0x9E3779B97F4A7C15ULL;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}

typedef struct { uint64_t key; int32_t col; } orc_colkey_t;

static int colkey_cmp(const void *x, const void *y) {
  const orc_colkey_t *u = (const orc_colkey_t *)x, *v = (const orc_colkey_t *)y;
  if (u->key != v->key) return (u->key < v->key) ? -1 : 1;
  if (u->col != v->col) return (u->col < v->col) ? -1 : 1;
  return 0;
}

/* colmap[n] receives the new column index or -1; the *_out arrays need capacity nnz.
 * Returns d through d_out and the number of kept entries through nnz_out. */
void orc_sample_template(int32_t m, int32_t n, int64_t nnz, double alpha, uint64_t seed,
                         const int32_t *rows, const int32_t *cols, const float *vals,
                         int32_t *colmap, int32_t *rows_out, int32_t *cols_out, float *vals_out,
                         int32_t *d_out, int64_t *nnz_out) {
  (void)m;
  double dd = ceil(alpha * (double)n);
  int32_t d = dd < 1.0 ? 1 : (dd > (double)n ? n : (int32_t)dd);
  orc_colkey_t *ck = (orc_colkey_t *)malloc(sizeof(orc_colkey_t) * (size_t)n);
  for (int32_t j = 0; j < n; ++j) { ck[j].key = orc_splitmix64_at(seed, (uint64_t)j + 1); ck[j].col = j; }
  qsort(ck, (size_t)n, sizeof(orc_colkey_t), colkey_cmp);
  for (int32_t j = 0; j < n; ++j) colmap[j] = -1;
  for (int32_t q = 0; q < d; ++q) colmap[ck[q].col] = 0;      /* chosen */
  int32_t next = 0;
  for (int32_t j = 0; j < n; ++j) if (colmap[j] == 0) colmap[j] = next++;
  int64_t o = 0;
  for (int64_t t = 0; t < nnz; ++t) {
    int32_t c = colmap[cols[t]];
    if (c >= 0) { rows_out[o] = rows[t]; cols_out[o] = c; vals_out[o] = vals[t]; ++o; }
  }
  *d_out = d;
  *nnz_out = o;
  free(ck);
}

/* ---- Stage II: template-conditioned extension (Sec. 5.2, Eq. 10) ---------------------------------
 * With the template estimate Rhat* = P Q^T (m x d) fixed, every column j of the full matrix gets a
 * coefficient vector C_j in R^d minimising
 *       L_j(C_j) = sum_{i in Omega^j} (R_ij - Rhat*_i C_j)^2 + lambda |C_j|^2        (Eq. 10, per column)
 * by gradient steps through Adam (Kingma & Ba, Algorithm 1):
 *       g = -2 Rhat*_{Omega^j}^T e + 2 lambda C_j,     e_i = R_ij - Rhat*_i C_j
 *       m <- b1 m + (1-b1) g,  v <- b2 v + (1-b2) g^2,  C_j <- C_j - eta (m/(1-b1^t)) / (sqrt(v/(1-b2^t)) + eps)
 * Readings: C starts at the values passed in (zeros in the tests and the bench); Adam's constants are
 * arguments (the paper names the optimiser only); the objective decomposes over columns, so a chunk is
 * just a set of columns and chunking cannot change the result; `iters` steps per column.
 * The loops below follow the definition with Rhat* materialised (no factored shortcut).
 * Layout: column-compressed input (col_ptr[ncols+1], row_idx, vals); C is stored one column after the
 * other, C[j*d + a].  sse_out (may be NULL) receives sum_Omega e^2 at the returned C. */
void orc_extend(int32_t m, int32_t d, int32_t k, int32_t ncols, const int64_t *col_ptr,
                const int32_t *row_idx, const float *vals, const float *P, const float *Q,
                double eta, double lambda, double b1, double b2, double eps, int32_t iters,
                double *C, double *sse_out) {
  double *Rhat = (double *)malloc(sizeof(double) * (size_t)m * d);
  for (int32_t i = 0; i < m; ++i)
    for (int32_t a = 0; a < d; ++a) {
      double s = 0.0;
      for (int32_t l = 0; l < k; ++l) s += (double)P[(size_t)i * k + l] * (double)Q[(size_t)a * k + l];
      Rhat[(size_t)i * d + a] = s;
    }
  double *g = (double *)malloc(sizeof(double) * (size_t)d);
  double *mo = (double *)malloc(sizeof(double) * (size_t)d);
  double *vo = (double *)malloc(sizeof(double) * (size_t)d);
  double sse = 0.0;
  for (int32_t j = 0; j < ncols; ++j) {
    double *Cj = C + (size_t)j * d;
    for (int32_t a = 0; a < d; ++a) { mo[a] = 0.0; vo[a] = 0.0; }
    double p1 = 1.0, p2 = 1.0;
    for (int32_t it = 1; it <= iters; ++it) {
      for (int32_t a = 0; a < d; ++a) g[a] = 2.0 * lambda * Cj[a];
      for (int64_t t = col_ptr[j]; t < col_ptr[j + 1]; ++t) {
        const double *rh = Rhat + (size_t)row_idx[t] * d;
        double pred = 0.0;
        for (int32_t a = 0; a < d; ++a) pred += rh[a] * Cj[a];
        double e = (double)vals[t] - pred;
        for (int32_t a = 0; a < d; ++a) g[a] -= 2.0 * e * rh[a];
      }
      p1 *= b1; p2 *= b2;
      for (int32_t a = 0; a < d; ++a) {
        mo[a] = b1 * mo[a] + (1.0 - b1) * g[a];
        vo[a] = b2 * vo[a] + (1.0 - b2) * g[a] * g[a];
        double mh = mo[a] / (1.0 - p1), vh = vo[a] / (1.0 - p2);
        Cj[a] -= eta * mh / (sqrt(vh) + eps);
      }
    }
    for (int64_t t = col_ptr[j]; t < col_ptr[j + 1]; ++t) {
      const double *rh = Rhat + (size_t)row_idx[t] * d;
      double pred = 0.0;
      for (int32_t a = 0; a < d; ++a) pred += rh[a] * Cj[a];
      double e = (double)vals[t] - pred;
      sse += e * e;
    }
  }
  if (sse_out) *sse_out = sse;
  free(Rhat); free(g); free(mo); free(vo);
}

/* Stage II in the paper's mixed precision (Sec. 5.2: the products of Stage II run with half-precision operands
 * and fp32 accumulation).  The same Adam iteration as orc_extend, but written in the factored form in which the
 * mixed-precision products appear, with the operands of exactly those two products rounded to bfloat16 (nearest
 * even) and every sum exact:
 *       W_j = Q^T bf(C_j)            first product   (k values: Rhat*_i C_j = p_i . W_j)
 *       e_i = R_ij - p_i . W_j ,  U_j = sum_i e_i p_i                         (full precision)
 *       g   = -2 bf(Q) bf(U_j) + 2 lambda C_j       second product
 * bf(.) = bfloat16 rounding; Q is rounded in both products; C, the Adam moments, the residuals and U stay in
 * full precision (C is rounded only where it enters the first product; it is first taken to fp32, the precision
 * the stored coefficients have).  With rounding switched off this is orc_extend re-associated, which is how it is
 * pinned (besides dense algebra with library casts for where the rounding sits). */
void orc_extend_mixed(int32_t m, int32_t d, int32_t k, int32_t ncols, const int64_t *col_ptr,
                      const int32_t *row_idx, const float *vals, const float *P, const float *Q,
                      double eta, double lambda, double b1, double b2, double eps, int32_t iters,
                      int round_operands, double *C, double *sse_out) {
  (void)m;
  double *Qr = (double *)malloc(sizeof(double) * (size_t)d * k);
  for (size_t a = 0; a < (size_t)d * k; ++a) Qr[a] = round_operands ? (double)orc_bf16_round(Q[a]) : (double)Q[a];
  double *W = (double *)malloc(sizeof(double) * (size_t)k);
  double *U = (double *)malloc(sizeof(double) * (size_t)k);
  double *mo = (double *)malloc(sizeof(double) * (size_t)d);
  double *vo = (double *)malloc(sizeof(double) * (size_t)d);
  double sse = 0.0;
  for (int32_t j = 0; j < ncols; ++j) {
    double *Cj = C + (size_t)j * d;
    for (int32_t a = 0; a < d; ++a) { mo[a] = 0.0; vo[a] = 0.0; }
    double p1 = 1.0, p2 = 1.0;
    for (int32_t it = 1; it <= iters + 1; ++it) {          /* the extra round only evaluates the SSE */
      for (int32_t l = 0; l < k; ++l) W[l] = 0.0;
      for (int32_t a = 0; a < d; ++a) {
        double c = round_operands ? (double)orc_bf16_round((float)Cj[a]) : Cj[a];
        for (int32_t l = 0; l < k; ++l) W[l] += c * Qr[(size_t)a * k + l];
      }
      for (int32_t l = 0; l < k; ++l) U[l] = 0.0;
      for (int64_t t = col_ptr[j]; t < col_ptr[j + 1]; ++t) {
        const float *pi = P + (size_t)row_idx[t] * k;
        double pred = 0.0;
        for (int32_t l = 0; l < k; ++l) pred += (double)pi[l] * W[l];
        double e = (double)vals[t] - pred;
        if (it > iters) sse += e * e;
        for (int32_t l = 0; l < k; ++l) U[l] += e * (double)pi[l];
      }
      if (it > iters) break;
      if (round_operands) for (int32_t l = 0; l < k; ++l) U[l] = (double)orc_bf16_round((float)U[l]);
      p1 *= b1; p2 *= b2;
      for (int32_t a = 0; a < d; ++a) {
        double qu = 0.0;
        for (int32_t l = 0; l < k; ++l) qu += Qr[(size_t)a * k + l] * U[l];
        double g = -2.0 * qu + 2.0 * lambda * Cj[a];
        mo[a] = b1 * mo[a] + (1.0 - b1) * g;
        vo[a] = b2 * vo[a] + (1.0 - b2) * g * g;
        double mh = mo[a] / (1.0 - p1), vh = vo[a] / (1.0 - p2);
        Cj[a] -= eta * mh / (sqrt(vh) + eps);
      }
    }
  }
  if (sse_out) *sse_out = sse;
  free(Qr); free(W); free(U); free(mo); free(vo);
}

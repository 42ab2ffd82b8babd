/*
 * star_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, obviously-correct CPU statement of the row-typed associative-algebra
 * projection Y = X *_q W and of the two-map FFN built from it.  Everything is fp64 (small
 * integers are therefore summed exactly).  It shares no code, header, table or helper with
 * the CUDA library; only tests, the smoke check and the benchmark's CPU-baseline leg may
 * call it.
 *
 * Notation (Section "Transformer Projections"): X is M x K, W is the ordinary K x N weight
 * bank, input features are split into q groups of widths s[0..q-1] (sum K), output features
 * into q groups of widths r[0..q-1] (sum N); W_{kj} is the s[k] x r[j] sub-block
 * W[S_k, R_j].  Row b has type t[b] in [0,q) (0-based here; the paper counts from 1).
 *
 * Pins (all in tests/test_oracle_pins.py): hand-derived scalar examples, the six-product
 * rule term by term, dense-minus-removed brute force, associativity/unit/edge-ideal on
 * integer block arrays, the 2q^2-q count and the MAC formulas, q=1 / dense table against
 * numpy.matmul, GELU and SiLU against closed-form values, the gated FFN against an
 * independent numpy composition, the two gradient maps against the displayed per-type equations
 * and against the adjoint identities <X * W, G> = <X, dX(G)> = <W, dW(X, G)>.
 * Parity unpinned by the paper: the FFN-level choices (erf-GELU, bias added before the
 * activation) come from the benchmark specification, not from a printed value; SwiGLU is
 * named by the paper without its formula (the standard one is taken).
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC star_oracle.c -o libstar_oracle.so -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_BAD_ARG 1
#define ORACLE_BAD_TYPE 2

int star_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ---------------------------------------------------------------------------------------
 * Support sets.  keep[(i*q + j)*q + k] = 1 iff group k belongs to B(i,j), i.e. a row of
 * type i adds x_k W_{kj} into output group j  (Eq. recursive-row-action).
 * ------------------------------------------------------------------------------------- */

/* Complete-graph law Q_q: B(i,j) = {i,j} as a set (Eqs. typed-diag / typed-off). */
int star_support_qq(int q, uint8_t *keep) {
  if (q < 1 || !keep) return ORACLE_BAD_ARG;
  memset(keep, 0, (size_t)q * q * q);
  for (int i = 0; i < q; ++i)
    for (int j = 0; j < q; ++j) {
      keep[((size_t)i * q + j) * q + i] = 1; /* x_i W_ij  */
      keep[((size_t)i * q + j) * q + j] = 1; /* x_j W_jj  (same entry when i == j) */
    }
  return ORACLE_OK;
}

/* Ordinary matrix product: every group meets every weight block (Eq. dense-two). */
int star_support_dense(int q, uint8_t *keep) {
  if (q < 1 || !keep) return ORACLE_BAD_ARG;
  memset(keep, 1, (size_t)q * q * q);
  return ORACLE_OK;
}

/* Tensor power Q_2^{(x)L}: groups and types are L-bit strings; beta is in B(alpha,delta)
 * iff every bit of beta equals the matching bit of alpha or of delta
 * (Appendix "The Tensor-Square Candidate", Eq. recursive-unequal-cost). q = 2^L. */
int star_support_q2_power(int L, uint8_t *keep) {
  if (L < 1 || L > 5 || !keep) return ORACLE_BAD_ARG;
  int q = 1 << L;
  for (int a = 0; a < q; ++a)
    for (int d = 0; d < q; ++d)
      for (int b = 0; b < q; ++b) {
        int ok = 1;
        for (int bit = 0; bit < L; ++bit) {
          int ab = (a >> bit) & 1, db = (d >> bit) & 1, bb = (b >> bit) & 1;
          if (bb != ab && bb != db) ok = 0;
        }
        keep[((size_t)a * q + d) * q + b] = (uint8_t)ok;
      }
  return ORACLE_OK;
}

/* Number of block GEMMs the rule keeps: |{(i,j,k): k in B(i,j)}|  (2q^2-q for Q_q). */
int64_t star_gemm_count(int q, const uint8_t *keep) {
  int64_t n = 0;
  for (size_t e = 0; e < (size_t)q * q * q; ++e) n += keep[e] ? 1 : 0;
  return n;
}

/* Forward MACs of a batch with rows_per_type[i] rows of type i: sum over kept (i,j,k) of
 * M_i * s_k * r_j, counted term by term (to be compared with Eq. rectangular-batch-cost). */
int64_t star_macs(int q, const uint8_t *keep, const int32_t *s, const int32_t *r,
                  const int64_t *rows_per_type) {
  int64_t macs = 0;
  for (int i = 0; i < q; ++i)
    for (int j = 0; j < q; ++j)
      for (int k = 0; k < q; ++k)
        if (keep[((size_t)i * q + j) * q + k]) macs += rows_per_type[i] * (int64_t)s[k] * r[j];
  return macs;
}

static void prefix(int q, const int32_t *w, int64_t *off) {
  off[0] = 0;
  for (int g = 0; g < q; ++g) off[g + 1] = off[g] + w[g];
}

/* ---------------------------------------------------------------------------------------
 * Row-typed projection, per-row form (Eq. recursive-row-action):
 *   for row b of type i, output group j:  y_j = bias_j + sum_{k in B(i,j)} x_k W_{kj}.
 * X: M x K (ldx), W: K x N (ldw), Y: M x N (ldy), all row-major, leading dims in elements.
 * bias: N values or NULL.  Y is overwritten.
 * ------------------------------------------------------------------------------------- */
int star_proj_rows(const double *X, int64_t ldx, const int32_t *types, int64_t M,
                   const double *W, int64_t ldw, const double *bias, double *Y, int64_t ldy,
                   int q, const int32_t *s, const int32_t *r, const uint8_t *keep) {
  if (q < 1 || M < 0 || !s || !r || !keep) return ORACLE_BAD_ARG;
  int64_t *so = (int64_t *)malloc(sizeof(int64_t) * (q + 1));
  int64_t *ro = (int64_t *)malloc(sizeof(int64_t) * (q + 1));
  prefix(q, s, so);
  prefix(q, r, ro);
  int bad = 0;
  for (int64_t b = 0; b < M; ++b)
    if (types[b] < 0 || types[b] >= q) bad = 1;
  if (!bad) {
#pragma omp parallel for schedule(static)
    for (int64_t b = 0; b < M; ++b) {
      const int i = types[b];
      const double *x = X + b * ldx;
      double *y = Y + b * ldy;
      for (int j = 0; j < q; ++j) {
        for (int64_t n = ro[j]; n < ro[j + 1]; ++n) y[n] = bias ? bias[n] : 0.0;
        for (int k = 0; k < q; ++k) {
          if (!keep[((size_t)i * q + j) * q + k]) continue;
          for (int64_t c = so[k]; c < so[k + 1]; ++c) {
            const double xv = x[c];
            const double *w = W + c * ldw;
            for (int64_t n = ro[j]; n < ro[j + 1]; ++n) y[n] += xv * w[n];
          }
        }
      }
    }
  }
  free(so);
  free(ro);
  return bad ? ORACLE_BAD_TYPE : ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------
 * Single output entries of the same projection, straight from the definition
 * (Eq. recursive-row-action): for e = 0..n_entries-1 with (b, n) = (rows[e], cols[e]), n in
 * output group j,   out[e] = bias[n] + sum_{k in B(t_b, j)} sum_{c in S_k} X[b,c] W[c,n].
 * Lets the tests sample outputs of problems far too large to compute in full.
 * ------------------------------------------------------------------------------------- */
int star_proj_entries(const double *X, int64_t ldx, const int32_t *types, int64_t M,
                      const double *W, int64_t ldw, const double *bias, int q,
                      const int32_t *s, const int32_t *r, const uint8_t *keep,
                      const int64_t *rows, const int64_t *cols, int64_t n_entries, double *out) {
  if (q < 1 || M < 0 || n_entries < 0 || !s || !r || !keep) return ORACLE_BAD_ARG;
  int64_t *so = (int64_t *)malloc(sizeof(int64_t) * (q + 1));
  int64_t *ro = (int64_t *)malloc(sizeof(int64_t) * (q + 1));
  prefix(q, s, so);
  prefix(q, r, ro);
  int rc = ORACLE_OK;
  for (int64_t e = 0; e < n_entries; ++e) {
    if (rows[e] < 0 || rows[e] >= M || cols[e] < 0 || cols[e] >= ro[q]) rc = ORACLE_BAD_ARG;
    else if (types[rows[e]] < 0 || types[rows[e]] >= q) rc = ORACLE_BAD_TYPE;
  }
  if (rc == ORACLE_OK) {
#pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < n_entries; ++e) {
      const int64_t b = rows[e], n = cols[e];
      const int i = types[b];
      int j = 0;
      while (n >= ro[j + 1]) ++j;
      double acc = bias ? bias[n] : 0.0;
      for (int k = 0; k < q; ++k) {
        if (!keep[((size_t)i * q + j) * q + k]) continue;
        for (int64_t c = so[k]; c < so[k + 1]; ++c) acc += X[b * ldx + c] * W[c * ldw + n];
      }
      out[e] = acc;
    }
  }
  free(so);
  free(ro);
  return rc;
}

/* ---------------------------------------------------------------------------------------
 * The same function evaluated type by type, as Algorithm 1 organises a batch: the rows of one
 * type are collected first, then every kept (input group, output group) pair of that type
 * contributes one rectangular product to those rows of Y (which starts from zero).
 * Written separately from star_proj_rows so the two can be tested against each other.
 * ------------------------------------------------------------------------------------- */
int star_proj_alg1(const double *X, int64_t ldx, const int32_t *types, int64_t M,
                   const double *W, int64_t ldw, double *Y, int64_t ldy, int q,
                   const int32_t *s, const int32_t *r, const uint8_t *keep) {
  if (q < 1 || M < 0 || !s || !r || !keep) return ORACLE_BAD_ARG;
  int64_t *so = (int64_t *)malloc(sizeof(int64_t) * (q + 1));
  int64_t *ro = (int64_t *)malloc(sizeof(int64_t) * (q + 1));
  int64_t *I = (int64_t *)malloc(sizeof(int64_t) * (M > 0 ? M : 1));
  prefix(q, s, so);
  prefix(q, r, ro);
  for (int64_t b = 0; b < M; ++b) {
    if (types[b] < 0 || types[b] >= q) {
      free(so); free(ro); free(I);
      return ORACLE_BAD_TYPE;
    }
    for (int64_t n = 0; n < ro[q]; ++n) Y[b * ldy + n] = 0.0;
  }
  for (int i = 0; i < q; ++i) {
    int64_t cnt = 0;
    for (int64_t b = 0; b < M; ++b)
      if (types[b] == i) I[cnt++] = b;
    for (int j = 0; j < q; ++j)
      for (int k = 0; k < q; ++k) {
        if (!keep[((size_t)i * q + j) * q + k]) continue;
        /* one rectangular GEMM: (|I_i| x s_k) times (s_k x r_j) */
        for (int64_t a = 0; a < cnt; ++a) {
          const int64_t b = I[a];
          for (int64_t n = ro[j]; n < ro[j + 1]; ++n) {
            double acc = 0.0;
            for (int64_t c = so[k]; c < so[k + 1]; ++c) acc += X[b * ldx + c] * W[c * ldw + n];
            Y[b * ldy + n] += acc;
          }
        }
      }
  }
  free(so); free(ro); free(I);
  return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------
 * Square block form (Eqs. q-product-diag / q-product-off):
 *   (A * B)_ii = A_ii B_ii,   (A * B)_ij = A_ii B_ij + A_ij B_jj  (i != j).
 * A is a q x q array of blocks, block (i,k) of size a[i] x c[k]; B has blocks (k,j) of
 * size c[k] x d[j]; C gets blocks (i,j) of size a[i] x d[j].  Dense row-major storage.
 * ------------------------------------------------------------------------------------- */
static void block_mac(const double *A, int64_t lda, const double *B, int64_t ldb, double *C,
                      int64_t ldc, int64_t m, int64_t kk, int64_t n) {
  for (int64_t x = 0; x < m; ++x)
    for (int64_t y = 0; y < n; ++y) {
      double acc = 0.0;
      for (int64_t z = 0; z < kk; ++z) acc += A[x * lda + z] * B[z * ldb + y];
      C[x * ldc + y] += acc;
    }
}

int star_square(const double *A, const double *B, double *C, int q, const int32_t *a,
                const int32_t *c, const int32_t *d) {
  if (q < 1) return ORACLE_BAD_ARG;
  int64_t *ao = (int64_t *)malloc(sizeof(int64_t) * (q + 1));
  int64_t *co = (int64_t *)malloc(sizeof(int64_t) * (q + 1));
  int64_t *dd = (int64_t *)malloc(sizeof(int64_t) * (q + 1));
  prefix(q, a, ao);
  prefix(q, c, co);
  prefix(q, d, dd);
  const int64_t lda = co[q], ldb = dd[q], ldc = dd[q];
  for (int64_t e = 0; e < ao[q] * ldc; ++e) C[e] = 0.0;
  for (int i = 0; i < q; ++i)
    for (int j = 0; j < q; ++j) {
      double *Cij = C + ao[i] * ldc + dd[j];
      const double *Aii = A + ao[i] * lda + co[i];
      const double *Bij = B + co[i] * ldb + dd[j];
      /* A_ii B_ij : present for every (i,j), and the only term when i == j */
      block_mac(Aii, lda, Bij, ldb, Cij, ldc, a[i], c[i], d[j]);
      if (i != j) {
        const double *Aij = A + ao[i] * lda + co[j];
        const double *Bjj = B + co[j] * ldb + dd[j];
        block_mac(Aij, lda, Bjj, ldb, Cij, ldc, a[i], c[j], d[j]);
      }
    }
  free(ao); free(co); free(dd);
  return ORACLE_OK;
}

/* Exact GELU, gelu(z) = z/2 (1 + erf(z / sqrt 2)). */
double star_gelu(double z) { return 0.5 * z * (1.0 + erf(z * 0.70710678118654752440)); }
/* The same, element by element over an array (in place). */
void star_gelu_array(double *z, int64_t n) {
#pragma omp parallel for schedule(static)
  for (int64_t e = 0; e < n; ++e) z[e] = star_gelu(z[e]);
}

/* ---------------------------------------------------------------------------------------
 * Two-map FFN: H = gelu(X * W_up + b_up),  Y = H * W_down + b_down, same row types for both
 * projections; H is kept in fp64 (never rounded).  d groups: dw[q] (sum D); f groups: fw[q]
 * (sum F).  W_up is D x F, W_down is F x D, both dense row-major; X M x D, Y M x D.
 * H (M x F) is caller-provided scratch so it can be inspected.
 * ------------------------------------------------------------------------------------- */
int star_ffn(const double *X, const int32_t *types, int64_t M, const double *W_up,
             const double *b_up, const double *W_down, const double *b_down, double *H,
             double *Y, int q, const int32_t *dw, const int32_t *fw, const uint8_t *keep) {
  int64_t D = 0, F = 0;
  for (int g = 0; g < q; ++g) { D += dw[g]; F += fw[g]; }
  int rc = star_proj_rows(X, D, types, M, W_up, F, b_up, H, F, q, dw, fw, keep);
  if (rc) return rc;
#pragma omp parallel for schedule(static)
  for (int64_t e = 0; e < M * F; ++e) H[e] = star_gelu(H[e]);
  return star_proj_rows(H, F, types, M, W_down, D, b_down, Y, D, q, fw, dw, keep);
}

/* ---------------------------------------------------------------------------------------
 * Gated FFN (SwiGLU), the FFN of the paper's pretraining pilot (Section "Projection Shapes":
 * two D x F weights and one F x D weight, the same row law on each; Appendix "Experimental
 * Details": bias-free SwiGLU):
 *     G = X * W_gate,   U = X * W_up,   H = silu(G) .* U,   Y = H * W_down,
 * silu(g) = g / (1 + exp(-g)), all three projections under the same support and row types,
 * H kept in fp64 (never rounded).  G, U (M x F each) and H are caller-provided scratch.
 * Parity unpinned by the paper: it names SwiGLU without writing the formula; the standard
 * definition is taken.
 * ------------------------------------------------------------------------------------- */
double star_silu(double g) { return g / (1.0 + exp(-g)); }

int star_ffn_swiglu(const double *X, const int32_t *types, int64_t M, const double *W_gate,
                    const double *W_up, const double *W_down, double *G, double *U, double *H,
                    double *Y, int q, const int32_t *dw, const int32_t *fw, const uint8_t *keep) {
  int64_t D = 0, F = 0;
  for (int g = 0; g < q; ++g) { D += dw[g]; F += fw[g]; }
  int rc = star_proj_rows(X, D, types, M, W_gate, F, NULL, G, F, q, dw, fw, keep);
  if (rc) return rc;
  rc = star_proj_rows(X, D, types, M, W_up, F, NULL, U, F, q, dw, fw, keep);
  if (rc) return rc;
#pragma omp parallel for schedule(static)
  for (int64_t e = 0; e < M * F; ++e) H[e] = star_silu(G[e]) * U[e];
  return star_proj_rows(H, F, types, M, W_down, D, NULL, Y, D, q, fw, dw, keep);
}

/* ---------------------------------------------------------------------------------------
 * Vector-Jacobian products of the row-typed projection (Appendix "Vector-Jacobian Products",
 * Eqs. vjp-xi ... vjp-wjj, written for a general support set): with G the gradient with respect
 * to Y,
 *     dX[b, S_k]   = sum_{j : k in B(t_b, j)} G[b, R_j] W[S_k, R_j]^T
 *     dW[S_k, R_j] = sum_{b : k in B(t_b, j)} X[b, S_k]^T G[b, R_j].
 * Both keep exactly the block support of the forward table; blocks of dW no row reaches stay 0.
 * ------------------------------------------------------------------------------------- */
int star_proj_vjp_x(const double *G, int64_t ldg, const int32_t *types, int64_t M, const double *W,
                    int64_t ldw, double *dX, int64_t lddx, int q, const int32_t *s,
                    const int32_t *r, const uint8_t *keep) {
  if (q < 1 || M < 0 || !s || !r || !keep) return ORACLE_BAD_ARG;
  int64_t *so = (int64_t *)malloc(sizeof(int64_t) * (q + 1));
  int64_t *ro = (int64_t *)malloc(sizeof(int64_t) * (q + 1));
  prefix(q, s, so);
  prefix(q, r, ro);
  int bad = 0;
  for (int64_t b = 0; b < M; ++b)
    if (types[b] < 0 || types[b] >= q) bad = 1;
  if (!bad) {
#pragma omp parallel for schedule(static)
    for (int64_t b = 0; b < M; ++b) {
      const int i = types[b];
      for (int k = 0; k < q; ++k)
        for (int64_t c = so[k]; c < so[k + 1]; ++c) {
          double acc = 0.0;
          for (int j = 0; j < q; ++j) {
            if (!keep[((size_t)i * q + j) * q + k]) continue;
            for (int64_t n = ro[j]; n < ro[j + 1]; ++n) acc += G[b * ldg + n] * W[c * ldw + n];
          }
          dX[b * lddx + c] = acc;
        }
    }
  }
  free(so);
  free(ro);
  return bad ? ORACLE_BAD_TYPE : ORACLE_OK;
}

int star_proj_vjp_w(const double *X, int64_t ldx, const double *G, int64_t ldg,
                    const int32_t *types, int64_t M, double *dW, int64_t lddw, int q,
                    const int32_t *s, const int32_t *r, const uint8_t *keep) {
  if (q < 1 || M < 0 || !s || !r || !keep) return ORACLE_BAD_ARG;
  int64_t *so = (int64_t *)malloc(sizeof(int64_t) * (q + 1));
  int64_t *ro = (int64_t *)malloc(sizeof(int64_t) * (q + 1));
  prefix(q, s, so);
  prefix(q, r, ro);
  int bad = 0;
  for (int64_t b = 0; b < M; ++b)
    if (types[b] < 0 || types[b] >= q) bad = 1;
  if (!bad) {
#pragma omp parallel for schedule(static)
    for (int64_t c = 0; c < so[q]; ++c) {
      int k = 0;
      while (c >= so[k + 1]) ++k;
      for (int j = 0; j < q; ++j)
        for (int64_t n = ro[j]; n < ro[j + 1]; ++n) {
          double acc = 0.0;
          for (int64_t b = 0; b < M; ++b)
            if (keep[((size_t)types[b] * q + j) * q + k]) acc += X[b * ldx + c] * G[b * ldg + n];
          dW[c * lddw + n] = acc;
        }
    }
  }
  free(so);
  free(ro);
  return bad ? ORACLE_BAD_TYPE : ORACLE_OK;
}

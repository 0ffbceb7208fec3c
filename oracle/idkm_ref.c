/*
 * idkm_ref.c -- float64 CPU oracle for the soft k-means fixed point of IDKM and its
 * implicit / Jacobian-free gradients.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of the paper's
 * method that the CUDA library is checked against and that the benchmark times as its
 * CPU baseline.  It shares no code with the CUDA path and the product never calls it.
 *
 * Notation (rows, not the paper's columns): W[m][d] weights w_i, C[k][d] centroids c_j,
 *   D_ij = ||w_i - c_j||_2                      (Algorithm 1, step 3; NOT squared)
 *   A_ij = exp(-D_ij/tau) / sum_l exp(-D_il/tau) (Eq. for a_j(w_i,C); Algorithm 1, step 4)
 *   S_j  = sum_i A_ij,   N_j = sum_i A_ij w_i
 *   F(C,W)_j = N_j / S_j                         (M-step; Eq. "C+ := diag(A^T 1)^-1 A^T W")
 *   Wq_i = sum_j A_ij c_j                        (soft quantiser r_tau, Eq. r_tau(w_i, C))
 *   n_ij = (w_i - c_j)/D_ij, and 0 when D_ij = 0 (a sub-gradient of the norm at its kink)
 *
 * Readings taken where the paper is silent:
 *   - stop rule ||C+ - C|| < eps: Frobenius norm relative to ||C+||_F, strict <, tol = 0
 *     disables the test (fixed iteration count);
 *   - a cluster with S_j < 1e-20 keeps its centroid; in the backward it contributes nothing;
 *   - Wq and all Jacobians are evaluated at the returned centroids C_T ("plug C* into F one
 *     time", Section 4.2): A, S and F_j = F(C_T, W)_j all come from C_T;
 *   - the backward iterates the adjoint vector u <- alpha (J^T u + g) + (1 - alpha) u from
 *     u = g, which has the same limit as the paper's k x k iteration M <- alpha G(M) + (1-alpha) M
 *     (u* = M*^T g); zero adjoint iterations is Jacobian-free backprop (M* = I);
 *   - dL/dC output := u.
 *
 * Variant (idkm_ref_set_squared(1)): the softmax takes the SQUARED distance, D_ij = ||w_i - c_j||^2, the quantity
 * the clustering objectives are written in (Section 3.1, the k-means objective; Section 3.2, the soft objective that
 * the iteration is derived from).  Everything below is written in terms of D_ij and its gradient
 * n_ij = dD_ij/dw_i = -dD_ij/dc_j, so the variant changes two lines: D_ij itself and n_ij = 2 (w_i - c_j), which has
 * no kink.  The method as published (Algorithm 1, step 3) is the default.
 *
 * Sums over i run in NCHUNK fixed row chunks (so that OpenMP may take one chunk per thread)
 * and the chunk sums are added in chunk order: the result does not depend on the thread count.
 * Nothing else is blocked, fused or reordered.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define IDKM_REF_S_MIN 1e-20
#define NCHUNK 64

int idkm_ref_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void idkm_ref_set_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

/* 0: D_ij is the Euclidean norm (Algorithm 1, step 3).  1: its square (the variant described above). */
static int g_squared = 0;

void idkm_ref_set_squared(int on) { g_squared = (on != 0); }
int idkm_ref_get_squared(void) { return g_squared; }

static void chunk_bounds(int64_t m, int c, int64_t *lo, int64_t *hi) {
  *lo = (m * (int64_t)c) / NCHUNK;
  *hi = (m * (int64_t)(c + 1)) / NCHUNK;
}

/* One row of the E-step: distances D_j (Algorithm 1 step 3) and attention A_j
 * (Algorithm 1 step 4 = softmax_tau of -D).  Subtracting the row minimum of D before the
 * exponential leaves A unchanged and avoids 0/0. */
static void attention_row(const double *w, const double *C, int k, int d, double tau, double *D, double *A) {
  double dmin = INFINITY;
  for (int j = 0; j < k; ++j) {
    double s = 0.0;
    for (int a = 0; a < d; ++a) {
      double t = w[a] - C[(int64_t)j * d + a];
      s += t * t;
    }
    D[j] = g_squared ? s : sqrt(s);
    if (D[j] < dmin) dmin = D[j];
  }
  double sum = 0.0;
  for (int j = 0; j < k; ++j) {
    A[j] = exp(-(D[j] - dmin) / tau);
    sum += A[j];
  }
  for (int j = 0; j < k; ++j) A[j] /= sum;
}

/* n_ij = dD_ij/dw_i: the unit vector (w_i - c_j) / D_ij, zero when D_ij == 0; for the squared distance 2 (w_i - c_j). */
static void unit_vector(const double *w, const double *cj, double Dj, int d, double *n) {
  if (g_squared) {
    for (int a = 0; a < d; ++a) n[a] = 2.0 * (w[a] - cj[a]);
    return;
  }
  for (int a = 0; a < d; ++a) n[a] = (Dj > 0.0) ? (w[a] - cj[a]) / Dj : 0.0;
}

/* Attention matrix A[m][k] = rowsoftmax_tau(-D(W,C))  (Eq. A(W,C) = rowsoftmax). */
void idkm_ref_attention(const double *W, int64_t m, int d, const double *C, int k, double tau, double *A_out) {
#pragma omp parallel for schedule(static)
  for (int c = 0; c < NCHUNK; ++c) {
    int64_t lo, hi;
    chunk_bounds(m, c, &lo, &hi);
    double *D = (double *)malloc(sizeof(double) * (size_t)k);
    for (int64_t i = lo; i < hi; ++i) attention_row(W + i * d, C, k, d, tau, D, A_out + i * k);
    free(D);
  }
}

/* S_j = sum_i A_ij and N_j = sum_i A_ij w_i: the two factors of the M-step. */
void idkm_ref_sums(const double *W, int64_t m, int d, const double *C, int k, double tau, double *S, double *N) {
  const int len = k * (d + 1);
  double *part = (double *)calloc((size_t)NCHUNK * (size_t)len, sizeof(double));
#pragma omp parallel for schedule(static)
  for (int c = 0; c < NCHUNK; ++c) {
    int64_t lo, hi;
    chunk_bounds(m, c, &lo, &hi);
    double *D = (double *)malloc(sizeof(double) * (size_t)k * 2);
    double *A = D + k;
    double *pS = part + (size_t)c * len, *pN = pS + k;
    for (int64_t i = lo; i < hi; ++i) {
      const double *w = W + i * d;
      attention_row(w, C, k, d, tau, D, A);
      for (int j = 0; j < k; ++j) {
        pS[j] += A[j];
        for (int a = 0; a < d; ++a) pN[j * d + a] += A[j] * w[a];
      }
    }
    free(D);
  }
  for (int j = 0; j < k; ++j) S[j] = 0.0;
  for (int t = 0; t < k * d; ++t) N[t] = 0.0;
  for (int c = 0; c < NCHUNK; ++c) {
    const double *pS = part + (size_t)c * len, *pN = pS + k;
    for (int j = 0; j < k; ++j) S[j] += pS[j];
    for (int t = 0; t < k * d; ++t) N[t] += pN[t];
  }
  free(part);
}

/* One application of the fixed-point map F(C, W) (Eq. F(C,W) := diag(rs(-D)^T 1)^-1 rs(-D)^T W).
 * Returns the number of clusters with S_j < S_MIN, whose centroid is kept. S_out may be NULL. */
int idkm_ref_step(const double *W, int64_t m, int d, const double *C, int k, double tau, double *C_plus,
                  double *S_out) {
  double *S = (double *)malloc(sizeof(double) * (size_t)k * (size_t)(d + 1));
  double *N = S + k;
  idkm_ref_sums(W, m, d, C, k, tau, S, N);
  int dead = 0;
  for (int j = 0; j < k; ++j) {
    if (S[j] >= IDKM_REF_S_MIN) {
      for (int a = 0; a < d; ++a) C_plus[j * d + a] = N[j * d + a] / S[j];
    } else {
      for (int a = 0; a < d; ++a) C_plus[j * d + a] = C[j * d + a];
      ++dead;
    }
    if (S_out) S_out[j] = S[j];
  }
  free(S);
  return dead;
}

static double rel_change(const double *X_new, const double *X_old, int n) {
  double num = 0.0, den = 0.0;
  for (int t = 0; t < n; ++t) {
    double e = X_new[t] - X_old[t];
    num += e * e;
    den += X_new[t] * X_new[t];
  }
  den = sqrt(den);
  if (den < 1e-300) den = 1e-300;
  return sqrt(num) / den;
}

/* Algorithm 1: repeat C <- F(C, W) until the relative change is below tol (tol > 0) or max_iter
 * applications were made.  Returns the last C+ (Algorithm 1, "return C+"). */
void idkm_ref_forward(const double *W, int64_t m, int d, const double *C0, int k, double tau, double tol,
                      int max_iter, double *C_out, int *iters_out, double *residual_out, int *dead_out) {
  const int n = k * d;
  double *Cp = (double *)malloc(sizeof(double) * (size_t)n);
  memcpy(C_out, C0, sizeof(double) * (size_t)n);
  int it = 0, dead = 0;
  double res = 0.0;
  while (it < max_iter) {
    dead = idkm_ref_step(W, m, d, C_out, k, tau, Cp, NULL);
    res = rel_change(Cp, C_out, n);
    memcpy(C_out, Cp, sizeof(double) * (size_t)n);
    ++it;
    if (tol > 0.0 && res < tol) break;
  }
  if (iters_out) *iters_out = it;
  if (residual_out) *residual_out = res;
  if (dead_out) *dead_out = dead;
  free(Cp);
}

/* Final pass at the returned centroids C: Wq_i = sum_j A_ij c_j (Eq. r_tau, Eq. r_tau(W,C) = C A^T),
 * optionally A itself, and the quantities of one more application of the map that the backward
 * needs: S_j and F_j = N_j / S_j (F_j := c_j for a dead cluster).  Any of Wq, A_out may be NULL. */
void idkm_ref_final(const double *W, int64_t m, int d, const double *C, int k, double tau, double *Wq,
                    double *A_out, double *S, double *F) {
#pragma omp parallel for schedule(static)
  for (int c = 0; c < NCHUNK; ++c) {
    int64_t lo, hi;
    chunk_bounds(m, c, &lo, &hi);
    double *D = (double *)malloc(sizeof(double) * (size_t)k * 2);
    double *A = D + k;
    for (int64_t i = lo; i < hi; ++i) {
      attention_row(W + i * d, C, k, d, tau, D, A);
      if (Wq) {
        for (int a = 0; a < d; ++a) {
          double s = 0.0;
          for (int j = 0; j < k; ++j) s += A[j] * C[j * d + a];
          Wq[i * d + a] = s;
        }
      }
      if (A_out) memcpy(A_out + i * k, A, sizeof(double) * (size_t)k);
    }
    free(D);
  }
  double *N = (double *)malloc(sizeof(double) * (size_t)k * (size_t)d);
  idkm_ref_sums(W, m, d, C, k, tau, S, N);
  for (int j = 0; j < k; ++j)
    for (int a = 0; a < d; ++a) F[j * d + a] = (S[j] >= IDKM_REF_S_MIN) ? N[j * d + a] / S[j] : C[j * d + a];
  free(N);
}

/* Direct codebook gradient g = (dWq/dC)^T G of L = <G, Wq(W, C)> with W fixed:
 *   g_l = sum_i [ A_il G_i + (1/tau) e_il(q) n_il ],  q_ij = G_i . c_j,
 *   e_ij(z) = A_ij (z_ij - sum_l A_il z_il).
 * From Wq_i = sum_j A_ij c_j, dA_ij/dD_il = -(1/tau) A_ij (delta_jl - A_il), dD_il/dc_l = -n_il. */
void idkm_ref_codebook_grad(const double *W, const double *G, int64_t m, int d, const double *C, int k,
                            double tau, double *g) {
  const int len = k * d;
  double *part = (double *)calloc((size_t)NCHUNK * (size_t)len, sizeof(double));
#pragma omp parallel for schedule(static)
  for (int c = 0; c < NCHUNK; ++c) {
    int64_t lo, hi;
    chunk_bounds(m, c, &lo, &hi);
    double *D = (double *)malloc(sizeof(double) * ((size_t)k * 3 + (size_t)d));
    double *A = D + k, *q = A + k, *n = q + k;
    double *pg = part + (size_t)c * len;
    for (int64_t i = lo; i < hi; ++i) {
      const double *w = W + i * d, *Gi = G + i * d;
      attention_row(w, C, k, d, tau, D, A);
      double t = 0.0;
      for (int j = 0; j < k; ++j) {
        q[j] = 0.0;
        for (int a = 0; a < d; ++a) q[j] += Gi[a] * C[j * d + a];
        t += A[j] * q[j];
      }
      for (int j = 0; j < k; ++j) {
        double e = A[j] * (q[j] - t);
        unit_vector(w, C + j * d, D[j], d, n);
        for (int a = 0; a < d; ++a) pg[j * d + a] += A[j] * Gi[a] + (e / tau) * n[a];
      }
    }
    free(D);
  }
  for (int t = 0; t < len; ++t) g[t] = 0.0;
  for (int c = 0; c < NCHUNK; ++c)
    for (int t = 0; t < len; ++t) g[t] += part[(size_t)c * len + t];
  free(part);
}

/* p_ij = u_j . (w_i - F_j) / S_j, zero for a dead cluster. */
static double p_term(const double *u, const double *w, const double *F, const double *S, int j, int d) {
  if (S[j] < IDKM_REF_S_MIN) return 0.0;
  double s = 0.0;
  for (int a = 0; a < d; ++a) s += u[j * d + a] * (w[a] - F[j * d + a]);
  return s / S[j];
}

/* Vector-Jacobian product with J_C = dF/dC at (C, W):
 *   (J_C^T u)_l = (1/tau) sum_i e_il(p) n_il,   p_ij = u_j . (w_i - F_j) / S_j.
 * From F_j = N_j/S_j: dF_j = (1/S_j) sum_i (w_i - F_j) dA_ij, dA_ij/dc_l = (1/tau) A_ij (delta_jl - A_il) n_il. */
void idkm_ref_adjoint_apply(const double *W, int64_t m, int d, const double *C, int k, double tau,
                            const double *S, const double *F, const double *u, double *JTu) {
  const int len = k * d;
  double *part = (double *)calloc((size_t)NCHUNK * (size_t)len, sizeof(double));
#pragma omp parallel for schedule(static)
  for (int c = 0; c < NCHUNK; ++c) {
    int64_t lo, hi;
    chunk_bounds(m, c, &lo, &hi);
    double *D = (double *)malloc(sizeof(double) * ((size_t)k * 3 + (size_t)d));
    double *A = D + k, *p = A + k, *n = p + k;
    double *pj = part + (size_t)c * len;
    for (int64_t i = lo; i < hi; ++i) {
      const double *w = W + i * d;
      attention_row(w, C, k, d, tau, D, A);
      double s = 0.0;
      for (int j = 0; j < k; ++j) {
        p[j] = p_term(u, w, F, S, j, d);
        s += A[j] * p[j];
      }
      for (int j = 0; j < k; ++j) {
        double e = A[j] * (p[j] - s);
        unit_vector(w, C + j * d, D[j], d, n);
        for (int a = 0; a < d; ++a) pj[j * d + a] += (e / tau) * n[a];
      }
    }
    free(D);
  }
  for (int t = 0; t < len; ++t) JTu[t] = 0.0;
  for (int c = 0; c < NCHUNK; ++c)
    for (int t = 0; t < len; ++t) JTu[t] += part[(size_t)c * len + t];
  free(part);
}

/* One step of the averaged iteration of Section 4.2 on the vector u: un = alpha (J^T u + g) + (1 - alpha) u. */
static void averaged_step(const double *Ju, const double *g, const double *u, double alpha, int n, double *un) {
  for (int t = 0; t < n; ++t) un[t] = alpha * (Ju[t] + g[t]) + (1.0 - alpha) * u[t];
}

/* Adjoint fixed point u = J_C^T u + g, the vector form of M* = (dF/dC) M* + I (Eq. for M*),
 * by the averaged iteration of Section 4.2: u <- alpha (J^T u + g) + (1 - alpha) u, u(0) = g.
 * Stops when the relative change is below adj_tol (adj_tol > 0) or after adj_max_iter steps. */
void idkm_ref_adjoint_solve(const double *W, int64_t m, int d, const double *C, int k, double tau,
                            const double *S, const double *F, const double *g, double alpha, double adj_tol,
                            int adj_max_iter, double *u, int *iters_out, double *residual_out) {
  const int n = k * d;
  double *Ju = (double *)malloc(sizeof(double) * (size_t)n * 2);
  double *un = Ju + n;
  memcpy(u, g, sizeof(double) * (size_t)n);
  int it = 0;
  double res = 0.0;
  while (it < adj_max_iter) {
    idkm_ref_adjoint_apply(W, m, d, C, k, tau, S, F, u, Ju);
    averaged_step(Ju, g, u, alpha, n, un);
    res = rel_change(un, u, n);
    memcpy(u, un, sizeof(double) * (size_t)n);
    ++it;
    if (adj_tol > 0.0 && res < adj_tol) break;
  }
  if (iters_out) *iters_out = it;
  if (residual_out) *residual_out = res;
  free(Ju);
}

/* The same iteration under the watch Section 4.2 asks for ("if we see the iteration diverge, we start over and divide
 * alpha by 2"; the paper gives no criterion, this is the reading taken): the iteration counts as diverged when u is
 * no longer finite, when the relative change has grown 10 steps running, or when ||u|| has passed 1e6 ||g|| (a
 * converging iteration stays below ||g|| / (1 - rho)).  Returns 1 if it diverged (u then holds the last iterate),
 * 0 otherwise. */
int idkm_ref_adjoint_solve_watched(const double *W, int64_t m, int d, const double *C, int k, double tau,
                                   const double *S, const double *F, const double *g, double alpha, double adj_tol,
                                   int adj_max_iter, double *u, int *iters_out, double *residual_out) {
  const int n = k * d;
  double *Ju = (double *)malloc(sizeof(double) * (size_t)n * 2);
  double *un = Ju + n;
  memcpy(u, g, sizeof(double) * (size_t)n);
  double g2 = 0.0;
  for (int t = 0; t < n; ++t) g2 += g[t] * g[t];
  int it = 0, up = 0, diverged = 0;
  double res = 0.0, prev = INFINITY;
  while (it < adj_max_iter) {
    idkm_ref_adjoint_apply(W, m, d, C, k, tau, S, F, u, Ju);
    double u2 = 0.0;
    int finite = 1;
    averaged_step(Ju, g, u, alpha, n, un);
    for (int t = 0; t < n; ++t) {
      u2 += un[t] * un[t];
      if (!isfinite(un[t])) finite = 0;
    }
    res = rel_change(un, u, n);
    memcpy(u, un, sizeof(double) * (size_t)n);
    ++it;
    up = (res > prev) ? up + 1 : 0;
    prev = res;
    if (!finite || up >= 10 || sqrt(u2) > 1e6 * sqrt(g2)) {
      diverged = 1;
      break;
    }
    if (adj_tol > 0.0 && res < adj_tol) break;
  }
  if (iters_out) *iters_out = it;
  if (residual_out) *residual_out = res;
  free(Ju);
  return diverged;
}

/* Section 4.2's safeguard as a policy: run the watched iteration with alpha0; each time it diverges start over from
 * u = g with half the alpha, at most max_halvings times.  Returns 1 if the last attempt diverged too.  alpha_used
 * receives the alpha of the last attempt, attempts_out the number of attempts made. */
int idkm_ref_adjoint_solve_restart(const double *W, int64_t m, int d, const double *C, int k, double tau,
                                   const double *S, const double *F, const double *g, double alpha0, int max_halvings,
                                   double adj_tol, int adj_max_iter, double *u, double *alpha_used, int *attempts_out,
                                   int *iters_out, double *residual_out) {
  double alpha = alpha0;
  int attempts = 0, diverged = 0;
  for (;;) {
    diverged = idkm_ref_adjoint_solve_watched(W, m, d, C, k, tau, S, F, g, alpha, adj_tol, adj_max_iter, u, iters_out,
                                              residual_out);
    ++attempts;
    if (!diverged || attempts > max_halvings) break;
    alpha *= 0.5;
  }
  if (alpha_used) *alpha_used = alpha;
  if (attempts_out) *attempts_out = attempts;
  return diverged;
}

/* dL/dW for L = <G, Wq>, given the adjoint u (the gradient equation dC/dW = (I - dF/dC)^-1 dF/dW at C*, contracted with g):
 *   dW_i = sum_j A_ij u_j / S_j  -  (1/tau) sum_j e_ij(q + p) n_ij
 * = (dWq/dW)^T G + (dF/dW)^T u.  With u = g this is the Jacobian-free gradient (the JFB equation dC/dW = dF/dW at C*). */
void idkm_ref_scatter(const double *W, const double *G, int64_t m, int d, const double *C, int k, double tau,
                      const double *S, const double *F, const double *u, double *dW) {
#pragma omp parallel for schedule(static)
  for (int c = 0; c < NCHUNK; ++c) {
    int64_t lo, hi;
    chunk_bounds(m, c, &lo, &hi);
    double *D = (double *)malloc(sizeof(double) * ((size_t)k * 3 + (size_t)d));
    double *A = D + k, *z = A + k, *n = z + k;
    for (int64_t i = lo; i < hi; ++i) {
      const double *w = W + i * d, *Gi = G + i * d;
      attention_row(w, C, k, d, tau, D, A);
      double zbar = 0.0;
      for (int j = 0; j < k; ++j) {
        double q = 0.0;
        for (int a = 0; a < d; ++a) q += Gi[a] * C[j * d + a];
        z[j] = q + p_term(u, w, F, S, j, d);
        zbar += A[j] * z[j];
      }
      for (int a = 0; a < d; ++a) dW[i * d + a] = 0.0;
      for (int j = 0; j < k; ++j) {
        double e = A[j] * (z[j] - zbar);
        unit_vector(w, C + j * d, D[j], d, n);
        double inv_s = (S[j] >= IDKM_REF_S_MIN) ? 1.0 / S[j] : 0.0;
        for (int a = 0; a < d; ++a) dW[i * d + a] += A[j] * u[j * d + a] * inv_s - (e / tau) * n[a];
      }
    }
    free(D);
  }
}

/* Whole backward at the returned centroids C.  mode 0: implicit (adjoint solve), mode 1: JFB (u = g).
 * S and F are those of idkm_ref_final at the same C. */
void idkm_ref_backward(const double *W, const double *G, int64_t m, int d, const double *C, int k, double tau,
                       const double *S, const double *F, int mode, double alpha, double adj_tol,
                       int adj_max_iter, double *dW, double *dC, int *iters_out, double *residual_out) {
  const int n = k * d;
  double *g = (double *)malloc(sizeof(double) * (size_t)n);
  idkm_ref_codebook_grad(W, G, m, d, C, k, tau, g);
  if (mode == 0) {
    idkm_ref_adjoint_solve(W, m, d, C, k, tau, S, F, g, alpha, adj_tol, adj_max_iter, dC, iters_out,
                           residual_out);
  } else {
    memcpy(dC, g, sizeof(double) * (size_t)n);
    if (iters_out) *iters_out = 0;
    if (residual_out) *residual_out = 0.0;
  }
  if (dW) idkm_ref_scatter(W, G, m, d, C, k, tau, S, F, dC, dW);
  free(g);
}

/*
 * dad_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, float64 CPU statement of what the distributed auto-differentiation
 * (dAD / rank-dAD) per-layer path computes, written from the paper so that the CUDA
 * library can be checked against it.  It shares no code with the CUDA path and is
 * only ever called by the tests, by the smoke check and by the benchmark's CPU
 * baseline leg.  Nothing here is blocked, fused or reordered beyond what the cited
 * definition states; the only parallelism is an OpenMP loop over independent sites
 * (or over independent output rows of a dense product).
 *
 * Notation (per linear layer, per site s of S):
 *   A  : N x h_in   layer input activations              (paper: A_{i-1})
 *   D  : N x h_out  back-propagated errors at the output  (paper: Delta_i)
 *   gradW = A^T D   : h_in x h_out local gradient          (Eq. "local_grad", Sec. 3.1)
 *   M  = gradW^T gradW = D^T A A^T D                       (Eq. "nabla_iter", Sec. 3.3.1)
 *   Q  : r x h_out  output-side factor, orthonormal rows   (the g vectors of Algorithm 2)
 *   P  : r x h_in   input-side factor, P_j = A^T (D Q_j)   (the un-normalised q of Algorithm 2)
 * All matrices are dense row-major arrays of double.
 *
 * Parity pins (tests/test_oracle_*.py): every function below is pinned to something
 * other than itself -- the pooled-batch gradient and autograd (full_grad), the
 * Eckart-Young theorem and a library SVD (spi), explicit Krylov spans, closed-form
 * byte counts.  No function is "parity unpinned"; what stays unpinned by a printed
 * example (the paper prints none) is the finite-iteration VALUE of spi_block, which
 * is fixed instead by the span identity span(Q) = span(M^iters Q0^T).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef int64_t i64;

int dad_oracle_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ------------------------------------------------------------------------------------
 * O-1  Uncompressed dAD gradient (Sec. 3.2; Eq. "local_grad"; Sec. 5.1):
 *      every site ships A_s and D_s, the aggregator concatenates them on the batch
 *      dimension and multiplies:  G[a][b] = sum_s sum_n A_s[n][a] * D_s[n][b].
 *      A: S*N*h_in, D: S*N*h_out (site-major), G: h_in*h_out (overwritten).
 * ---------------------------------------------------------------------------------- */
void dad_oracle_full_grad(int S, i64 N, i64 h_in, i64 h_out,
                          const double* A, const double* D, double* G) {
#pragma omp parallel for schedule(static)
  for (i64 a = 0; a < h_in; ++a) {
    double* g = G + a * h_out;
    for (i64 b = 0; b < h_out; ++b) g[b] = 0.0;
    for (int s = 0; s < S; ++s)
      for (i64 n = 0; n < N; ++n) {
        const double x = A[((i64)s * N + n) * h_in + a];
        const double* d = D + ((i64)s * N + n) * h_out;
        for (i64 b = 0; b < h_out; ++b) g[b] += x * d[b];
      }
  }
}

/* ------------------------------------------------------------------------------------
 * O-2  Reconstruction from stacked factors (Algorithm 1, the "P^T Q" step after the
 *      vertcat of all sites' factors):  G[a][b] = sum_k Pcat[k][a] * Qcat[k][b],
 *      k running over the K = S*r stacked rows, i.e. the sum over sites of the outer
 *      products of their factors.
 * ---------------------------------------------------------------------------------- */
void dad_oracle_reconstruct(i64 K, i64 h_in, i64 h_out,
                            const double* Pcat, const double* Qcat, double* G) {
#pragma omp parallel for schedule(static)
  for (i64 a = 0; a < h_in; ++a) {
    double* g = G + a * h_out;
    for (i64 b = 0; b < h_out; ++b) g[b] = 0.0;
    for (i64 k = 0; k < K; ++k) {
      const double p = Pcat[k * h_in + a];
      const double* q = Qcat + k * h_out;
      for (i64 b = 0; b < h_out; ++b) g[b] += p * q[b];
    }
  }
}

/* ------------------------------------------------------------------------------------
 * The four structured products of one application of M (Eq. "reduced_iter": the
 * recurrence g <- gradW^T gradW g evaluated right to left through D and A, never
 * forming gradW).  F holds r vectors as rows.
 * ---------------------------------------------------------------------------------- */
/* Y[n][j] = sum_c X[n][c] * F[j][c]        (X: N x h, F: r x h, Y: N x r) */
static void rows_dot(i64 N, i64 h, i64 r, const double* X, const double* F, double* Y) {
  for (i64 n = 0; n < N; ++n)
    for (i64 j = 0; j < r; ++j) {
      double acc = 0.0;
      for (i64 c = 0; c < h; ++c) acc += X[n * h + c] * F[j * h + c];
      Y[n * r + j] = acc;
    }
}
/* Z[j][c] = sum_n Y[n][j] * X[n][c]        (Y: N x r, X: N x h, Z: r x h) */
static void cols_acc(i64 N, i64 h, i64 r, const double* Y, const double* X, double* Z) {
  for (i64 j = 0; j < r; ++j) {
    for (i64 c = 0; c < h; ++c) Z[j * h + c] = 0.0;
    for (i64 n = 0; n < N; ++n) {
      const double y = Y[n * r + j];
      for (i64 c = 0; c < h; ++c) Z[j * h + c] += y * X[n * h + c];
    }
  }
}

static double norm2(const double* v, i64 h) {
  double s = 0.0;
  for (i64 c = 0; c < h; ++c) s += v[c] * v[c];
  return sqrt(s);
}
static double dot(const double* u, const double* v, i64 h) {
  double s = 0.0;
  for (i64 c = 0; c < h; ++c) s += u[c] * v[c];
  return s;
}

/* ------------------------------------------------------------------------------------
 * orth: orthonormalise the r rows of G (r x h) in place, in order -- a thin QR with a
 * positive diagonal, by Gram-Schmidt with every projection sweep applied twice.  This
 * is the block form of the deflation ("peeling") of Eq. "peel": removing from a
 * vector its components along the already-found directions.  A row whose remainder is
 * not larger than 1e-12 times its length before projection carries no new direction
 * (the true rank can be below r, Sec. 3.3.1) and is set to exactly zero, so that it
 * adds nothing to P^T Q.  Rdiag (length r, may be NULL) receives the remainders.
 * ---------------------------------------------------------------------------------- */
void dad_oracle_orth(i64 r, i64 h, double* G, double* Rdiag) {
  for (i64 j = 0; j < r; ++j) {
    double* v = G + j * h;
    const double before = norm2(v, h);
    for (int sweep = 0; sweep < 2; ++sweep)
      for (i64 l = 0; l < j; ++l) {
        const double* q = G + l * h;
        const double c = dot(q, v, h);
        for (i64 b = 0; b < h; ++b) v[b] -= c * q[b];
      }
    const double after = norm2(v, h);
    if (before == 0.0 || after <= 1e-12 * before) {
      for (i64 b = 0; b < h; ++b) v[b] = 0.0;
      if (Rdiag) Rdiag[j] = 0.0;
    } else {
      for (i64 b = 0; b < h; ++b) v[b] /= after;
      if (Rdiag) Rdiag[j] = after;
    }
  }
}

/* ------------------------------------------------------------------------------------
 * O-3  Blocked structured power iteration for ONE site (Algorithm 2 with all r
 *      vectors advanced together):
 *        G <- Q0                                  (random start, Algorithm 2 "g_0 ~ N(0,1)")
 *        repeat iters times:
 *          Y = D G^T ; Z = (A^T Y)^T              (gradW applied to the r vectors)
 *          W = A Z^T ; Gt = (D^T W)^T             (gradW^T applied: Gt = (M G^T)^T)
 *          G <- orth(Gt)
 *        P = (A^T (D G^T))^T ; Q = G ; sigma_j = ||P_j||
 *      (v = D g, q = A^T v and sigma = sqrt(v^T A A^T v) = ||A^T v|| of Algorithm 2; the
 *      division of q by sigma is not made, so P carries the singular values.)
 *      A: N x h_in, D: N x h_out, Q0/Q: r x h_out, P: r x h_in, sigma: r (may be NULL).
 *      Returns 0, or 1 if memory could not be had.
 * ---------------------------------------------------------------------------------- */
int dad_oracle_spi_block_site(i64 N, i64 h_in, i64 h_out, i64 r, int iters,
                              const double* A, const double* D, const double* Q0,
                              double* P, double* Q, double* sigma) {
  double* Y = (double*)malloc(sizeof(double) * (size_t)(N * r));
  double* Z = (double*)malloc(sizeof(double) * (size_t)(r * h_in));
  if (!Y || !Z) { free(Y); free(Z); return 1; }
  memcpy(Q, Q0, sizeof(double) * (size_t)(r * h_out));
  for (int k = 0; k < iters; ++k) {
    rows_dot(N, h_out, r, D, Q, Y);  /* Y = D G^T          */
    cols_acc(N, h_in, r, Y, A, Z);   /* Z = Y^T A          */
    rows_dot(N, h_in, r, A, Z, Y);   /* W = A Z^T  (in Y)  */
    cols_acc(N, h_out, r, Y, D, Q);  /* Gt = W^T D (in Q)  */
    dad_oracle_orth(r, h_out, Q, NULL);
  }
  rows_dot(N, h_out, r, D, Q, Y);
  cols_acc(N, h_in, r, Y, A, P);
  if (sigma)
    for (i64 j = 0; j < r; ++j) sigma[j] = norm2(P + j * h_in, h_in);
  free(Y); free(Z);
  return 0;
}

/* All S sites, independent of one another (Algorithm 1, the per-site SPI call). */
int dad_oracle_spi_block(int S, i64 N, i64 h_in, i64 h_out, i64 r, int iters,
                         const double* A, const double* D, const double* Q0,
                         double* P, double* Q, double* sigma) {
  int err = 0;
#pragma omp parallel for schedule(dynamic, 1) reduction(| : err)
  for (int s = 0; s < S; ++s)
    err |= dad_oracle_spi_block_site(N, h_in, h_out, r, iters,
                                     A + (i64)s * N * h_in, D + (i64)s * N * h_out,
                                     Q0 + (i64)s * r * h_out,
                                     P + (i64)s * r * h_in, Q + (i64)s * r * h_out,
                                     sigma ? sigma + (i64)s * r : NULL);
  return err;
}

/* ------------------------------------------------------------------------------------
 * O-4  Algorithm 2 taken one vector at a time, for ONE site, with the repairs that
 *      make its peel term well defined: the deflated operator is
 *      M - sum_{l<j} sigma_l^2 g_l g_l^T (the found part of M = V Sigma^2 V^T), the
 *      iterate is kept orthogonal to the found g_l and of unit length, exactly r
 *      vectors are produced, each with n applications of M, and the early stop is not
 *      taken.  Used to show that the blocked form O-3 and the paper's sequential form
 *      find the same subspace.
 * ---------------------------------------------------------------------------------- */
static void project_out(i64 j, i64 h, const double* Qfound, double* g) {
  for (int sweep = 0; sweep < 2; ++sweep)
    for (i64 l = 0; l < j; ++l) {
      const double c = dot(Qfound + l * h, g, h);
      for (i64 b = 0; b < h; ++b) g[b] -= c * Qfound[l * h + b];
    }
}

int dad_oracle_spi_paper_site(i64 N, i64 h_in, i64 h_out, i64 r, int n_iter,
                              const double* A, const double* D, const double* Q0,
                              double* P, double* Q, double* sigma_out) {
  double* v = (double*)malloc(sizeof(double) * (size_t)N);
  double* z = (double*)malloc(sizeof(double) * (size_t)h_in);
  double* g = (double*)malloc(sizeof(double) * (size_t)h_out);
  double* t = (double*)malloc(sizeof(double) * (size_t)h_out);
  double* sig = (double*)malloc(sizeof(double) * (size_t)r);
  if (!v || !z || !g || !t || !sig) { free(v); free(z); free(g); free(t); free(sig); return 1; }
  for (i64 j = 0; j < r; ++j) {
    memcpy(g, Q0 + j * h_out, sizeof(double) * (size_t)h_out);
    project_out(j, h_out, Q, g);
    double nrm = norm2(g, h_out);
    int dead = (nrm == 0.0);
    if (!dead) for (i64 b = 0; b < h_out; ++b) g[b] /= nrm;
    for (int k = 0; k < n_iter && !dead; ++k) {
      /* t = M g = D^T (A (A^T (D g))) */
      rows_dot(N, h_out, 1, D, g, v);
      cols_acc(N, h_in, 1, v, A, z);
      rows_dot(N, h_in, 1, A, z, v);
      cols_acc(N, h_out, 1, v, D, t);
      const double before = norm2(t, h_out);
      /* peel: subtract sigma_l^2 g_l (g_l . g) for the found components */
      for (i64 l = 0; l < j; ++l) {
        const double c = sig[l] * sig[l] * dot(Q + l * h_out, g, h_out);
        for (i64 b = 0; b < h_out; ++b) t[b] -= c * Q[l * h_out + b];
      }
      project_out(j, h_out, Q, t);
      nrm = norm2(t, h_out);
      if (before == 0.0 || nrm <= 1e-12 * before) { dead = 1; break; }
      for (i64 b = 0; b < h_out; ++b) g[b] = t[b] / nrm;
    }
    if (dead) for (i64 b = 0; b < h_out; ++b) g[b] = 0.0;
    memcpy(Q + j * h_out, g, sizeof(double) * (size_t)h_out);
    rows_dot(N, h_out, 1, D, g, v);              /* v = D g            */
    cols_acc(N, h_in, 1, v, A, P + j * h_in);    /* p = A^T v          */
    sig[j] = norm2(P + j * h_in, h_in);          /* = sqrt(v^T A A^T v) */
    if (sigma_out) sigma_out[j] = sig[j];
  }
  free(v); free(z); free(g); free(t); free(sig);
  return 0;
}

/* ------------------------------------------------------------------------------------
 * O-5  Bytes one site transmits for one layer.
 *   dAD      : the two component matrices, N*(h_in+h_out) elements of e bytes (Sec. 3.1,
 *              the "m+n versus m*n" argument; Sec. 3.2).
 *   rank-dAD : the two rank-r factors, r*(h_in+h_out) fp32 values (Sec. 2, the
 *              Theta(r(h_i+h_{i+1})) bandwidth of rank methods; Sec. 3.3).
 *   dSGD     : the full fp32 gradient, h_in*h_out values (Sec. 1).
 * ---------------------------------------------------------------------------------- */
uint64_t dad_oracle_bytes_dad(i64 N, i64 h_in, i64 h_out, int elem_bytes) {
  return (uint64_t)N * (uint64_t)(h_in + h_out) * (uint64_t)elem_bytes;
}
uint64_t dad_oracle_bytes_rank(i64 r, i64 h_in, i64 h_out) {
  return (uint64_t)r * (uint64_t)(h_in + h_out) * 4u;
}
uint64_t dad_oracle_bytes_dsgd(i64 h_in, i64 h_out) {
  return (uint64_t)h_in * (uint64_t)h_out * 4u;
}

/* ------------------------------------------------------------------------------------
 * Gather (Algorithm 1, the two vertcat lines at the aggregator): site s's factors
 * become rows s*r .. s*r+r-1 of the stacks; every site is charged the bytes of its
 * two factors.  P: S*r*h_in, Q: S*r*h_out -> Pcat (S*r) x h_in, Qcat (S*r) x h_out.
 * ---------------------------------------------------------------------------------- */
void dad_oracle_gather(int S, i64 r, i64 h_in, i64 h_out,
                       const double* P, const double* Q,
                       double* Pcat, double* Qcat, uint64_t* bytes_tx) {
  for (int s = 0; s < S; ++s) {
    for (i64 j = 0; j < r; ++j) {
      for (i64 a = 0; a < h_in; ++a)
        Pcat[((i64)s * r + j) * h_in + a] = P[((i64)s * r + j) * h_in + a];
      for (i64 b = 0; b < h_out; ++b)
        Qcat[((i64)s * r + j) * h_out + b] = Q[((i64)s * r + j) * h_out + b];
    }
    if (bytes_tx) bytes_tx[s] = dad_oracle_bytes_rank(r, h_in, h_out);
  }
}

/* ------------------------------------------------------------------------------------
 * Effective rank of a site's factors (Sec. 3.3.1, last paragraph; the early stop of
 * Algorithm 2, theta = 1e-3).  As printed the stop test compares consecutive components,
 * which are orthogonal to each other, and can never fire; the reading taken is: keep the
 * leading components while sigma_j > theta * sigma_1, drop that one and all later ones.
 * The decision is an integer taken on fp32 values, so it is made in fp32 here exactly as
 * the library makes it (fp32 product, fp32 comparison).
 *   sigma: S x r fp32, r_eff: S (out).
 * ---------------------------------------------------------------------------------- */
void dad_oracle_effective_rank(int S, i64 r, const float* sigma, float theta, int32_t* r_eff) {
  for (int s = 0; s < S; ++s) {
    const float* sg = sigma + (i64)s * r;
    const float bar = theta * sg[0];
    int keep = 0;
    while (keep < r && sg[keep] > bar) ++keep;
    r_eff[s] = keep;
  }
}

/* ------------------------------------------------------------------------------------
 * Algorithm 2 with its precomputed matrices, for ONE site: C = A A^T (N x N) and
 * B = D^T C (h_out x N) are formed explicitly, every iteration is G~ = B (D G^T)
 * (Eq. "reduced_iter") for all r vectors at once, followed by the same orthonormalisation as
 * spi_block; at the end v_j = D g_j, sigma_j = sqrt(v_j^T C v_j) and P_j = A^T v_j (the
 * division by sigma is again not made).  This is the form whose cost is O(h N) per vector and
 * iteration when N << h (Sec. 3.3.1).  Returns 0, or 1 if memory could not be had.
 * ---------------------------------------------------------------------------------- */
int dad_oracle_spi_gram_site(i64 N, i64 h_in, i64 h_out, i64 r, int iters,
                             const double* A, const double* D, const double* Q0,
                             double* P, double* Q, double* sigma) {
  double* C = (double*)malloc(sizeof(double) * (size_t)(N * N));
  double* B = (double*)malloc(sizeof(double) * (size_t)(h_out * N));
  double* V = (double*)malloc(sizeof(double) * (size_t)(N * r));
  if (!C || !B || !V) { free(C); free(B); free(V); return 1; }
  for (i64 n = 0; n < N; ++n)
    for (i64 m = 0; m < N; ++m) C[n * N + m] = dot(A + n * h_in, A + m * h_in, h_in);
  for (i64 b = 0; b < h_out; ++b)
    for (i64 m = 0; m < N; ++m) {
      double acc = 0.0;
      for (i64 n = 0; n < N; ++n) acc += D[n * h_out + b] * C[n * N + m];
      B[b * N + m] = acc;
    }
  memcpy(Q, Q0, sizeof(double) * (size_t)(r * h_out));
  for (int k = 0; k < iters; ++k) {
    rows_dot(N, h_out, r, D, Q, V);               /* V = D G^T            */
    for (i64 j = 0; j < r; ++j)                   /* G~_j = B v_j         */
      for (i64 b = 0; b < h_out; ++b) {
        double acc = 0.0;
        for (i64 m = 0; m < N; ++m) acc += B[b * N + m] * V[m * r + j];
        Q[j * h_out + b] = acc;
      }
    dad_oracle_orth(r, h_out, Q, NULL);
  }
  rows_dot(N, h_out, r, D, Q, V);
  cols_acc(N, h_in, r, V, A, P);                  /* P_j = A^T v_j        */
  if (sigma)
    for (i64 j = 0; j < r; ++j) {                 /* sigma_j = sqrt(v^T C v) */
      double acc = 0.0;
      for (i64 n = 0; n < N; ++n)
        for (i64 m = 0; m < N; ++m) acc += V[n * r + j] * C[n * N + m] * V[m * r + j];
      sigma[j] = sqrt(acc > 0.0 ? acc : 0.0);
    }
  free(C); free(B); free(V);
  return 0;
}

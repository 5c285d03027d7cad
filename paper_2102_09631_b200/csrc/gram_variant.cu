// Structured power iterations in the form Algorithm 2 prints them, for the regime the paper assumes
// (batch much smaller than the layer width, N << h): precompute C = A A^T (N x N) once, then every
// application of the operator touches only D and C,
//     g  <-  D^T ( C ( D g ) )          (Eq. "reduced_iter" with B = D^T C),
// and the singular value is sigma = sqrt(v^T C v), v = D g.  A is read twice in all (for C and for the
// final P = A^T v) instead of 2*iters + 1 times.  fp32 inputs, fp64 accumulation, general kernels.
#include "common.cuh"

namespace dad {

namespace {

// C[s][n][m] = sum_c A[s][n][c] * A[s][m][c]; one CTA per (site, 16 rows n), all N columns m.
__global__ void __launch_bounds__(256)
gram_rows_kernel(const float* __restrict__ A, int64_t ld, int64_t stride, int N, int64_t h, double* __restrict__ C) {
  extern __shared__ float tile[];  // [N][65]
  const int s = blockIdx.y, n0 = blockIdx.x * 16;
  const int nl = threadIdx.x / 16, mg = threadIdx.x % 16;
  const float* As = A + (int64_t)s * stride;
  double acc[DAD_MAX_GRAM_ROWS / 16];
#pragma unroll
  for (int k = 0; k < DAD_MAX_GRAM_ROWS / 16; ++k) acc[k] = 0.0;
  for (int64_t c0 = 0; c0 < h; c0 += 64) {
    for (int idx = threadIdx.x; idx < N * 64; idx += 256) {
      const int n = idx / 64, cc = idx % 64;
      tile[n * 65 + cc] = (c0 + cc < h) ? As[(int64_t)n * ld + c0 + cc] : 0.f;
    }
    __syncthreads();
    if (n0 + nl < N) {
      for (int cc = 0; cc < 64; ++cc) {
        const double a = (double)tile[(n0 + nl) * 65 + cc];
#pragma unroll
        for (int k = 0; k < DAD_MAX_GRAM_ROWS / 16; ++k) {
          const int m = mg + 16 * k;
          if (m < N) acc[k] += a * (double)tile[m * 65 + cc];
        }
      }
    }
    __syncthreads();
  }
  if (n0 + nl < N) {
#pragma unroll
    for (int k = 0; k < DAD_MAX_GRAM_ROWS / 16; ++k) {
      const int m = mg + 16 * k;
      if (m < N) C[((int64_t)s * N + n0 + nl) * N + m] = acc[k];
    }
  }
}

// T[s][n][j] = sum_m C[s][n][m] * Y[s][m][j]; one CTA per (site, row n), one thread per j.
__global__ void __launch_bounds__(DAD_MAX_RANK)
apply_gram_kernel(const double* __restrict__ C, const double* __restrict__ Y, int N, int r, double* __restrict__ T) {
  const int s = blockIdx.y, n = blockIdx.x, j = threadIdx.x;
  if (j >= r) return;
  const double* Cr = C + ((int64_t)s * N + n) * N;
  const double* Ys = Y + (int64_t)s * N * r;
  double acc[4] = {0.0, 0.0, 0.0, 0.0};
  int m = 0;
  for (; m + 4 <= N; m += 4) {
#pragma unroll
    for (int u = 0; u < 4; ++u) acc[u] += Cr[m + u] * Ys[(int64_t)(m + u) * r + j];
  }
  for (; m < N; ++m) acc[0] += Cr[m] * Ys[(int64_t)m * r + j];
  T[((int64_t)s * N + n) * r + j] = (acc[0] + acc[1]) + (acc[2] + acc[3]);
}

// sigma[s][j] = sqrt( sum_n Y[s][n][j] * T[s][n][j] ) = sqrt(v^T C v) with v = D g_j, T = C v.
__global__ void __launch_bounds__(DAD_MAX_RANK)
sigma_from_gram_kernel(const double* __restrict__ Y, const double* __restrict__ T, int N, int r, float* __restrict__ sigma) {
  const int s = blockIdx.x, j = threadIdx.x;
  if (j >= r) return;
  double acc = 0.0;
  for (int n = 0; n < N; ++n) acc += Y[((int64_t)s * N + n) * r + j] * T[((int64_t)s * N + n) * r + j];
  sigma[(int64_t)s * r + j] = (float)sqrt(acc > 0.0 ? acc : 0.0);
}

struct GramWs {
  CompressWs base;
  size_t C, T, total;
};

GramWs gram_ws_layout(const dad_layer& L, int r) {
  GramWs w;
  w.base = compress_ws_layout(L, r, true, false, 0);
  size_t off = w.base.total;
  w.C = off;
  off = align_up(off + (size_t)L.S * L.N * L.N * 8, 256);
  w.T = off;
  off = align_up(off + (size_t)L.S * L.N * r * 8, 256);
  w.total = off;
  return w;
}

bool gram_variant_takes(const dad_layer& L) { return L.dtype == DAD_F32 && L.N <= DAD_MAX_GRAM_ROWS; }

}  // namespace
}  // namespace dad

using namespace dad;

extern "C" {

size_t dad_rank_compress_gram_workspace_bytes(const dad_layer* L, int r, int iters) {
  if (dad_workspace_bytes(L, r, iters) == 0 || !gram_variant_takes(*L)) return 0;
  return gram_ws_layout(*L, r).total;
}

dad_status dad_rank_compress_gram(const dad_layer* L, const void* A, const void* D, int r, int iters, const float* Q0,
                                  float* P, float* Q, float* sigma, void* ws, size_t ws_bytes, void* cuda_stream) {
  if (!L) return DAD_ERR_NULL;
  if (L->dtype != DAD_F32) return DAD_ERR_DTYPE;
  if (!A || !D || !Q0 || !P || !Q || !ws) return DAD_ERR_NULL;
  if (dad_workspace_bytes(L, r, iters) == 0) {  // same shape, stride and rank rules as dad_rank_compress
    if (r < 1 || r > DAD_MAX_RANK || r > L->h_in || r > L->h_out) return DAD_ERR_RANK;
    return DAD_ERR_SHAPE;
  }
  if (L->N > DAD_MAX_GRAM_ROWS) return DAD_ERR_SHAPE;
  const uintptr_t bits = reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(D) | reinterpret_cast<uintptr_t>(Q0) |
                         reinterpret_cast<uintptr_t>(P) | reinterpret_cast<uintptr_t>(Q);
  if (bits % 16 || reinterpret_cast<uintptr_t>(ws) % 256) return DAD_ERR_ALIGN;
  const GramWs w = gram_ws_layout(*L, r);
  if (ws_bytes < w.total) return DAD_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  char* base = static_cast<char*>(ws);
  const CompressWs& b = w.base;
  const int S = L->S, N = (int)L->N;
  const int64_t hi = L->h_in, ho = L->h_out;
  cudaError_t err = cudaMemsetAsync(base + b.status, 0, b.counters + b.n_counters * sizeof(unsigned) - b.status, st);
  if (err != cudaSuccess) return DAD_ERR_CUDA;
  int* status = reinterpret_cast<int*>(base + b.status);
  unsigned* ctr_cols = reinterpret_cast<unsigned*>(base + b.counters);
  unsigned* ctr_gram = ctr_cols + (b.n_counters - (size_t)S);
  double* G = reinterpret_cast<double*>(base + b.G);
  double* Y = reinterpret_cast<double*>(base + b.Y);
  double* Z = reinterpret_cast<double*>(base + b.Z);
  double* part = reinterpret_cast<double*>(base + b.partial);
  double* gram_partial = reinterpret_cast<double*>(base + b.gram_partial);
  double* gram = reinterpret_cast<double*>(base + b.gram);
  double* tratio = reinterpret_cast<double*>(base + b.tratio);
  unsigned char* dead = reinterpret_cast<unsigned char*>(base + b.dead);
  int* need2 = reinterpret_cast<int*>(base + b.dead + align_up((size_t)S * r, 16));
  double* C = reinterpret_cast<double*>(base + w.C);
  double* T = reinterpret_cast<double*>(base + w.T);
  const double tol = 1e-12;
#define DAD_STEP(call)                            \
  do {                                            \
    err = (call);                                 \
    if (err != cudaSuccess) return DAD_ERR_CUDA;  \
  } while (0)
  DAD_STEP(widen_f32_to_f64(Q0, G, (size_t)S * r * ho, st));
  if (iters == 0 && Q != Q0)
    DAD_STEP(cudaMemcpyAsync(Q, Q0, sizeof(float) * (size_t)S * r * ho, cudaMemcpyDeviceToDevice, st));
  // C = A A^T
  DAD_LAUNCH(err, "gram_rows", gram_rows_kernel, dim3((unsigned)ceil_div(N, 16), (unsigned)S), 256,
             sizeof(float) * (size_t)N * 65, st, (const float*)A, L->ldA, L->strideA, N, hi, C);
  if (err != cudaSuccess) return DAD_ERR_CUDA;
  for (int k = 0; k < iters; ++k) {
    DAD_STEP(rows_dot<double>(DAD_F32, D, L->ldD, L->strideD, S, N, ho, G, r, Y, st));  // v = D g
    DAD_LAUNCH(err, "apply_gram", apply_gram_kernel, dim3((unsigned)N, (unsigned)S), DAD_MAX_RANK, 0, st, C, Y, N, r, T);  // C v
    if (err != cudaSuccess) return DAD_ERR_CUDA;
    DAD_STEP(cols_acc<double>(DAD_F32, D, L->ldD, L->strideD, S, N, ho, T, r, G, nullptr, part, ctr_cols, st));  // D^T (C v)
    float* q32 = (k == iters - 1) ? Q : nullptr;
    if (orth_cluster_fits(r, ho, sizeof(double))) {
      DAD_STEP(orth_cluster<double>(G, S, r, ho, tol, status, q32, nullptr, 0, st));
      continue;
    }
    DAD_STEP(cholqr_pass<double>(G, S, r, ho, 0, tol, gram_partial, gram, tratio, dead, need2, ctr_gram, status, q32,
                                 nullptr, 0, st));
    DAD_STEP(cholqr_pass<double>(G, S, r, ho, 1, tol, gram_partial, gram, tratio, dead, need2, ctr_gram, status, q32,
                                 nullptr, 0, st));
  }
  DAD_STEP(rows_dot<double>(DAD_F32, D, L->ldD, L->strideD, S, N, ho, G, r, Y, st));
  DAD_STEP(cols_acc<double>(DAD_F32, A, L->ldA, L->strideA, S, N, hi, Y, r, Z, P, part, ctr_cols, st));  // P = (A^T v)^T
  if (sigma) {
    DAD_LAUNCH(err, "apply_gram", apply_gram_kernel, dim3((unsigned)N, (unsigned)S), DAD_MAX_RANK, 0, st, C, Y, N, r, T);
    DAD_LAUNCH(err, "sigma_from_gram", sigma_from_gram_kernel, (unsigned)S, DAD_MAX_RANK, 0, st, Y, T, N, r, sigma);
    if (err != cudaSuccess) return DAD_ERR_CUDA;
  }
#undef DAD_STEP
  return DAD_OK;
}

}  // extern "C"

// Algorithm 2 in the order the paper prints it: the r components of a site are found ONE AFTER THE OTHER, each by
// its own power iteration on M = gradW^T gradW applied through D and A (Eq. "reduced_iter"), with the components
// already found peeled off (Eq. "peel": subtract sigma_l^2 g_l (g_l . g)) and projected out, the iterate normalised
// after every application.  r times as many passes over A and D as the block form dad_rank_compress takes: this
// entry point exists to compare the two orders on the device, not for speed.  fp64 accumulation and fp64
// intermediates for both input types; sites run side by side in every launch.
#include "common.cuh"

namespace dad {
namespace {

constexpr int kSeqThreads = 256;

// Sum over the CTA in a fixed order (shuffle tree inside a warp, then the eight warp sums in warp order); every
// thread returns the same value.
__device__ double block_sum(double v, double* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  double t = 0.0;
#pragma unroll
  for (int w = 0; w < kSeqThreads / 32; ++w) t += red[w];
  __syncthreads();
  return t;
}

__device__ double block_dot(const double* a, const double* b, int64_t h, double* red) {
  double acc = 0.0;
  for (int64_t c = threadIdx.x; c < h; c += kSeqThreads) acc += a[c] * b[c];
  return block_sum(acc, red);
}

// x <- x minus its components along the j found unit vectors, two sweeps of modified Gram-Schmidt.
__device__ void project_out(int j, int64_t h, const double* found, double* x, double* red) {
  for (int sweep = 0; sweep < 2; ++sweep)
    for (int l = 0; l < j; ++l) {
      const double* gl = found + (int64_t)l * h;
      const double c = block_dot(gl, x, h, red);
      for (int64_t b = threadIdx.x; b < h; b += kSeqThreads) x[b] -= c * gl[b];
      __syncthreads();
    }
}

// g <- start vector j of the site, projected on the complement of the found components and normalised; a start
// vector inside their span leaves g = 0 and the component dead.
__global__ void __launch_bounds__(kSeqThreads)
seq_start_kernel(const float* __restrict__ Q0, int r, int64_t h, int j, const double* __restrict__ found,
                 double* __restrict__ g, int* __restrict__ dead) {
  __shared__ double red[kSeqThreads / 32];
  const int s = blockIdx.x;
  double* x = g + (int64_t)s * h;
  const float* q0 = Q0 + ((int64_t)s * r + j) * h;
  for (int64_t b = threadIdx.x; b < h; b += kSeqThreads) x[b] = (double)q0[b];
  __syncthreads();
  project_out(j, h, found + (int64_t)s * r * h, x, red);
  const double nrm = sqrt(block_dot(x, x, h, red));
  const bool is_dead = (nrm == 0.0);
  for (int64_t b = threadIdx.x; b < h; b += kSeqThreads) x[b] = is_dead ? 0.0 : x[b] / nrm;
  if (threadIdx.x == 0) dead[s] = is_dead ? 1 : 0;
}

// One iteration's tail: t = M g arrives from the column product; peel, project, normalise -> g.
__global__ void __launch_bounds__(kSeqThreads)
seq_step_kernel(double* __restrict__ t_all, double* __restrict__ g_all, int r, int64_t h, int j,
                const double* __restrict__ found_all, const double* __restrict__ sig_all, int* __restrict__ dead) {
  __shared__ double red[kSeqThreads / 32];
  const int s = blockIdx.x;
  double* t = t_all + (int64_t)s * h;
  double* g = g_all + (int64_t)s * h;
  const double* found = found_all + (int64_t)s * r * h;
  const double* sig = sig_all + (int64_t)s * r;
  if (dead[s]) return;  // g is zero already and stays zero
  const double before = sqrt(block_dot(t, t, h, red));
  for (int l = 0; l < j; ++l) {  // Eq. "peel"
    const double* gl = found + (int64_t)l * h;
    const double c = sig[l] * sig[l] * block_dot(gl, g, h, red);
    for (int64_t b = threadIdx.x; b < h; b += kSeqThreads) t[b] -= c * gl[b];
    __syncthreads();
  }
  project_out(j, h, found, t, red);
  const double nrm = sqrt(block_dot(t, t, h, red));
  const bool is_dead = (before == 0.0 || nrm <= 1e-12 * before);
  for (int64_t b = threadIdx.x; b < h; b += kSeqThreads) g[b] = is_dead ? 0.0 : t[b] / nrm;
  if (is_dead && threadIdx.x == 0) dead[s] = 1;
}

// Component j is done: g joins the found vectors and goes out as row j of Q; p = A^T (D g) goes out as row j of
// P; sigma_j = ||p|| = sqrt(v^T C v).
__global__ void __launch_bounds__(kSeqThreads)
seq_store_kernel(const double* __restrict__ g_all, const double* __restrict__ p_all, int r, int64_t h_in, int64_t h_out,
                 int j, double* __restrict__ found_all, double* __restrict__ sig_all, float* __restrict__ P,
                 float* __restrict__ Q, float* __restrict__ sigma) {
  __shared__ double red[kSeqThreads / 32];
  const int s = blockIdx.x;
  const double* g = g_all + (int64_t)s * h_out;
  const double* p = p_all + (int64_t)s * h_in;
  double* fj = found_all + ((int64_t)s * r + j) * h_out;
  for (int64_t b = threadIdx.x; b < h_out; b += kSeqThreads) {
    fj[b] = g[b];
    Q[((int64_t)s * r + j) * h_out + b] = (float)g[b];
  }
  for (int64_t a = threadIdx.x; a < h_in; a += kSeqThreads) P[((int64_t)s * r + j) * h_in + a] = (float)p[a];
  const double sg = sqrt(block_dot(p, p, h_in, red));
  if (threadIdx.x == 0) {
    sig_all[(int64_t)s * r + j] = sg;
    if (sigma) sigma[(int64_t)s * r + j] = (float)sg;
  }
}

struct SeqWs {
  CompressWs base;  // the r = 1 layout of the general pipeline: g (as G), Y, Z, split partials, counters
  size_t T, found, sig, dead, total;
};

SeqWs seq_ws_layout(const dad_layer& L, int r) {
  SeqWs w;
  w.base = compress_ws_layout(L, 1, true, false, 0);
  size_t off = w.base.total;
  w.T = off;
  off = align_up(off + (size_t)L.S * L.h_out * 8, 256);
  w.found = off;
  off = align_up(off + (size_t)L.S * r * L.h_out * 8, 256);
  w.sig = off;
  off = align_up(off + (size_t)L.S * r * 8, 256);
  w.dead = off;
  off = align_up(off + (size_t)L.S * sizeof(int), 256);
  w.total = off;
  return w;
}

}  // namespace
}  // namespace dad

using namespace dad;

extern "C" {

size_t dad_rank_compress_sequential_workspace_bytes(const dad_layer* L, int r, int iters) {
  if (dad_workspace_bytes(L, r, iters) == 0) return 0;
  return seq_ws_layout(*L, r).total;
}

dad_status dad_rank_compress_sequential(const dad_layer* L, const void* A, const void* D, int r, int iters,
                                        const float* Q0, float* P, float* Q, float* sigma, void* ws, size_t ws_bytes,
                                        void* cuda_stream) {
  if (!L) return DAD_ERR_NULL;
  if (L->dtype != DAD_F32 && L->dtype != DAD_BF16) return DAD_ERR_DTYPE;
  if (!A || !D || !Q0 || !P || !Q || !ws) return DAD_ERR_NULL;
  if (dad_workspace_bytes(L, r, iters) == 0) {  // same shape, stride and rank rules as dad_rank_compress
    if (r < 1 || r > DAD_MAX_RANK || r > L->h_in || r > L->h_out) return DAD_ERR_RANK;
    return DAD_ERR_SHAPE;
  }
  const uintptr_t bits = reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(D) | reinterpret_cast<uintptr_t>(Q0) |
                         reinterpret_cast<uintptr_t>(P) | reinterpret_cast<uintptr_t>(Q);
  if (bits % 16 || reinterpret_cast<uintptr_t>(ws) % 256) return DAD_ERR_ALIGN;
  const SeqWs w = seq_ws_layout(*L, r);
  if (ws_bytes < w.total) return DAD_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  char* base = static_cast<char*>(ws);
  const CompressWs& b = w.base;
  const int S = L->S;
  const int64_t N = L->N, hi = L->h_in, ho = L->h_out;
  cudaError_t err = cudaMemsetAsync(base + b.status, 0, b.counters + b.n_counters * sizeof(unsigned) - b.status, st);
  if (err != cudaSuccess) return DAD_ERR_CUDA;
  unsigned* ctr = reinterpret_cast<unsigned*>(base + b.counters);
  double* g = reinterpret_cast<double*>(base + b.G);
  double* Y = reinterpret_cast<double*>(base + b.Y);
  double* Z = reinterpret_cast<double*>(base + b.Z);
  double* part = reinterpret_cast<double*>(base + b.partial);
  double* T = reinterpret_cast<double*>(base + w.T);
  double* found = reinterpret_cast<double*>(base + w.found);
  double* sig = reinterpret_cast<double*>(base + w.sig);
  int* dead = reinterpret_cast<int*>(base + w.dead);
#define DAD_STEP(call)                            \
  do {                                            \
    err = (call);                                 \
    if (err != cudaSuccess) return DAD_ERR_CUDA;  \
  } while (0)
  for (int j = 0; j < r; ++j) {
    DAD_LAUNCH(err, "seq_vector", seq_start_kernel, (unsigned)S, kSeqThreads, 0, st, Q0, r, ho, j, (const double*)found, g,
               dead);
    if (err != cudaSuccess) return DAD_ERR_CUDA;
    for (int k = 0; k < iters; ++k) {
      DAD_STEP(rows_dot<double>(L->dtype, D, L->ldD, L->strideD, S, N, ho, g, 1, Y, st));                        // v = D g
      DAD_STEP(cols_acc<double>(L->dtype, A, L->ldA, L->strideA, S, N, hi, Y, 1, Z, nullptr, part, ctr, st));    // z = A^T v
      DAD_STEP(rows_dot<double>(L->dtype, A, L->ldA, L->strideA, S, N, hi, Z, 1, Y, st));                        // w = A z
      DAD_STEP(cols_acc<double>(L->dtype, D, L->ldD, L->strideD, S, N, ho, Y, 1, T, nullptr, part, ctr, st));    // t = D^T w
      DAD_LAUNCH(err, "seq_vector", seq_step_kernel, (unsigned)S, kSeqThreads, 0, st, T, g, r, ho, j, (const double*)found,
                 (const double*)sig, dead);
      if (err != cudaSuccess) return DAD_ERR_CUDA;
    }
    DAD_STEP(rows_dot<double>(L->dtype, D, L->ldD, L->strideD, S, N, ho, g, 1, Y, st));
    DAD_STEP(cols_acc<double>(L->dtype, A, L->ldA, L->strideA, S, N, hi, Y, 1, Z, nullptr, part, ctr, st));      // p = A^T (D g)
    DAD_LAUNCH(err, "seq_vector", seq_store_kernel, (unsigned)S, kSeqThreads, 0, st, (const double*)g, (const double*)Z, r, hi,
               ho, j, found, sig, P, Q, sigma);
    if (err != cudaSuccess) return DAD_ERR_CUDA;
  }
#undef DAD_STEP
  return DAD_OK;
}

}  // extern "C"

// Orthonormalisation of the r iterate vectors of a site (the block form of the deflation of
// Eq. "peel": each vector loses its components along the ones before it), as Cholesky-QR:
//   Gram = G G^T (fp64, r x r)  ->  Gram = L L^T  ->  rows of G <- L^{-1} G.
// This is the thin QR with positive diagonal (R = L^T).  One pass leaves an orthogonality
// defect of about 1e-16 * cond(G)^2, so a second pass follows whenever the first one shows that
// some vector lost more than three digits to the projection (R_jj < 1e-3 ||g_j||); otherwise the
// second pass's kernels return at once.  Pivots are kept from collapsing: a pivot below (1e-7)^2
// of the vector's squared length is raised to that value in the first pass (the vector then comes
// out short instead of wrong), and the second pass, which sees a well-conditioned matrix, decides
// from the product of both passes' diagonals whether the vector carried any new direction; if not
// it is set to exactly zero.
#include "common.cuh"

namespace dad {

constexpr double kPivotFloor = 1e-14;   // (1e-7)^2, relative to the squared length of the vector
constexpr double kSecondPassBelow = 1e-3;

template <typename T>
__global__ void __launch_bounds__(256)
gram_cholesky_kernel(const T* __restrict__ G, int r, int64_t h, int chunks, int pass, double tol,
                     double* __restrict__ partial, double* __restrict__ Lout, double* __restrict__ tratio,
                     unsigned char* __restrict__ dead, int* __restrict__ need2, unsigned* __restrict__ counters,
                     int* __restrict__ status) {
  extern __shared__ double sm[];  // tile of T [r][kGramChunk + 1], later the r x (r + 1) factor in fp64
  const int s = blockIdx.y, chunk = blockIdx.x, tid = threadIdx.x;
  if (pass == 1 && need2[s] == 0) return;
  T* tile = reinterpret_cast<T*>(sm);
  const T* Gs = G + (int64_t)s * r * h;
  const int64_t c0 = (int64_t)chunk * kGramChunk;
  constexpr int LD = kGramChunk + 1;
  for (int idx = tid; idx < r * kGramChunk; idx += 256) {
    const int j = idx / kGramChunk, cc = idx % kGramChunk;
    tile[j * LD + cc] = (c0 + cc < h) ? Gs[(int64_t)j * h + c0 + cc] : T(0);
  }
  __syncthreads();
  double* mine = partial + ((int64_t)s * chunks + chunk) * r * r;
  for (int p = tid; p < r * r; p += 256) {
    const int i = p / r, j = p % r;
    if (j <= i) {
      double acc = 0.0;
#pragma unroll 8
      for (int cc = 0; cc < kGramChunk; ++cc) acc += (double)tile[i * LD + cc] * (double)tile[j * LD + cc];
      mine[p] = acc;
    }
  }
  __shared__ bool is_last;
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned old = atomicAdd(counters + s, 1u);
    is_last = (old == (unsigned)chunks - 1u);
    if (is_last) counters[s] = 0u;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  // Sum the chunk partials in chunk order (loads issued eight at a time), then factor in shared memory.
  const int LR = r + 1;
  const double* src = partial + (int64_t)s * chunks * r * r;
  const int64_t rr = (int64_t)r * r;
  for (int p = tid; p < r * r; p += 256) {
    const int i = p / r, j = p % r;
    if (j <= i) {
      double v = 0.0;
      int q = 0;
      for (; q + 8 <= chunks; q += 8) {
        double t[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) t[u] = __ldcg(src + (q + u) * rr + p);
#pragma unroll
        for (int u = 0; u < 8; ++u) v += t[u];
      }
      for (; q < chunks; ++q) v += __ldcg(src + q * rr + p);
      sm[i * LR + j] = v;
    }
  }
  __shared__ double ljj;
  __shared__ int col_dead;
  __shared__ double min_ratio;
  if (tid == 0) min_ratio = 1.0;
  __syncthreads();
  double* Ls = Lout + (int64_t)s * r * r;
  for (int j = 0; j < r; ++j) {
    if (tid == 0) {
      const double d = sm[j * LR + j];
      // squared length of vector j before projection = remaining pivot + what the earlier columns took
      double orig = d;
      for (int l = 0; l < j; ++l) orig += sm[j * LR + l] * sm[j * LR + l];
      int is_dead = 0;
      double piv = d;
      if (!(orig == orig) || orig > 1.7e308) {
        *status = (int)DAD_ERR_NUMERIC;
        is_dead = 1;
      } else if (!(orig > 0.0)) {
        is_dead = 1;
      } else {
        const double floor_ = kPivotFloor * orig;
        if (!(piv > floor_)) piv = floor_;
      }
      const double l = is_dead ? 1.0 : sqrt(piv);
      if (!is_dead) {
        if (pass == 0) {
          const double t = l / sqrt(orig);
          tratio[(int64_t)s * r + j] = t;
          if (t < min_ratio) min_ratio = t;
        } else {
          // total remainder relative to the vector's length before the first pass
          const double total = tratio[(int64_t)s * r + j] * l;
          if (!(total > tol)) is_dead = 1;
        }
      } else if (pass == 0) {
        tratio[(int64_t)s * r + j] = 0.0;
      }
      ljj = l;
      col_dead = is_dead;
      dead[(int64_t)s * r + j] = (unsigned char)is_dead;
      sm[j * LR + j] = l;
    }
    __syncthreads();
    const double l = ljj;
    const int dd = col_dead;
    for (int i = j + 1 + tid; i < r; i += 256) sm[i * LR + j] = dd ? 0.0 : sm[i * LR + j] / l;
    __syncthreads();
    const int m = r - j - 1;  // trailing block rows j+1..r-1
    for (int p = tid; p < m * m; p += 256) {
      const int i = j + 1 + p / m, k = j + 1 + p % m;
      if (k <= i) sm[i * LR + k] -= sm[i * LR + j] * sm[k * LR + j];
    }
    __syncthreads();
  }
  for (int p = tid; p < r * r; p += 256) {
    const int i = p / r, j = p % r;
    Ls[p] = (j <= i) ? sm[i * LR + j] : 0.0;
  }
  if (tid == 0 && pass == 0) need2[s] = (min_ratio < kSecondPassBelow) ? 1 : 0;
}

template <typename T>
__global__ void __launch_bounds__(128)
tri_solve_kernel(T* __restrict__ G, int r, int64_t h, int pass, const double* __restrict__ L,
                 const unsigned char* __restrict__ dead, const int* __restrict__ need2, float* __restrict__ out32,
                 __nv_bfloat16* __restrict__ planes, int plane_rows) {
  extern __shared__ double sm[];  // r*r (L) + r*128 (column values, solved in place)
  double* Ls = sm;
  double* qs = sm + r * r;
  const int s = blockIdx.y, tid = threadIdx.x;
  if (pass == 1 && need2[s] == 0) return;
  const int64_t b = (int64_t)blockIdx.x * 128 + tid;
  T* Gs = G + (int64_t)s * r * h;
  if (b < h)
    for (int j = 0; j < r; ++j) qs[j * 128 + tid] = (double)Gs[(int64_t)j * h + b];  // independent loads, all in flight
  for (int p = tid; p < r * r; p += 128) Ls[p] = L[(int64_t)s * r * r + p];
  __syncthreads();
  if (b >= h) return;
  const unsigned char* ds = dead + (int64_t)s * r;
  for (int j = 0; j < r; ++j) {
    double v = qs[j * 128 + tid];
    for (int l = 0; l < j; ++l) v -= Ls[j * r + l] * qs[l * 128 + tid];
    v = ds[j] ? 0.0 : v / Ls[j * r + j];
    qs[j * 128 + tid] = v;
    Gs[(int64_t)j * h + b] = (T)v;
    if (out32) out32[((int64_t)s * r + j) * h + b] = (float)v;
    if (planes) {  // hi + lo bf16 terms of the fp32 value, for the tensor-core product that reads it next
      const float f = (float)v;
      const __nv_bfloat16 hi = __float2bfloat16_rn(f);
      planes[(((int64_t)s * 2 + 0) * plane_rows + j) * h + b] = hi;
      planes[(((int64_t)s * 2 + 1) * plane_rows + j) * h + b] = __float2bfloat16_rn(f - __bfloat162float(hi));
    }
  }
}

template <typename T>
cudaError_t cholqr_pass(T* G, int S, int r, int64_t h, int pass, double tol, double* gram_partial,
                        double* gram, double* tratio, unsigned char* dead, int* need2, unsigned* counters,
                        int* status, float* out32, __nv_bfloat16* planes, int plane_rows, cudaStream_t st) {
  cudaError_t err = cudaSuccess;
  const int chunks = (int)ceil_div(h, kGramChunk);
  const size_t a = sizeof(T) * (size_t)r * (kGramChunk + 1), b = sizeof(double) * (size_t)r * (r + 1);
  const size_t smem1 = a > b ? a : b;
  const size_t smem2 = sizeof(double) * (size_t)(r * r + r * 128);
  // the opt-in is per device and cheap, so it is simply made on every call
  if (smem1 > 48 * 1024) {
    err = cudaFuncSetAttribute(gram_cholesky_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1);
    if (err != cudaSuccess) return err;
  }
  if (smem2 > 48 * 1024) {
    err = cudaFuncSetAttribute(tri_solve_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2);
    if (err != cudaSuccess) return err;
  }
  DAD_LAUNCH(err, "gram_cholesky", (gram_cholesky_kernel<T>), dim3((unsigned)chunks, (unsigned)S), 256, smem1, st, G, r,
             h, chunks, pass, tol, gram_partial, gram, tratio, dead, need2, counters, status);
  DAD_LAUNCH(err, "tri_solve", (tri_solve_kernel<T>), dim3((unsigned)ceil_div(h, 128), (unsigned)S), 128, smem2, st, G, r,
             h, pass, gram, dead, need2, out32, planes, plane_rows);
  return err;
}
template cudaError_t cholqr_pass<float>(float*, int, int, int64_t, int, double, double*, double*, double*,
                                        unsigned char*, int*, unsigned*, int*, float*, __nv_bfloat16*, int,
                                        cudaStream_t);
template cudaError_t cholqr_pass<double>(double*, int, int, int64_t, int, double, double*, double*, double*,
                                         unsigned char*, int*, unsigned*, int*, float*, __nv_bfloat16*, int,
                                         cudaStream_t);

}  // namespace dad

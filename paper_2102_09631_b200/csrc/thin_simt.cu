// General (any shape, any alignment) kernels for the two tall-skinny products of a structured
// power iteration (Eq. "reduced_iter": the operator gradW^T gradW applied right to left through
// D and A):
//   rows_dot : Y = X F^T   (N x h by h x r)  -- one warp per row pair, reduction along h by
//              warp shuffles;
//   cols_acc : Z = Y^T X   (r x N by N x h)  -- one thread per column, rows split over CTAs,
//              partial slabs summed in a fixed order by the last CTA to arrive (deterministic).
// fp32 inputs accumulate in fp64, bf16 inputs in fp32 (TAcc).
#include "common.cuh"

namespace dad {

int cols_acc_splits(int S, int64_t N, int64_t h) {
  const int64_t colblocks = ceil_div(h, kColsAccThreads);
  const int64_t target = 148 * 8;  // CTAs wanted in flight
  int64_t splits = ceil_div(target, colblocks * S);
  const int64_t max_by_rows = ceil_div(N, 16);  // at least 16 rows per split
  if (splits > max_by_rows) splits = max_by_rows;
  if (splits > 32) splits = 32;
  if (splits < 1) splits = 1;
  return (int)splits;
}

template <typename TIn, typename TAcc, int RT, int ROWS>
__global__ void __launch_bounds__(256)
rows_dot_kernel(const TIn* __restrict__ X, int64_t ld, int64_t stride, int64_t N, int64_t h,
                const TAcc* __restrict__ F, int r, TAcc* __restrict__ Y) {
  const int s = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t row0 = ((int64_t)blockIdx.x * 8 + warp) * ROWS;
  if (row0 >= N) return;
  const TIn* Xs = X + (int64_t)s * stride;
  const TAcc* Fs = F + (int64_t)s * r * h;
  TAcc* Ys = Y + (int64_t)s * N * r;
  for (int j0 = 0; j0 < r; j0 += RT) {
    TAcc acc[ROWS][RT];
#pragma unroll
    for (int q = 0; q < ROWS; ++q)
#pragma unroll
      for (int jj = 0; jj < RT; ++jj) acc[q][jj] = TAcc(0);
#pragma unroll 4
    for (int64_t c = lane; c < h; c += 32) {  // unrolled: several columns' loads in flight per lane
      TAcc x[ROWS];
#pragma unroll
      for (int q = 0; q < ROWS; ++q)
        x[q] = (row0 + q < N) ? TAcc(to_float(Xs[(row0 + q) * ld + c])) : TAcc(0);
#pragma unroll
      for (int jj = 0; jj < RT; ++jj) {
        if (j0 + jj < r) {
          const TAcc f = Fs[(int64_t)(j0 + jj) * h + c];
#pragma unroll
          for (int q = 0; q < ROWS; ++q) acc[q][jj] += x[q] * f;
        }
      }
    }
#pragma unroll
    for (int q = 0; q < ROWS; ++q)
#pragma unroll
      for (int jj = 0; jj < RT; ++jj) {
        TAcc v = acc[q][jj];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0 && row0 + q < N && j0 + jj < r) Ys[(row0 + q) * r + j0 + jj] = v;
      }
  }
}

template <typename TAcc>
cudaError_t rows_dot(dad_dtype dt, const void* X, int64_t ld, int64_t stride, int S, int64_t N, int64_t h,
                     const TAcc* F, int r, TAcc* Y, cudaStream_t st) {
  constexpr int ROWS = 2, RT = 8;
  dim3 grid((unsigned)ceil_div(N, 8 * ROWS), (unsigned)S);
  cudaError_t err = cudaSuccess;
  if (dt == DAD_F32)
    DAD_LAUNCH(err, "rows_dot_simt", (rows_dot_kernel<float, TAcc, RT, ROWS>), grid, 256, 0, st, (const float*)X, ld, stride, N, h, F, r, Y);
  else
    DAD_LAUNCH(err, "rows_dot_simt", (rows_dot_kernel<__nv_bfloat16, TAcc, RT, ROWS>), grid, 256, 0, st, (const __nv_bfloat16*)X, ld,
               stride, N, h, F, r, Y);
  return err;
}
template cudaError_t rows_dot<float>(dad_dtype, const void*, int64_t, int64_t, int, int64_t, int64_t, const float*, int,
                                     float*, cudaStream_t);
template cudaError_t rows_dot<double>(dad_dtype, const void*, int64_t, int64_t, int, int64_t, int64_t, const double*,
                                      int, double*, cudaStream_t);

template <typename TIn, typename TAcc, int RT>
__global__ void __launch_bounds__(kColsAccThreads)
cols_acc_kernel(const TIn* __restrict__ X, int64_t ld, int64_t stride, int64_t N, int64_t h,
                const TAcc* __restrict__ Y, int r, TAcc* __restrict__ Z, float* __restrict__ out32,
                TAcc* __restrict__ partial, unsigned* __restrict__ counters, int splits, int64_t rows_per_split) {
  const int s = blockIdx.z, split = blockIdx.y;
  const int64_t c = (int64_t)blockIdx.x * kColsAccThreads + threadIdx.x;
  const int64_t n0 = (int64_t)split * rows_per_split;
  const int64_t n1 = (n0 + rows_per_split < N) ? n0 + rows_per_split : N;
  const TIn* Xs = X + (int64_t)s * stride;
  const TAcc* Ys = Y + (int64_t)s * N * r;
  TAcc* Zs = Z + (int64_t)s * r * h;
  TAcc* dst = (splits == 1) ? Zs : partial + ((int64_t)s * splits + split) * r * h;
  for (int j0 = 0; j0 < r; j0 += RT) {
    TAcc acc[RT];
#pragma unroll
    for (int jj = 0; jj < RT; ++jj) acc[jj] = TAcc(0);
#pragma unroll 4
    for (int64_t n = n0; n < n1; ++n) {
      const TAcc x = (c < h) ? TAcc(to_float(Xs[n * ld + c])) : TAcc(0);
#pragma unroll
      for (int jj = 0; jj < RT; ++jj)
        if (j0 + jj < r) acc[jj] += Ys[n * r + j0 + jj] * x;
    }
    if (c < h) {
#pragma unroll
      for (int jj = 0; jj < RT; ++jj)
        if (j0 + jj < r) {
          dst[(int64_t)(j0 + jj) * h + c] = acc[jj];
          if (splits == 1 && out32) out32[((int64_t)s * r + j0 + jj) * h + c] = (float)acc[jj];
        }
    }
  }
  if (splits == 1) return;
  // Last CTA of this (site, column block) to arrive sums the partial slabs in split order.
  __shared__ bool is_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned* ctr = counters + (int64_t)s * gridDim.x + blockIdx.x;
    const unsigned old = atomicAdd(ctr, 1u);
    is_last = (old == (unsigned)splits - 1u);
    if (is_last) *ctr = 0u;  // ready for the next launch on this stream
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  if (c < h) {
    const TAcc* src = partial + (int64_t)s * splits * r * h;
    for (int j = 0; j < r; ++j) {
      TAcc v = TAcc(0);
      for (int p = 0; p < splits; ++p) v += __ldcg(src + ((int64_t)p * r + j) * h + c);
      Zs[(int64_t)j * h + c] = v;
      if (out32) out32[((int64_t)s * r + j) * h + c] = (float)v;
    }
  }
}

template <typename TAcc>
cudaError_t cols_acc(dad_dtype dt, const void* X, int64_t ld, int64_t stride, int S, int64_t N, int64_t h,
                     const TAcc* Y, int r, TAcc* Z, float* out32, TAcc* partial, unsigned* counters,
                     cudaStream_t st) {
  constexpr int RT = 8;
  const int splits = cols_acc_splits(S, N, h);
  const int64_t rows_per_split = ceil_div(N, splits);
  dim3 grid((unsigned)ceil_div(h, kColsAccThreads), (unsigned)splits, (unsigned)S);
  cudaError_t err = cudaSuccess;
  if (dt == DAD_F32)
    DAD_LAUNCH(err, "cols_acc_simt", (cols_acc_kernel<float, TAcc, RT>), grid, kColsAccThreads, 0, st, (const float*)X, ld, stride, N, h,
               Y, r, Z, out32, partial, counters, splits, rows_per_split);
  else
    DAD_LAUNCH(err, "cols_acc_simt", (cols_acc_kernel<__nv_bfloat16, TAcc, RT>), grid, kColsAccThreads, 0, st,
               (const __nv_bfloat16*)X, ld, stride, N, h, Y, r, Z, out32, partial, counters, splits, rows_per_split);
  return err;
}
template cudaError_t cols_acc<float>(dad_dtype, const void*, int64_t, int64_t, int, int64_t, int64_t, const float*, int,
                                     float*, float*, float*, unsigned*, cudaStream_t);
template cudaError_t cols_acc<double>(dad_dtype, const void*, int64_t, int64_t, int, int64_t, int64_t, const double*,
                                      int, double*, float*, double*, unsigned*, cudaStream_t);

}  // namespace dad

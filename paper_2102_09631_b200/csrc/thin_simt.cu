// General (any shape, any alignment) kernels for the two tall-skinny products of a structured
// power iteration (Eq. "reduced_iter": the operator gradW^T gradW applied right to left through
// D and A):
//   rows_dot : Y = X F^T   (N x h by h x r)  -- one CTA per 8 rows, columns split over its warps,
//              reduction along h by a shuffle reduce-scatter and a fixed-order sum over the warps;
//   cols_acc : Z = Y^T X   (r x N by N x h)  -- one CTA per 128 columns, rows split over its warps and over
//              CTAs, partial slabs summed in a fixed order by the last CTA to arrive (deterministic).
// fp32 inputs accumulate in fp64, bf16 inputs in fp32 (TAcc).
#include "bounds.cuh"
#include "common.cuh"
#include "warp_reduce.cuh"

namespace dad {

// Row splits of the general column-slab product: about two CTAs per SM, at least 32 rows per split (four per
// warp), at most 16 (measured on stacks of 32 ... 1024 rows: more splits only add slabs for the finishing CTA).
int cols_acc_splits(int S, int64_t N, int64_t h) {
  const int64_t colblocks = ceil_div(h, kColsAccThreads);
  const int64_t target = 148 * 2;
  int64_t splits = ceil_div(target, colblocks * S);
  const int64_t max_by_rows = N / 32;
  if (splits > max_by_rows) splits = max_by_rows;
  if (splits > 16) splits = 16;
  if (splits < 1) splits = 1;
  return (int)splits;
}

// One CTA per RB rows and RT factor rows: its 8 warps split the columns (warp w takes columns 32 w .. 32 w + 31 of every 256), every
// lane accumulates RB x RT products, the warp sums them with the reduce-scatter above, and the 8 warp sums are
// added in warp order through shared memory.  Each element of F is read once per RB rows.
template <typename TIn, typename TAcc, int RT, int RB>
__global__ void __launch_bounds__(256)
rows_dot_kernel(const TIn* __restrict__ X, int64_t ld, int64_t stride, int64_t N, int64_t h,
                const TAcc* __restrict__ F, int r, TAcc* __restrict__ Y) {
  constexpr int NV = RB * RT;
  __shared__ TAcc red[8][NV];
  const int s = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t row0 = (int64_t)blockIdx.x * RB;
  const TIn* Xs = X + (int64_t)s * stride;
  const TAcc* Fs = F + (int64_t)s * r * h;
  TAcc* Ys = Y + (int64_t)s * N * r;
  {
    const int j0 = blockIdx.z * RT;  // one block of RT factor rows per CTA
    TAcc acc[NV];  // [q * RT + jj]
#pragma unroll
    for (int i = 0; i < NV; ++i) acc[i] = TAcc(0);
#pragma unroll 4
    for (int64_t c = warp * 32 + lane; c < h; c += 256) {
      TAcc x[RB];
#pragma unroll
      for (int q = 0; q < RB; ++q) x[q] = (row0 + q < N) ? TAcc(to_float(DAD_LD(&Xs[(row0 + q) * ld + c]))) : TAcc(0);
#pragma unroll
      for (int jj = 0; jj < RT; ++jj) {
        if (j0 + jj < r) {
          const TAcc f = DAD_LD(&Fs[(int64_t)(j0 + jj) * h + c]);
#pragma unroll
          for (int q = 0; q < RB; ++q) acc[q * RT + jj] += x[q] * f;
        }
      }
    }
    warp_reduce_scatter<TAcc, NV>(acc, lane);
#pragma unroll
    for (int i = 0; i < NV / 32; ++i) red[warp][reduced_index<NV>(lane, i)] = acc[i];
    __syncthreads();
    if (threadIdx.x < NV) {
      TAcc v = red[0][threadIdx.x];
#pragma unroll
      for (int w = 1; w < 8; ++w) v += red[w][threadIdx.x];
      const int q = threadIdx.x / RT, jj = threadIdx.x % RT;
      if (row0 + q < N && j0 + jj < r) DAD_ST(&Ys[(row0 + q) * r + j0 + jj], v);
    }
  }
}

template <typename TAcc>
cudaError_t rows_dot(dad_dtype dt, const void* X, int64_t ld, int64_t stride, int S, int64_t N, int64_t h,
                     const TAcc* F, int r, TAcc* Y, cudaStream_t st) {
  constexpr int RB = 8, RT = 8;
  dim3 grid((unsigned)ceil_div(N, RB), (unsigned)S, (unsigned)ceil_div(r, RT));
  cudaError_t err = cudaSuccess;
  if (dt == DAD_F32)
    DAD_LAUNCH(err, "rows_dot_simt", (rows_dot_kernel<float, TAcc, RT, RB>), grid, 256, 0, st, (const float*)X, ld, stride, N, h, F, r, Y);
  else
    DAD_LAUNCH(err, "rows_dot_simt", (rows_dot_kernel<__nv_bfloat16, TAcc, RT, RB>), grid, 256, 0, st, (const __nv_bfloat16*)X, ld,
               stride, N, h, F, r, Y);
  return err;
}
template cudaError_t rows_dot<float>(dad_dtype, const void*, int64_t, int64_t, int, int64_t, int64_t, const float*, int,
                                     float*, cudaStream_t);
template cudaError_t rows_dot<double>(dad_dtype, const void*, int64_t, int64_t, int, int64_t, int64_t, const double*,
                                      int, double*, cudaStream_t);

// One CTA per (site, block of 128 columns, split of the rows): its 8 warps take every 8th row of the split, each
// lane four columns 32 apart (coalesced 128-byte rows of X per warp), and the warps' sums are added in warp
// order through shared memory.  With a split contraction the slab goes to `partial`, and the last CTA of the
// column block to arrive adds the slabs in split order.
template <typename TIn, typename TAcc, int RT>
__global__ void __launch_bounds__(256)
cols_acc_kernel(const TIn* __restrict__ X, int64_t ld, int64_t stride, int64_t N, int64_t h,
                const TAcc* __restrict__ Y, int r, TAcc* __restrict__ Z, float* __restrict__ out32,
                TAcc* __restrict__ partial, unsigned* __restrict__ counters, int splits, int64_t rows_per_split) {
  __shared__ TAcc red[RT][kColsAccThreads];
  const int s = blockIdx.z, split = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t cb = (int64_t)blockIdx.x * kColsAccThreads;
  const int64_t n0 = (int64_t)split * rows_per_split;
  const int64_t n1 = (n0 + rows_per_split < N) ? n0 + rows_per_split : N;
  const TIn* Xs = X + (int64_t)s * stride;
  const TAcc* Ys = Y + (int64_t)s * N * r;
  TAcc* Zs = Z + (int64_t)s * r * h;
  TAcc* dst = (splits == 1) ? Zs : partial + ((int64_t)s * splits + split) * r * h;
  for (int j0 = 0; j0 < r; j0 += RT) {
    TAcc acc[4][RT];
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
      for (int jj = 0; jj < RT; ++jj) acc[q][jj] = TAcc(0);
#pragma unroll 2
    for (int64_t n = n0 + warp; n < n1; n += 8) {
      TAcc x[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int64_t c = cb + q * 32 + lane;
        x[q] = (c < h) ? TAcc(to_float(DAD_LD(&Xs[n * ld + c]))) : TAcc(0);
      }
#pragma unroll
      for (int jj = 0; jj < RT; ++jj) {
        if (j0 + jj < r) {
          const TAcc y = DAD_LD(&Ys[n * r + j0 + jj]);
#pragma unroll
          for (int q = 0; q < 4; ++q) acc[q][jj] += y * x[q];
        }
      }
    }
    for (int w = 0; w < 8; ++w) {  // warp order: a fixed summation order
      if (warp == w) {
#pragma unroll
        for (int q = 0; q < 4; ++q)
#pragma unroll
          for (int jj = 0; jj < RT; ++jj) {
            TAcc* cell = &red[jj][q * 32 + lane];
            *cell = (w == 0) ? acc[q][jj] : *cell + acc[q][jj];
          }
      }
      __syncthreads();
    }
    for (int idx = threadIdx.x; idx < RT * kColsAccThreads; idx += 256) {
      const int jj = idx / kColsAccThreads;
      const int64_t c = cb + idx % kColsAccThreads;
      if (c < h && j0 + jj < r) {
        const TAcc v = red[jj][idx % kColsAccThreads];
        DAD_ST(&dst[(int64_t)(j0 + jj) * h + c], v);
        if (splits == 1 && out32) DAD_ST(&out32[((int64_t)s * r + j0 + jj) * h + c], (float)v);
      }
    }
    __syncthreads();
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
  const TAcc* src = partial + (int64_t)s * splits * r * h;
  for (int idx = threadIdx.x; idx < r * kColsAccThreads; idx += 256) {
    const int j = idx / kColsAccThreads;
    const int64_t c = cb + idx % kColsAccThreads;
    if (c >= h) continue;
    TAcc v = TAcc(0);
    int p = 0;
    for (; p + 4 <= splits; p += 4) {  // four loads in flight, added in split order
      TAcc t[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) t[u] = DAD_LDCG(src + ((int64_t)(p + u) * r + j) * h + c);
#pragma unroll
      for (int u = 0; u < 4; ++u) v += t[u];
    }
    for (; p < splits; ++p) v += DAD_LDCG(src + ((int64_t)p * r + j) * h + c);
    DAD_ST(&Zs[(int64_t)j * h + c], v);
    if (out32) DAD_ST(&out32[((int64_t)s * r + j) * h + c], (float)v);
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
    DAD_LAUNCH(err, "cols_acc_simt", (cols_acc_kernel<float, TAcc, RT>), grid, 256, 0, st, (const float*)X, ld, stride, N, h,
               Y, r, Z, out32, partial, counters, splits, rows_per_split);
  else
    DAD_LAUNCH(err, "cols_acc_simt", (cols_acc_kernel<__nv_bfloat16, TAcc, RT>), grid, 256, 0, st,
               (const __nv_bfloat16*)X, ld, stride, N, h, Y, r, Z, out32, partial, counters, splits, rows_per_split);
  return err;
}
template cudaError_t cols_acc<float>(dad_dtype, const void*, int64_t, int64_t, int, int64_t, int64_t, const float*, int,
                                     float*, float*, float*, unsigned*, cudaStream_t);
template cudaError_t cols_acc<double>(dad_dtype, const void*, int64_t, int64_t, int, int64_t, int64_t, const double*,
                                      int, double*, float*, double*, unsigned*, cudaStream_t);

}  // namespace dad

// General fp32-FMA kernel for the two dense products of the path, both of the form
//   C[a][b] = sum_k X[k][a] * Y[k][b]
// with the contraction index k as the row index of both operands:
//   - the uncompressed dAD gradient sum_s A_s^T D_s (Sec. 3.2; k runs over all sites' rows),
//   - the reconstruction Pcat^T Qcat (Algorithm 1; k runs over the S*r stacked factor rows).
// Used for fp32 inputs (where bf16 tensor-core products would miss the 1e-5 parity bound) and
// for layouts the tensor-core kernel does not take.  Also small helpers: factor gather copy,
// fp32 -> fp64 widening, row norms.
#include "bounds.cuh"
#include "common.cuh"

namespace dad {

constexpr int BM = 64, BN = 64, BK = 16;

template <typename TIn>
__global__ void __launch_bounds__(256)
gemm_tn_kernel(const TIn* __restrict__ X, int64_t ldX, int64_t strideX, const TIn* __restrict__ Y, int64_t ldY,
               int64_t strideY, int64_t N, int64_t Ktot, int64_t hx, int64_t hy, float* __restrict__ C) {
  __shared__ __align__(16) float Xs[BK][BM];
  __shared__ __align__(16) float Ys[BK][BN];
  const int tid = threadIdx.x;
  const int tx = tid % 16, ty = tid / 16;
  const int64_t a0 = (int64_t)blockIdx.y * BM, b0 = (int64_t)blockIdx.x * BN;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  for (int64_t k0 = 0; k0 < Ktot; k0 += BK) {
#pragma unroll
    for (int i = 0; i < (BK * BM) / 256; ++i) {
      const int idx = tid + i * 256;
      const int kk = idx / BM, col = idx % BM;
      const int64_t k = k0 + kk;
      float xv = 0.f, yv = 0.f;
      if (k < Ktot) {
        const int64_t s = k / N, n = k % N;
        if (a0 + col < hx) xv = to_float(DAD_LD(&X[s * strideX + n * ldX + a0 + col]));
        if (b0 + col < hy) yv = to_float(DAD_LD(&Y[s * strideY + n * ldY + b0 + col]));
      }
      Xs[kk][col] = xv;
      Ys[kk][col] = yv;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      const float4 xa = *reinterpret_cast<const float4*>(&Xs[kk][ty * 4]);
      const float4 yb = *reinterpret_cast<const float4*>(&Ys[kk][tx * 4]);
      const float xr[4] = {xa.x, xa.y, xa.z, xa.w};
      const float yr[4] = {yb.x, yb.y, yb.z, yb.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(xr[i], yr[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t a = a0 + ty * 4 + i;
    if (a >= hx) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t b = b0 + tx * 4 + j;
      if (b < hy) DAD_ST(&C[a * hy + b], acc[i][j]);
    }
  }
}

cudaError_t gemm_tn_simt(dad_dtype dt, const void* X, int64_t ldX, int64_t strideX, const void* Y,
                         int64_t ldY, int64_t strideY, int S, int64_t N, int64_t hx, int64_t hy, float* C,
                         cudaStream_t st) {
  dim3 grid((unsigned)ceil_div(hy, BN), (unsigned)ceil_div(hx, BM));
  cudaError_t err = cudaSuccess;
  const int64_t Ktot = (int64_t)S * N;
  if (dt == DAD_F32)
    DAD_LAUNCH(err, "gemm_tn_simt", (gemm_tn_kernel<float>), grid, 256, 0, st, (const float*)X, ldX, strideX, (const float*)Y, ldY,
               strideY, N, Ktot, hx, hy, C);
  else
    DAD_LAUNCH(err, "gemm_tn_simt", (gemm_tn_kernel<__nv_bfloat16>), grid, 256, 0, st, (const __nv_bfloat16*)X, ldX, strideX,
               (const __nv_bfloat16*)Y, ldY, strideY, N, Ktot, hx, hy, C);
  return err;
}

// ---- small helpers ---------------------------------------------------------------------------
__global__ void copy_two_kernel(const float* __restrict__ a, float* __restrict__ a_out, size_t na,
                                const float* __restrict__ b, float* __restrict__ b_out, size_t nb) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < na + nb; i += stride) {
    if (i < na) {
      if (a_out != a) DAD_ST(&a_out[i], DAD_LD(&a[i]));
    } else {
      if (b_out != b) DAD_ST(&b_out[i - na], DAD_LD(&b[i - na]));
    }
  }
}

// The same with 16-byte accesses: na and nb count float4 elements.
__global__ void copy_two_vec_kernel(const float4* __restrict__ a, float4* __restrict__ a_out, size_t na,
                                    const float4* __restrict__ b, float4* __restrict__ b_out, size_t nb) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < na + nb; i += stride) {
    if (i < na) {
      if (a_out != a) DAD_ST(&a_out[i], DAD_LD(&a[i]));
    } else {
      if (b_out != b) DAD_ST(&b_out[i - na], DAD_LD(&b[i - na]));
    }
  }
}

cudaError_t copy_two(const float* a, float* a_out, size_t na, const float* b, float* b_out, size_t nb,
                     cudaStream_t st) {
  cudaError_t err = cudaSuccess;
  const bool vec = na % 4 == 0 && nb % 4 == 0 &&
                   ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(a_out) | reinterpret_cast<uintptr_t>(b) |
                     reinterpret_cast<uintptr_t>(b_out)) & 15) == 0;
  const size_t items = vec ? (na + nb) / 4 : na + nb;
  size_t blocks = (items + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  if (vec) {
    DAD_LAUNCH(err, "gather_copy", copy_two_vec_kernel, (unsigned)blocks, 256, 0, st, reinterpret_cast<const float4*>(a),
               reinterpret_cast<float4*>(a_out), na / 4, reinterpret_cast<const float4*>(b),
               reinterpret_cast<float4*>(b_out), nb / 4);
  } else {
    DAD_LAUNCH(err, "gather_copy", copy_two_kernel, (unsigned)blocks, 256, 0, st, a, a_out, na, b, b_out, nb);
  }
  return err;
}

__global__ void widen_kernel(const float* __restrict__ in, double* __restrict__ out, size_t n) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) out[i] = (double)in[i];
}

cudaError_t widen_f32_to_f64(const float* in, double* out, size_t n, cudaStream_t st) {
  cudaError_t err = cudaSuccess;
  size_t blocks = (n + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  DAD_LAUNCH(err, "widen", widen_kernel, (unsigned)blocks, 256, 0, st, in, out, n);
  return err;
}

__global__ void split_planes_kernel(const float* __restrict__ in, int r, int64_t h, __nv_bfloat16* __restrict__ planes,
                                    int plane_rows, size_t n) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const size_t c = i % (size_t)h, sj = i / (size_t)h;
    const size_t j = sj % (size_t)r, s = sj / (size_t)r;
    const float f = in[i];
    const __nv_bfloat16 hi = __float2bfloat16_rn(f);
    planes[((s * 2 + 0) * plane_rows + j) * h + c] = hi;
    planes[((s * 2 + 1) * plane_rows + j) * h + c] = __float2bfloat16_rn(f - __bfloat162float(hi));
  }
}

// Four elements per thread (h a multiple of four, `in` 16-byte and `planes` 8-byte aligned); n counts quads.
__global__ void split_planes_vec_kernel(const float4* __restrict__ in, int r, int64_t h4, __nv_bfloat16* __restrict__ planes,
                                        int plane_rows, size_t n) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const size_t c = i % (size_t)h4, sj = i / (size_t)h4;
    const size_t j = sj % (size_t)r, s = sj / (size_t)r;
    const float4 v = in[i];
    const float f[4] = {v.x, v.y, v.z, v.w};
    __align__(8) __nv_bfloat16 hi[4], lo[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      hi[u] = __float2bfloat16_rn(f[u]);
      lo[u] = __float2bfloat16_rn(f[u] - __bfloat162float(hi[u]));
    }
    uint2* ph = reinterpret_cast<uint2*>(planes + ((s * 2 + 0) * plane_rows + j) * (size_t)(h4 * 4)) + c;
    uint2* pl = reinterpret_cast<uint2*>(planes + ((s * 2 + 1) * plane_rows + j) * (size_t)(h4 * 4)) + c;
    *ph = *reinterpret_cast<const uint2*>(hi);
    *pl = *reinterpret_cast<const uint2*>(lo);
  }
}

cudaError_t split_planes(const float* in, int S, int r, int64_t h, __nv_bfloat16* planes, int plane_rows,
                         cudaStream_t st) {
  cudaError_t err = cudaSuccess;
  const size_t n = (size_t)S * r * h;
  const bool vec = h % 4 == 0 && (reinterpret_cast<uintptr_t>(in) & 15) == 0 && (reinterpret_cast<uintptr_t>(planes) & 7) == 0;
  const size_t items = vec ? n / 4 : n;
  size_t blocks = (items + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  if (vec) {
    DAD_LAUNCH(err, "split_planes", split_planes_vec_kernel, (unsigned)blocks, 256, 0, st,
               reinterpret_cast<const float4*>(in), r, h / 4, planes, plane_rows, items);
  } else {
    DAD_LAUNCH(err, "split_planes", split_planes_kernel, (unsigned)blocks, 256, 0, st, in, r, h, planes, plane_rows, n);
  }
  return err;
}

// Operands of the reconstruction sum_k P_k^T Q_k (Algorithm 1, the P^T Q step; Section 3.3) for a bf16 tensor-core product that keeps
// fp32-level accuracy: with x = hi(x) + lo(x) (two bf16 terms), P^T Q ~= hi^T hi + hi^T lo + lo^T hi, the
// dropped lo^T lo term being 2^-16 relative.  The three products become one contraction of length 3K over
//     X3 = [hi(P); hi(P); lo(P)]   and   Y3 = [hi(Q); lo(Q); hi(Q)].
// Four elements per thread; nP and nQ are multiples of 4 and all pointers 8-byte aligned.  `batch` independent
// factor stacks lie one after the other in P and Q; each gets its own three-term stack in X3 and Y3.
// With terms == 1 only the hi terms are stored (X = hi(P), Y = hi(Q)): one product, about 8 significant bits of
// each factor.
__global__ void stack_split3_kernel(const float* __restrict__ P, size_t nP, __nv_bfloat16* __restrict__ X3,
                                    const float* __restrict__ Q, size_t nQ, __nv_bfloat16* __restrict__ Y3, int batch,
                                    int terms) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  const size_t qP = nP / 4, qQ = nQ / 4;
  const size_t allP = qP * (size_t)batch, all = (qP + qQ) * (size_t)batch;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < all; i += stride) {
    const bool isP = i < allP;
    const size_t lin = isP ? i : i - allP;     // quad index over all batch entries of this operand
    const size_t plane = isP ? qP : qQ;        // quads per term of one batch entry
    const size_t b = lin / plane, q = lin % plane;
    const float4 v = reinterpret_cast<const float4*>(isP ? P : Q)[lin];
    const float f[4] = {v.x, v.y, v.z, v.w};
    __align__(8) __nv_bfloat16 hi[4], lo[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      hi[u] = __float2bfloat16_rn(f[u]);
      lo[u] = __float2bfloat16_rn(f[u] - __bfloat162float(hi[u]));
    }
    const uint2 h2 = *reinterpret_cast<const uint2*>(hi), l2 = *reinterpret_cast<const uint2*>(lo);
    uint2* out = reinterpret_cast<uint2*>(isP ? X3 : Y3) + b * terms * plane;
    out[q] = h2;
    if (terms == 3) {
      out[plane + q] = isP ? h2 : l2;
      out[2 * plane + q] = isP ? l2 : h2;
    }
  }
}

cudaError_t stack_split3(const float* P, size_t nP, __nv_bfloat16* X3, const float* Q, size_t nQ, __nv_bfloat16* Y3,
                         int batch, int terms, cudaStream_t st) {
  cudaError_t err = cudaSuccess;
  size_t blocks = ((nP + nQ) / 4 * (size_t)batch + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  DAD_LAUNCH(err, "stack_split3", stack_split3_kernel, (unsigned)blocks, 256, 0, st, P, nP, X3, Q, nQ, Y3, batch, terms);
  return err;
}

// out[row] = || M[row] ||_2, one warp per row (sigma_j = ||P_j||, Algorithm 2's sqrt(v^T C v)).
template <typename T>
__global__ void __launch_bounds__(256) row_norms_kernel(const T* __restrict__ M, int64_t rows, int64_t h,
                                                        float* __restrict__ out) {
  const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;  // four partial sums per lane: loads and additions overlap
  const T* Mr = M + row * h;
  int64_t c = lane;
  if constexpr (sizeof(T) == 4) {
    if ((h & 3) == 0 && (reinterpret_cast<uintptr_t>(M) & 15) == 0) {  // 16-byte loads, two in flight per lane
      const float4* M4 = reinterpret_cast<const float4*>(Mr);
      const int64_t h4 = h / 4;
      int64_t q = lane;
      for (; q + 32 < h4; q += 64) {
        const float4 u = M4[q], w = M4[q + 32];
        a0 += (double)u.x * u.x + (double)u.y * u.y;
        a1 += (double)u.z * u.z + (double)u.w * u.w;
        a2 += (double)w.x * w.x + (double)w.y * w.y;
        a3 += (double)w.z * w.z + (double)w.w * w.w;
      }
      for (; q < h4; q += 32) {
        const float4 u = M4[q];
        a0 += (double)u.x * u.x + (double)u.y * u.y;
        a1 += (double)u.z * u.z + (double)u.w * u.w;
      }
      c = h;  // nothing left for the scalar loops
    }
  }
  for (; c + 96 < h; c += 128) {
    const double v0 = (double)Mr[c], v1 = (double)Mr[c + 32], v2 = (double)Mr[c + 64], v3 = (double)Mr[c + 96];
    a0 += v0 * v0;
    a1 += v1 * v1;
    a2 += v2 * v2;
    a3 += v3 * v3;
  }
  for (; c < h; c += 32) {
    const double v = (double)Mr[c];
    a0 += v * v;
  }
  double acc = (a0 + a1) + (a2 + a3);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) out[row] = (float)sqrt(acc);
}

template <typename T>
cudaError_t row_norms(const T* M, int64_t rows, int64_t h, float* out, cudaStream_t st) {
  cudaError_t err = cudaSuccess;
  DAD_LAUNCH(err, "row_norms", (row_norms_kernel<T>), (unsigned)ceil_div(rows, 8), 256, 0, st, M, rows, h, out);
  return err;
}
template cudaError_t row_norms<float>(const float*, int64_t, int64_t, float*, cudaStream_t);
template cudaError_t row_norms<double>(const double*, int64_t, int64_t, float*, cudaStream_t);

}  // namespace dad

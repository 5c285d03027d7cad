// One-launch compress for small sites: a thread-block cluster owns a site for the WHOLE structured power
// iteration (Algorithm 2): every application of the operator gradW^T gradW through D and A (Eq. "reduced_iter"),
// the orthonormalisation of the r vectors after each (Eq. "peel" as block deflation), and the final input-side
// factor P = (A^T (D G^T))^T with sigma_j = ||P_j||.
//
// The N rows of the site are dealt out to the C CTAs of the cluster.  The two row-wise products of an application,
//     Y = D G^T   and   W = A Z^T            (N x r: a row of the result needs only that row of D or A),
// are local to a CTA; the two column-wise products,
//     Z = Y^T A   and   G~ = W^T D           (r x h: sums over all rows),
// leave every CTA with a partial sum over its own rows.  The partials meet in a scratch area (global memory, i.e.
// L2): after a cluster barrier CTA q adds the C partials of its own slice of the columns in rank order -- the same
// order whatever the timing, so two runs agree bit for bit -- and publishes the slice for everybody.  The slice of
// G~ stays in the CTA's shared memory for the Cholesky-QR (orth_slab.cuh), whose r x r Gram matrix is summed over
// distributed shared memory.  The only synchronisation is the hardware cluster barrier; no wait is a spin.
//
// Y and W live in shared memory; A_s and D_s are re-read from L2 / L1 on every pass (a site this kernel takes is a
// few hundred KB per CTA at most).  fp32 inputs accumulate in fp64 and keep fp64 intermediates; bf16 inputs in fp32.
#include "bounds.cuh"
#include "orth_slab.cuh"
#include "warp_reduce.cuh"

namespace dad {
using namespace orthslab;

struct FusedParams {
  const void* A;
  const void* D;
  int64_t ldA, ldD, strideA, strideD;
  int N, h_in, h_out, r, iters, C;
  const float* Q0;
  float* P;
  float* Q;
  float* sigma;
  void* FG;          // S x r x h_out  accumulator type: the iterate G, complete, republished after every orthonormalisation
  void* FZ;          // S x r x h_in   accumulator type: Z, complete
  void* part;        // S x C x r x hmax accumulator type: per-CTA partial sums of the column-wise products
  double* sig_part;  // S x C x r: squared lengths of the slices of P
  int* status;
  double tol;
};

namespace {

constexpr int kRowGroup = 4;   // rows a warp advances together in the row-wise products
constexpr int kVecBlock = 8;   // vectors (rows of the factor) per register block

__device__ __forceinline__ void cluster_barrier(cg::cluster_group& cluster) {
  __threadfence();  // what this thread wrote to global memory is visible before the barrier releases anybody
  cluster.sync();
}

// Y[n][j] = sum_c X[n][c] F[j][c] for this CTA's rows.  A warp takes kRowGroup rows x kVecBlock vectors at a
// time, its lanes stride over the columns (coalesced rows of X and F), and the 32 sums are completed with the
// exchange tree of warp_reduce.cuh.  Y has `rpad` (a multiple of kVecBlock) entries per row, those >= r zero.
template <typename TIn, typename TAcc>
__device__ __forceinline__ void fused_rows_dot(const TIn* __restrict__ X, int64_t ld, int nrows, int h, const TAcc* F,
                                               int r, int rpad, TAcc* Y) {
  constexpr int NV = kRowGroup * kVecBlock;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_jb = rpad / kVecBlock;
  const int items = ((nrows + kRowGroup - 1) / kRowGroup) * n_jb;
  for (int item = warp; item < items; item += kThreads / 32) {
    const int row0 = (item / n_jb) * kRowGroup, j0 = (item % n_jb) * kVecBlock;
    TAcc acc[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) acc[i] = TAcc(0);
#pragma unroll 2
    for (int c = lane; c < h; c += 32) {
      TAcc x[kRowGroup];
#pragma unroll
      for (int q = 0; q < kRowGroup; ++q) x[q] = (row0 + q < nrows) ? TAcc(to_float(DAD_LD(&X[(int64_t)(row0 + q) * ld + c]))) : TAcc(0);
#pragma unroll
      for (int jj = 0; jj < kVecBlock; ++jj) {
        if (j0 + jj < r) {
          const TAcc f = DAD_LD(&F[(int64_t)(j0 + jj) * h + c]);
#pragma unroll
          for (int q = 0; q < kRowGroup; ++q) acc[q * kVecBlock + jj] += x[q] * f;
        }
      }
    }
    warp_reduce_scatter<TAcc, NV>(acc, lane);
    const int idx = reduced_index<NV>(lane, 0);
    const int q = idx / kVecBlock, jj = idx % kVecBlock;
    if (row0 + q < nrows) Y[(row0 + q) * rpad + j0 + jj] = (j0 + jj < r) ? acc[0] : TAcc(0);
  }
}

// out[j][c] = sum over this CTA's rows of Y[n][j] X[n][c]: a thread owns CG columns 256 apart, and adds the rows
// in their order (one fixed summation order).  Rows of X are read coalesced, Y is broadcast from shared memory.
template <typename TIn, typename TAcc, int CG>
__device__ __forceinline__ void fused_cols_acc(const TIn* __restrict__ X, int64_t ld, int nrows, int h, const TAcc* Y,
                                               int r, int rpad, TAcc* __restrict__ out) {
  for (int cb = threadIdx.x; cb < h; cb += kThreads * CG) {
    for (int j0 = 0; j0 < rpad; j0 += kVecBlock) {
      TAcc acc[CG][kVecBlock];
#pragma unroll
      for (int g = 0; g < CG; ++g)
#pragma unroll
        for (int jj = 0; jj < kVecBlock; ++jj) acc[g][jj] = TAcc(0);
#pragma unroll 2
      for (int n = 0; n < nrows; ++n) {
        TAcc x[CG];
#pragma unroll
        for (int g = 0; g < CG; ++g) {
          const int c = cb + g * kThreads;
          x[g] = (c < h) ? TAcc(to_float(DAD_LD(&X[(int64_t)n * ld + c]))) : TAcc(0);
        }
#pragma unroll
        for (int jj = 0; jj < kVecBlock; ++jj) {
          const TAcc y = Y[n * rpad + j0 + jj];
#pragma unroll
          for (int g = 0; g < CG; ++g) acc[g][jj] += y * x[g];
        }
      }
#pragma unroll
      for (int g = 0; g < CG; ++g) {
        const int c = cb + g * kThreads;
        if (c < h) {
#pragma unroll
          for (int jj = 0; jj < kVecBlock; ++jj)
            if (j0 + jj < r) DAD_ST(&out[(int64_t)(j0 + jj) * h + c], acc[g][jj]);
        }
      }
    }
  }
}

// Complete sums of this CTA's slice [c0, c0 + W) of the columns: value (j, c) = sum over the C partials in rank
// order (the partial of CTA q is a compact r x h matrix at part_site + q * part_stride).  A warp takes whole vectors j, its lanes stride over the slice; sink(j, cc, c, v) receives every element
// of the slice (cc = c - c0; v = 0 beyond column h), in increasing cc for a lane.
template <typename TAcc, typename Sink>
__device__ __forceinline__ void fused_reduce_slice(const TAcc* part_site, int64_t part_stride, int C, int r, int h, int c0,
                                                   int W, Sink&& sink) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int j = warp; j < r; j += kThreads / 32) {
    for (int cc = lane; cc < W; cc += 32) {
      const int c = c0 + cc;
      TAcc v = TAcc(0);
      if (c < h) {
        TAcc t[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) t[q] = (q < C) ? DAD_LDCG(part_site + q * part_stride + (int64_t)j * h + c) : TAcc(0);
        v = t[0];
#pragma unroll
        for (int q = 1; q < 8; ++q) v += t[q];
      }
      sink(j, cc, c, v);
    }
  }
}

}  // namespace

template <typename TIn, typename TAcc, int BS>
__global__ void __launch_bounds__(kThreads)
fused_site_kernel(const FusedParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  cg::cluster_group cluster = cg::this_cluster();
  const int C = p.C, r = p.r, h_in = p.h_in, h_out = p.h_out;
  const OrthGeom g = orth_geom<BS>(r, h_out, C, sizeof(TAcc));
  TAcc* slab = reinterpret_cast<TAcc*>(smem_raw);
  TAcc* Ybuf = reinterpret_cast<TAcc*>(smem_raw + (g.total + 15) / 16 * 16);
  __shared__ OrthShared orth_sh;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int s = blockIdx.y;
  const int rank = (int)cluster.block_rank();
  const int rpad = (r + kVecBlock - 1) / kVecBlock * kVecBlock;
  const int hmax = h_in > h_out ? h_in : h_out;
  // rows of this CTA
  const int Nc = (p.N + C - 1) / C;
  const int n0 = rank * Nc;
  const int nrows = n0 >= p.N ? 0 : (n0 + Nc <= p.N ? Nc : p.N - n0);
  const TIn* As = reinterpret_cast<const TIn*>(p.A) + (int64_t)s * p.strideA + (int64_t)n0 * p.ldA;
  const TIn* Ds = reinterpret_cast<const TIn*>(p.D) + (int64_t)s * p.strideD + (int64_t)n0 * p.ldD;
  TAcc* FG = reinterpret_cast<TAcc*>(p.FG) + (int64_t)s * r * h_out;
  TAcc* FZ = reinterpret_cast<TAcc*>(p.FZ) + (int64_t)s * r * h_in;
  TAcc* part_site = reinterpret_cast<TAcc*>(p.part) + (int64_t)s * C * r * hmax;
  // slices of the columns this CTA completes: of h_out (the slab of the Cholesky-QR) and of h_in
  const int Wg = g.W, Wp = g.Wp, cg0 = rank * Wg;
  const int Wz = ((h_in + C - 1) / C + 3) / 4 * 4, cz0 = rank * Wz;
  const float* Q0s = p.Q0 + (int64_t)s * r * h_out;
  float* Qs = p.Q + (int64_t)s * r * h_out;
  float* Ps = p.P + (int64_t)s * r * h_in;

  // G <- Q0 (this CTA's slice); with no iteration Q is the start block as it came
  for (int j = warp; j < r; j += kThreads / 32)
    for (int cc = lane; cc < Wg; cc += 32) {
      const int c = cg0 + cc;
      if (c < h_out) {
        const float q0 = DAD_LD(&Q0s[(int64_t)j * h_out + c]);
        DAD_ST(&FG[(int64_t)j * h_out + c], TAcc(q0));
        if (p.iters == 0 && p.Q != p.Q0) DAD_ST(&Qs[(int64_t)j * h_out + c], q0);
      }
    }
  cluster_barrier(cluster);

  auto cols_acc = [&](const TIn* X, int64_t ld, int h, TAcc* out) {
    if (h >= 4 * kThreads)
      fused_cols_acc<TIn, TAcc, 4>(X, ld, nrows, h, Ybuf, r, rpad, out);
    else
      fused_cols_acc<TIn, TAcc, 1>(X, ld, nrows, h, Ybuf, r, rpad, out);
  };
  TAcc* my_part = part_site + (int64_t)rank * r * hmax;  // partial of a product over h columns: [r][h], compact

  for (int k = 0; k < p.iters; ++k) {
    fused_rows_dot<TIn, TAcc>(Ds, p.ldD, nrows, h_out, FG, r, rpad, Ybuf);  // Y = D G^T
    __syncthreads();
    cols_acc(As, p.ldA, h_in, my_part);                                      // partial of Z = Y^T A
    cluster_barrier(cluster);
    fused_reduce_slice<TAcc>(part_site, (int64_t)r * hmax, C, r, h_in, cz0, Wz, [&](int j, int, int c, TAcc v) {
      if (c < h_in) DAD_ST(&FZ[(int64_t)j * h_in + c], v);
    });
    cluster_barrier(cluster);
    fused_rows_dot<TIn, TAcc>(As, p.ldA, nrows, h_in, FZ, r, rpad, Ybuf);   // W = A Z^T
    __syncthreads();
    cols_acc(Ds, p.ldD, h_out, my_part);                                     // partial of G~ = W^T D
    cluster_barrier(cluster);
    fused_reduce_slice<TAcc>(part_site, (int64_t)r * hmax, C, r, h_out, cg0, Wg, [&](int j, int cc, int, TAcc v) { slab[j * Wp + cc] = v; });
    for (int idx = tid; idx < (g.rp - r) * Wg; idx += kThreads) slab[(r + idx / Wg) * Wp + idx % Wg] = TAcc(0);
    // (orth_slab_passes starts with a CTA barrier)
    orth_slab_passes<BS, TAcc>(slab, smem_raw, g, C, p.tol, p.status, &orth_sh);
    const bool last = k == p.iters - 1;
    for (int j = warp; j < r; j += kThreads / 32)
      for (int cc = lane; cc < Wg; cc += 32) {
        const int c = cg0 + cc;
        if (c < h_out) {
          const TAcc v = slab[j * Wp + cc];
          DAD_ST(&FG[(int64_t)j * h_out + c], v);
          if (last) DAD_ST(&Qs[(int64_t)j * h_out + c], (float)v);
        }
      }
    cluster_barrier(cluster);
  }

  // P = (A^T (D G^T))^T and the lengths of its rows
  fused_rows_dot<TIn, TAcc>(Ds, p.ldD, nrows, h_out, FG, r, rpad, Ybuf);
  __syncthreads();
  cols_acc(As, p.ldA, h_in, my_part);
  cluster_barrier(cluster);
  {
    double sq = 0.0;  // this lane's share of ||P_j slice||^2; a warp owns whole vectors j
    int cur_j = -1;
    auto flush = [&](int j) {
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
      if (lane == 0 && p.sig_part) DAD_ST(&p.sig_part[((int64_t)s * C + rank) * r + j], sq);
      sq = 0.0;
    };
    for (int j = warp; j < r; j += kThreads / 32) {
      for (int cc = lane; cc < Wz; cc += 32) {
        const int c = cz0 + cc;
        double v = 0.0;
        if (c < h_in) {
          TAcc t[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) t[q] = (q < C) ? DAD_LDCG(part_site + (int64_t)q * r * hmax + (int64_t)j * h_in + c) : TAcc(0);
          TAcc a = t[0];
#pragma unroll
          for (int q = 1; q < 8; ++q) a += t[q];
          DAD_ST(&Ps[(int64_t)j * h_in + c], (float)a);
          v = (double)a;
        }
        sq += v * v;
      }
      cur_j = j;
      flush(cur_j);
    }
  }
  if (p.sigma) {
    cluster_barrier(cluster);
    if (rank == 0 && tid < r) {
      double t = 0.0;
      for (int q = 0; q < C; ++q) t += DAD_LDCG(p.sig_part + ((int64_t)s * C + q) * r + tid);
      DAD_ST(&p.sigma[(int64_t)s * r + tid], (float)sqrt(t));
    }
  }
}

// ---- host side ---------------------------------------------------------------------------------------------------
namespace {

template <int BS>
size_t fused_smem_bytes(int64_t N, int64_t h_out, int r, int C, size_t acc) {
  const int64_t Nc = (N + C - 1) / C;
  const int rpad = (r + kVecBlock - 1) / kVecBlock * kVecBlock;
  return (orth_geom<BS>(r, h_out, C, acc).total + 15) / 16 * 16 + (size_t)Nc * rpad * acc;
}

size_t fused_smem_for(int64_t N, int64_t h_out, int r, int C, size_t acc) {
  return r >= 32 ? fused_smem_bytes<8>(N, h_out, r, C, acc) : fused_smem_bytes<2>(N, h_out, r, C, acc);
}

template <typename TIn, typename TAcc, int BS>
cudaError_t launch_fused(const FusedParams& p, int S, size_t smem, cudaStream_t st) {
  auto kernel = fused_site_kernel<TIn, TAcc, BS>;
  static FirstUse first;  // the opt-in to large dynamic shared memory is per function and device, not per launch
  if (first.on_this_device()) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) {
      first.forget();
      return e;
    }
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)p.C, (unsigned)S, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)p.C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const bool timed = g_timing.load(std::memory_order_relaxed);
  if (timed) timing_mark("fused_site", st, true);
  cudaError_t err = cudaLaunchKernelEx(&cfg, kernel, p);
  if (timed) timing_mark("fused_site", st, false);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return err;
}

}  // namespace

// CTAs per site of the one-launch compress, or 0 when the shape is left to the multi-launch pipelines.
//
// Measured on B200 (fp32 inputs, fp64 accumulation): a pass of the one-launch kernel over A or D costs about 8 us
// of barriers, exchanges and dependent memory round trips however small the site, plus about 40 ns per thousand
// multiply-adds of a CTA's share (20 ns with fp32 accumulation); a pass of the multi-launch pipelines costs about
// 24 us of launches (general kernels) or 15 us (tensor-core kernels) while the GPU is not yet full.  A GPU holds
// about 15 clusters of 8 CTAs at a time (two per GPC), 32 of 4, 70 of 2; more sites than that run in waves.  The
// cluster size with the smallest estimate is taken, if it beats the multi-launch estimate.
int fused_cluster_size(const dad_layer& L, int r, int iters) {
  if (L.N > (1 << 20) || L.h_in > (1 << 20) || L.h_out > (1 << 20)) return 0;
  const size_t acc = L.dtype == DAD_F32 ? 8 : 4;
  const double ns_per_kfma = L.dtype == DAD_F32 ? 40.0 : 20.0;
  const double multi_us = tc_eligible(L) ? 15.0 : 24.0;
  const double fma_per_pass = (double)L.N * r * (double)(L.h_in + L.h_out);
  int best = 0;
  double best_us = multi_us;  // per pass
  for (int C = 8; C >= 1; C /= 2) {
    if (C > 1 && L.N < 4 * C) continue;  // at least 4 rows per CTA
    if (fused_smem_for(L.N, L.h_out, r, C, acc) > 200 * 1024 && !fused_dsm_fits(L, r, C, nullptr)) continue;
    const int at_once = C == 8 ? 15 : C == 4 ? 32 : C == 2 ? 70 : 148;
    const double waves = (double)((L.S + at_once - 1) / at_once);
    const double us = waves * (8.0 + ns_per_kfma * 1e-6 * fma_per_pass / C);
    if (us < best_us) {
      best_us = us;
      best = C;
    }
  }
  return best;
}

cudaError_t fused_compress(const dad_layer& L, const void* A, const void* D, int r, int iters, const float* Q0, float* P,
                           float* Q, float* sigma, void* FG, void* FZ, void* part, double* sig_part, int* status, int C,
                           cudaStream_t st) {
  FusedParams p{};
  p.A = A;
  p.D = D;
  p.ldA = L.ldA;
  p.ldD = L.ldD;
  p.strideA = L.strideA;
  p.strideD = L.strideD;
  p.N = (int)L.N;
  p.h_in = (int)L.h_in;
  p.h_out = (int)L.h_out;
  p.r = r;
  p.iters = iters;
  p.C = C;
  p.Q0 = Q0;
  p.P = P;
  p.Q = Q;
  p.sigma = sigma;
  p.FG = FG;
  p.FZ = FZ;
  p.part = part;
  p.sig_part = sig_part;
  p.status = status;
  const bool f32in = L.dtype == DAD_F32;
  p.tol = f32in ? 1e-12 : 1e-6;
  const size_t smem = fused_smem_for(L.N, L.h_out, r, C, f32in ? 8 : 4);
  if (f32in) {
    if (r >= 32) return launch_fused<float, double, 8>(p, L.S, smem, st);
    return launch_fused<float, double, 2>(p, L.S, smem, st);
  }
  if (r >= 32) return launch_fused<__nv_bfloat16, float, 8>(p, L.S, smem, st);
  return launch_fused<__nv_bfloat16, float, 2>(p, L.S, smem, st);
}

}  // namespace dad

// Orthonormalisation of the r iterate vectors of a site in ONE launch (vectors stored as fp32, or as fp64 in
// the pipeline of fp32 inputs):
// a thread-block cluster of C CTAs per site, each holding a slab of r x W columns in shared
// memory for the whole Cholesky-QR (both passes), so the vectors are read from and written to
// global memory exactly once.
//
//   pass:  partial Gram of the slab (fp64, BS x BS register blocks)  ->  sum of the C partials
//          over distributed shared memory, in rank order, by every CTA (all CTAs get the identical
//          r x r matrix)  ->  Cholesky in shared memory (same pivot floor and zeroing rule as
//          orth.cu)  ->  forward substitution down each column of the slab, in place, four rows
//          at a time.
//   A second pass runs when the first shows R_jj < 1e-5 ||g_j|| for some vector (one fp64 pass leaves
//   an orthogonality defect of about 1e-16 cond^2 <= 1e-6, the level of the fp32 storage itself); the
//   decision is identical in all CTAs of the cluster because they factor the same matrix.
//
// The substitution reads the already-solved vectors back in fp32; that perturbs the right-hand
// side by one fp32 rounding, the same size as the rounding of the stored input itself.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace dad {

namespace {
constexpr double kPivotFloor = 1e-14;          // (1e-7)^2 of the squared length
// Ratio of squared lengths R_jj^2 / ||g_j||^2 below which a second pass is asked for: (1e-5)^2 for fp32 storage (one
// fp64 pass leaves a defect of 1e-16 cond^2 <= 1e-6, the level of the storage), (1e-3)^2 for fp64 storage (<= 1e-10).
template <typename T>
constexpr double second_pass_below_sq() { return sizeof(T) == 4 ? 1e-10 : 1e-6; }
template <typename T> struct Vec2;
template <> struct Vec2<float> { using type = float2; };
template <> struct Vec2<double> { using type = double2; };
constexpr int kThreads = 256;

struct OrthGeom {
  int rp;       // r rounded up to the register block (a multiple of 4)
  int W;        // columns per CTA (multiple of 4)
  int Wp;       // padded row length of the slab in floats
  int nblocks;  // lower-triangular register blocks of the Gram matrix
  int cgs;      // column groups the slab is split into for the Gram phase
  size_t off_gram, off_L, off_vec, total;  // byte offsets after the slab (of elements of `esize` bytes)
};

template <int BS>
__host__ __device__ inline OrthGeom orth_geom(int r, int64_t h, int C, size_t esize) {
  OrthGeom g;
  constexpr int RB = BS < 4 ? 4 : BS;
  g.rp = (r + RB - 1) / RB * RB;
  int W = (int)((h + C - 1) / C);
  g.W = (W + 3) / 4 * 4;
  g.Wp = g.W + 2;  // even (two-element vector accesses), and rows 8 apart do not share a bank
  const int nb = g.rp / BS;
  g.nblocks = nb * (nb + 1) / 2;
  g.cgs = kThreads / g.nblocks;
  if (g.cgs < 1) g.cgs = 1;
  if (g.cgs > 8) g.cgs = 8;
  size_t off = esize * (size_t)g.rp * g.Wp;
  off = (off + 15) / 16 * 16;
  g.off_gram = off;  // this CTA's partial Gram, rp x rp doubles (read by the other CTAs of the cluster)
  off += sizeof(double) * (size_t)g.rp * g.rp;
  g.off_L = off;  // rp x (rp + 1) doubles
  off += sizeof(double) * (size_t)g.rp * (g.rp + 1);
  g.off_vec = off;  // 4 x rp doubles: squared lengths, first-pass pivots, inverse diagonal, first-pass lengths
  off += sizeof(double) * 4 * (size_t)g.rp;
  g.total = off;
  return g;
}

template <int BS>
inline bool slab_fits(int r, int64_t h, int C, size_t esize) { return orth_geom<BS>(r, h, C, esize).total <= 200 * 1024; }

// CTAs per site.  Every CTA of a cluster repeats the r x r factorisation, so the cluster is kept as small as
// still fills the GPU with S sites (and as the slab of h / C columns allows); with few sites it grows to 8.
inline int cluster_size_for(int r, int64_t h, int S, size_t esize) {
  int best = 0;
  for (int C = 1; C <= 8; C *= 2) {
    if (C > 1 && h / C < 128) break;
    const bool fits = r >= 32 ? slab_fits<8>(r, h, C, esize) : slab_fits<2>(r, h, C, esize);
    if (!fits) continue;
    best = C;
    if ((int64_t)S * C >= 2 * 148) break;
  }
  return best;  // 0: no cluster size fits
}
}  // namespace

template <int BS, typename T>
__global__ void __launch_bounds__(kThreads)
orth_cluster_kernel(T* __restrict__ G, int r, int64_t h, int C, double tol, int* __restrict__ status,
                    float* __restrict__ out32, __nv_bfloat16* __restrict__ planes, int plane_rows) {
  using T2 = typename Vec2<T>::type;
  constexpr bool kF32 = sizeof(T) == 4;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  cg::cluster_group cluster = cg::this_cluster();
  const OrthGeom g = orth_geom<BS>(r, h, C, sizeof(T));
  T* slab = reinterpret_cast<T*>(smem_raw);
  double* gram = reinterpret_cast<double*>(smem_raw + g.off_gram);
  double* Lm = reinterpret_cast<double*>(smem_raw + g.off_L);
  double* diag0 = reinterpret_cast<double*>(smem_raw + g.off_vec);
  double* piv1 = diag0 + g.rp;   // first-pass pivots (squared R_jj)
  double* inv_l = piv1 + g.rp;
  double* orig1 = inv_l + g.rp;  // squared lengths before the first pass
  __shared__ int need2_s;
  __shared__ unsigned char dead_row[DAD_MAX_RANK];

  const int tid = threadIdx.x;
  const int s = blockIdx.y;
  const int rank = (int)cluster.block_rank();
  const int rp = g.rp, W = g.W, Wp = g.Wp, LR = rp + 1;
  const int64_t c0 = (int64_t)rank * W;
  T* Gs = G + (int64_t)s * r * h;
  const double tol2 = tol * tol;

  // the next kernel in the stream may begin its set-up now; it waits for this grid before touching memory
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // ---- load the slab (rows >= r and columns >= h are zero) ----
  // Loads are issued eight at a time per thread before any is stored, so that their latencies overlap.
  if (kF32 && (h & 3) == 0) {
    const float* Gf = reinterpret_cast<const float*>(Gs);
    float* slabf = reinterpret_cast<float*>(slab);
    const int W4 = W / 4, total = rp * W4;
    for (int base = 0; base < total; base += kThreads * 8) {
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int idx = base + u * kThreads + tid;
        const int j = idx / W4, c = (idx % W4) * 4;
        v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (idx < total && j < r && c0 + c < h) v[u] = *reinterpret_cast<const float4*>(Gf + (int64_t)j * h + c0 + c);
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int idx = base + u * kThreads + tid;
        if (idx < total) {
          float* dst = slabf + (idx / W4) * Wp + (idx % W4) * 4;  // 8-byte aligned (Wp is even)
          *reinterpret_cast<float2*>(dst) = make_float2(v[u].x, v[u].y);
          *reinterpret_cast<float2*>(dst + 2) = make_float2(v[u].z, v[u].w);
        }
      }
    }
  } else {
    const int total = rp * W;
    for (int base = 0; base < total; base += kThreads * 8) {
      T v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int idx = base + u * kThreads + tid;
        const int j = idx / W, c = idx % W;
        v[u] = (idx < total && j < r && c0 + c < h) ? Gs[(int64_t)j * h + c0 + c] : T(0);
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int idx = base + u * kThreads + tid;
        if (idx < total) slab[(idx / W) * Wp + idx % W] = v[u];
      }
    }
  }
  if (tid < DAD_MAX_RANK) dead_row[tid] = 0;
  __syncthreads();

  for (int pass = 0; pass < 2; ++pass) {
    // ---- partial Gram of the slab: BS x BS register blocks of the lower triangle, fp64.  The slab is cut
    //      into column groups; the groups add their blocks into `gram` one after the other (fixed order). ----
    {
      const int Wc = ((W + g.cgs - 1) / g.cgs + 3) / 4 * 4;
      const int item = tid;
      const bool active = item < g.nblocks * g.cgs;  // nblocks * cgs <= kThreads by construction, or cgs == 1
      const int rounds = (g.nblocks + kThreads - 1) / kThreads;  // > 1 only when cgs == 1
      for (int round = 0; round < rounds; ++round) {
        const int b = (g.cgs > 1) ? item % g.nblocks : item + round * kThreads;
        const int grp = (g.cgs > 1) ? item / g.nblocks : 0;
        const bool mine = (g.cgs > 1) ? active : b < g.nblocks;
        int bi = 0, bj = 0;
        double acc[BS][BS];
#pragma unroll
        for (int u = 0; u < BS; ++u)
#pragma unroll
          for (int v = 0; v < BS; ++v) acc[u][v] = 0.0;
        if (mine) {
          while ((bi + 1) * (bi + 2) / 2 <= b) ++bi;  // block row: bi(bi+1)/2 <= b
          bj = b - bi * (bi + 1) / 2;
          const int cbeg = grp * Wc, cend = (cbeg + Wc < W) ? cbeg + Wc : W;
          const T* ra = slab + (bi * BS) * Wp;
          const T* rb = slab + (bj * BS) * Wp;
          for (int c = cbeg; c < cend; ++c) {
            double a[BS], bb[BS];
#pragma unroll
            for (int u = 0; u < BS; ++u) a[u] = (double)ra[u * Wp + c];
#pragma unroll
            for (int v = 0; v < BS; ++v) bb[v] = (double)rb[v * Wp + c];
#pragma unroll
            for (int u = 0; u < BS; ++u)
#pragma unroll
              for (int v = 0; v < BS; ++v) acc[u][v] += a[u] * bb[v];
          }
        }
        for (int turn = 0; turn < g.cgs; ++turn) {
          if (mine && grp == turn) {
#pragma unroll
            for (int u = 0; u < BS; ++u)
#pragma unroll
              for (int v = 0; v < BS; ++v) {
                double* dst = gram + (bi * BS + u) * rp + bj * BS + v;
                *dst = (turn == 0) ? acc[u][v] : *dst + acc[u][v];
              }
          }
          __syncthreads();
        }
      }
    }
    // ---- sum the partials of all CTAs of the cluster, in rank order ----
    cluster.sync();
    for (int e = tid; e < rp * rp; e += kThreads) {
      const int i = e / rp, j = e % rp;
      if (j <= i) {
        double t[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) t[q] = (q < C) ? cluster.map_shared_rank(gram, q)[e] : 0.0;
        double v = t[0];
#pragma unroll
        for (int q = 1; q < 8; ++q) v += t[q];
        Lm[i * LR + j] = v;
      }
    }
    cluster.sync();  // nobody rewrites its partial while a neighbour still reads it
    if (tid < rp) diag0[tid] = Lm[tid * LR + tid];
    if (tid == 0) need2_s = 0;
    __syncthreads();

    // ---- Cholesky, left-looking, one barrier per column: thread i owns row i; for column j it forms
    //      c_ij = G_ij - sum_{l<j} L_il L_jl, and (redundantly, so that no second barrier is needed) the
    //      pivot of row j, on which every thread takes the same decisions ----
    for (int j = 0; j < rp; ++j) {
      const int i = tid;
      if (i >= j && i < rp) {
        // the diagonal is read from its saved copy: thread j overwrites Lm[j][j] in this very step
        // four partial sums per dot product: the fp64 dependency chain is a quarter as long
        double dd[4] = {0.0, 0.0, 0.0, 0.0}, cc[4] = {0.0, 0.0, 0.0, 0.0};
        int l = 0;
        for (; l + 4 <= j; l += 4) {
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const double a = Lm[j * LR + l + u];
            dd[u] += a * a;
            cc[u] += Lm[i * LR + l + u] * a;
          }
        }
        for (; l < j; ++l) {
          const double a = Lm[j * LR + l];
          dd[0] += a * a;
          cc[0] += Lm[i * LR + l] * a;
        }
        const double d = diag0[j] - ((dd[0] + dd[1]) + (dd[2] + dd[3]));
        const double c = Lm[i * LR + j] - ((cc[0] + cc[1]) + (cc[2] + cc[3]));
        const double orig = diag0[j];
        double piv = d;
        int is_dead = 0, bad = 0;
        if (!(orig == orig) || orig > 1.7e308) {
          bad = 1;
          is_dead = 1;
        } else if (!(orig > 0.0)) {
          is_dead = 1;
        } else {
          const double floor_ = kPivotFloor * orig;
          if (!(piv > floor_)) piv = floor_;
          // second pass: total remainder (R1_jj R2_jj)^2 against tol^2 of the squared length before pass one
          if (pass == 1 && !(piv1[j] * piv > tol2 * orig1[j])) is_dead = 1;
        }
        if (is_dead) piv = 1.0;
        const double il = rsqrt(piv);  // one reciprocal square root instead of a square root and divisions
        if (i == j) {
          if (bad && status) *status = (int)DAD_ERR_NUMERIC;
          if (pass == 0) {
            piv1[j] = is_dead ? 0.0 : piv;
            orig1[j] = orig;
            if (!is_dead && piv < second_pass_below_sq<T>() * orig) need2_s = 1;
          }
          if (is_dead) dead_row[j] = 1;
          Lm[j * LR + j] = piv * il;
          inv_l[j] = il;
        } else {
          Lm[i * LR + j] = is_dead ? 0.0 : c * il;
        }
      }
      __syncthreads();
    }

    // ---- forward substitution down each column of the slab, in place: two adjacent columns per thread,
    //      four rows at a time so that every solved value is read (and widened) once per row block ----
    for (int c = 2 * tid; c < W; c += 2 * kThreads) {
      for (int j0 = 0; j0 < rp; j0 += 4) {
        double v[4][2];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const T2 x = *reinterpret_cast<const T2*>(slab + (j0 + u) * Wp + c);
          v[u][0] = (double)x.x;
          v[u][1] = (double)x.y;
        }
        for (int l = 0; l < j0; ++l) {
          const T2 q = *reinterpret_cast<const T2*>(slab + l * Wp + c);
          const double q0 = (double)q.x, q1 = (double)q.y;
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const double a = Lm[(j0 + u) * LR + l];
            v[u][0] -= a * q0;
            v[u][1] -= a * q1;
          }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int j = j0 + u;
          const double il = dead_row[j] ? 0.0 : inv_l[j];
          // the value stored (and used by the rows below) is the one rounded to the storage type
          const T o0 = (T)(v[u][0] * il), o1 = (T)(v[u][1] * il);
          T2 o;
          o.x = o0;
          o.y = o1;
          *reinterpret_cast<T2*>(slab + j * Wp + c) = o;
#pragma unroll
          for (int w = u + 1; w < 4; ++w) {
            const double a = Lm[(j0 + w) * LR + j];
            v[w][0] -= a * (double)o0;
            v[w][1] -= a * (double)o1;
          }
        }
      }
    }
    __syncthreads();
    if (need2_s == 0) break;  // same matrix, same decision in every CTA of the cluster
  }

  // ---- write the orthonormal vectors (and their bf16 hi/lo planes) ----
  if (kF32 && (h & 3) == 0) {
    float* Gf = reinterpret_cast<float*>(Gs);
    const float* slabf = reinterpret_cast<const float*>(slab);
    const int W4 = W / 4;
    for (int idx = tid; idx < r * W4; idx += kThreads) {
      const int j = idx / W4, c = (idx % W4) * 4;
      const int64_t col = c0 + c;
      if (col < h) {
        const float2 lo2 = *reinterpret_cast<const float2*>(slabf + j * Wp + c);
        const float2 hi2 = *reinterpret_cast<const float2*>(slabf + j * Wp + c + 2);
        const float f[4] = {lo2.x, lo2.y, hi2.x, hi2.y};
        *reinterpret_cast<float4*>(Gf + (int64_t)j * h + col) = make_float4(f[0], f[1], f[2], f[3]);
        if (out32) *reinterpret_cast<float4*>(out32 + ((int64_t)s * r + j) * h + col) = make_float4(f[0], f[1], f[2], f[3]);
        if (planes) {
          __nv_bfloat16 hi[4], lo[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            hi[u] = __float2bfloat16_rn(f[u]);
            lo[u] = __float2bfloat16_rn(f[u] - __bfloat162float(hi[u]));
          }
          __nv_bfloat16* ph = planes + (((int64_t)s * 2 + 0) * plane_rows + j) * h + col;  // 8-byte aligned
          __nv_bfloat16* pl = planes + (((int64_t)s * 2 + 1) * plane_rows + j) * h + col;
          *reinterpret_cast<uint2*>(ph) = *reinterpret_cast<const uint2*>(hi);
          *reinterpret_cast<uint2*>(pl) = *reinterpret_cast<const uint2*>(lo);
        }
      }
    }
  } else {
    for (int idx = tid; idx < r * W; idx += kThreads) {
      const int j = idx / W, c = idx % W;
      if (c0 + c < h) {
        const T g_out = slab[j * Wp + c];
        const float f = (float)g_out;
        const int64_t col = c0 + c;
        Gs[(int64_t)j * h + col] = g_out;
        if (out32) out32[((int64_t)s * r + j) * h + col] = f;
        if (planes) {
          const __nv_bfloat16 hi = __float2bfloat16_rn(f);
          planes[(((int64_t)s * 2 + 0) * plane_rows + j) * h + col] = hi;
          planes[(((int64_t)s * 2 + 1) * plane_rows + j) * h + col] = __float2bfloat16_rn(f - __bfloat162float(hi));
        }
      }
    }
  }
}

template <int BS, typename T>
static cudaError_t launch_orth_cluster(T* G, int S, int r, int64_t h, int C, double tol, int* status, float* out32,
                                       __nv_bfloat16* planes, int plane_rows, size_t smem, cudaStream_t st) {
  auto kernel = orth_cluster_kernel<BS, T>;
  cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return err;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)C, (unsigned)S, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const bool timed = g_timing.load(std::memory_order_relaxed);
  if (timed) timing_mark("orth_cluster", st, true);
  err = cudaLaunchKernelEx(&cfg, kernel, G, r, h, C, tol, status, out32, planes, plane_rows);
  if (timed) timing_mark("orth_cluster", st, false);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return err;
}

// Whether the one-launch kernel takes this shape (the slab of a CTA has to fit in shared memory).
bool orth_cluster_fits(int r, int64_t h, size_t elem_bytes) {
  if (h > (int64_t)1 << 30) return false;
  return cluster_size_for(r, h, 1 << 20, elem_bytes) > 0;  // the largest admissible cluster decides
}

// Cholesky-QR (one or two passes, decided on the device) of the rows of G (S x r x h, in place).
template <typename T>
cudaError_t orth_cluster(T* G, int S, int r, int64_t h, double tol, int* status, float* out32, __nv_bfloat16* planes,
                         int plane_rows, cudaStream_t st) {
  const int C = cluster_size_for(r, h, S, sizeof(T));
  if (C == 0) return cudaErrorInvalidValue;
  if (r >= 32)
    return launch_orth_cluster<8, T>(G, S, r, h, C, tol, status, out32, planes, plane_rows,
                                     orth_geom<8>(r, h, C, sizeof(T)).total, st);
  return launch_orth_cluster<2, T>(G, S, r, h, C, tol, status, out32, planes, plane_rows,
                                   orth_geom<2>(r, h, C, sizeof(T)).total, st);
}
template cudaError_t orth_cluster<float>(float*, int, int, int64_t, double, int*, float*, __nv_bfloat16*, int, cudaStream_t);
template cudaError_t orth_cluster<double>(double*, int, int, int64_t, double, int*, float*, __nv_bfloat16*, int, cudaStream_t);

}  // namespace dad

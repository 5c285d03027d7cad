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
#include "orth_slab.cuh"

namespace dad {
using namespace orthslab;

namespace {
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
  __shared__ OrthShared orth_sh;

  const int tid = threadIdx.x;
  const int s = blockIdx.y;
  const int rank = (int)cluster.block_rank();
  const int rp = g.rp, W = g.W, Wp = g.Wp;
  const int64_t c0 = (int64_t)rank * W;
  T* Gs = G + (int64_t)s * r * h;


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
  orth_slab_passes<BS, T>(slab, smem_raw, g, C, tol, status, &orth_sh);


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

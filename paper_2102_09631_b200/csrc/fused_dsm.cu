// One-launch compress, on-chip form: as fused_site.cu a thread-block cluster owns a site for the whole structured
// power iteration (Algorithm 2; Eq. "reduced_iter", Eq. "peel" as block deflation), but here everything the CTAs
// exchange travels over distributed shared memory and nothing but the inputs is read from global memory:
//
//   row-wise products     Y = D G^T, W = A Z^T : CTA q owns rows [q Nc, (q+1) Nc) of the site.  Its rows of A and D
//                         sit in its shared memory for the whole kernel (when they fit), the factor (G or Z) too.
//                         Each finished row of Y / W is stored into the Y buffer of EVERY CTA of the cluster.
//   column-wise products  Z = Y^T A, G~ = W^T D : CTA q owns a slice of the columns and sums over ALL rows of the
//                         site (Y complete in shared memory, the column slab of A / D streamed from L2), so its
//                         slice is complete: no partial sums cross CTAs.  The slice of Z is stored into the factor
//                         buffer of every CTA; the slice of G~ stays at home as the slab of the Cholesky-QR
//                         (orth_slab.cuh), after which the orthonormal slice goes to every factor buffer.
//
// Every output element is summed by one thread (or a fixed tree of threads) in a fixed order: two runs agree bit
// for bit.  The only synchronisation is the hardware cluster barrier, whose release/acquire orders the remote
// shared-memory stores; no wait is a spin.  fp32 inputs accumulate in fp64 and keep fp64 intermediates, bf16
// inputs in fp32.
#include "bounds.cuh"
#include "orth_slab.cuh"
#include "warp_reduce.cuh"

namespace dad {
using namespace orthslab;

struct DsmParams {
  const void* A;
  const void* D;
  int64_t ldA, ldD, strideA, strideD;
  int N, h_in, h_out, r, iters, C;
  int x_resident;  // this CTA's rows of A and D are copied to shared memory once
  const float* Q0;
  float* P;
  float* Q;
  float* sigma;
  int* status;
  double tol;
};

namespace {

constexpr int kRowGroup = 4;  // rows a warp advances together in the row-wise products
constexpr int kVecBlock = 8;  // vectors (rows of the factor) per register block
constexpr int kMaxColSplit = 4;  // warps that may share the columns of one row group in the row-wise products

// Shared-memory carve of a CTA (bytes), identical on host and device.
struct DsmGeom {
  OrthGeom og;
  int rpad, hF, Nc, Wz;
  size_t off_F, off_Y, off_red, off_sig, off_stage, off_X, total;
};

template <int BS>
__host__ __device__ inline DsmGeom dsm_geom(int N, int h_in, int h_out, int r, int C, size_t acc, size_t in_bytes,
                                            bool x_resident) {
  DsmGeom d;
  d.og = orth_geom<BS>(r, h_out, C, acc);
  d.rpad = (r + kVecBlock - 1) / kVecBlock * kVecBlock;
  d.hF = ((h_in > h_out ? h_in : h_out) + 3) / 4 * 4;  // row length of the factor buffer (16-byte rows)
  d.Nc = (N + C - 1) / C;
  d.Wz = ((h_in + C - 1) / C + 3) / 4 * 4;
  size_t off = (d.og.total + 15) / 16 * 16;
  d.off_F = off;  // rpad x hF accumulator type: the factor of the row-wise products (G, then Z), complete
  off += acc * (size_t)d.rpad * d.hF;
  d.off_Y = off;  // (C * Nc) x rpad: Y (then W), complete
  off += acc * (size_t)C * d.Nc * d.rpad;
  // scratch of the column-wise products (kThreads x kVecBlock: the row groups' sums) and, at other times, of the
  // row-wise products (kMaxColSplit x Nc x rpad: the column shares' sums)
  d.off_red = off;
  {
    const size_t a = (size_t)kThreads * kVecBlock, b = (size_t)kMaxColSplit * d.Nc * d.rpad;
    off += acc * (a > b ? a : b);
  }
  d.off_sig = off;  // C x rpad doubles: squared lengths of the slices of P (used on rank 0)
  off += sizeof(double) * (size_t)C * d.rpad;
  d.off_stage = d.off_red;
  off = (off + 15) / 16 * 16;
  d.off_X = off;  // Nc x h_in, then Nc x h_out, input type
  if (x_resident) off += in_bytes * (size_t)d.Nc * ((size_t)h_in + h_out);
  d.total = off;
  return d;
}

// The building blocks below are deliberately NOT inlined and exist once per kernel: the kernel runs each of them for
// a few microseconds at a time, and a body that is unrolled and duplicated at every call site spends longer
// fetching instructions than executing them.

// Two adjacent input elements (a row of the site starts on an even element; widths are even), widened.
template <typename TAcc>
__device__ __forceinline__ void load_pair(const float* p, TAcc& a, TAcc& b) {
  if (!DAD_RANGE_OK(p, 8)) {
    a = b = TAcc(0);
    return;
  }
  const float2 t = *reinterpret_cast<const float2*>(p);
  a = TAcc(t.x);
  b = TAcc(t.y);
}
template <typename TAcc>
__device__ __forceinline__ void load_pair(const __nv_bfloat16* p, TAcc& a, TAcc& b) {
  if (!DAD_RANGE_OK(p, 4)) {
    a = b = TAcc(0);
    return;
  }
  const float2 t = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(p));
  a = TAcc(t.x);
  b = TAcc(t.y);
}
__device__ __forceinline__ void load_pair(const double* p, double& a, double& b) {
  const double2 t = *reinterpret_cast<const double2*>(p);
  a = t.x;
  b = t.y;
}

template <typename T> struct PairOf;
template <> struct PairOf<float> { using type = float2; };
template <> struct PairOf<__nv_bfloat16> { using type = __nv_bfloat162; };
template <typename TAcc>
__device__ __forceinline__ void widen_pair(float2 t, TAcc& a, TAcc& b) {
  a = TAcc(t.x);
  b = TAcc(t.y);
}
template <typename TAcc>
__device__ __forceinline__ void widen_pair(__nv_bfloat162 v, TAcc& a, TAcc& b) {
  const float2 t = __bfloat1622float2(v);
  a = TAcc(t.x);
  b = TAcc(t.y);
}
// A pair of inputs requested NOW: the volatile asm keeps the compiler from sinking the load to its use, which would
// turn a batch of requests into as many dependent round trips to L2.
__device__ __forceinline__ float2 request_pair(const float* p) {
  float2 v;
  if (!DAD_RANGE_OK(p, 8)) return make_float2(0.f, 0.f);
  asm volatile("ld.global.nc.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "l"(p));
  return v;
}
__device__ __forceinline__ __nv_bfloat162 request_pair(const __nv_bfloat16* p) {
  uint32_t w = 0;
  if (!DAD_RANGE_OK(p, 4)) return *reinterpret_cast<__nv_bfloat162*>(&w);
  asm volatile("ld.global.nc.b32 %0, [%1];" : "=r"(w) : "l"(p));
  return *reinterpret_cast<__nv_bfloat162*>(&w);
}
constexpr int kRowBatch = 32;  // rows of the column slab a thread requests from L2 at once

// What the row-wise / column-wise products read and where their results go.
template <typename TIn, typename TAcc>
struct DsmCtx {
  TAcc* Fbuf;   // factor buffer of this CTA: rpad x hF
  TAcc* Ybuf;   // Y of the whole site: (C Nc) x rpad
  TAcc* stage;  // kMaxColSplit x Nc x rpad
  TAcc* red;    // kThreads x kVecBlock
  TAcc* slab;   // rp x Wp
  float* Ps;    // this site's P (global)
  int hF, r, rpad, Nc, C, Wp, h_in;
  int nrows, row_base;
};

// A block of this CTA's shared memory -- `rows` rows of `width` elements starting at base[col0], `stride` apart --
// copied to the same place in every OTHER CTA of the cluster, 16 bytes per store, the stores dealt over all threads.
// (A store into a neighbour's shared memory keeps its warp busy for about a hundred cycles, so few wide stores
// spread over all warps, not many narrow ones from the warps that happen to hold the results.)  base + col0, stride
// and width are multiples of 16 bytes.
template <typename TAcc>
__device__ __forceinline__ void dsm_push(TAcc* base, int rows, int stride, int col0, int width, int C) {
  cg::cluster_group cluster = cg::this_cluster();
  constexpr int E = 16 / (int)sizeof(TAcc);
  const int rank = (int)cluster.block_rank();
  const int wv = width / E;
  if (wv <= 0) return;
  const int per_peer = rows * wv;
#pragma unroll 1
  for (int idx = threadIdx.x; idx < per_peer * (C - 1); idx += kThreads) {
    const int hop = idx / per_peer, rem = idx - hop * per_peer;
    const int peer = (rank + 1 + hop) % C;  // every CTA starts with a different neighbour
    const int row = rem / wv, i = rem - row * wv;
    const int at = row * stride + col0 + i * E;
    const uint4 v = *reinterpret_cast<const uint4*>(base + at);
    *reinterpret_cast<uint4*>(cluster.map_shared_rank(base, peer) + at) = v;
  }
}

// Y[n][j] = sum_c X[n][c] F[j][c] for this CTA's nrows rows; every finished row goes to the Y buffer of all C CTAs
// at row row_base + n.  A warp takes kRowGroup rows x kVecBlock vectors and one of `ks` equal shares of the columns
// (ks chosen so that all eight warps have work), two adjacent columns per lane and step, and completes its 32 sums
// with the exchange tree of warp_reduce.cuh; the shares are then added in share order through `stage`.
template <typename TIn, typename TAcc>
__device__ __noinline__ void dsm_rows_dot(const DsmCtx<TIn, TAcc>& cx, const TIn* X, int64_t ld, int h) {
  cg::cluster_group cluster = cg::this_cluster();
  constexpr int NV = kRowGroup * kVecBlock;
  constexpr int kWarps = kThreads / 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nrows = cx.nrows, rpad = cx.rpad, hF = cx.hF;
  const int n_jb = rpad / kVecBlock;
  const int items = ((nrows + kRowGroup - 1) / kRowGroup) * n_jb;
  int ks = 1;
  while (ks < kMaxColSplit && items * ks * 2 <= kWarps && h >= 64 * ks * 2) ks *= 2;
  const int hshare = ((h + ks - 1) / ks + 63) / 64 * 64;
#pragma unroll 1
  for (int wi = warp; wi < items * ks; wi += kWarps) {
    const int item = wi / ks, share = wi % ks;
    const int row0 = (item / n_jb) * kRowGroup, j0 = (item % n_jb) * kVecBlock;
    const int cbeg = share * hshare, cend = (cbeg + hshare < h) ? cbeg + hshare : h;
    const TIn* xr[kRowGroup];  // rows past the end alias a valid row; their sums are dropped below
#pragma unroll
    for (int q = 0; q < kRowGroup; ++q) xr[q] = X + (int64_t)(row0 + q < nrows ? row0 + q : row0) * ld;
    const TAcc* fr = cx.Fbuf + j0 * hF;
    TAcc acc[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) acc[i] = TAcc(0);
#pragma unroll 2
    for (int c = cbeg + 2 * lane; c < cend; c += 64) {
      TAcc x[kRowGroup][2], f[kVecBlock][2];
#pragma unroll
      for (int q = 0; q < kRowGroup; ++q) load_pair(xr[q] + c, x[q][0], x[q][1]);
#pragma unroll
      for (int jj = 0; jj < kVecBlock; ++jj) load_pair(fr + jj * hF + c, f[jj][0], f[jj][1]);
#pragma unroll
      for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int jj = 0; jj < kVecBlock; ++jj)
#pragma unroll
          for (int q = 0; q < kRowGroup; ++q) acc[q * kVecBlock + jj] += x[q][u] * f[jj][u];
    }
    warp_reduce_scatter<TAcc, NV>(acc, lane);
#pragma unroll
    for (int i = 0; i < NV / 32; ++i) {
      const int idx = reduced_index<NV>(lane, i);
      const int q = idx / kVecBlock, jj = idx % kVecBlock;
      if (row0 + q < nrows) cx.stage[(share * cx.Nc + row0 + q) * rpad + j0 + jj] = acc[i];
    }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < nrows * rpad; idx += kThreads) {
    TAcc v = cx.stage[idx];
    for (int sh = 1; sh < ks; ++sh) v += cx.stage[sh * cx.Nc * rpad + idx];
    cx.Ybuf[cx.row_base * rpad + idx] = v;
  }
  __syncthreads();
  dsm_push<TAcc>(cx.Ybuf, 1, 0, cx.row_base * rpad, nrows * rpad, cx.C);
}

constexpr int kMaxParts = 8;
enum : int { SINK_FACTOR = 0, SINK_SLAB = 1, SINK_P = 2, SINK_P_KEEP = 3 };

// One finished element (vector j, column c = c0 + cc of the product) to where `sink` says.
template <typename TIn, typename TAcc>
__device__ __noinline__ void dsm_emit(const DsmCtx<TIn, TAcc>& cx, int sink, int j, int cc, int c, TAcc v) {
  if (sink == SINK_FACTOR) {
    cx.Fbuf[j * cx.hF + c] = v;  // this CTA's copy; dsm_cols_slice sends the finished slice to the others
  } else if (sink == SINK_SLAB) {
    cx.slab[j * cx.Wp + cc] = v;
  } else {
    DAD_ST(&cx.Ps[(int64_t)j * cx.h_in + c], (float)v);
    if (sink == SINK_P_KEEP) cx.slab[j * cx.Wp + cc] = v;
  }
}

// The CTA's slice [c0, c0 + W) of a column-wise product over ALL N rows of the site:
//     v(j, c) = sum_n Y[n][j] X[n][c].
// The threads form `parts` groups of `cols` threads; a group takes a contiguous share of the rows, a thread two
// adjacent columns (coalesced rows of X from global memory -- L2, several hundred cycles per dependent batch, so
// eight rows are requested at a time -- and Y broadcast from shared memory).  The groups' sums are added in group
// order through `red`.  The finished element goes, by `sink`, to the factor buffer of every CTA (Z), to this CTA's
// Cholesky-QR slab (G~), or to P in global memory (and the slab, for the lengths).
template <typename TIn, typename TAcc>
__device__ __noinline__ void dsm_cols_slice(const DsmCtx<TIn, TAcc>& cx, const TIn* __restrict__ Xsite, int64_t ld, int N,
                                            int h, int c0, int W, int sink) {
  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x;
  const int rpad = cx.rpad, r = cx.r;
  const int Wt = W / 2;  // threads that cover the slice (W is a multiple of 4)
  const int cols = Wt < kThreads / 2 ? Wt : kThreads / 2;
  int parts = kThreads / cols;
  if (parts > kMaxParts) parts = kMaxParts;  // the groups' sums are added one after the other
  if (parts > N) parts = N;
  const int rows_per = (N + parts - 1) / parts;
  const int part = tid / cols, col = tid % cols;
  const bool active = part < parts;
  const int nb = part * rows_per, ne = (nb + rows_per < N) ? nb + rows_per : N;
#pragma unroll 1
  for (int cb = 0; cb < Wt; cb += cols) {
    const int cc = (cb + col) * 2, c = c0 + cc;
    const bool live = active && cc < W && c < h;  // h is even: c < h implies c + 1 < h
#pragma unroll 1
    for (int j0 = 0; j0 < rpad; j0 += kVecBlock) {
      TAcc acc[2][kVecBlock];
#pragma unroll
      for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int jj = 0; jj < kVecBlock; ++jj) acc[u][jj] = TAcc(0);
      if (live) {
        const TIn* row = Xsite + c + (int64_t)nb * ld;
        const TAcc* y = cx.Ybuf + j0;
        int n = nb;
#pragma unroll 1
        for (; n + kRowBatch <= ne; n += kRowBatch, row += kRowBatch * ld) {
          typename PairOf<TIn>::type raw[kRowBatch];  // all requested before any is used: one L2 latency per batch
#pragma unroll
          for (int u = 0; u < kRowBatch; ++u) raw[u] = request_pair(row + (int64_t)u * ld);
#pragma unroll
          for (int u = 0; u < kRowBatch; ++u) {
            TAcc x0, x1;
            widen_pair(raw[u], x0, x1);
            TAcc yy[kVecBlock];
#pragma unroll
            for (int jj = 0; jj < kVecBlock; jj += 2) load_pair(y + (n + u) * rpad + jj, yy[jj], yy[jj + 1]);
#pragma unroll
            for (int jj = 0; jj < kVecBlock; ++jj) {
              acc[0][jj] += yy[jj] * x0;
              acc[1][jj] += yy[jj] * x1;
            }
          }
        }
#pragma unroll 1
        for (; n < ne; ++n, row += ld) {
          TAcc x0, x1;
          load_pair(row, x0, x1);
#pragma unroll
          for (int jj = 0; jj < kVecBlock; ++jj) {
            const TAcc yv = y[n * rpad + jj];
            acc[0][jj] += yv * x0;
            acc[1][jj] += yv * x1;
          }
        }
      }
      if (parts > 1) {
        // `red` holds one value set per thread (kVecBlock x kThreads, a thread's values kThreads apart so that a warp's
        // stores fall into different banks): the two columns of a thread take turns
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          if (u > 0) __syncthreads();
          if (active) {
#pragma unroll
            for (int jj = 0; jj < kVecBlock; ++jj) cx.red[jj * kThreads + part * cols + col] = acc[u][jj];
          }
          __syncthreads();
          if (part == 0) {
#pragma unroll 1
            for (int q = 1; q < parts; ++q)
#pragma unroll
              for (int jj = 0; jj < kVecBlock; ++jj) acc[u][jj] += cx.red[jj * kThreads + q * cols + col];
          }
        }
      }
      if (part == 0 && cc < W && c < h) {
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
          for (int jj = 0; jj < kVecBlock; ++jj)
            if (j0 + jj < r) dsm_emit(cx, sink, j0 + jj, cc + u, c + u, acc[u][jj]);
      }
      if (parts > 1) __syncthreads();  // red is reused by the next block
    }
  }
  if (sink == SINK_FACTOR) {
    __syncthreads();
    const int room = cx.hF - c0;
    dsm_push<TAcc>(cx.Fbuf, r, cx.hF, c0, W < room ? W : room, cx.C);
  }
}

}  // namespace

template <typename TIn, typename TAcc, int BS>
__global__ void __launch_bounds__(kThreads)
fused_dsm_kernel(const DsmParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  cg::cluster_group cluster = cg::this_cluster();
  const int C = p.C, r = p.r, h_in = p.h_in, h_out = p.h_out, N = p.N;
  const DsmGeom d = dsm_geom<BS>(N, h_in, h_out, r, C, sizeof(TAcc), sizeof(TIn), p.x_resident != 0);
  const OrthGeom& g = d.og;
  TAcc* slab = reinterpret_cast<TAcc*>(smem_raw);
  TAcc* Fbuf = reinterpret_cast<TAcc*>(smem_raw + d.off_F);
  double* sigbuf = reinterpret_cast<double*>(smem_raw + d.off_sig);
  TIn* Xa = reinterpret_cast<TIn*>(smem_raw + d.off_X);
  TIn* Xd = Xa + (size_t)d.Nc * h_in;
  __shared__ OrthShared orth_sh;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int s = blockIdx.y;
  const int rank = (int)cluster.block_rank();
  const int rpad = d.rpad, hF = d.hF, Nc = d.Nc;
  const int n0 = rank * Nc;
  const int nrows = n0 >= N ? 0 : (n0 + Nc <= N ? Nc : N - n0);
  const TIn* Asite = reinterpret_cast<const TIn*>(p.A) + (int64_t)s * p.strideA;
  const TIn* Dsite = reinterpret_cast<const TIn*>(p.D) + (int64_t)s * p.strideD;
  const int Wg = g.W, Wp = g.Wp, cg0 = rank * Wg;
  const int Wz = d.Wz, cz0 = rank * Wz;
  const float* Q0s = p.Q0 + (int64_t)s * r * h_out;
  float* Qs = p.Q + (int64_t)s * r * h_out;

  __shared__ DsmCtx<TIn, TAcc> cx;  // read by the building blocks below (shared memory: they are real calls)
  if (tid == 0) {
    cx.Fbuf = Fbuf;
    cx.Ybuf = reinterpret_cast<TAcc*>(smem_raw + d.off_Y);
    cx.stage = reinterpret_cast<TAcc*>(smem_raw + d.off_stage);
    cx.red = reinterpret_cast<TAcc*>(smem_raw + d.off_red);
    cx.slab = slab;
    cx.Ps = p.P + (int64_t)s * r * h_in;
    cx.hF = hF;
    cx.r = r;
    cx.rpad = rpad;
    cx.Nc = Nc;
    cx.C = C;
    cx.Wp = Wp;
    cx.h_in = h_in;
    cx.nrows = nrows;
    cx.row_base = n0;
  }
  __syncthreads();

  // ---- set-up: rows of A and D to shared memory (asynchronous 16-byte copies where the layout allows, all in
  //      flight at once), factor buffer <- Q0 (every CTA reads the whole start block) ----
  const TIn* Arows = Asite + (int64_t)n0 * p.ldA;
  const TIn* Drows = Dsite + (int64_t)n0 * p.ldD;
  int64_t ldAr = p.ldA, ldDr = p.ldD;
  if (p.x_resident) {
    constexpr int V = 16 / (int)sizeof(TIn);  // elements per 16-byte piece
#pragma unroll 1
    for (int which = 0; which < 2; ++which) {
      TIn* dst = which ? Xa : Xd;
      const TIn* src = which ? Arows : Drows;
      const int64_t ld = which ? p.ldA : p.ldD;
      const int h = which ? h_in : h_out;
      const bool vec = (h % V) == 0 && (ld % V) == 0 && (reinterpret_cast<uintptr_t>(src) & 15) == 0;
      if (vec) {
        const int hv = h / V;
#pragma unroll 1
        for (int idx = tid; idx < nrows * hv; idx += kThreads) {
          const int n = idx / hv, c = (idx - n * hv) * V;
          if (!DAD_RANGE_OK(src + (int64_t)n * ld + c, 16)) continue;
          const uint32_t d32 = (uint32_t)__cvta_generic_to_shared(dst + (size_t)n * h + c);
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d32), "l"(src + (int64_t)n * ld + c) : "memory");
        }
      } else {
#pragma unroll 1
        for (int idx = tid; idx < nrows * h; idx += kThreads) dst[idx] = DAD_LD(&src[(int64_t)(idx / h) * ld + idx % h]);
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    Arows = Xa;
    Drows = Xd;
    ldAr = h_in;
    ldDr = h_out;
  }
#pragma unroll 4
  for (int idx = tid; idx < rpad * hF; idx += kThreads) {
    const int j = idx / hF, c = idx - j * hF;
    Fbuf[idx] = (j < r && c < h_out) ? TAcc(DAD_LD(&Q0s[(int64_t)j * h_out + c])) : TAcc(0);
  }
  if (p.iters == 0 && p.Q != p.Q0) {
    for (int j = warp; j < r; j += kThreads / 32)
      for (int cc = lane; cc < Wg; cc += 32)
        if (cg0 + cc < h_out) DAD_ST(&Qs[(int64_t)j * h_out + cg0 + cc], DAD_LD(&Q0s[(int64_t)j * h_out + cg0 + cc]));
  }
  if (p.x_resident) asm volatile("cp.async.wait_all;" ::: "memory");
  cluster.sync();  // every CTA of the cluster is running (its shared memory may be written) and set up

#pragma unroll 1
  for (int k = 0; k < p.iters; ++k) {
    dsm_rows_dot<TIn, TAcc>(cx, Drows, ldDr, h_out);                           // Y = D G^T
    cluster.sync();
    dsm_cols_slice<TIn, TAcc>(cx, Asite, p.ldA, N, h_in, cz0, Wz, SINK_FACTOR);  // Z = Y^T A, to every factor buffer
    cluster.sync();
    dsm_rows_dot<TIn, TAcc>(cx, Arows, ldAr, h_in);                            // W = A Z^T
    cluster.sync();
    for (int idx = tid; idx < g.rp * Wg; idx += kThreads) slab[(idx / Wg) * Wp + idx % Wg] = TAcc(0);
    __syncthreads();
    dsm_cols_slice<TIn, TAcc>(cx, Dsite, p.ldD, N, h_out, cg0, Wg, SINK_SLAB);   // G~ = W^T D, this CTA's slab
    // (orth_slab_passes starts with a CTA barrier and contains the cluster barriers of the Gram exchange)
    orth_slab_passes<BS, TAcc>(slab, smem_raw, g, C, p.tol, p.status, &orth_sh);
    const bool last = k == p.iters - 1;
    // the orthonormal slice goes to the factor buffer of every CTA (and, after the last application, to Q)
    for (int j = warp; j < r; j += kThreads / 32)
      for (int cc = lane; cc < Wg; cc += 32) {
        const int c = cg0 + cc;
        if (c < h_out) {
          const TAcc v = slab[j * Wp + cc];
          Fbuf[j * hF + c] = v;
          if (last) DAD_ST(&Qs[(int64_t)j * h_out + c], (float)v);
        }
      }
    __syncthreads();
    dsm_push<TAcc>(Fbuf, r, hF, cg0, Wg < hF - cg0 ? Wg : hF - cg0, C);
    cluster.sync();
  }

  // ---- P = (A^T (D G^T))^T and the lengths of its rows ----
  dsm_rows_dot<TIn, TAcc>(cx, Drows, ldDr, h_out);
  cluster.sync();
  // the slice of P goes to global memory and, for sigma, into the (now free) slab as well
  for (int idx = tid; idx < g.rp * Wg; idx += kThreads) slab[(idx / Wg) * Wp + idx % Wg] = TAcc(0);
  __syncthreads();
  const bool keep = p.sigma != nullptr && Wz <= Wg;  // the slab has room for the slice of h_in
  dsm_cols_slice<TIn, TAcc>(cx, Asite, p.ldA, N, h_in, cz0, Wz, keep ? SINK_P_KEEP : SINK_P);
  if (p.sigma) {
    __syncthreads();
    // squared length of every vector's slice: a warp per vector, fixed tree; sent to rank 0
    for (int j = warp; j < r; j += kThreads / 32) {
      double sq = 0.0;
      for (int cc = lane; cc < Wz; cc += 32) {
        double v = 0.0;
        if (keep) {
          v = (double)slab[j * Wp + cc];
        } else if (cz0 + cc < h_in) {
          v = (double)DAD_LD(&cx.Ps[(int64_t)j * h_in + cz0 + cc]);  // written by this CTA above (visible after the CTA barrier)
        }
        sq += v * v;
      }
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
      if (lane == 0) cluster.map_shared_rank(sigbuf, 0)[rank * rpad + j] = sq;
    }
    cluster.sync();
    if (rank == 0 && tid < r) {
      double t = 0.0;
      for (int q = 0; q < C; ++q) t += sigbuf[q * rpad + tid];
      DAD_ST(&p.sigma[(int64_t)s * r + tid], (float)sqrt(t));
    }
  } else {
    cluster.sync();  // no CTA leaves while a neighbour may still store into its shared memory
  }
}

// ---- host side ---------------------------------------------------------------------------------------------------
namespace {

constexpr size_t kSmemLimit = 226 * 1024;  // dynamic shared memory a CTA may opt in to, less the static part

size_t dsm_smem_for(const dad_layer& L, int r, int C, bool x_resident) {
  const size_t acc = L.dtype == DAD_F32 ? 8 : 4, in_bytes = L.dtype == DAD_F32 ? 4 : 2;
  if (r >= 32) return dsm_geom<8>((int)L.N, (int)L.h_in, (int)L.h_out, r, C, acc, in_bytes, x_resident).total;
  return dsm_geom<2>((int)L.N, (int)L.h_in, (int)L.h_out, r, C, acc, in_bytes, x_resident).total;
}

template <typename TIn, typename TAcc, int BS>
cudaError_t launch_dsm(const DsmParams& p, int S, size_t smem, cudaStream_t st) {
  auto kernel = fused_dsm_kernel<TIn, TAcc, BS>;
  static FirstUse first;
  if (first.on_this_device()) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit);
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

// Whether the on-chip form takes a site handled by a cluster of C CTAs: the factor, Y and the Cholesky-QR slab have to
// fit in a CTA's shared memory; *x_resident tells whether the CTA's rows of A and D fit beside them.
bool fused_dsm_fits(const dad_layer& L, int r, int C, bool* x_resident) {
  // the kernel reads pairs of adjacent elements: even widths, rows and sites that start on even elements
  if ((L.h_in | L.h_out | L.ldA | L.ldD) & 1) return false;
  if (L.S > 1 && ((L.strideA | L.strideD) & 1)) return false;
  if (dsm_smem_for(L, r, C, false) > kSmemLimit) return false;
  if (x_resident) *x_resident = dsm_smem_for(L, r, C, true) <= kSmemLimit;
  return true;
}

cudaError_t fused_dsm_compress(const dad_layer& L, const void* A, const void* D, int r, int iters, const float* Q0, float* P,
                               float* Q, float* sigma, int* status, int C, cudaStream_t st) {
  bool xres = false;
  if (!fused_dsm_fits(L, r, C, &xres)) return cudaErrorInvalidValue;
  DsmParams p{};
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
  p.x_resident = xres ? 1 : 0;
  p.Q0 = Q0;
  p.P = P;
  p.Q = Q;
  p.sigma = sigma;
  p.status = status;
  const bool f32in = L.dtype == DAD_F32;
  p.tol = f32in ? 1e-12 : 1e-6;
  const size_t smem = dsm_smem_for(L, r, C, xres);
  if (f32in) {
    if (r >= 32) return launch_dsm<float, double, 8>(p, L.S, smem, st);
    return launch_dsm<float, double, 2>(p, L.S, smem, st);
  }
  if (r >= 32) return launch_dsm<__nv_bfloat16, float, 8>(p, L.S, smem, st);
  return launch_dsm<__nv_bfloat16, float, 2>(p, L.S, smem, st);
}

}  // namespace dad

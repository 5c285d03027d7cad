// Cholesky-QR of a slab of the r iterate vectors held in shared memory by the CTAs of a thread-block cluster
// (each CTA owns W of the h columns): the geometry of the slab and the pass loop shared by the stand-alone
// orthonormalisation kernel and by the one-launch compress kernel.
//
//   pass:  partial Gram of the slab (fp64, BS x BS register blocks)  ->  sum of the C partials over distributed
//          shared memory, in rank order, by every CTA (all CTAs get the identical r x r matrix)  ->  Cholesky in
//          shared memory (pivot floor, zeroing rule)  ->  forward substitution down each column of the slab.
//   A second pass runs when the first shows a pivot far below the vector's length; every CTA of the cluster
//   factors the same matrix and so takes the same decision.
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"

namespace dad {
namespace orthslab {

namespace cg = cooperative_groups;

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

// Shared-memory state of the pass loop beside the slab itself.
struct OrthShared {
  int need2;
  unsigned char dead_row[DAD_MAX_RANK];
};

// Both passes on `slab` (rp x Wp elements of T, rows >= r and columns beyond the CTA's share zero), in place.
// Every thread of every CTA of the cluster calls it (it contains cluster-wide barriers).
template <int BS, typename T>
__device__ __forceinline__ void orth_slab_passes(T* slab, unsigned char* smem_raw, const OrthGeom& g, int C, double tol,
                                                 int* __restrict__ status, OrthShared* sh) {
  using T2 = typename Vec2<T>::type;
  cg::cluster_group cluster = cg::this_cluster();
  double* gram = reinterpret_cast<double*>(smem_raw + g.off_gram);
  double* Lm = reinterpret_cast<double*>(smem_raw + g.off_L);
  double* diag0 = reinterpret_cast<double*>(smem_raw + g.off_vec);
  double* piv1 = diag0 + g.rp;   // first-pass pivots (squared R_jj)
  double* inv_l = piv1 + g.rp;
  double* orig1 = inv_l + g.rp;  // squared lengths before the first pass
  int& need2_s = sh->need2;
  unsigned char* dead_row = sh->dead_row;
  const int tid = threadIdx.x;
  const int rp = g.rp, W = g.W, Wp = g.Wp, LR = rp + 1;
  const double tol2 = tol * tol;
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
}

}  // namespace orthslab
}  // namespace dad

// Orthonormalisation of the r iterate vectors of a site (fp32 storage), with the two fp64-heavy phases
// of Cholesky-QR on the fp64 matrix-multiply unit (mma.sync m8n8k4).  Phases, on a slab of rp x W
// columns of the vectors held in shared memory (rp = r rounded up to 8; rows >= r and columns >= h zero):
//
//   Gram:      8 x 8 tiles of the lower triangle of slab slab^T, four columns per MMA; row blocks are
//              paired (i, nb-1-i) over the warps so that every warp owns about the same number of tiles;
//   Cholesky:  panels of four columns, two threads per row on the first four warps.  A thread brings two
//              panel entries of its row up to date (dot products over the columns already factored,
//              four partial sums each); after a barrier every row's threads factor their own copy of
//              the 4 x 4 diagonal block in registers.  The reciprocal square root of a pivot starts
//              before the floor test on that pivot is known (the test compares bit patterns, off the
//              fp64 pipe) and is replaced afterwards if the test says so; floor and zeroing rule are
//              those of orth.cu;
//   solve:     rows <- L^{-1} rows as block forward substitution in product form,
//              X_b = sum_{k<=b} M_bk Src_k with M_bb = L_bb^{-1}, M_bk = -L_bb^{-1} L_bk, Src_k = X_k
//              (already solved, read back in fp32) for k < b and the unsolved rows for k = b; every warp
//              owns whole columns, so the substitution needs no barrier.
//   A second pass runs when the first shows R_jj < 1e-5 ||g_j|| for some vector.
//
// Two arrangements of these phases:
//   * one launch, a thread-block cluster of C CTAs per site, each keeping its slab in shared memory
//     throughout; the C partial Gram matrices are added over distributed shared memory in rank order by
//     every CTA, so all CTAs factor the identical matrix and take identical decisions.  Vectors cross
//     HBM once each way.  Every CTA repeats the factorisation, which is a latency chain: right for few
//     sites.
//   * two launches per pass for many sites at large r: (1) partial Gram per 256-column chunk, the last
//     CTA of a site to arrive adds the partials in chunk order, factors and stores the M matrices;
//     (2) every chunk applies them.  The factorisation runs once per site and under other sites' Gram
//     work.
// All sums run in a fixed order: two runs give identical bits.
#include <cooperative_groups.h>

#include <algorithm>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace dad {

namespace {
constexpr double kPivotFloor = 1e-14;         // (1e-7)^2 of the squared length
constexpr double kSecondPassBelowSq = 1e-10;  // (1e-5)^2: one fp64 pass leaves a defect of 1e-16 cond^2 <= 1e-6
constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr size_t kSmemLimit = 200 * 1024;
constexpr int kFactorW = 256;  // columns per CTA of the two-launch arrangement: Gram + factorisation kernel
constexpr int kApplyW = 128;   // ... and substitution kernel

struct MmaGeom {
  int rp, nb, nt;  // padded rank, row blocks of 8, tiles of the lower triangle
  int W, Wp, LR;   // columns per CTA (multiple of 8), slab row stride (floats), row stride of L (doubles)
  size_t off_tiles, off_L, off_vec, total;
};

__host__ __device__ inline MmaGeom mma_geom(int r, int W) {
  MmaGeom g;
  g.rp = (r + 7) / 8 * 8;
  g.nb = g.rp / 8;
  g.nt = g.nb * (g.nb + 1) / 2;
  g.W = W;
  g.Wp = (W + 31) / 32 * 32 + 12;  // 12 mod 32: the 8 x 4 fragment loads of the Gram phase hit 32 different banks
  g.LR = g.rp + 1;                 // odd: the sixteen rows a warp of the factorisation serves fall into different banks
  size_t off = sizeof(float) * (size_t)g.rp * g.Wp;
  off = (off + 15) / 16 * 16;
  g.off_tiles = off;  // nt tiles of 64 doubles: this CTA's partial Gram (read by the cluster), later the matrices M_bk
  off += sizeof(double) * 64 * (size_t)g.nt;
  g.off_L = off;
  off += sizeof(double) * (size_t)g.rp * g.LR;
  g.off_vec = off;  // 5 x rp doubles: see FactorState
  off += sizeof(double) * 5 * (size_t)g.rp;
  g.total = off;
  return g;
}

inline int columns_per_cta(int64_t h, int C) { return (int)((ceil_div(h, C) + 7) / 8 * 8); }

// CTAs per site of the one-launch arrangement: as few as still give every SM a CTA (each CTA of a cluster repeats the
// r x r factorisation, and a launch that fits the GPU in one wave beats a finer one in two: 256 sites at r = 16,
// h = 1024 take 25 us as 256 CTAs, 36 us as 512), more if the slab would not fit otherwise; no slabs narrower than
// 128 columns.
inline int mma_cluster_size(int r, int64_t h, int S) {
  int best = 0;
  for (int C = 1; C <= 8; C *= 2) {
    if (C > 1 && h / C < 128) break;
    if (mma_geom(r, columns_per_cta(h, C)).total > kSmemLimit) continue;
    best = C;
    if ((int64_t)S * C >= 148) break;
  }
  return best;
}

__device__ __forceinline__ void dmma(double (&c)[2], double a, double b) {
  asm("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
      : "+d"(c[0]), "+d"(c[1])
      : "d"(a), "d"(b));
}

// Index of element (row g, column k) of an 8 x 8 tile stored in the order the A fragments of two MMAs read it.
__device__ __forceinline__ int afrag_index(int g, int k) { return (k >> 2) * 32 + g * 4 + (k & 3); }

// Per-column state of the factorisation, rp doubles each, in shared memory.
struct FactorState {
  double* diag0;    // squared lengths of the vectors (diagonal of the Gram matrix)
  double* p1;       // in: factor of the zeroing test, 1 in the first pass
  double* bar;      // in: threshold of the zeroing test, -1 in the first pass: zero when !(p1 * pivot > bar)
  double* piv_out;  // out: pivot used (squared R_jj), 0 for a zeroed vector
  double* inv_l;    // out: 1 / R_jj (1 for a zeroed vector)
  unsigned char* dead_row;  // out: 1 for a zeroed vector (set, never cleared)
  int* need2;               // out: set to 1 when some pivot fell below kSecondPassBelowSq of its squared length
};

__device__ __forceinline__ FactorState factor_state(double* base, int rp, unsigned char* dead_row, int* need2) {
  FactorState f;
  f.diag0 = base;
  f.p1 = base + rp;
  f.bar = base + 2 * rp;
  f.piv_out = base + 3 * rp;
  f.inv_l = base + 4 * rp;
  f.dead_row = dead_row;
  f.need2 = need2;
  return f;
}

// ---- load a slab: columns [c0, c0 + W) of the r vectors of a site; rows >= r and columns >= h are zero ----
__device__ __forceinline__ void load_slab(float* __restrict__ slab, const float* __restrict__ Gs, int r, int rp, int64_t h,
                                          int64_t c0, int W, int Wp, int tid) {
  if ((h & 3) == 0) {
    const int W4 = W / 4, total = rp * W4;
    for (int base = 0; base < total; base += kThreads * 8) {  // loads issued eight at a time per thread
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int idx = base + u * kThreads + tid;
        const int j = idx / W4, c = (idx % W4) * 4;
        v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (idx < total && j < r && c0 + c < h) v[u] = *reinterpret_cast<const float4*>(Gs + (int64_t)j * h + c0 + c);
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int idx = base + u * kThreads + tid;
        if (idx < total) *reinterpret_cast<float4*>(slab + (idx / W4) * Wp + (idx % W4) * 4) = v[u];
      }
    }
  } else {
    const int total = rp * W;
    for (int base = 0; base < total; base += kThreads * 8) {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int idx = base + u * kThreads + tid;
        const int j = idx / W, c = idx % W;
        v[u] = (idx < total && j < r && c0 + c < h) ? Gs[(int64_t)j * h + c0 + c] : 0.f;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int idx = base + u * kThreads + tid;
        if (idx < total) slab[(idx / W) * Wp + idx % W] = v[u];
      }
    }
  }
}

// ---- write a slab back (and its bf16 hi/lo planes) ----
__device__ __forceinline__ void store_slab(const float* __restrict__ slab, float* __restrict__ Gs, int s, int r, int64_t h,
                                           int64_t c0, int W, int Wp, float* __restrict__ out32,
                                           __nv_bfloat16* __restrict__ planes, int plane_rows, int tid) {
  if ((h & 3) == 0) {
    const int W4 = W / 4;
    for (int idx = tid; idx < r * W4; idx += kThreads) {
      const int j = idx / W4, c = (idx % W4) * 4;
      const int64_t col = c0 + c;
      if (col < h) {
        const float4 v = *reinterpret_cast<const float4*>(slab + j * Wp + c);
        const float f[4] = {v.x, v.y, v.z, v.w};
        *reinterpret_cast<float4*>(Gs + (int64_t)j * h + col) = v;
        if (out32) *reinterpret_cast<float4*>(out32 + ((int64_t)s * r + j) * h + col) = v;
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
        const float f = slab[j * Wp + c];
        const int64_t col = c0 + c;
        Gs[(int64_t)j * h + col] = f;
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

// ---- partial Gram of the slab into `tiles` (tile (bi, bj), bj <= bi, at (bi (bi + 1) / 2 + bj) * 64, row-major 8 x 8).
//      Warp (pair, cgi): row blocks lo = pair and hi = NB-1-pair, the cgi-th part of the columns.  The column
//      parts add their tiles one after the other (fixed order).  Ends with a barrier. ----
template <int NB>
__device__ __forceinline__ void gram_tiles(const float* __restrict__ slab, int W, int Wp, double* __restrict__ tiles,
                                           int warp, int lane) {
  constexpr int TG = (NB + 1) / 2;   // row-block pairs
  constexpr int CG = kWarps / TG;    // column parts
  constexpr int NLO = (NB + 1) / 2;  // tiles of the lower row block of a pair: at most this many
  const int g = lane >> 2, t = lane & 3;
  const int pair = warp % TG, cgi = warp / TG;
  const bool working = cgi < CG;
  const int lo = pair, hi = NB - 1 - pair;
  double acc_hi[NB][2], acc_lo[NLO][2];
#pragma unroll
  for (int b = 0; b < NB; ++b) acc_hi[b][0] = acc_hi[b][1] = 0.0;
#pragma unroll
  for (int b = 0; b < NLO; ++b) acc_lo[b][0] = acc_lo[b][1] = 0.0;
  if (working) {
    const int KS = W / 4, per = (KS + CG - 1) / CG;
    const int ks_end = min(KS, (cgi + 1) * per);
    const float* row_g = slab + g * Wp + t;
    for (int ks = cgi * per; ks < ks_end; ++ks) {
      const float* p = row_g + ks * 4;
      double f[NB];
#pragma unroll
      for (int b = 0; b < NB; ++b) f[b] = (b <= hi) ? (double)p[b * 8 * Wp] : 0.0;
      const double a_hi = (double)p[hi * 8 * Wp];
      const double a_lo = (double)p[lo * 8 * Wp];
#pragma unroll
      for (int b = 0; b < NB; ++b)
        if (b <= hi) dmma(acc_hi[b], a_hi, f[b]);
      if (lo != hi) {
#pragma unroll
        for (int b = 0; b < NLO; ++b)
          if (b <= lo) dmma(acc_lo[b], a_lo, f[b]);
      }
    }
  }
  for (int turn = 0; turn < CG; ++turn) {
    if (working && cgi == turn) {
#pragma unroll
      for (int b = 0; b < NB; ++b)
        if (b <= hi) {
          double2* dst = reinterpret_cast<double2*>(tiles + (size_t)(hi * (hi + 1) / 2 + b) * 64 + lane * 2);
          double2 v = make_double2(acc_hi[b][0], acc_hi[b][1]);
          if (turn > 0) {
            const double2 o = *dst;
            v.x += o.x;
            v.y += o.y;
          }
          *dst = v;
        }
      if (lo != hi) {
#pragma unroll
        for (int b = 0; b < NLO; ++b)
          if (b <= lo) {
            double2* dst = reinterpret_cast<double2*>(tiles + (size_t)(lo * (lo + 1) / 2 + b) * 64 + lane * 2);
            double2 v = make_double2(acc_lo[b][0], acc_lo[b][1]);
            if (turn > 0) {
              const double2 o = *dst;
              v.x += o.x;
              v.y += o.y;
            }
            *dst = v;
          }
      }
    }
    __syncthreads();
  }
}

// ---- Cholesky of the rp x rp matrix whose lower triangle is in Lm (row stride LR), in place, in panels of four
//      columns.  Threads 2i and 2i+1 (the first four warps: one per scheduler, so that the dependent fp64 chains do
//      not queue behind one another) serve row i, two panel columns each; the other threads only join the barriers.
//      All threads of the CTA call it; f.diag0, f.p1, f.bar are filled and visible.  Ends with a barrier. ----
template <bool FIRST>
__device__ __forceinline__ void cholesky_panels(double* __restrict__ Lm, int LR, int rp, const FactorState& f,
                                                double (*Dblk)[4], int* __restrict__ status, int tid) {
  const int i = tid >> 1, q = tid & 1;
  const bool in_rows = i < rp;  // rp <= 64: rows live in threads 0..127
  double* Li = Lm + (in_rows ? i : 0) * LR;
  // What the thread of a diagonal entry decided for its column is written out one panel later, when its row is
  // finished and the thread would idle: the stores stay off the critical path.
  bool pend = false, pend_dead = false, pend_bad = false, pend_need2 = false;
  double pend_piv = 0.0, pend_il = 0.0;
  auto record = [&]() {
    if (pend_bad && status) *status = (int)DAD_ERR_NUMERIC;
    f.piv_out[i] = pend_piv;
    f.inv_l[i] = pend_il;
    if (pend_need2) *f.need2 = 1;
    if (pend_dead) f.dead_row[i] = 1;
    pend = false;
  };
  for (int k0 = 0; k0 < rp; k0 += 4) {
    const bool mine = in_rows && i >= k0;
    if (pend) record();
    if (mine) {
      // entries (i, k0 + 2q) and (i, k0 + 2q + 1) of the panel, brought up to date: G_in - sum_{l<k0} L_il L_(k0+n)l
      const double* La = Lm + (k0 + 2 * q) * LR;
      const double* Lb = La + LR;
      double sa0 = 0.0, sa1 = 0.0, sa2 = 0.0, sa3 = 0.0, sb0 = 0.0, sb1 = 0.0, sb2 = 0.0, sb3 = 0.0;
      for (int l = 0; l < k0; l += 4) {  // four partial sums per entry
        const double x0 = Li[l], x1 = Li[l + 1], x2 = Li[l + 2], x3 = Li[l + 3];
        sa0 += x0 * La[l];
        sa1 += x1 * La[l + 1];
        sa2 += x2 * La[l + 2];
        sa3 += x3 * La[l + 3];
        sb0 += x0 * Lb[l];
        sb1 += x1 * Lb[l + 1];
        sb2 += x2 * Lb[l + 2];
        sb3 += x3 * Lb[l + 3];
      }
      const double va = Li[k0 + 2 * q] - ((sa0 + sa1) + (sa2 + sa3));
      const double vb = Li[k0 + 2 * q + 1] - ((sb0 + sb1) + (sb2 + sb3));
      Li[k0 + 2 * q] = va;
      Li[k0 + 2 * q + 1] = vb;
      if (i < k0 + 4) {  // the diagonal block, for everybody
        Dblk[i - k0][2 * q] = va;
        Dblk[i - k0][2 * q + 1] = vb;
      }
    }
    // what the decisions on the four pivots need, fetched ahead of the barrier
    double orig[4], floor_[4], il_floor[4], p1[4], bar[4], thr2[4];
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      orig[jj] = f.diag0[k0 + jj];
      floor_[jj] = kPivotFloor * orig[jj];
      il_floor[jj] = rsqrt(floor_[jj]);
      thr2[jj] = kSecondPassBelowSq * orig[jj];
      p1[jj] = f.p1[k0 + jj];
      bar[jj] = f.bar[k0 + jj];
    }
    __syncthreads();
    double a[4] = {0.0, 0.0, 0.0, 0.0};
    if (mine) {
      double D[4][4], piv_rec[4], il_rec[4];
      unsigned dead_mask = 0, bad_mask = 0;
#pragma unroll
      for (int m = 0; m < 4; ++m)
#pragma unroll
        for (int n = 0; n <= m; ++n) D[m][n] = Dblk[m][n];
#pragma unroll
      for (int n = 0; n < 4; ++n) a[n] = Li[k0 + n];
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        const bool bad = !(orig[jj] == orig[jj]) || orig[jj] > 1.7e308;
        const bool usable = !bad && orig[jj] > 0.0;
        const double d = D[jj][jj];
        const double il_raw = rsqrt(d);  // started at once; the decisions below run beside it
        // A pivot at or below the floor is raised to it.  Both are compared as integers (same order as the values for
        // a positive floor; a negative pivot has the sign bit set and is smaller): the fp64 comparison would take
        // longer than the reciprocal square root beside it and hold up the choice between the two candidates.
        // (A floor that is not positive or not a number belongs to an unusable vector, which is zeroed whatever ok is.)
        const bool ok = __double_as_longlong(d) > __double_as_longlong(floor_[jj]);
        const double piv = ok ? d : floor_[jj];
        // zeroing rule: first pass never (known ahead, so the choice of the scale below waits for the floor test
        // only); second pass: total remainder (R1_jj R2_jj)^2 against tol^2 of the squared length before the first
        const bool is_dead = FIRST ? !usable : (!usable || !(p1[jj] * piv > bar[jj]));
        const double il = ok ? il_raw : il_floor[jj];
        const double scale = is_dead ? 0.0 : il;
        // column jj of the diagonal block, then its effect on the columns to the right
#pragma unroll
        for (int m = jj + 1; m < 4; ++m) D[m][jj] *= scale;
#pragma unroll
        for (int m = jj + 1; m < 4; ++m)
#pragma unroll
          for (int n = jj + 1; n <= m; ++n) D[m][n] -= D[m][jj] * D[n][jj];
        // the same for this thread's own row
        const double l_ij = a[jj] * scale;
#pragma unroll
        for (int n = jj + 1; n < 4; ++n) a[n] -= l_ij * D[n][jj];
        a[jj] = (i == k0 + jj) ? (is_dead ? 1.0 : piv * il) : l_ij;
        piv_rec[jj] = is_dead ? 0.0 : piv;
        il_rec[jj] = is_dead ? 1.0 : il;
        dead_mask |= (is_dead ? 1u : 0u) << jj;
        bad_mask |= (bad ? 1u : 0u) << jj;
      }
      if (i < k0 + 4 && q == 0) {  // the thread of the diagonal entry notes what was decided for its column
        // one path for the four diagonal threads (they share a warp): values selected by column, not branched on
        const int jj = i - k0;
        pend_piv = jj == 0 ? piv_rec[0] : jj == 1 ? piv_rec[1] : jj == 2 ? piv_rec[2] : piv_rec[3];
        pend_il = jj == 0 ? il_rec[0] : jj == 1 ? il_rec[1] : jj == 2 ? il_rec[2] : il_rec[3];
        const double thr = jj == 0 ? thr2[0] : jj == 1 ? thr2[1] : jj == 2 ? thr2[2] : thr2[3];
        pend_dead = (dead_mask >> jj) & 1u;
        pend_bad = (bad_mask >> jj) & 1u;
        pend_need2 = FIRST && !pend_dead && pend_piv < thr;
        pend = true;
      }
    }
    __syncwarp();  // the two threads of a row have both read the row's panel entries
    // (selected, not indexed: an index known only at run time would push a[] out of the registers)
    if (mine) {
      if (k0 + 2 * q <= i) Li[k0 + 2 * q] = q == 0 ? a[0] : a[2];
      if (k0 + 2 * q + 1 <= i) Li[k0 + 2 * q + 1] = q == 0 ? a[1] : a[3];
    }
    __syncthreads();
  }
  if (pend) record();
  __syncthreads();
}

// ---- the matrices of the substitution into `tiles` (fragment order): M_bb = L_bb^{-1}, M_bk = -L_bb^{-1} L_bk;
//      rows of zeroed vectors are zero.  Ends with a barrier. ----
__device__ __forceinline__ void build_m(double* __restrict__ tiles, const double* __restrict__ Lm, int LR, int rp, int nt,
                                        const FactorState& f, const unsigned char* tile_bi, const unsigned char* tile_bj,
                                        int tid) {
  if (tid < rp) {  // thread (b, c): column c of the inverse of diagonal block b, by forward substitution
    const int b = tid >> 3, c = tid & 7;
    const double* Lb = Lm + (b * 8) * LR + b * 8;
    double x[8];
#pragma unroll
    for (int m = 0; m < 8; ++m) {
      double v = (m == c) ? 1.0 : 0.0;
#pragma unroll
      for (int l = 0; l < m; ++l) v -= Lb[m * LR + l] * x[l];
      x[m] = (m < c) ? 0.0 : v * f.inv_l[b * 8 + m];
    }
    double* Mbb = tiles + (size_t)(b * (b + 1) / 2 + b) * 64;
#pragma unroll
    for (int m = 0; m < 8; ++m) Mbb[afrag_index(m, c)] = f.dead_row[b * 8 + m] ? 0.0 : x[m];
  }
  __syncthreads();
  for (int e = tid; e < nt * 64; e += kThreads) {
    const int T = e >> 6, m = (e >> 3) & 7, c = e & 7;
    const int b = tile_bi[T], k = tile_bj[T];
    if (k < b) {
      const double* Mbb = tiles + (size_t)(b * (b + 1) / 2 + b) * 64;
      const double* Lbk = Lm + (b * 8) * LR + k * 8 + c;
      double v = 0.0;
#pragma unroll
      for (int l = 0; l < 8; ++l) v -= Mbb[afrag_index(m, l)] * Lbk[l * LR];  // entries right of the diagonal of M_bb are zero
      tiles[(size_t)T * 64 + afrag_index(m, c)] = v;  // a zero row of M_bb gives a zero row here
    }
  }
  __syncthreads();
}

// X_b rows of NT column tiles (8 columns each, starting at col[.]) for all row blocks b, in place.
template <int NT>
__device__ __forceinline__ void solve_tiles(float* __restrict__ slab, const double* __restrict__ Mt, int nb, int Wp,
                                            const int (&col)[NT], int lane) {
  const int g = lane >> 2, t = lane & 3;
  for (int b = 0; b < nb; ++b) {
    double acc[NT][2];
#pragma unroll
    for (int n = 0; n < NT; ++n) acc[n][0] = acc[n][1] = 0.0;
    const double* Mrow = Mt + (size_t)(b * (b + 1) / 2) * 64;
    for (int k = 0; k <= b; ++k) {
#pragma unroll
      for (int kk = 0; kk < 2; ++kk) {
        const double a = Mrow[k * 64 + kk * 32 + lane];
        const float* src = slab + (k * 8 + kk * 4 + t) * Wp + g;
#pragma unroll
        for (int n = 0; n < NT; ++n) dmma(acc[n], a, (double)src[col[n]]);
      }
    }
    __syncwarp();  // every lane has read the unsolved rows of block b
#pragma unroll
    for (int n = 0; n < NT; ++n)
      *reinterpret_cast<float2*>(slab + (b * 8 + g) * Wp + col[n] + 2 * t) = make_float2((float)acc[n][0], (float)acc[n][1]);
    __syncwarp();  // the rows below read them back
  }
}

// ---- block forward substitution over the whole slab: every warp takes whole column tiles, up to four at a time ----
__device__ __forceinline__ void solve_slab(float* __restrict__ slab, const double* __restrict__ tiles, int nb, int W, int Wp,
                                           int warp, int lane) {
  const int ntile = W / 8;
  int tile = warp;
  for (; tile + 3 * kWarps < ntile; tile += 4 * kWarps) {
    const int col[4] = {tile * 8, (tile + kWarps) * 8, (tile + 2 * kWarps) * 8, (tile + 3 * kWarps) * 8};
    solve_tiles<4>(slab, tiles, nb, Wp, col, lane);
  }
  for (; tile + kWarps < ntile; tile += 2 * kWarps) {
    const int col[2] = {tile * 8, (tile + kWarps) * 8};
    solve_tiles<2>(slab, tiles, nb, Wp, col, lane);
  }
  for (; tile < ntile; tile += kWarps) {
    const int col[1] = {tile * 8};
    solve_tiles<1>(slab, tiles, nb, Wp, col, lane);
  }
}

__device__ __forceinline__ void fill_tile_table(unsigned char* tile_bi, unsigned char* tile_bj, int nt, int tid) {
  if (tid < nt) {
    int bi = 0;
    while ((bi + 1) * (bi + 2) / 2 <= tid) ++bi;
    tile_bi[tid] = (unsigned char)bi;
    tile_bj[tid] = (unsigned char)(tid - bi * (bi + 1) / 2);
  }
}
}  // namespace

// =====================================================================================================================
// One launch: a cluster of C CTAs per site.
// =====================================================================================================================
template <int NB>
__global__ void __launch_bounds__(kThreads, 2)
orth_mma_kernel(float* __restrict__ G, int r, int64_t h, int C, int W, double tol, int* __restrict__ status,
                float* __restrict__ out32, __nv_bfloat16* __restrict__ planes, int plane_rows) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  cg::cluster_group cluster = cg::this_cluster();
  const MmaGeom geo = mma_geom(r, W);
  float* slab = reinterpret_cast<float*>(smem_raw);
  double* tiles = reinterpret_cast<double*>(smem_raw + geo.off_tiles);
  double* Lm = reinterpret_cast<double*>(smem_raw + geo.off_L);
  __shared__ int need2_s;
  __shared__ unsigned char dead_row[DAD_MAX_RANK];
  __shared__ unsigned char tile_bi[36], tile_bj[36];
  __shared__ double Dblk[4][4];  // diagonal block of the Cholesky panel being factored

  constexpr int rp = NB * 8, nt = NB * (NB + 1) / 2;
  const FactorState f = factor_state(reinterpret_cast<double*>(smem_raw + geo.off_vec), rp, dead_row, &need2_s);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int s = blockIdx.y;
  const int rank = (int)cluster.block_rank();
  const int Wp = geo.Wp, LR = geo.LR;
  const int64_t c0 = (int64_t)rank * W;
  float* Gs = G + (int64_t)s * r * h;
  const double tol2 = tol * tol;

  // the next kernel in the stream may begin its set-up now; it waits for this grid before touching memory
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  load_slab(slab, Gs, r, rp, h, c0, W, Wp, tid);
  if (tid < DAD_MAX_RANK) dead_row[tid] = 0;
  fill_tile_table(tile_bi, tile_bj, nt, tid);
  if (tid < rp) {
    f.p1[tid] = 1.0;
    f.bar[tid] = -1.0;
  }
  __syncthreads();

  for (int pass = 0; pass < 2; ++pass) {
    gram_tiles<NB>(slab, W, Wp, tiles, warp, lane);
    // ---- sum the partials of all CTAs of the cluster, in rank order, into L (lower triangle incl. whole diagonal tiles) ----
    cluster.sync();
    for (int e = tid; e < nt * 64; e += kThreads) {
      double v[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) v[q] = (q < C) ? cluster.map_shared_rank(tiles, q)[e] : 0.0;
      double sum = v[0];
#pragma unroll
      for (int q = 1; q < 8; ++q) sum += v[q];
      const int T = e >> 6, w = e & 63;
      Lm[(tile_bi[T] * 8 + (w >> 3)) * LR + tile_bj[T] * 8 + (w & 7)] = sum;
    }
    cluster.sync();  // nobody rewrites its partial while a neighbour still reads it
    if (tid < rp) f.diag0[tid] = Lm[tid * LR + tid];
    if (tid == 0) need2_s = 0;
    __syncthreads();

    if (pass == 0) {
      cholesky_panels<true>(Lm, LR, rp, f, Dblk, status, tid);
    } else {
      cholesky_panels<false>(Lm, LR, rp, f, Dblk, status, tid);
    }
    build_m(tiles, Lm, LR, rp, nt, f, tile_bi, tile_bj, tid);
    solve_slab(slab, tiles, NB, W, Wp, warp, lane);
    __syncthreads();
    if (need2_s == 0) break;  // same matrix, same decision in every CTA of the cluster
    if (tid < rp) {           // second pass: (R1_jj R2_jj)^2 against tol^2 of the squared length before the first
      f.p1[tid] = f.piv_out[tid];
      f.bar[tid] = tol2 * f.diag0[tid];
    }
    __syncthreads();
  }

  store_slab(slab, Gs, s, r, h, c0, W, Wp, out32, planes, plane_rows, tid);
}

// =====================================================================================================================
// Two launches per pass: Gram + factorisation (last CTA of a site), then the substitution.
//   partial: S x chunks x nt x 64 doubles; Mt: S x nt x 64 doubles; ratio1: S x r doubles (first-pass pivot over the
//   squared length); dead: S x r bytes; need2: S ints; counters: S arrival counters (zero on entry, left zero).
// =====================================================================================================================
template <int NB>
__global__ void __launch_bounds__(kThreads, 2)
orth_split_factor_kernel(const float* __restrict__ G, int S, int r, int64_t h, int chunks, int pass, double tol,
                         double* __restrict__ partial, double* __restrict__ Mt, double* __restrict__ ratio1,
                         unsigned char* __restrict__ dead, int* __restrict__ need2, unsigned* __restrict__ counters,
                         int* __restrict__ status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int rp = NB * 8, nt = NB * (NB + 1) / 2;
  const int chunk = blockIdx.x;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const MmaGeom geo = mma_geom(r, kFactorW);
  // the factorisation (last CTA only) reuses the slab's place for L: the slab is spent by then
  float* slab = reinterpret_cast<float*>(smem_raw);
  double* Lm = reinterpret_cast<double*>(smem_raw);
  const size_t lbytes = sizeof(double) * (size_t)rp * geo.LR, sbytes = geo.off_tiles;
  double* tiles = reinterpret_cast<double*>(smem_raw + (lbytes > sbytes ? lbytes : sbytes));
  double* vec = tiles + (size_t)nt * 64;
  __shared__ int need2_s;
  __shared__ bool is_last;
  __shared__ unsigned char dead_row[DAD_MAX_RANK];
  __shared__ unsigned char tile_bi[36], tile_bj[36];
  __shared__ double Dblk[4][4];
  const FactorState f = factor_state(vec, rp, dead_row, &need2_s);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int Wp = geo.Wp, LR = geo.LR;
  fill_tile_table(tile_bi, tile_bj, nt, tid);

  // First pass: one site per CTA row.  Second pass: a small grid walks over the sites and skips those that do not
  // need it (nearly always all of them), so the launch costs next to nothing.
  for (int s = blockIdx.y; s < S; s += gridDim.y) {
  if (pass == 1 && need2[s] == 0) continue;
  __syncthreads();  // the previous site's shared memory is no longer in use
  load_slab(slab, G + (int64_t)s * r * h, r, rp, h, (int64_t)chunk * kFactorW, kFactorW, Wp, tid);
  __syncthreads();
  gram_tiles<NB>(slab, kFactorW, Wp, tiles, warp, lane);
  double* mine = partial + ((size_t)s * chunks + chunk) * nt * 64;
  for (int e = tid; e < nt * 64; e += kThreads) mine[e] = tiles[e];
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned old = atomicAdd(counters + s, 1u);
    is_last = (old == (unsigned)chunks - 1u);
    if (is_last) counters[s] = 0u;
  }
  __syncthreads();
  if (!is_last) continue;
  __threadfence();

  // ---- sum the chunk partials in chunk order (loads issued eight at a time) into L ----
  const double* src = partial + (size_t)s * chunks * nt * 64;
  for (int e = tid; e < nt * 64; e += kThreads) {
    double v = 0.0;
    int q = 0;
    for (; q + 8 <= chunks; q += 8) {
      double t[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) t[u] = __ldcg(src + (size_t)(q + u) * nt * 64 + e);
#pragma unroll
      for (int u = 0; u < 8; ++u) v += t[u];
    }
    for (; q < chunks; ++q) v += __ldcg(src + (size_t)q * nt * 64 + e);
    const int T = e >> 6, w = e & 63;
    Lm[(tile_bi[T] * 8 + (w >> 3)) * LR + tile_bj[T] * 8 + (w & 7)] = v;
  }
  if (tid < DAD_MAX_RANK) dead_row[tid] = 0;
  if (tid == 0) need2_s = 0;
  __syncthreads();
  if (tid < rp) {
    f.diag0[tid] = Lm[tid * LR + tid];
    const bool second = pass == 1 && tid < r;
    f.p1[tid] = second ? ratio1[(size_t)s * r + tid] : 1.0;
    f.bar[tid] = second ? tol * tol : -1.0;
  }
  __syncthreads();
  if (pass == 0) {
    cholesky_panels<true>(Lm, LR, rp, f, Dblk, status, tid);
  } else {
    cholesky_panels<false>(Lm, LR, rp, f, Dblk, status, tid);
  }
  build_m(tiles, Lm, LR, rp, nt, f, tile_bi, tile_bj, tid);
  double* Ms = Mt + (size_t)s * nt * 64;
  for (int e = tid; e < nt * 64; e += kThreads) Ms[e] = tiles[e];
  if (tid < r) {
    if (pass == 0) {
      const double o = f.diag0[tid];
      ratio1[(size_t)s * r + tid] = (f.dead_row[tid] || !(o > 0.0)) ? 0.0 : f.piv_out[tid] / o;
    }
    dead[(size_t)s * r + tid] = f.dead_row[tid];
  }
  if (tid == 0 && pass == 0) need2[s] = need2_s;
  }
}

template <int NB>
__global__ void __launch_bounds__(kThreads, 3)
orth_split_apply_kernel(float* __restrict__ G, int S, int r, int64_t h, int pass, const double* __restrict__ Mt,
                        const int* __restrict__ need2, float* __restrict__ out32, __nv_bfloat16* __restrict__ planes,
                        int plane_rows) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int rp = NB * 8, nt = NB * (NB + 1) / 2;
  const int chunk = blockIdx.x;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const MmaGeom geo = mma_geom(r, kApplyW);
  float* slab = reinterpret_cast<float*>(smem_raw);
  double* tiles = reinterpret_cast<double*>(smem_raw + geo.off_tiles);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t c0 = (int64_t)chunk * kApplyW;
  for (int s = blockIdx.y; s < S; s += gridDim.y) {  // second pass: a small grid walks over the sites
  if (pass == 1 && need2[s] == 0) continue;
  __syncthreads();
  float* Gs = G + (int64_t)s * r * h;
  const double* Ms = Mt + (size_t)s * nt * 64;
  for (int e = tid; e < nt * 64; e += kThreads) tiles[e] = Ms[e];
  load_slab(slab, Gs, r, rp, h, c0, kApplyW, geo.Wp, tid);
  __syncthreads();
  solve_slab(slab, tiles, NB, kApplyW, geo.Wp, warp, lane);
  __syncthreads();
  store_slab(slab, Gs, s, r, h, c0, kApplyW, geo.Wp, out32, planes, plane_rows, tid);
  }
}

template <int NB>
static cudaError_t launch_orth_mma(float* G, int S, int r, int64_t h, int C, int W, double tol, int* status, float* out32,
                                   __nv_bfloat16* planes, int plane_rows, size_t smem, cudaStream_t st) {
  auto kernel = orth_mma_kernel<NB>;
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
  if (timed) timing_mark("orth_mma", st, true);
  err = cudaLaunchKernelEx(&cfg, kernel, G, r, h, C, W, tol, status, out32, planes, plane_rows);
  if (timed) timing_mark("orth_mma", st, false);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return err;
}

template <int NB>
static cudaError_t launch_orth_split(float* G, int S, int r, int64_t h, double tol, double* partial, double* Mt,
                                     double* ratio1, unsigned char* dead, int* need2, unsigned* counters, int* status,
                                     float* out32, __nv_bfloat16* planes, int plane_rows, cudaStream_t st) {
  const MmaGeom geo = mma_geom(r, kFactorW), geo_a = mma_geom(r, kApplyW);
  const int chunks = (int)ceil_div(h, kFactorW), chunks_a = (int)ceil_div(h, kApplyW);
  const size_t lbytes = sizeof(double) * (size_t)geo.rp * geo.LR;
  const size_t smem_f =
      (lbytes > geo.off_tiles ? lbytes : geo.off_tiles) + sizeof(double) * (64 * (size_t)geo.nt + 5 * (size_t)geo.rp);
  const size_t smem_a = geo_a.off_tiles + sizeof(double) * 64 * (size_t)geo_a.nt;
  cudaError_t err =
      cudaFuncSetAttribute(orth_split_factor_kernel<NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_f);
  if (err != cudaSuccess) return err;
  err = cudaFuncSetAttribute(orth_split_apply_kernel<NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_a);
  if (err != cudaSuccess) return err;
  for (int pass = 0; pass < 2; ++pass) {
    // second pass: about two CTAs per SM in all, each walking over the sites
    const int rows_f = pass == 0 ? S : (int)std::max<int64_t>(1, std::min<int64_t>(S, 2 * 148 / chunks));
    const int rows_a = pass == 0 ? S : (int)std::max<int64_t>(1, std::min<int64_t>(S, 2 * 148 / chunks_a));
    DAD_LAUNCH(err, "orth_split_factor", (orth_split_factor_kernel<NB>), dim3((unsigned)chunks, (unsigned)rows_f), kThreads,
               smem_f, st, G, S, r, h, chunks, pass, tol, partial, Mt, ratio1, dead, need2, counters, status);
    DAD_LAUNCH(err, "orth_split_apply", (orth_split_apply_kernel<NB>), dim3((unsigned)chunks_a, (unsigned)rows_a), kThreads,
               smem_a, st, G, S, r, h, pass, Mt, need2, out32, planes, plane_rows);
  }
  return err;
}

// Whether the one-launch kernel takes this shape (the slab of a CTA of the largest admissible cluster has to fit).
bool orth_mma_fits(int r, int64_t h) {
  if (r < 1 || r > DAD_MAX_RANK || h > (int64_t)1 << 30) return false;
  return mma_cluster_size(r, h, 1 << 20) > 0;
}

// Whether the two-launch arrangement is the better one: more CTAs than fit on the GPU at once at a rank where every
// CTA of the one-launch kernel would repeat a long factorisation -- and its scratch fits the workspace regions that
// are sized for the multi-kernel Cholesky-QR (S x ceil(h / 64) x r x r doubles of partials, S x r x r of factor).
bool orth_split_preferred(int r, int64_t h, int S) {
  if (r < 32 || r > DAD_MAX_RANK) return false;
  const MmaGeom geo = mma_geom(r, kFactorW);
  if ((size_t)geo.nt * 64 > (size_t)r * r) return false;
  const int C = mma_cluster_size(r, h, S);
  return C == 0 || (int64_t)S * C > 2 * 148;
}

// Cholesky-QR (one or two passes, decided on the device) of the rows of G (S x r x h fp32, in place), one launch.
cudaError_t orth_mma(float* G, int S, int r, int64_t h, double tol, int* status, float* out32, __nv_bfloat16* planes,
                     int plane_rows, cudaStream_t st) {
  const int C = mma_cluster_size(r, h, S);
  if (C == 0) return cudaErrorInvalidValue;
  const int W = columns_per_cta(h, C);
  const size_t smem = mma_geom(r, W).total;
#define DAD_ORTH_MMA_CASE(NB) \
  case NB: return launch_orth_mma<NB>(G, S, r, h, C, W, tol, status, out32, planes, plane_rows, smem, st)
  switch ((r + 7) / 8) {
    DAD_ORTH_MMA_CASE(1);
    DAD_ORTH_MMA_CASE(2);
    DAD_ORTH_MMA_CASE(3);
    DAD_ORTH_MMA_CASE(4);
    DAD_ORTH_MMA_CASE(5);
    DAD_ORTH_MMA_CASE(6);
    DAD_ORTH_MMA_CASE(7);
    DAD_ORTH_MMA_CASE(8);
  }
#undef DAD_ORTH_MMA_CASE
  return cudaErrorInvalidValue;
}

// The same in two launches per pass (four in all; those of the second pass return at once for sites that do not need it).
cudaError_t orth_split(float* G, int S, int r, int64_t h, double tol, double* partial, double* Mt, double* ratio1,
                       unsigned char* dead, int* need2, unsigned* counters, int* status, float* out32,
                       __nv_bfloat16* planes, int plane_rows, cudaStream_t st) {
#define DAD_ORTH_SPLIT_CASE(NB)                                                                                       \
  case NB:                                                                                                            \
    return launch_orth_split<NB>(G, S, r, h, tol, partial, Mt, ratio1, dead, need2, counters, status, out32, planes, \
                                 plane_rows, st)
  switch ((r + 7) / 8) {
    DAD_ORTH_SPLIT_CASE(4);
    DAD_ORTH_SPLIT_CASE(5);
    DAD_ORTH_SPLIT_CASE(6);
    DAD_ORTH_SPLIT_CASE(7);
    DAD_ORTH_SPLIT_CASE(8);
  }
#undef DAD_ORTH_SPLIT_CASE
  return cudaErrorInvalidValue;
}

}  // namespace dad

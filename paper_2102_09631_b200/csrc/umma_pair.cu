// One application of half the operator of Eq. "reduced_iter" in ONE launch, for sites of a few MB (bf16 inputs):
//
//     Z = (X1 F^T)^T X2          X1: N x h1, X2: N x h2 (the same N rows of one site), F: r x h1, Z: r x h2
//
// i.e. the pair  Y = D G^T, Z = Y^T A   (X1 = D, X2 = A)  or  W = A Z^T, G~ = W^T D   (X1 = A, X2 = D)  of Algorithm 2's
// structured power iteration, which the streaming pipeline runs as two launches with Y^T handed on through global
// memory.  Here a CTA owns 128 rows of a site:
//
//   phase A  Y[128 x r] = X1[rows] F^T: X1 tiles (K-major) and the hi/lo planes of F stream through the stage ring,
//            one MMA of width 2 rp per k-step multiplies by both planes, accumulator in tensor memory;
//   phase B  the four epilogue warps read Y, add the two halves, split it into bf16 hi + lo and lay it out in shared
//            memory exactly as a TMA load of Y^T planes would (K-major rows of 128 bytes, 128-byte swizzle);
//   phase C  for every 128-column chunk of X2: D2[128 columns x 2 rp] = X2[rows, chunk]^T Y (X2 tiles M/N-major
//            through the same ring), one accumulator per chunk, all of them side by side in tensor memory;
//   phase D  the epilogue drains chunk after chunk while the MMAs of later chunks run, adds the hi and lo halves and
//            stores the CTA's partial r x 128 block;
//   phase E  the sum over the row blocks of a site.  The CTAs of up to 8 consecutive row blocks form a thread-block
//            cluster; after the cluster's hardware barrier CTA q of the cluster sums the chunks q, q + size, ... over
//            the cluster's blocks in row-block order, so the work is dealt out by rank, not by who happens to finish
//            last (with arrival counters alone one slow CTA ended up summing every chunk of its site: 20-30 us).
//            A site of more row blocks than one cluster holds adds a second, light step: the cluster's sums are
//            stored, an arrival counter per (site, chunk) finds the last cluster, and that one adds the clusters'
//            sums in cluster order.  Every sum has a fixed order: two runs are bit-identical.
//
// Y never leaves the SM, and a launch, its pipeline ramp and its tail are paid once per pair.  Roles, bounded waits and
// teardown as in umma_kernel; the cluster barrier is a hardware barrier that every thread reaches whatever happened
// before it.
//
// Measured on one encoder layer (d = 512, FFN 2048, 4 sites of 2048 rows, r = 10; per launch, caches as a training step
// leaves them): 24 us for the four stacked 512 -> 512 projections (256 CTAs; the two streaming kernels: 8 + 13 us),
// 29 us for X1 2048 wide and 39 us for X2 2048 wide (64 CTAs; 14 + 11 and 7 + 13 us).  What bounds all of them is the
// same thing: a CTA pulls about 40 GB/s from L2 / HBM, a site of 2048 rows is 16 row blocks, and 64 CTAs on 148 SMs
// cannot stream faster than 2.5 TB/s whatever they fuse, while the second streaming kernel re-deals the same bytes over
// 128 CTAs.  So the paired form is an OPTION (dad_pair_enable), off by default, taken only while the row blocks of a
// call are few (the partial blocks are r / 32 of the bytes streamed).
#include "common.cuh"
#include "umma.cuh"

namespace dad {
using namespace sm100;

constexpr int kPairMaxChunks = 16;
constexpr int kPairMaxCluster = 8;

struct PairParams {
  int n_rows;        // N
  int h2;            // columns of X2 (= of Z)
  int r;
  int kb_a;          // 64-wide blocks of h1
  int chunks;        // 128-wide chunks of h2
  int nbp;           // row blocks per site, padded to a multiple of the cluster size (= gridDim.x)
  int cs;            // cluster size
  uint32_t tmem_cols;
  float* out_f32;    // [S][r][ld_out] or null
  float* out2_f32;   // second copy, same layout, or null
  int64_t ld_out;
  __nv_bfloat16* out_planes;  // [S][2][plane_rows][ld_planes] or null
  int64_t ld_planes;
  int plane_rows;
  float* partial;    // [S][chunks][nbp][r][128] block sums
  float* partial2;   // [S][chunks][nbp / cs][r][128] cluster sums (sites of more than one cluster)
  unsigned* counters;  // [S][chunks], zero on entry, zero again on exit
  int* status;
  uint32_t wait_limit;
};

__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <int RP, int STAGES>
__global__ void __launch_bounds__(192)
umma_pair_kernel(const __grid_constant__ CUtensorMap tmX1, const __grid_constant__ CUtensorMap tmF,
                 const __grid_constant__ CUtensorMap tmX2, const PairParams p) {
  constexpr int X_BYTES = 128 * 64 * 2;          // X1 tile [128 rows][64 k] or X2 tile 2 x [64 rows][64 columns]
  constexpr int F_BYTES = 2 * RP * 128;          // hi and lo plane, [RP rows][64 k] each
  constexpr int SLOT_BYTES = X_BYTES + F_BYTES;
  constexpr uint32_t IDESC_A = instr_desc(128, 2 * RP, false, false);
  constexpr uint32_t IDESC_C = instr_desc(128, 2 * RP, true, false);
  static_assert(F_BYTES % 1024 == 0, "operand tiles start on 1024-byte boundaries");

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* ysm = smem + (size_t)STAGES * SLOT_BYTES;  // Y planes: two k-blocks (rows 0-63, 64-127) of [2 RP][64 k]
  __shared__ uint64_t full_bar[STAGES], empty_bar[STAGES], y_full, y_smem, chunk_bar[kPairMaxChunks], flush_bar;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag, issued_s, flush_s, epi_bad, is_last_s[kPairMaxChunks];
  const uint32_t wlim = p.wait_limit ? p.wait_limit : kWaitLimit;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int blk = blockIdx.x, site = blockIdx.z;
  const int row0 = blk * 128;  // padded blocks (row0 >= N) load zeros and contribute zero blocks
  const int n_items = p.kb_a + 2 * p.chunks;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(&y_full, 1);
    mbar_init(&y_smem, 128);
    for (int c = 0; c < kPairMaxChunks; ++c) mbar_init(&chunk_bar[c], 1);
    mbar_init(&flush_bar, 1);
    abort_flag = 0;
    issued_s = 0;
    flush_s = 0;
    epi_bad = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(&tmem_base_s, p.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  volatile int* abortp = &abort_flag;

  // everything above touched only this CTA's own shared and tensor memory (see umma_kernel)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  const int q = warp & 3;
  const int row = q * 32 + lane;  // epilogue threads: row of the block in phase B, column of the chunk afterwards
  const int r = p.r;

  if (warp == 0) {
    if (lane == 0) {
      prefetch_tmap(&tmX1);
      prefetch_tmap(&tmF);
      prefetch_tmap(&tmX2);
      for (int g = 0; g < n_items; ++g) {
        const int stage = g % STAGES;
        const uint32_t ph = (uint32_t)(g / STAGES) & 1u;
        if (!mbar_wait(&empty_bar[stage], ph ^ 1u, abortp, wlim)) break;
        uint8_t* dst = smem + (size_t)stage * SLOT_BYTES;
        if (g < p.kb_a) {
          mbar_expect_tx(&full_bar[stage], SLOT_BYTES);
          tma_load_3d(dst, &tmX1, &full_bar[stage], g * 64, row0, site);
          tma_load_3d(dst + X_BYTES, &tmF, &full_bar[stage], g * 64, 0, site * 2);
          tma_load_3d(dst + X_BYTES + RP * 128, &tmF, &full_bar[stage], g * 64, 0, site * 2 + 1);
        } else {
          const int c = (g - p.kb_a) >> 1, kb = (g - p.kb_a) & 1;
          mbar_expect_tx(&full_bar[stage], X_BYTES);
          tma_load_3d(dst, &tmX2, &full_bar[stage], c * 128, row0 + kb * 64, site);
          tma_load_3d(dst + 8192, &tmX2, &full_bar[stage], c * 128 + 64, row0 + kb * 64, site);
        }
        issued_s = g + 1;
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      bool go = true;
      int g = 0;
      for (; g < p.kb_a; ++g) {  // phase A
        const int stage = g % STAGES;
        const uint32_t ph = (uint32_t)(g / STAGES) & 1u;
        if (!mbar_wait(&full_bar[stage], ph, abortp, wlim)) {
          go = false;
          break;
        }
        tc_fence_after();
        const uint32_t a_addr = smem_u32(smem + (size_t)stage * SLOT_BYTES);
        const uint32_t b_addr = a_addr + X_BYTES;
#pragma unroll
        for (int k16 = 0; k16 < 4; ++k16)
          umma_bf16(tmem_base, desc_k_major(a_addr, k16), desc_k_major(b_addr, k16), IDESC_A, (g | k16) != 0 ? 1u : 0u);
        umma_commit(&empty_bar[stage]);
      }
      if (go) {
        umma_commit(&y_full);
        go = mbar_wait(&y_smem, 0u, abortp, wlim);  // Y is in shared memory as bf16 planes, its accumulator is free
        tc_fence_after();
      }
      const uint32_t y_addr = smem_u32(ysm);
      for (int c = 0; go && c < p.chunks; ++c) {  // phase C
        const uint32_t acc = tmem_base + (uint32_t)(c * 2 * RP);
        for (int kb = 0; kb < 2; ++kb, ++g) {
          const int stage = g % STAGES;
          const uint32_t ph = (uint32_t)(g / STAGES) & 1u;
          if (!mbar_wait(&full_bar[stage], ph, abortp, wlim)) {
            go = false;
            break;
          }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem + (size_t)stage * SLOT_BYTES);
          const uint32_t b_addr = y_addr + (uint32_t)kb * F_BYTES;
#pragma unroll
          for (int k16 = 0; k16 < 4; ++k16)
            umma_bf16(acc, desc_mn_major(a_addr, k16), desc_k_major(b_addr, k16), IDESC_C, (kb | k16) != 0 ? 1u : 0u);
          umma_commit(&empty_bar[stage]);
        }
        if (go) umma_commit(&chunk_bar[c]);
      }
      if (*abortp) {  // giving up: the teardown waits on this for the MMAs issued so far before tensor memory is freed
        umma_commit(&flush_bar);
        flush_s = 1;
      }
    }
  } else {
    const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
    // ---- phase B: Y -> bf16 hi / lo planes in shared memory, the K-major B operand of phase C ----
    if (!mbar_wait(&y_full, 0u, abortp, wlim)) epi_bad = 1;
    asm volatile("bar.sync 1, 128;" ::: "memory");  // the four warps go on, or stop, together
    const bool alive = *reinterpret_cast<volatile int*>(&epi_bad) == 0;
    if (alive) {
      tc_fence_after();
      const int kb = row >> 6, kk = row & 63;
      uint8_t* tile = ysm + kb * F_BYTES;
#pragma unroll 1
      for (int c16 = 0; c16 < RP / 16; ++c16) {
        float v[16], w[16];
        tmem_ld16(lane_base + c16 * 16, v);
        tmem_ld16(lane_base + RP + c16 * 16, w);  // the product with the lo plane of F
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int j = c16 * 16 + i;
          const float y = j < r ? v[i] + w[i] : 0.f;
          const __nv_bfloat16 hi = __float2bfloat16_rn(y);
          const __nv_bfloat16 lo = __float2bfloat16_rn(y - __bfloat162float(hi));
          // element (n, k) of a K-major tile: row n at n * 128 bytes, 16-byte pieces XOR-swizzled with n % 8
          const int off = (((kk >> 3) ^ (j & 7)) << 4) + ((kk & 7) << 1);
          *reinterpret_cast<__nv_bfloat16*>(tile + j * 128 + off) = hi;
          *reinterpret_cast<__nv_bfloat16*>(tile + (RP + j) * 128 + off) = lo;  // (RP + j) % 8 == j % 8
        }
      }
      fence_async_proxy();  // the tensor cores read shared memory through the asynchronous proxy
      tc_fence_before();
      mbar_arrive(&y_smem);
      // ---- phase D: this block's r x 128 sums, chunk after chunk ----
#pragma unroll 1
      for (int c = 0; c < p.chunks; ++c) {
        if (!mbar_wait(&chunk_bar[c], 0u, abortp, wlim)) break;
        tc_fence_after();
        float* mine = p.partial + ((((int64_t)site * p.chunks + c) * p.nbp + blk) * r) * 128 + row;
#pragma unroll
        for (int c16 = 0; c16 < RP / 16; ++c16) {
          float v[16], w[16];
          tmem_ld16(lane_base + c * 2 * RP + c16 * 16, v);
          tmem_ld16(lane_base + c * 2 * RP + RP + c16 * 16, w);
#pragma unroll
          for (int i = 0; i < 16; ++i)
            if (c16 * 16 + i < r) mine[(c16 * 16 + i) * 128] = v[i] + w[i];
        }
      }
    }
  }
  // ---- phase E: the sum over the row blocks of the site ----
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // every CTA of the cluster has stored its blocks (or has given up): all threads, unconditionally
  if (warp >= 2 && abort_flag == 0) {
    const int cs = p.cs, qc = blk % cs, cl = blk / cs, ncl = p.nbp / cs;
    auto emit = [&](int c, const float (&z)[RP]) {  // column c * 128 + row of Z, all r rows
      const int64_t gm = (int64_t)c * 128 + row;
      if (gm >= p.h2) return;
#pragma unroll
      for (int j = 0; j < RP; ++j) {
        if (j < r) {
          if (p.out_f32) p.out_f32[((int64_t)site * r + j) * p.ld_out + gm] = z[j];
          if (p.out2_f32) p.out2_f32[((int64_t)site * r + j) * p.ld_out + gm] = z[j];
          if (p.out_planes) {
            const __nv_bfloat16 hi = __float2bfloat16_rn(z[j]);
            const __nv_bfloat16 lo = __float2bfloat16_rn(z[j] - __bfloat162float(hi));
            p.out_planes[(((int64_t)site * 2 + 0) * p.plane_rows + j) * p.ld_planes + gm] = hi;
            p.out_planes[(((int64_t)site * 2 + 1) * p.plane_rows + j) * p.ld_planes + gm] = lo;
          }
        }
      }
    };
    auto sum_blocks = [&](const float* src, int count, float (&z)[RP]) {  // `count` consecutive r x 128 blocks, in order
#pragma unroll
      for (int j = 0; j < RP; ++j) z[j] = 0.f;
#pragma unroll 4
      for (int b = 0; b < count; ++b) {
#pragma unroll
        for (int j = 0; j < RP; ++j)
          if (j < r) z[j] += __ldcg(src + ((int64_t)b * r + j) * 128);
      }
    };
    int owned = 0;
#pragma unroll 1
    for (int c = qc; c < p.chunks; c += cs, ++owned) {
      float z[RP];
      sum_blocks(p.partial + ((((int64_t)site * p.chunks + c) * p.nbp + (int64_t)cl * cs) * r) * 128 + row, cs, z);
      if (ncl == 1) {
        emit(c, z);
      } else {
        float* dst = p.partial2 + ((((int64_t)site * p.chunks + c) * ncl + cl) * r) * 128 + row;
#pragma unroll
        for (int j = 0; j < RP; ++j)
          if (j < r) dst[j * 128] = z[j];
      }
    }
    if (ncl > 1) {
      __threadfence();
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (row < owned) {  // one arrival per owned chunk, all of them in flight at once
        unsigned* ctr = p.counters + (int64_t)site * p.chunks + qc + row * cs;
        const unsigned old = atomicAdd(ctr, 1u);
        const int is_last = (old == (unsigned)ncl - 1u);
        if (is_last) *ctr = 0u;
        is_last_s[row] = is_last;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      bool fenced = false;
#pragma unroll 1
      for (int t = 0; t < owned; ++t) {
        if (!is_last_s[t]) continue;
        if (!fenced) __threadfence();  // the other clusters' sums, stored before their arrivals
        fenced = true;
        const int c = qc + t * cs;
        float z[RP];
        sum_blocks(p.partial2 + ((((int64_t)site * p.chunks + c) * ncl) * r) * 128 + row, ncl, z);
        emit(c, z);
      }
    }
  }

  // ---- teardown ----
  __syncthreads();
  if (abort_flag) {
    if (threadIdx.x == 0) {
      const int issued = issued_s;
      const int first = issued > STAGES ? issued - STAGES : 0;
      for (int i = first; i < issued; ++i) {  // copies already issued into this CTA's shared memory
        uint64_t* bar = &full_bar[i % STAGES];
        const uint32_t ph = (uint32_t)(i / STAGES) & 1u;
        for (uint32_t t = 0; t < kWaitLimit && !mbar_try_wait(bar, ph); ++t) {
        }
      }
      if (flush_s) {  // MMAs already issued
        for (uint32_t t = 0; t < kWaitLimit && !mbar_try_wait(&flush_bar, 0u); ++t) {
        }
      }
      if (p.status) *p.status = (int)DAD_ERR_TIMEOUT;
    }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, p.tmem_cols);
  }
}

// ---- host side ---------------------------------------------------------------------------------
// Cluster size and padded row-block count for N rows per site: the largest cluster of 8, 4, 2 or 1 CTAs whose padding
// (CTAs that stream zeros) stays within an eighth of the real blocks.
static void pair_geometry(int64_t N, int* cs_out, int* nbp_out) {
  const int64_t nb = ceil_div(N, 128);
  for (int cs = kPairMaxCluster; cs >= 1; cs /= 2) {
    const int64_t nbp = ceil_div(nb, cs) * cs;
    if (cs == 1 || nbp - nb <= nb / 8) {
      *cs_out = cs;
      *nbp_out = (int)nbp;
      return;
    }
  }
}

// Whether one launch takes the pair for this shape: the accumulators of all chunks of X2 have to fit the 512 columns of
// tensor memory beside one another, and the call has to be small -- at most four row blocks per SM -- since every row
// block leaves an r x h2 partial block behind (r / 32 of the bytes it streams from X2).
bool umma_pair_fits(int S, int64_t N, int64_t h2, int r) {
  const int rp = umma_rank_pad(r);
  if (rp > 32) return false;
  const int64_t chunks = ceil_div(h2, 128);
  if (chunks > kPairMaxChunks || chunks * 2 * rp > 512) return false;
  int cs, nbp;
  pair_geometry(N, &cs, &nbp);
  return (int64_t)S * nbp <= 4 * 148;
}

size_t umma_pair_partial_bytes(int S, int64_t N, int64_t h2, int r) {
  int cs, nbp;
  pair_geometry(N, &cs, &nbp);
  const size_t block = (size_t)S * (size_t)ceil_div(h2, 128) * (size_t)r * 128 * sizeof(float);
  return block * (size_t)nbp + block * (size_t)(nbp / cs);
}

template <int RP, int STAGES>
static cudaError_t launch_pair(const CUtensorMap& tmX1, const CUtensorMap& tmF, const CUtensorMap& tmX2, const PairParams& p,
                               dim3 grid, cudaStream_t st) {
  constexpr size_t smem = (size_t)STAGES * (128 * 64 * 2 + 2 * RP * 128) + 4 * RP * 128 + 1024;
  auto kernel = umma_pair_kernel<RP, STAGES>;
  cudaError_t err = cudaSuccess;
  static FirstUse first;
  if (first.on_this_device()) {
    err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) {
      first.forget();
      return err;
    }
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(192, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = (unsigned)p.cs;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  const bool timed = g_timing.load(std::memory_order_relaxed);
  if (timed) timing_mark("pair_tc", st, true);
  err = cudaLaunchKernelEx(&cfg, kernel, tmX1, tmF, tmX2, p);
  if (timed) timing_mark("pair_tc", st, false);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return err;
}

// Z <- (X1 F^T)^T X2.  tmX1: X1 as (h1, N, S) with box 64 x 128; tmF: factor planes as (h1, rp, 2S) with box 64 x rp;
// tmX2: X2 as (h2, N, S) with box 64 x 64.  `partial`: umma_pair_partial_bytes; `counters` (S * chunks words) must be
// zero and are left zero.
cudaError_t umma_pair(const CUtensorMap& tmX1, const CUtensorMap& tmF, const CUtensorMap& tmX2, int S, int64_t N, int64_t h1,
                      int64_t h2, int r, float* out, float* out2, __nv_bfloat16* planes, int64_t ld_planes, float* partial,
                      unsigned* counters, int* status, cudaStream_t st) {
  const int rp = umma_rank_pad(r);
  PairParams p{};
  p.n_rows = (int)N;
  p.h2 = (int)h2;
  p.r = r;
  p.kb_a = (int)ceil_div(h1, 64);
  p.chunks = (int)ceil_div(h2, 128);
  pair_geometry(N, &p.cs, &p.nbp);
  uint32_t cols = 32;
  while (cols < (uint32_t)(p.chunks * 2 * rp)) cols *= 2;
  p.tmem_cols = cols;
  p.out_f32 = out;
  p.out2_f32 = out2;
  p.ld_out = h2;
  p.out_planes = planes;
  p.ld_planes = ld_planes;
  p.plane_rows = rp;
  p.partial = partial;
  p.partial2 = partial + (size_t)S * p.chunks * p.nbp * r * 128;
  p.counters = counters;
  p.status = status;
  dim3 grid((unsigned)p.nbp, 1, (unsigned)S);
  // One CTA per SM with everything it streams in flight while the launch fits the GPU in one wave; two shallower ones
  // per SM (tensor memory permitting) beyond that.
  const bool deep = (int64_t)p.nbp * S <= 148 || cols > 256;
  if (rp == 16) {
    if (deep) return launch_pair<16, 8>(tmX1, tmF, tmX2, p, grid, st);
    return launch_pair<16, 4>(tmX1, tmF, tmX2, p, grid, st);
  }
  if (deep) return launch_pair<32, 8>(tmX1, tmF, tmX2, p, grid, st);
  return launch_pair<32, 4>(tmX1, tmF, tmX2, p, grid, st);
}

}  // namespace dad

// Tensor-core (tcgen05 / TMEM) kernel family for bf16 inputs.  One kernel template computes a
// 128 x BN tile  D[m][n] = sum_k Aop[m][k] * Bop[n][k]  with fp32 accumulation in tensor memory,
// operands staged by TMA into 128-byte-swizzled shared memory behind an mbarrier ring:
//
//   rows_dot  Y = X F^T     (Eq. "reduced_iter", the products D g and A z of a power iteration):
//             A operand = X tile, K-major (row-major X, contraction along its columns);
//             B operand = the r x h factor as two bf16 planes (hi + lo split of fp32), K-major.
//             Epilogue writes Y transposed as bf16 hi/lo planes, the layout cols_acc reads.
//   cols_acc  Z = Y^T X     (the products A^T v and D^T w):
//             A operand = X tile read as its transpose, M/N-major (contraction along rows);
//             B operand = Y^T planes, K-major.  Rows are split over CTAs; partial tiles are summed
//             in split order by the last CTA to arrive (deterministic).  Epilogue writes Z as fp32
//             and, if asked, as bf16 hi/lo planes for the next rows_dot.
//   gemm_tn   C = X^T Y     (the dAD gradient sum_s A_s^T D_s of Sec. 3.2 and the reconstruction
//             Pcat^T Qcat of Algorithm 1): both operands M/N-major, optional split over the
//             contraction with the same ordered reduction.
//
// Warp roles (192 threads): warp 0 issues TMA loads, warp 1 owns tensor memory and issues the
// MMAs, warps 2-5 drain the accumulator (each warp reads its own quarter of the 128 TMEM lanes).
// Every mbarrier wait is bounded; if one runs out the CTA raises an abort flag, all roles leave
// their loops, outstanding copies are waited for (bounded), tensor memory is freed, and the status
// word in the workspace is set to DAD_ERR_TIMEOUT.
#include <cstdlib>

#include "common.cuh"
#include "umma.cuh"

namespace dad {
using namespace sm100;

enum : int { EPI_YT = 0, EPI_Z = 1, EPI_C = 2 };

// 256 x 256 dense-product kernel: contraction rows per stage, stages (3 x 64 KB of shared memory), and the
// shortest contraction it is used for (below that the output write dominates and 128-row tiles fill more SMs).
constexpr int kGemm256BK = 64;
constexpr int kGemm256Stages = 3;
constexpr int kGemm256MinRows = 4096;

struct UmmaParams {
  int m_extent;      // valid rows of D: N (rows_dot), h (cols_acc), h_in (gemm_tn)
  int n_extent;      // valid columns of D: r, or h_out
  int k_blocks;      // 64-wide blocks of the contraction (per batch entry)
  int kb_per_split;
  int splits;
  int kb_per_site;   // gemm_tn over sites: blocks per site (site = block / kb_per_site); 0 = batch from blockIdx.z
  int rem_ctas;      // 256 x 256 kernel: CTAs that each take the last blocks of the contraction of several tiles
  int tiles_m, tiles_n;  // 256 x 256 kernel: tile grid (its launch is one-dimensional)
  float* out_f32;    // EPI_Z: [batch][r][ld_out];  EPI_C: [m][ld_out]
  float* out2_f32;   // EPI_Z: optional second copy, same layout
  int64_t ld_out;
  int64_t out_batch_stride;   // EPI_C: elements between the outputs of consecutive batch entries
  __nv_bfloat16* out_planes;  // EPI_YT / EPI_Z: [batch][2][plane_rows][ld_planes] (hi plane, lo plane), or null
  int64_t ld_planes;
  int plane_rows;    // rows per plane (r rounded up to the MMA width); rows >= r are never written
  float* partial;    // split partial tiles [tile][split][128][BN]
  unsigned* counters;
  int* status;
  int batch_count;      // persistent dense-product kernels and the 256 x 256 kernel: products in the launch
  int sites_per_product;  // 256 x 256 kernel: sites of each product (product g reads sites g * sites_per_product ...)
  int tma_store;        // EPI_C without a split contraction: the tile leaves through shared memory and TMA stores (tmC)
  uint32_t wait_limit;  // polls a bounded wait may take; 0 = kWaitLimit
  int expect_extra_kb;  // self-test only: the MMA role waits for this many blocks more than the producer loads
};

template <int BN, bool A_MN, bool B_MN, int TERMS, int EPI, int STAGES>
__global__ void __launch_bounds__(192)
umma_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmC, const UmmaParams p) {
  constexpr int A_BYTES = 128 * 64 * 2;
  constexpr int B_BYTES = B_MN ? (BN / 64) * 8192 : TERMS * BN * 128;
  constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  // The hi and lo planes of a K-major B operand lie one after the other in a stage, so one MMA of width
  // TERMS * BN multiplies A by both at once (A is read from shared memory once per k-step); the two halves
  // of the accumulator are added in the epilogue.
  constexpr int MMA_N = B_MN ? BN : TERMS * BN;
  constexpr uint32_t TMEM_COLS = MMA_N < 32 ? 32 : MMA_N;
  constexpr uint32_t IDESC = instr_desc(128, MMA_N, A_MN, B_MN);
  static_assert(!B_MN || (BN % 64 == 0 && TERMS == 1), "M/N-major B comes in 64-wide chunks, one term");

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ uint64_t full_bar[STAGES], empty_bar[STAGES], accum_bar, flush_bar;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag, issued_s, last_flag, flush_s;
  const uint32_t wlim = p.wait_limit ? p.wait_limit : kWaitLimit;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m_tile = blockIdx.x;
  const int n_tile = blockIdx.y / p.splits, split = blockIdx.y % p.splits;
  const int batch = blockIdx.z;
  const int m0 = m_tile * 128, n0 = n_tile * BN;
  const int kb0 = split * p.kb_per_split;
  const int kb1 = (kb0 + p.kb_per_split < p.k_blocks) ? kb0 + p.kb_per_split : p.k_blocks;
  const int nkb = kb1 > kb0 ? kb1 - kb0 : 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(&accum_bar, 1);
    mbar_init(&flush_bar, 1);
    abort_flag = 0;
    issued_s = 0;
    last_flag = 0;
    flush_s = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(&tmem_base_s, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  volatile int* abortp = &abort_flag;

  // Programmatic dependent launch: everything above touched only this CTA's own shared and tensor
  // memory, so it may overlap the tail of the previous kernel in the stream.  From here on the kernel
  // reads what earlier kernels wrote (and overwrites what they read): wait for them to finish.  The
  // next kernel in the stream is allowed to start its own set-up right away.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (warp == 0) {
    if (lane == 0) {
      prefetch_tmap(&tmA);
      prefetch_tmap(&tmB);
      int i = 0;
      for (; i < nkb; ++i) {
        const int stage = i % STAGES;
        const uint32_t ph = (uint32_t)(i / STAGES) & 1u;
        if (!mbar_wait(&empty_bar[stage], ph ^ 1u, abortp, wlim)) break;
        mbar_expect_tx(&full_bar[stage], STAGE_BYTES);
        uint8_t* a_dst = smem + (size_t)stage * STAGE_BYTES;
        uint8_t* b_dst = a_dst + A_BYTES;
        const int kb = kb0 + i;
        int kcoord = kb * 64, bz = batch;
        if (p.kb_per_site > 0) {
          bz = kb / p.kb_per_site;
          kcoord = (kb % p.kb_per_site) * 64;
        }
        if constexpr (A_MN) {
          tma_load_3d(a_dst, &tmA, &full_bar[stage], m0, kcoord, bz);
          tma_load_3d(a_dst + 8192, &tmA, &full_bar[stage], m0 + 64, kcoord, bz);
        } else {
          tma_load_3d(a_dst, &tmA, &full_bar[stage], kcoord, m0, bz);
        }
        if constexpr (B_MN) {
#pragma unroll
          for (int c = 0; c < BN / 64; ++c) tma_load_3d(b_dst + c * 8192, &tmB, &full_bar[stage], n0 + c * 64, kcoord, bz);
        } else {
#pragma unroll
          for (int t = 0; t < TERMS; ++t) tma_load_3d(b_dst + t * BN * 128, &tmB, &full_bar[stage], kcoord, n0, bz * TERMS + t);
        }
        issued_s = i + 1;
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      for (int i = 0; i < nkb + p.expect_extra_kb; ++i) {
        const int stage = i % STAGES;
        const uint32_t ph = (uint32_t)(i / STAGES) & 1u;
        if (!mbar_wait(&full_bar[stage], ph, abortp, wlim)) break;
        tc_fence_after();
        const uint32_t a_addr = smem_u32(smem + (size_t)stage * STAGE_BYTES);
        const uint32_t b_addr = a_addr + A_BYTES;
#pragma unroll
        for (int k16 = 0; k16 < 4; ++k16) {
          const uint64_t adesc = A_MN ? desc_mn_major(a_addr, k16) : desc_k_major(a_addr, k16);
          const uint64_t bdesc = B_MN ? desc_mn_major(b_addr, k16) : desc_k_major(b_addr, k16);
          umma_bf16(tmem_base, adesc, bdesc, IDESC, (i | k16) != 0 ? 1u : 0u);
        }
        umma_commit(&empty_bar[stage]);
      }
      umma_commit(&accum_bar);
      if (*abortp) {  // giving up: the teardown waits on this for the MMAs issued so far before tensor memory is freed
        umma_commit(&flush_bar);
        flush_s = 1;
      }
    }
  } else {
    // ---- epilogue: 4 warps, warp (id % 4) owns TMEM lanes 32*(id % 4) .. +31 ----
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
    const bool ok = mbar_wait(&accum_bar, 0u, abortp, wlim);
    tc_fence_after();
    const int tiles_n = gridDim.y / p.splits;
    const int64_t tile_lin = ((int64_t)batch * gridDim.x + m_tile) * tiles_n + n_tile;
    float* my_partial = p.partial ? p.partial + ((tile_lin * p.splits + split) * 128 + row) * BN : nullptr;
    bool finish = ok;
    if (ok && p.splits > 1) {
#pragma unroll 1
      for (int c = 0; c < BN / 16; ++c) {
        float v[16];
        if (nkb > 0) {
          tmem_ld16(lane_base + c * 16, v);
          if constexpr (MMA_N > BN) {  // add the product with the lo plane
            float w[16];
            tmem_ld16(lane_base + BN + c * 16, w);
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] += w[i];
          }
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) v[i] = 0.f;
        }
        float4* dst = reinterpret_cast<float4*>(my_partial + c * 16);
#pragma unroll
        for (int i = 0; i < 4; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
      }
      __threadfence();
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (warp == 2 && lane == 0) {
        unsigned* ctr = p.counters + tile_lin;
        const unsigned old = atomicAdd(ctr, 1u);
        const int is_last = (old == (unsigned)p.splits - 1u);
        if (is_last) *ctr = 0u;
        last_flag = is_last;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      finish = last_flag != 0;
      if (finish) __threadfence();
    }
    if constexpr (EPI == EPI_YT) {
      // Y^T planes: thread `row` holds one row of the tile, but a plane row (fixed j) is contiguous along the tile's
      // rows.  The tile is turned in shared memory -- the stages are free once the accumulator is complete -- and
      // written out in 16-byte pieces (rows_dot at r = 64: 16 stores per thread instead of 128 two-byte ones).
      static_assert(2 * BN * 128 * 2 <= STAGES * STAGE_BYTES, "the staging tile has to fit in the stages");
      __nv_bfloat16* stg = reinterpret_cast<__nv_bfloat16*>(smem);  // [plane][j][128 rows]
      if (finish) {
#pragma unroll 1
        for (int c = 0; c < BN / 16; ++c) {
          float v[16];
          if (nkb > 0) {
            tmem_ld16(lane_base + c * 16, v);
            if constexpr (MMA_N > BN) {
              float w[16];
              tmem_ld16(lane_base + BN + c * 16, w);
#pragma unroll
              for (int i = 0; i < 16; ++i) v[i] += w[i];
            }
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = 0.f;
          }
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int j = c * 16 + i;
            const __nv_bfloat16 hi = __float2bfloat16_rn(v[i]);
            stg[j * 128 + row] = hi;
            stg[(BN + j) * 128 + row] = __float2bfloat16_rn(v[i] - __bfloat162float(hi));
          }
        }
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");  // all four epilogue warps, whatever they decided above
      if (finish && p.out_planes) {
        const int et = (warp - 2) * 32 + lane, seg = et & 15;
        const int r = p.n_extent;
        const int64_t g0 = (int64_t)m0 + seg * 8;  // first of the eight tile rows of this piece
        for (int o = et >> 4; o < 2 * r; o += 8) {
          const int plane = o >= r ? 1 : 0, j = o - plane * r;
          const __nv_bfloat16* src = stg + (plane * BN + j) * 128 + seg * 8;
          __nv_bfloat16* dst = p.out_planes + (((int64_t)batch * 2 + plane) * p.plane_rows + j) * p.ld_planes + g0;
          if (g0 + 8 <= p.m_extent && (p.ld_planes & 7) == 0) {
            *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
          } else {
            for (int e = 0; e < 8; ++e)
              if (g0 + e < p.m_extent) dst[e] = src[e];
          }
        }
      }
    } else if (EPI == EPI_C && p.tma_store != 0) {
      // The 128 x BN fp32 tile leaves through shared memory: 32 columns at a time every thread puts its row's 128
      // bytes into a [128 rows][128 bytes] box (16-byte pieces swizzled as the tensor map expects, so the 32 lanes of
      // a warp spread over all banks), and one thread hands the box to a TMA store, which writes whole lines and
      // clips at the edges of C.  Two boxes alternate (the pipeline stages are free once the accumulator is complete),
      // so the stores of one run under the TMEM reads of the next.  The contraction is not split here (splits == 1).
      static_assert(EPI != EPI_C || 2 * 16384 <= STAGES * STAGE_BYTES, "two staging boxes have to fit in the stages");
      const bool issuer = warp == 2 && lane == 0;
      if (issuer) prefetch_tmap(&tmC);
#pragma unroll 1
      for (int c32 = 0; c32 < BN / 32; ++c32) {
        uint8_t* box = smem + (c32 & 1) * 16384;
        if (c32 >= 2) {  // the store that read this box two rounds ago has to be done with it
          if (issuer) bulk_wait_read<1>();
          asm volatile("bar.sync 1, 128;" ::: "memory");
        }
        if (ok) {
          float v[32];
          tmem_ld16(lane_base + c32 * 32, *reinterpret_cast<float(*)[16]>(&v[0]));
          tmem_ld16(lane_base + c32 * 32 + 16, *reinterpret_cast<float(*)[16]>(&v[16]));
#pragma unroll
          for (int k = 0; k < 8; ++k)
            *reinterpret_cast<float4*>(box + row * 128 + ((k ^ (row & 7)) * 16)) =
                make_float4(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
        }
        fence_async_proxy();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (issuer && ok && n0 + c32 * 32 < p.n_extent) {
          tma_store_3d(&tmC, box, n0 + c32 * 32, m0, batch);
          bulk_commit();
        }
      }
      if (issuer) bulk_wait_all();
    } else if (finish) {
      const int64_t gm = (int64_t)m0 + row;  // global row of D
#pragma unroll 1
      for (int c = 0; c < BN / 16; ++c) {
        float v[16];
        if (p.splits > 1) {
#pragma unroll
          for (int i = 0; i < 16; ++i) v[i] = 0.f;
          const float* src = p.partial + (tile_lin * p.splits * 128 + row) * BN + c * 16;
          for (int s = 0; s < p.splits; ++s) {
            const float4* s4 = reinterpret_cast<const float4*>(src + (int64_t)s * 128 * BN);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float4 t = __ldcg(s4 + i);
              v[4 * i] += t.x;
              v[4 * i + 1] += t.y;
              v[4 * i + 2] += t.z;
              v[4 * i + 3] += t.w;
            }
          }
        } else if (nkb > 0) {
          tmem_ld16(lane_base + c * 16, v);
          if constexpr (MMA_N > BN) {
            float w[16];
            tmem_ld16(lane_base + BN + c * 16, w);
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] += w[i];
          }
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) v[i] = 0.f;
        }
        if (gm < p.m_extent) {
          if constexpr (EPI == EPI_C) {
            float* dst = p.out_f32 + (int64_t)batch * p.out_batch_stride + gm * p.ld_out + n0 + c * 16;
            if (n0 + c * 16 + 16 <= p.n_extent && (p.ld_out & 3) == 0) {
#pragma unroll
              for (int i = 0; i < 4; ++i)
                reinterpret_cast<float4*>(dst)[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            } else {
#pragma unroll
              for (int i = 0; i < 16; ++i)
                if (n0 + c * 16 + i < p.n_extent) dst[i] = v[i];
            }
          } else {
            const int r = p.n_extent;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const int j = c * 16 + i;
              if (j < r) {
                if constexpr (EPI == EPI_Z) {
                  if (p.out_f32) p.out_f32[((int64_t)batch * r + j) * p.ld_out + gm] = v[i];
                  if (p.out2_f32) p.out2_f32[((int64_t)batch * r + j) * p.ld_out + gm] = v[i];
                }
                if (p.out_planes) {
                  const __nv_bfloat16 hi = __float2bfloat16_rn(v[i]);
                  const __nv_bfloat16 lo = __float2bfloat16_rn(v[i] - __bfloat162float(hi));
                  p.out_planes[(((int64_t)batch * 2 + 0) * p.plane_rows + j) * p.ld_planes + gm] = hi;
                  p.out_planes[(((int64_t)batch * 2 + 1) * p.plane_rows + j) * p.ld_planes + gm] = lo;
                }
              }
            }
          }
        }
      }
    }
  }

  // ---- teardown ----
  tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    if (threadIdx.x == 0) {
      // wait (bounded) for copies already issued into this CTA's shared memory
      const int issued = issued_s;
      const int first = issued > STAGES ? issued - STAGES : 0;
      for (int i = first; i < issued; ++i) {
        uint64_t* bar = &full_bar[i % STAGES];
        const uint32_t ph = (uint32_t)(i / STAGES) & 1u;
        for (uint32_t t = 0; t < kWaitLimit && !mbar_try_wait(bar, ph); ++t) {
        }
      }
      // ... and for the MMAs already issued (they read shared memory and write the accumulator)
      for (uint32_t t = 0; t < kWaitLimit && !mbar_try_wait(&accum_bar, 0u); ++t) {  // committed after the last MMA issued
      }
      if (flush_s) {
        for (uint32_t t = 0; t < kWaitLimit && !mbar_try_wait(&flush_bar, 0u); ++t) {
        }
      }
      if (p.status) *p.status = (int)DAD_ERR_TIMEOUT;
    }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// Dense product C = X^T Y for long contractions (the dAD gradient, K = S*N): one CTA owns a 256 x 256
// tile as two 128 x 256 accumulators that fill tensor memory (512 columns).  Both MMAs of a k-step read
// the same B operand, so a CTA fetches 64 KB per 64-deep block for 2 * 256 * 256 * 64 flops: two thirds of
// the bytes per flop of the 128 x 256 tile, and the same bytes in flight cover a 1.5x longer stretch of
// MMA time.  Stages are BK contraction rows deep (BK = 32: more, finer stages in the same shared memory).
// Same roles, bounded waits, split reduction and teardown as umma_kernel.
template <int BK, int STAGES>
__global__ void __launch_bounds__(192)
umma_gemm256_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const UmmaParams p) {
  constexpr int CHUNK = BK * 128;          // [BK k-rows][64 bf16 along M or N]
  constexpr int A_BYTES = 4 * CHUNK;       // 256 rows of the tile
  constexpr int STAGE_BYTES = 8 * CHUNK;   // A and B
  constexpr uint32_t TMEM_COLS = 512;
  constexpr uint32_t IDESC = instr_desc(128, 256, true, true);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ uint64_t full_bar[STAGES], empty_bar[STAGES], accum_bar, drained_bar, flush_bar;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag, issued_s, flush_s;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Work of this CTA.  The first tiles * splits CTAs each own one tile and one of the `splits` equal parts of the
  // first splits * kb_per_split blocks of the contraction (m fastest, so neighbours share a B panel at the same k).
  // The rem_ctas CTAs after them take what is left of the contraction, the same block range for every tile, each for
  // the tiles t = j, j + rem_ctas, ... one after the other: they fill the SMs that tiles * splits leaves empty.
  const int tiles_per_product = p.tiles_m * p.tiles_n;
  const int n_tiles = tiles_per_product * p.batch_count;  // several products of one shape share a launch
  const int n_main = n_tiles * p.splits;
  const bool is_rem = (int)blockIdx.x >= n_main;
  const int rem_j = (int)blockIdx.x - n_main;
  const int slots = p.splits + (p.rem_ctas > 0 ? 1 : 0);  // partial tiles per output tile
  struct Item {
    int m0, n0, kb0, kb1, slot, product;
    int64_t tile_lin;
  };
  auto item_at = [&](int it, Item& w) -> bool {
    int tile, split;
    if (!is_rem) {
      if (it > 0) return false;
      const int rest = (int)blockIdx.x / p.tiles_m;
      tile = (rest / p.splits) * p.tiles_m + (int)blockIdx.x % p.tiles_m;  // n_tile * tiles_m + m_tile
      split = rest % p.splits;
      w.kb0 = split * p.kb_per_split;
      const int end = p.rem_ctas > 0 ? p.splits * p.kb_per_split : p.k_blocks;
      w.kb1 = (w.kb0 + p.kb_per_split < end) ? w.kb0 + p.kb_per_split : end;
    } else {
      tile = rem_j + it * p.rem_ctas;
      if (tile >= n_tiles) return false;
      split = p.splits;
      w.kb0 = p.splits * p.kb_per_split;
      w.kb1 = p.k_blocks;
    }
    if (w.kb1 < w.kb0) w.kb1 = w.kb0;
    w.product = tile / tiles_per_product;
    const int rem = tile - w.product * tiles_per_product;
    const int m_tile = rem % p.tiles_m, n_tile = rem / p.tiles_m;
    w.m0 = m_tile * 256;
    w.n0 = n_tile * 256;
    w.slot = split;
    w.tile_lin = (int64_t)w.product * tiles_per_product + (int64_t)m_tile * p.tiles_n + n_tile;
    return true;
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(&accum_bar, 1);
    mbar_init(&drained_bar, 128);
    mbar_init(&flush_bar, 1);
    abort_flag = 0;
    issued_s = 0;
    flush_s = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(&tmem_base_s, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  volatile int* abortp = &abort_flag;

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (warp == 0) {
    if (lane == 0) {
      prefetch_tmap(&tmA);
      prefetch_tmap(&tmB);
      int g = 0;  // blocks issued so far, over all items: the stage ring runs on across items
      bool go = true;
      Item w;
      for (int it = 0; go && item_at(it, w); ++it) {
        for (int kb = w.kb0; kb < w.kb1; ++kb, ++g) {
          const int stage = g % STAGES;
          const uint32_t ph = (uint32_t)(g / STAGES) & 1u;
          if (!mbar_wait(&empty_bar[stage], ph ^ 1u, abortp)) {
            go = false;
            break;
          }
          mbar_expect_tx(&full_bar[stage], STAGE_BYTES);
          uint8_t* a_dst = smem + (size_t)stage * STAGE_BYTES;
          uint8_t* b_dst = a_dst + A_BYTES;
          const int bz = w.product * p.sites_per_product + kb / p.kb_per_site;
          const int kcoord = (kb % p.kb_per_site) * BK;
#pragma unroll
          for (int c = 0; c < 4; ++c) tma_load_3d(a_dst + c * CHUNK, &tmA, &full_bar[stage], w.m0 + c * 64, kcoord, bz);
#pragma unroll
          for (int c = 0; c < 4; ++c) tma_load_3d(b_dst + c * CHUNK, &tmB, &full_bar[stage], w.n0 + c * 64, kcoord, bz);
          issued_s = g + 1;
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      int g = 0;
      bool go = true;
      Item w;
      for (int it = 0; go && item_at(it, w); ++it) {
        // the accumulators of the previous item have been read out
        if (it > 0 && !mbar_wait(&drained_bar, (uint32_t)(it - 1) & 1u, abortp)) break;
        tc_fence_after();
        for (int kb = w.kb0; kb < w.kb1; ++kb, ++g) {
          const int stage = g % STAGES;
          const uint32_t ph = (uint32_t)(g / STAGES) & 1u;
          if (!mbar_wait(&full_bar[stage], ph, abortp)) {
            go = false;
            break;
          }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem + (size_t)stage * STAGE_BYTES);
          const uint32_t b_addr = a_addr + A_BYTES;
#pragma unroll
          for (int k16 = 0; k16 < BK / 16; ++k16) {
            const uint64_t bdesc = smem_desc(b_addr + (uint32_t)k16 * 2048u, CHUNK, 1024u);
            const uint32_t acc = (kb != w.kb0 || k16 != 0) ? 1u : 0u;
            umma_bf16(tmem_base, smem_desc(a_addr + (uint32_t)k16 * 2048u, CHUNK, 1024u), bdesc, IDESC, acc);
            umma_bf16(tmem_base + 256u, smem_desc(a_addr + 2u * CHUNK + (uint32_t)k16 * 2048u, CHUNK, 1024u), bdesc, IDESC, acc);
          }
          umma_commit(&empty_bar[stage]);
        }
        if (go) umma_commit(&accum_bar);
      }
      if (*abortp) {  // giving up: the teardown waits on this for the MMAs issued so far before tensor memory is freed
        umma_commit(&flush_bar);
        flush_s = 1;
      }
    }
  } else {
    const int q = warp & 3;
    const int row = q * 32 + lane;  // row inside each 128-row half
    const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
    Item w;
    for (int it = 0; item_at(it, w); ++it) {
      if (!mbar_wait(&accum_bar, (uint32_t)it & 1u, abortp)) break;
      tc_fence_after();
      const int nkb = w.kb1 - w.kb0;
      // With several partial tiles per output tile every CTA stores its own and gemm256_reduce sums them in slot order;
      // otherwise the tile goes straight to C.
      float* my_partial = slots > 1 ? p.partial + (w.tile_lin * slots + w.slot) * (int64_t)(256 * 256) : nullptr;
#pragma unroll 1
      for (int c = 0; c < 32; ++c) {  // chunk c: half c / 16 of the tile, columns (c % 16) * 16 .. +15
        const int half = c / 16, col = (c % 16) * 16;
        float v[16];
        if (nkb > 0) {
          tmem_ld16(lane_base + (uint32_t)c * 16u, v);
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) v[i] = 0.f;
        }
        if (my_partial) {
          float4* dst = reinterpret_cast<float4*>(my_partial + (half * 128 + row) * 256 + col);
#pragma unroll
          for (int i = 0; i < 4; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
        } else {
          const int64_t gm = (int64_t)w.m0 + half * 128 + row;
          if (gm < p.m_extent) {
            float* dst = p.out_f32 + (int64_t)w.product * p.out_batch_stride + gm * p.ld_out + w.n0 + col;
            if (w.n0 + col + 16 <= p.n_extent && (p.ld_out & 3) == 0) {
#pragma unroll
              for (int i = 0; i < 4; ++i)
                reinterpret_cast<float4*>(dst)[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            } else {
#pragma unroll
              for (int i = 0; i < 16; ++i)
                if (w.n0 + col + i < p.n_extent) dst[i] = v[i];
            }
          }
        }
      }
      // this thread's part of the accumulators is in registers or memory: the next item may overwrite them
      tc_fence_before();
      mbar_arrive(&drained_bar);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    if (threadIdx.x == 0) {
      const int issued = issued_s;
      const int first = issued > STAGES ? issued - STAGES : 0;
      for (int i = first; i < issued; ++i) {
        uint64_t* bar = &full_bar[i % STAGES];
        const uint32_t ph = (uint32_t)(i / STAGES) & 1u;
        for (uint32_t t = 0; t < kWaitLimit && !mbar_try_wait(bar, ph); ++t) {
        }
      }
      // ... and for the MMAs already issued (they read shared memory and write the accumulator)
      if (flush_s) {
        for (uint32_t t = 0; t < kWaitLimit && !mbar_try_wait(&flush_bar, 0u); ++t) {
        }
      }
      if (p.status) *p.status = (int)DAD_ERR_TIMEOUT;
    }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// Dense product C = X^T Y for SHORT contractions (the reconstruction P^T Q of Algorithm 1, K = S r), persistent form:
// one CTA per SM walks over 128 x 256 output tiles (all products of a batched call), with TWO accumulators in tensor
// memory (2 x 256 columns), so that the tensor cores fill one while the epilogue drains the other.  With K of a few
// hundred a tile's MMAs last about a microsecond and its 128 KB of fp32 output two or three: what bounds the product
// is writing C, and per-tile CTAs spend as long starting, filling their pipeline and waiting for their last stores
// as they spend on the tile.  Here the set-up happens once per SM, the stage ring runs on across tiles, and the
// output leaves through two staging boxes and TMA stores (whole lines, clipped at the edges of C) that never block
// the next tile.  Measured against the per-tile CTAs (two per SM) on 144 reconstructions of 1024 x 1024 ... 4096 per
// step: 4 blocks per tile 0.453 against 0.466 ms, 12 blocks 0.725 against 0.703, 16 blocks 1.03 against 0.94 -- so it
// takes the products of at most 8 blocks only.  (Staging the whole tile at once -- one proxy fence and two barriers
// per tile instead of per 32 columns, with two pipeline stages -- was slower still: 0.507 ms.)  Roles, bounded waits and teardown as in umma_kernel; the contraction is never split.
template <int STAGES>
__global__ void __launch_bounds__(192)
umma_gemm_persist_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                         const __grid_constant__ CUtensorMap tmC, const UmmaParams p) {
  constexpr int BN = 256;
  constexpr int A_BYTES = 2 * 8192, B_BYTES = 4 * 8192, STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr int BOX_BYTES = 128 * 128;  // [128 rows][32 fp32]
  constexpr uint32_t TMEM_COLS = 512;
  constexpr uint32_t IDESC = instr_desc(128, BN, true, true);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* boxes = smem + (size_t)STAGES * STAGE_BYTES;
  __shared__ uint64_t full_bar[STAGES], empty_bar[STAGES], acc_full[2], acc_empty[2], flush_bar;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag, issued_s, flush_s, epi_bad;
  const uint32_t wlim = p.wait_limit ? p.wait_limit : kWaitLimit;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int per_product = p.tiles_m * p.tiles_n;
  const int n_tiles = per_product * p.batch_count;
  const int nkb = p.k_blocks;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&acc_full[b], 1);
      mbar_init(&acc_empty[b], 128);
    }
    mbar_init(&flush_bar, 1);
    abort_flag = 0;
    issued_s = 0;
    flush_s = 0;
    epi_bad = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(&tmem_base_s, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  volatile int* abortp = &abort_flag;

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // tile t: product t / per_product; inside it m fastest, so that CTAs working side by side share a panel of Y
  auto tile_at = [&](int t, int& m0, int& n0, int& bz) {
    bz = t / per_product;
    const int rem = t - bz * per_product;
    n0 = (rem / p.tiles_m) * BN;
    m0 = (rem % p.tiles_m) * 128;
  };

  if (warp == 0) {
    if (lane == 0) {
      prefetch_tmap(&tmA);
      prefetch_tmap(&tmB);
      int g = 0;
      bool go = true;
      for (int t = blockIdx.x; go && t < n_tiles; t += gridDim.x) {
        int m0, n0, bz;
        tile_at(t, m0, n0, bz);
        for (int kb = 0; kb < nkb; ++kb, ++g) {
          const int stage = g % STAGES;
          const uint32_t ph = (uint32_t)(g / STAGES) & 1u;
          if (!mbar_wait(&empty_bar[stage], ph ^ 1u, abortp, wlim)) {
            go = false;
            break;
          }
          mbar_expect_tx(&full_bar[stage], STAGE_BYTES);
          uint8_t* a_dst = smem + (size_t)stage * STAGE_BYTES;
          uint8_t* b_dst = a_dst + A_BYTES;
          const int kcoord = kb * 64;
          tma_load_3d(a_dst, &tmA, &full_bar[stage], m0, kcoord, bz);
          tma_load_3d(a_dst + 8192, &tmA, &full_bar[stage], m0 + 64, kcoord, bz);
#pragma unroll
          for (int c = 0; c < 4; ++c) tma_load_3d(b_dst + c * 8192, &tmB, &full_bar[stage], n0 + c * 64, kcoord, bz);
          issued_s = g + 1;
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      int g = 0, it = 0;
      bool go = true;
      for (int t = blockIdx.x; go && t < n_tiles; t += gridDim.x, ++it) {
        const int buf = it & 1;
        const uint32_t uses = (uint32_t)(it >> 1);
        // the epilogue has read this accumulator's previous tile out (passes at once on its first use)
        if (!mbar_wait(&acc_empty[buf], (uses & 1u) ^ 1u, abortp, wlim)) break;
        tc_fence_after();
        const uint32_t acc = tmem_base + (uint32_t)buf * BN;
        for (int kb = 0; kb < nkb; ++kb, ++g) {
          const int stage = g % STAGES;
          const uint32_t ph = (uint32_t)(g / STAGES) & 1u;
          if (!mbar_wait(&full_bar[stage], ph, abortp, wlim)) {
            go = false;
            break;
          }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem + (size_t)stage * STAGE_BYTES);
          const uint32_t b_addr = a_addr + A_BYTES;
#pragma unroll
          for (int k16 = 0; k16 < 4; ++k16)
            umma_bf16(acc, desc_mn_major(a_addr, k16), desc_mn_major(b_addr, k16), IDESC, (kb | k16) != 0 ? 1u : 0u);
          umma_commit(&empty_bar[stage]);
        }
        if (go) umma_commit(&acc_full[buf]);
      }
      if (*abortp) {  // giving up: the teardown waits on this for the MMAs issued so far before tensor memory is freed
        umma_commit(&flush_bar);
        flush_s = 1;
      }
    }
  } else {
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const bool issuer = warp == 2 && lane == 0;
    if (issuer) prefetch_tmap(&tmC);
    int it = 0, boxes_used = 0;
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++it) {
      int m0, n0, bz;
      tile_at(t, m0, n0, bz);
      const int buf = it & 1;
      const uint32_t uses = (uint32_t)(it >> 1);
      if (!mbar_wait(&acc_full[buf], uses & 1u, abortp, wlim)) epi_bad = 1;
      asm volatile("bar.sync 1, 128;" ::: "memory");  // the four warps go on, or stop, together
      if (*reinterpret_cast<volatile int*>(&epi_bad)) break;
      tc_fence_after();
      const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)buf * BN;
#pragma unroll 1
      for (int c32 = 0; c32 < BN / 32; ++c32, ++boxes_used) {
        uint8_t* box = boxes + (boxes_used & 1) * BOX_BYTES;
        if (boxes_used >= 2) {  // the store that read this box two rounds ago has to be done with it
          if (issuer) bulk_wait_read<1>();
          asm volatile("bar.sync 1, 128;" ::: "memory");
        }
        float v[32];
        tmem_ld16(lane_base + c32 * 32, *reinterpret_cast<float(*)[16]>(&v[0]));
        tmem_ld16(lane_base + c32 * 32 + 16, *reinterpret_cast<float(*)[16]>(&v[16]));
#pragma unroll
        for (int k = 0; k < 8; ++k)
          *reinterpret_cast<float4*>(box + row * 128 + ((k ^ (row & 7)) * 16)) =
              make_float4(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
        fence_async_proxy();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (issuer) {
          if (n0 + c32 * 32 < p.n_extent) tma_store_3d(&tmC, box, n0 + c32 * 32, m0, bz);
          bulk_commit();  // (an empty group where the box lies beyond C, so that the count of groups stays in step)
        }
      }
      // this thread's part of the accumulator is in shared memory: the tensor cores may overwrite it
      tc_fence_before();
      mbar_arrive(&acc_empty[buf]);
    }
    if (issuer) bulk_wait_all();
  }

  tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    if (threadIdx.x == 0) {
      const int issued = issued_s;
      const int first = issued > STAGES ? issued - STAGES : 0;
      for (int i = first; i < issued; ++i) {
        uint64_t* bar = &full_bar[i % STAGES];
        const uint32_t ph = (uint32_t)(i / STAGES) & 1u;
        for (uint32_t t = 0; t < kWaitLimit && !mbar_try_wait(bar, ph); ++t) {
        }
      }
      if (flush_s) {
        for (uint32_t t = 0; t < kWaitLimit && !mbar_try_wait(&flush_bar, 0u); ++t) {
        }
      }
      if (p.status) *p.status = (int)DAD_ERR_TIMEOUT;
    }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}


// Dense product C = X^T Y for short contractions, persistent form on CTA PAIRS (cta_group::2): two CTAs of a cluster,
// on neighbouring SMs, own a 256 x 256 output tile together.  Each loads its own 128 columns of X (rows of the tile)
// and only HALF of the tile's 256 columns of Y per 64-deep block -- 32 KB instead of the 48 KB a lone CTA needs for a
// 128 x 256 tile -- and the tensor cores of both SMs read the two halves of Y out of both shared memories.  The
// reconstruction (Algorithm 1, P^T Q) is bound by exactly those bytes: at a contraction of a few hundred rows a CTA
// spends longer pulling its operands through its SM's L2 port than multiplying or storing.  One thread of the leader
// (cluster rank 0) issues the MMAs for both CTAs; every CTA fetches its own tiles with plain TMA loads (no cluster
// multicast), whose completion is counted on the leader's barrier; a commit arrives on the barriers of both CTAs.
// Each CTA holds two accumulators of 128 x 256 in its tensor memory, so the epilogue of one tile (through two staging
// boxes and TMA stores, as in umma_gemm_persist_kernel) runs under the MMAs of the next.  Waits are bounded as
// everywhere; whatever happens, every thread of both CTAs reaches the cluster barrier before tensor memory is freed.
template <int STAGES>
__global__ void __launch_bounds__(192)
umma_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                      const __grid_constant__ CUtensorMap tmC, const UmmaParams p) {
  constexpr int A_BYTES = 2 * 8192, B_BYTES = 2 * 8192, STAGE_BYTES = A_BYTES + B_BYTES;  // per CTA
  constexpr int BOX_BYTES = 128 * 128;  // [128 rows][32 fp32]
  constexpr uint32_t TMEM_COLS = 512;
  constexpr uint32_t IDESC = instr_desc(256, 256, true, true);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* boxes = smem + (size_t)STAGES * STAGE_BYTES;
  // full / acc_empty are used in the leader only (they count both CTAs); empty / acc_full in each CTA
  __shared__ uint64_t full_bar[STAGES], empty_bar[STAGES], acc_full[2], acc_empty[2], flush_bar;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag, issued_s, flush_s, epi_bad;
  const uint32_t wlim = p.wait_limit ? p.wait_limit : kWaitLimit;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int per_product = p.tiles_m * p.tiles_n;  // 256 x 256 tiles
  const int n_tiles = per_product * p.batch_count;
  const int nkb = p.k_blocks;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&acc_full[b], 1);
      mbar_init(&acc_empty[b], 256);  // the epilogue threads of both CTAs
    }
    mbar_init(&flush_bar, 1);
    abort_flag = 0;
    issued_s = 0;
    flush_s = 0;
    epi_bad = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(&tmem_base_s, TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_barrier_all();  // both CTAs' barriers are initialised before either signals the other's
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  volatile int* abortp = &abort_flag;

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // tile t: product t / per_product; inside it m fastest, so that pairs working side by side share a panel of Y
  auto tile_at = [&](int t, int& m0, int& n0, int& bz) {
    bz = t / per_product;
    const int rem = t - bz * per_product;
    n0 = (rem / p.tiles_m) * 256;
    m0 = (rem % p.tiles_m) * 256;
  };

  if (warp == 0) {
    if (lane == 0) {
      prefetch_tmap(&tmA);
      prefetch_tmap(&tmB);
      int g = 0;
      bool go = true;
      for (int t = pair; go && t < n_tiles; t += n_pairs) {
        int m0, n0, bz;
        tile_at(t, m0, n0, bz);
        m0 += 128 * (int)rank;  // this CTA's rows of the tile
        n0 += 128 * (int)rank;  // ... and its half of the tile's columns of Y
        for (int kb = 0; kb < nkb; ++kb, ++g) {
          const int stage = g % STAGES;
          const uint32_t ph = (uint32_t)(g / STAGES) & 1u;
          if (!mbar_wait(&empty_bar[stage], ph ^ 1u, abortp, wlim)) {
            go = false;
            break;
          }
          if (leader) mbar_expect_tx(&full_bar[stage], 2 * STAGE_BYTES);  // the tiles of both CTAs
          const uint32_t bar = cluster_map(smem_u32(&full_bar[stage]), 0);
          uint8_t* a_dst = smem + (size_t)stage * STAGE_BYTES;
          uint8_t* b_dst = a_dst + A_BYTES;
          const int kcoord = kb * 64;
          tma_load_3d_pair(a_dst, &tmA, bar, m0, kcoord, bz);
          tma_load_3d_pair(a_dst + 8192, &tmA, bar, m0 + 64, kcoord, bz);
          tma_load_3d_pair(b_dst, &tmB, bar, n0, kcoord, bz);
          tma_load_3d_pair(b_dst + 8192, &tmB, bar, n0 + 64, kcoord, bz);
          issued_s = g + 1;
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && leader) {
      int g = 0, it = 0;
      bool go = true;
      for (int t = pair; go && t < n_tiles; t += n_pairs, ++it) {
        const int buf = it & 1;
        const uint32_t uses = (uint32_t)(it >> 1);
        // both epilogues have read this accumulator's previous tile out (passes at once on its first use)
        if (!mbar_wait(&acc_empty[buf], (uses & 1u) ^ 1u, abortp, wlim)) break;
        tc_fence_after();
        const uint32_t acc = tmem_base + (uint32_t)buf * 256u;
        for (int kb = 0; kb < nkb; ++kb, ++g) {
          const int stage = g % STAGES;
          const uint32_t ph = (uint32_t)(g / STAGES) & 1u;
          if (!mbar_wait(&full_bar[stage], ph, abortp, wlim)) {
            go = false;
            break;
          }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem + (size_t)stage * STAGE_BYTES);
          const uint32_t b_addr = a_addr + A_BYTES;
#pragma unroll
          for (int k16 = 0; k16 < 4; ++k16)
            umma_bf16_pair(acc, desc_mn_major(a_addr, k16), desc_mn_major(b_addr, k16), IDESC, (kb | k16) != 0 ? 1u : 0u);
          umma_commit_pair(&empty_bar[stage]);
        }
        if (go) umma_commit_pair(&acc_full[buf]);
      }
      if (*abortp) {  // giving up: the teardown waits on this for the MMAs issued so far before tensor memory is freed
        umma_commit_pair(&flush_bar);
        flush_s = 1;
      }
    }
  } else {
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const bool issuer = warp == 2 && lane == 0;
    if (issuer) prefetch_tmap(&tmC);
    int it = 0, boxes_used = 0;
    for (int t = pair; t < n_tiles; t += n_pairs, ++it) {
      int m0, n0, bz;
      tile_at(t, m0, n0, bz);
      m0 += 128 * (int)rank;
      const int buf = it & 1;
      const uint32_t uses = (uint32_t)(it >> 1);
      if (!mbar_wait(&acc_full[buf], uses & 1u, abortp, wlim)) epi_bad = 1;
      asm volatile("bar.sync 1, 128;" ::: "memory");  // the four warps go on, or stop, together
      if (*reinterpret_cast<volatile int*>(&epi_bad)) break;
      tc_fence_after();
      const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)buf * 256u;
#pragma unroll 1
      for (int c32 = 0; c32 < 8; ++c32, ++boxes_used) {
        uint8_t* box = boxes + (boxes_used & 1) * BOX_BYTES;
        if (boxes_used >= 2) {  // the store that read this box two rounds ago has to be done with it
          if (issuer) bulk_wait_read<1>();
          asm volatile("bar.sync 1, 128;" ::: "memory");
        }
        float v[32];
        tmem_ld16(lane_base + c32 * 32, *reinterpret_cast<float(*)[16]>(&v[0]));
        tmem_ld16(lane_base + c32 * 32 + 16, *reinterpret_cast<float(*)[16]>(&v[16]));
#pragma unroll
        for (int k = 0; k < 8; ++k)
          *reinterpret_cast<float4*>(box + row * 128 + ((k ^ (row & 7)) * 16)) =
              make_float4(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
        fence_async_proxy();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (issuer) {
          if (n0 + c32 * 32 < p.n_extent && m0 < p.m_extent) tma_store_3d(&tmC, box, n0 + c32 * 32, m0, bz);
          bulk_commit();  // (an empty group where the box lies beyond C, so that the count of groups stays in step)
        }
      }
      // this thread's part of the accumulator is in shared memory: the tensor cores may overwrite it
      tc_fence_before();
      mbar_arrive_remote(cluster_map(smem_u32(&acc_empty[buf]), 0));
    }
    if (issuer) bulk_wait_all();
  }

  tc_fence_before();
  __syncthreads();
  // Neither CTA goes on to free tensor memory, or leaves, while its peer may still read its shared memory, arrive on
  // its barriers or multiply into its accumulators.
  if (abort_flag) {
    if (threadIdx.x == 0) {
      const int issued = issued_s;
      const int first = issued > STAGES ? issued - STAGES : 0;
      if (leader) {
        for (int i = first; i < issued; ++i) {
          uint64_t* bar = &full_bar[i % STAGES];
          const uint32_t ph = (uint32_t)(i / STAGES) & 1u;
          for (uint32_t t = 0; t < kWaitLimit && !mbar_try_wait(bar, ph); ++t) {
          }
        }
      }
      if (flush_s) {
        for (uint32_t t = 0; t < kWaitLimit && !mbar_try_wait(&flush_bar, 0u); ++t) {
        }
      }
      if (p.status) *p.status = (int)DAD_ERR_TIMEOUT;
    }
    __syncthreads();
  }
  cluster_barrier_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
}

// C[m][n] = sum over splits, in split order, of the partial tiles umma_gemm256_kernel stored
// ([tile][split][256][256] fp32): four columns per thread, the whole GPU instead of one CTA per tile.
__global__ void __launch_bounds__(256)
gemm256_reduce_kernel(const float* __restrict__ partial, int splits, int m_extent, int n_extent, float* __restrict__ C) {
  const int n4 = n_extent / 4;  // n_extent is a multiple of 8 on this path
  const int tiles_n = (n_extent + 255) / 256;
  const int64_t total = (int64_t)m_extent * n4;
  // one product per blockIdx.y: its partial tiles and its C follow the previous product's
  partial += (int64_t)blockIdx.y * ((m_extent + 255) / 256) * tiles_n * splits * (int64_t)(256 * 256);
  C += (int64_t)blockIdx.y * m_extent * n_extent;
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    const int m = (int)(idx / n4), n = (int)(idx % n4) * 4;
    const int64_t tile = (int64_t)(m / 256) * tiles_n + n / 256;
    const float* src = partial + tile * splits * (int64_t)(256 * 256) + (m % 256) * 256 + n % 256;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < splits; ++s) {
      const float4 t = __ldcg(reinterpret_cast<const float4*>(src + (int64_t)s * (256 * 256)));
      acc.x += t.x;
      acc.y += t.y;
      acc.z += t.z;
      acc.w += t.w;
    }
    *reinterpret_cast<float4*>(C + (int64_t)m * n_extent + n) = acc;
  }
}

// ---- host side ---------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

bool tmap_encoder_available() { return encode_fn() != nullptr; }

// Whether short dense products may run on CTA pairs (on unless DAD_NO_PAIR_GEMM is set in the environment, for A/B timing).
static const bool g_pair_gemm = getenv("DAD_NO_PAIR_GEMM") == nullptr;

// bf16 tensor (d0 innermost, contiguous) x d1 x d2 with byte strides s1, s2; box = box0 x box1 x 1,
// 128-byte swizzle, out-of-range elements read as zero.
bool make_tmap_bf16_3d(CUtensorMap* map, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t s1_bytes,
                       uint64_t s2_bytes, uint32_t box0, uint32_t box1) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  if (d2 <= 1 && s2_bytes < s1_bytes) s2_bytes = s1_bytes * d1;
  // A map is a pure function of these nine numbers, and callers ask for the same few again and again (the planes
  // of a workspace never move, a layer's inputs rarely do): the last encodings of this thread are kept.
  struct Key {
    const void* base;
    uint64_t d0, d1, d2, s1, s2;
    uint32_t b0, b1;
    bool operator==(const Key& o) const {
      return base == o.base && d0 == o.d0 && d1 == o.d1 && d2 == o.d2 && s1 == o.s1 && s2 == o.s2 && b0 == o.b0 && b1 == o.b1;
    }
  };
  constexpr int kSlots = 64;
  struct Slot {
    Key key;
    CUtensorMap map;
    bool used;
  };
  static thread_local Slot cache[kSlots] = {};
  static thread_local unsigned next = 0;
  const Key key{base, d0, d1, d2, s1_bytes, s2_bytes, box0, box1};
  for (int i = 0; i < kSlots; ++i)
    if (cache[i].used && cache[i].key == key) {
      *map = cache[i].map;
      return true;
    }
  cuuint64_t dims[3] = {d0, d1, d2};
  cuuint64_t strides[2] = {s1_bytes, s2_bytes};
  cuuint32_t box[3] = {box0, box1, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  Slot& slot = cache[next++ % kSlots];
  slot.key = key;
  slot.map = *map;
  slot.used = true;
  return true;
}

// fp32 tensor (d0 innermost, contiguous) x d1 x d2 with byte strides s1, s2; box = 32 x box1 x 1 (128 bytes wide),
// 128-byte swizzle: the output tiles of the TMA-store epilogue.
bool make_tmap_f32_3d(CUtensorMap* map, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t s1_bytes,
                      uint64_t s2_bytes, uint32_t box1) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {d0, d1, d2};
  if (d2 <= 1 && s2_bytes < s1_bytes) s2_bytes = s1_bytes * d1;
  cuuint64_t strides[2] = {s1_bytes, s2_bytes};
  cuuint32_t box[3] = {32, box1, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

int umma_rank_pad(int r) { return r <= 16 ? 16 : (r <= 32 ? 32 : 64); }

// CTAs that share the rows of one 128-column tile of Z = Y^T X.  A CTA streams its rows at about one SM's
// share of the HBM bandwidth whatever the grid, and every extra split costs a partial tile and a pass of the
// finishing CTA over it, so the rows are split only while tiles alone leave SMs empty: about one CTA per SM,
// at most 8 splits, at least 256 rows each (measured on 8 ... 512 tiles: best at 148 / tiles, rounded; aiming at 1.5, 2
// or 3 CTAs per SM instead made 128-tile launches 8-14 % and an encoder layer's step 2-11 % slower).
int umma_cols_acc_splits(int S, int64_t N, int64_t h) {
  const int64_t tiles = ceil_div(h, 128) * S;
  const int64_t kb = ceil_div(N, 64);
  int64_t splits = (148 + tiles / 2) / tiles;
  if (splits > 8) splits = 8;
  if (splits > kb / 4) splits = kb / 4;
  if (splits < 1) splits = 1;
  const int64_t per = ceil_div(kb, splits);
  return (int)ceil_div(kb, per);  // no empty split
}

template <int BN, bool A_MN, bool B_MN, int TERMS, int EPI, int STAGES>
static cudaError_t launch_umma(const CUtensorMap& tmA, const CUtensorMap& tmB, const UmmaParams& p, dim3 grid,
                               const char* tag, cudaStream_t st, const CUtensorMap* tmC = nullptr) {
  constexpr int A_BYTES = 128 * 64 * 2;
  constexpr int B_BYTES = B_MN ? (BN / 64) * 8192 : TERMS * BN * 128;
  constexpr size_t smem = (size_t)STAGES * (A_BYTES + B_BYTES) + 1024;
  auto kernel = umma_kernel<BN, A_MN, B_MN, TERMS, EPI, STAGES>;
  cudaError_t err = cudaSuccess;
  static FirstUse first;  // the opt-in to large dynamic shared memory is per function and device, not per launch
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
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see griddepcontrol in the kernel
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const bool timed = g_timing.load(std::memory_order_relaxed);
  if (timed) timing_mark(tag, st, true);
  err = cudaLaunchKernelEx(&cfg, kernel, tmA, tmB, tmC ? *tmC : tmA, p);  // without tmC the kernel never touches it
  if (timed) timing_mark(tag, st, false);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return err;
}

// Y^T planes <- split(X F^T).  tmX: X as (h, N, S) with box 64 x 128; tmF: factor planes as (h, rp, 2S) with box 64 x rp,
// rp = umma_rank_pad(r).  Stage counts are measured: a CTA of this kernel is short (h / 64 blocks, then an epilogue that
// loads nothing), so several shallow CTAs per SM that cover one another's epilogues stream better than two deep ones
// (r <= 16: 5 CTAs of 2 stages 31.9 ms per benchmark step, 3 of 3 stages 32.4, 2 of 5 stages 32.9).
cudaError_t umma_rows_dot(const CUtensorMap& tmX, const CUtensorMap& tmF, int S, int64_t N, int64_t h, int r,
                          __nv_bfloat16* yt_planes, int64_t ld_planes, int* status, cudaStream_t st) {
  UmmaParams p{};
  p.m_extent = (int)N;
  p.n_extent = r;
  p.k_blocks = (int)ceil_div(h, 64);
  p.kb_per_split = p.k_blocks;
  p.splits = 1;
  p.out_planes = yt_planes;
  p.ld_planes = ld_planes;
  p.plane_rows = umma_rank_pad(r);
  p.status = status;
  dim3 grid((unsigned)ceil_div(N, 128), 1, (unsigned)S);
  // A launch of at most two CTAs per SM has few neighbours to cover a CTA's load latency: there the CTA keeps four
  // stages in flight itself (64 CTAs streaming 2048-wide rows: 17.4 us with two stages, 15 with four, 14.2 with eight).
  // Not eight: a 161 KB CTA takes its SM for itself, and such launches come from calls small enough to be run side by
  // side on several streams (one encoder layer, three calls on three streams: 0.369 ms per step with eight stages,
  // 0.359 with five, 0.354 with four, 0.365-0.388 with three).
  const int64_t ctas = (int64_t)grid.x * grid.z;
  switch (umma_rank_pad(r)) {
    case 16:
      if (ctas <= 2 * 148) return launch_umma<16, false, false, 2, EPI_YT, 4>(tmX, tmF, p, grid, "rows_dot_tc", st);
      return launch_umma<16, false, false, 2, EPI_YT, 2>(tmX, tmF, p, grid, "rows_dot_tc", st);
    case 32: return launch_umma<32, false, false, 2, EPI_YT, 4>(tmX, tmF, p, grid, "rows_dot_tc", st);
    default:
      if (ctas <= 148) return launch_umma<64, false, false, 2, EPI_YT, 6>(tmX, tmF, p, grid, "rows_dot_tc", st);
      return launch_umma<64, false, false, 2, EPI_YT, 2>(tmX, tmF, p, grid, "rows_dot_tc", st);
  }
}

// Self-test of the bounded waits: one 128 x 64 tile of Y = X F^T whose MMA role is told to expect one block more than
// the producer loads, with a wait limit of 1024 polls.  The extra wait runs out, the CTA raises its abort flag, waits
// (bounded) for the copies and MMAs it has issued, frees its tensor memory, sets *status = DAD_ERR_TIMEOUT and
// returns.  `area` is 64 KB of zeroed device memory for the operands and the result.
cudaError_t umma_selftest_timeout(char* area, int* status, cudaStream_t st) {
  __nv_bfloat16* X = reinterpret_cast<__nv_bfloat16*>(area);             // 128 x 64
  __nv_bfloat16* F = reinterpret_cast<__nv_bfloat16*>(area + 16384);     // 2 planes x 16 x 64
  __nv_bfloat16* Yt = reinterpret_cast<__nv_bfloat16*>(area + 32768);    // 2 planes x 16 x 128
  CUtensorMap tmX, tmF;
  if (!make_tmap_bf16_3d(&tmX, X, 64, 128, 1, 128, 128 * 128, 64, 128) ||
      !make_tmap_bf16_3d(&tmF, F, 64, 16, 2, 128, 16 * 128, 64, 16))
    return cudaErrorInvalidValue;
  UmmaParams p{};
  p.m_extent = 128;
  p.n_extent = 16;
  p.k_blocks = 1;
  p.kb_per_split = 1;
  p.splits = 1;
  p.out_planes = Yt;
  p.ld_planes = 128;
  p.plane_rows = 16;
  p.status = status;
  p.wait_limit = 1024;
  p.expect_extra_kb = 1;
  return launch_umma<16, false, false, 2, EPI_YT, 2>(tmX, tmF, p, dim3(1, 1, 1), "selftest", st);
}

// Z <- Y^T X.  tmX: X as (h, N, S) with box 64 x 64; tmYt: Y^T planes as (N, rp, 2S) with box 64 x rp.
cudaError_t umma_cols_acc(const CUtensorMap& tmX, const CUtensorMap& tmYt, int S, int64_t N, int64_t h, int r, float* out,
                          float* out2, __nv_bfloat16* planes, int64_t ld_planes, float* partial, unsigned* counters,
                          int* status, cudaStream_t st) {
  UmmaParams p{};
  p.m_extent = (int)h;
  p.n_extent = r;
  p.k_blocks = (int)ceil_div(N, 64);
  p.splits = umma_cols_acc_splits(S, N, h);
  p.kb_per_split = (int)ceil_div(p.k_blocks, p.splits);
  p.out_f32 = out;
  p.out2_f32 = out2;
  p.ld_out = h;
  p.out_planes = planes;
  p.ld_planes = ld_planes;
  p.plane_rows = umma_rank_pad(r);
  p.partial = partial;
  p.counters = counters;
  p.status = status;
  dim3 grid((unsigned)ceil_div(h, 128), (unsigned)p.splits, (unsigned)S);
  switch (umma_rank_pad(r)) {
    // r <= 16: when the launch has CTAs for many waves, five shallow CTAs per SM stream better than two deep ones, as
    // in rows_dot (2 / 3 / 4 / 5 stages: 30.8 / 31.0 / 31.2 / 31.5 ms per benchmark step of 2048-CTA launches); with
    // fewer CTAs the 740 slots of the shallow form leave a nearly empty last wave (768 CTAs: 9.2 -> 10.7 ms).  CTAs of
    // at most 16 blocks -- the launches of small calls, which run side by side with other calls' kernels on several
    // streams -- take three stages: they never fill five, and a smaller CTA leaves more of the SM to the neighbours
    // (one encoder layer, three calls on three streams: 0.354 -> 0.344 ms per step; 0.363 with two stages).  Long
    // CTAs that have an SM to themselves keep five (128 CTAs of 64 blocks: 48.2 ms per step with three, 41.4 with five).
    case 16:
      if ((int64_t)grid.x * grid.y * grid.z >= 12 * 148)
        return launch_umma<16, true, false, 2, EPI_Z, 2>(tmX, tmYt, p, grid, "cols_acc_tc", st);
      if (p.kb_per_split <= 16) return launch_umma<16, true, false, 2, EPI_Z, 3>(tmX, tmYt, p, grid, "cols_acc_tc", st);
      return launch_umma<16, true, false, 2, EPI_Z, 5>(tmX, tmYt, p, grid, "cols_acc_tc", st);
    case 32: return launch_umma<32, true, false, 2, EPI_Z, 4>(tmX, tmYt, p, grid, "cols_acc_tc", st);
    default: return launch_umma<64, true, false, 2, EPI_Z, 3>(tmX, tmYt, p, grid, "cols_acc_tc", st);
  }
}

// Geometry of the dense product.  Long contractions (the dAD gradient) over outputs at least 256 x 256 take
// the 256 x 256 two-accumulator kernel; everything else 128 x BN tiles, BN = 256 where the output is wide
// enough (a 128 x 128 x 16 MMA needs 128 B/clk of operands from shared memory, a 128 x 256 x 16 one
// 96 B/clk).  Splits of the contraction fill the 148 SMs when the tiles alone do not.
GemmPlan umma_gemm_plan(int64_t hx, int64_t hy, int S, int64_t N, int batch, int products) {
  GemmPlan g;
  g.products = products;
  const bool big = batch == 1 && hx >= 256 && hy >= 256 && N * S >= kGemm256MinRows;
  int64_t min_blocks;
  if (big) {
    g.bm = 256;
    g.bn = 256;
    g.bk = kGemm256BK;
    g.tiles = ceil_div(hx, 256) * ceil_div(hy, 256) * products;  // of all the products of the launch
    min_blocks = 512 / g.bk;
  } else {
    g.bm = 128;
    g.bn = (hy > 128 && ceil_div(hx, 128) * ceil_div(hy, 256) * batch >= 74) ? 256 : 128;  // narrow tiles while SMs would idle
    g.bk = 64;
    g.tiles = ceil_div(hx, 128) * ceil_div(hy, g.bn);
    min_blocks = 8;
  }
  g.kb_per_site = ceil_div(N, g.bk);
  g.k_blocks = g.kb_per_site * S;
  g.batch = batch;
  int64_t splits = 148 / (g.tiles * batch);
  if (splits > g.k_blocks / min_blocks) splits = g.k_blocks / min_blocks;
  if (splits > 32) splits = 32;
  if (splits < 1) splits = 1;
  const int64_t per = ceil_div(g.k_blocks, splits);
  g.splits = (int)ceil_div(g.k_blocks, per);  // no empty split
  g.kb_per_split = per;
  g.rem_ctas = 0;
  if (big) {
    // SMs that tiles * splits leaves empty (64 tiles x 2 splits: 20 of 148) take the tail of every tile's contraction,
    // each for ceil(tiles / R) tiles in turn.  Balance: a CTA of the main part runs kb_main blocks and one epilogue, a
    // remainder CTA tpr times (kb_rem blocks and an epilogue); the epilogue and the refill of the pipeline are put at
    // the time of 30 blocks (measured on the 1024 x 4096 gradient over 65 536 rows: 0 / 12 / 30 / 60 / 100 blocks give
    // 383 / 370 / 369 / 373 / 376 us, 378 us without remainder CTAs -- the 20 extra SMs buy 2.4 %, not their 13.5 %
    // share: with every SM multiplying the clock settles lower under the power limit).
    const int64_t R = 148 - g.tiles * g.splits;
    if (R >= 8) {
      const int64_t tpr = ceil_div(g.tiles, R), ovh = 30;
      const int64_t kb_rem = (g.k_blocks - g.splits * (tpr - 1) * ovh) / (g.splits * tpr + 1);
      const int64_t kb_main = ceil_div(g.k_blocks - kb_rem, g.splits);
      if (kb_rem >= 32 && g.k_blocks - g.splits * kb_main >= 16) {
        g.rem_ctas = (int)R;
        g.kb_per_split = kb_main;
      }
    }
  }
  return g;
}

template <int BK, int STAGES>
static cudaError_t launch_gemm256(const CUtensorMap& tmA, const CUtensorMap& tmB, const UmmaParams& p, dim3 grid,
                                  cudaStream_t st) {
  constexpr size_t smem = (size_t)STAGES * 8 * BK * 128 + 1024;
  auto kernel = umma_gemm256_kernel<BK, STAGES>;
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
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const bool timed = g_timing.load(std::memory_order_relaxed);
  if (timed) timing_mark("gemm_tn_tc", st, true);
  err = cudaLaunchKernelEx(&cfg, kernel, tmA, tmB, p);
  if (timed) timing_mark("gemm_tn_tc", st, false);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return err;
}

template <int STAGES>
static cudaError_t launch_gemm_persist(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC,
                                       const UmmaParams& p, unsigned ctas, cudaStream_t st) {
  constexpr size_t smem = (size_t)STAGES * (6 * 8192) + 2 * 128 * 128 + 1024;
  auto kernel = umma_gemm_persist_kernel<STAGES>;
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
  cfg.gridDim = dim3(ctas, 1, 1);
  cfg.blockDim = dim3(192, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const bool timed = g_timing.load(std::memory_order_relaxed);
  if (timed) timing_mark("gemm_tn_tc", st, true);
  err = cudaLaunchKernelEx(&cfg, kernel, tmA, tmB, tmC, p);
  if (timed) timing_mark("gemm_tn_tc", st, false);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return err;
}


template <int STAGES>
static cudaError_t launch_gemm_pair(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC,
                                    const UmmaParams& p, unsigned ctas, cudaStream_t st) {
  constexpr size_t smem = (size_t)STAGES * (4 * 8192) + 2 * 128 * 128 + 1024;
  auto kernel = umma_gemm_pair_kernel<STAGES>;
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
  cfg.gridDim = dim3(ctas, 1, 1);
  cfg.blockDim = dim3(192, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = 2;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  const bool timed = g_timing.load(std::memory_order_relaxed);
  if (timed) timing_mark("gemm_tn_tc", st, true);
  err = cudaLaunchKernelEx(&cfg, kernel, tmA, tmB, tmC, p);
  if (timed) timing_mark("gemm_tn_tc", st, false);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return err;
}

// C (hx x hy, fp32) <- sum over sites and rows of X^T Y.  tmX: (hx, N, S), tmY: (hy, N, S), boxes 64 x plan.bk.
// With plan.batch > 1 (and S = 1) the third tensor dimension counts independent products instead: C is batch x hx x hy.
cudaError_t umma_gemm_tn(const CUtensorMap& tmX, const CUtensorMap& tmY, const GemmPlan& g, int64_t hx, int64_t hy,
                         float* C, float* partial, unsigned* counters, int* status, cudaStream_t st) {
  UmmaParams p{};
  p.m_extent = (int)hx;
  p.n_extent = (int)hy;
  p.kb_per_site = g.batch > 1 ? 0 : (int)g.kb_per_site;  // batched: one site per entry, the entry from blockIdx.z
  p.k_blocks = (int)g.k_blocks;
  p.splits = g.splits;
  p.kb_per_split = (int)g.kb_per_split;
  p.rem_ctas = g.rem_ctas;
  p.tiles_m = (int)ceil_div(hx, g.bm);
  p.tiles_n = (int)ceil_div(hy, g.bn);
  p.out_f32 = C;
  p.ld_out = hy;
  p.out_batch_stride = hx * hy;
  p.partial = partial;
  p.counters = counters;
  p.status = status;
  dim3 grid((unsigned)ceil_div(hx, g.bm), (unsigned)(ceil_div(hy, g.bn) * g.splits), (unsigned)g.batch);
  if (g.bm == 256) {
    p.batch_count = g.products;
    p.sites_per_product = (int)(g.k_blocks / g.kb_per_site);
    const int slots = g.splits + (g.rem_ctas > 0 ? 1 : 0);
    const dim3 grid1((unsigned)(g.tiles * g.splits + g.rem_ctas), 1, 1);
    cudaError_t err = launch_gemm256<kGemm256BK, kGemm256Stages>(tmX, tmY, p, grid1, st);
    if (err != cudaSuccess || slots == 1) return err;
    const int64_t quads = hx * hy / 4;
    unsigned blocks = (unsigned)(quads / 256 < 148 * 8 ? ceil_div(quads, 256) : 148 * 8);
    blocks = (blocks + g.products - 1) / g.products;
    if (blocks < 1) blocks = 1;
    DAD_LAUNCH(err, "gemm_tn_reduce", gemm256_reduce_kernel, dim3(blocks, (unsigned)g.products, 1), 256, 0, st,
               (const float*)partial, slots, (int)hx, (int)hy, C);
    return err;
  }
  // Short contractions (the reconstruction: 3 S r rows) spend as long in the epilogue -- 128 KB of fp32 per tile -- as in
  // the MMAs: two shallow CTAs per SM, one draining its accumulator while the other multiplies, instead of one deep one.
  const bool shallow = p.kb_per_split <= 64;
  // Without a split contraction the tile goes out through TMA stores (whole lines, asynchronous); C is hx x hy fp32,
  // contiguous, one matrix per batch entry.
  CUtensorMap tmC;
  const CUtensorMap* pC = nullptr;
  if (g.splits == 1 && make_tmap_f32_3d(&tmC, C, (uint64_t)hy, (uint64_t)hx, (uint64_t)g.batch, (uint64_t)hy * 4,
                                        (uint64_t)hx * hy * 4, 128)) {
    p.tma_store = 1;
    pC = &tmC;
  }
  // Many 128 x 256 tiles of a short contraction over one site per product: the persistent kernel (one CTA per SM, two
  // accumulators).  Its blocks are numbered per product, so a contraction over several sites keeps the per-tile CTAs.
  const int64_t all_tiles = g.tiles * g.batch;
  // Enough 256 x 256 tiles for every pair of SMs: the pair kernel, which needs a third fewer operand bytes per SM.
  const int64_t tiles256 = ceil_div(hx, 256) * ceil_div(hy, 256) * g.batch;
  if (pC && g.bn == 256 && tiles256 >= 74 && g_pair_gemm && (g.batch > 1 || g.k_blocks == g.kb_per_site)) {
    p.batch_count = g.batch;
    p.tiles_m = (int)ceil_div(hx, 256);
    p.tiles_n = (int)ceil_div(hy, 256);
    return launch_gemm_pair<5>(tmX, tmY, tmC, p, 148u, st);
  }
  if (pC && g.bn == 256 && all_tiles >= 148 && p.k_blocks <= 8 && (g.batch > 1 || g.k_blocks == g.kb_per_site)) {
    p.batch_count = g.batch;
    return launch_gemm_persist<3>(tmX, tmY, tmC, p, 148u, st);
  }
  if (g.bn == 256) {
    if (shallow) return launch_umma<256, true, true, 1, EPI_C, 2>(tmX, tmY, p, grid, "gemm_tn_tc", st, pC);
    return launch_umma<256, true, true, 1, EPI_C, 4>(tmX, tmY, p, grid, "gemm_tn_tc", st, pC);
  }
  if (shallow) return launch_umma<128, true, true, 1, EPI_C, 3>(tmX, tmY, p, grid, "gemm_tn_tc", st, pC);
  return launch_umma<128, true, true, 1, EPI_C, 6>(tmX, tmY, p, grid, "gemm_tn_tc", st, pC);
}

}  // namespace dad

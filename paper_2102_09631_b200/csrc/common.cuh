// Shared declarations of the libdad translation units: launch accounting, the workspace
// layout of dad_rank_compress, and the host-side launchers of every kernel family.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <atomic>

#include "dad.h"

namespace dad {

extern std::atomic<uint64_t> g_launches;

// Optional per-kernel timing (dad_timing_*): CUDA events recorded around every launch on the
// launching stream, summed per tag when collected.  Off by default; no cost when off.
extern std::atomic<bool> g_timing;
void timing_mark(const char* tag, cudaStream_t st, bool begin);

// Launch a kernel under a tag, count it and fold its launch error into `err` (first error wins).
#define DAD_LAUNCH(err, tag, kernel, grid, block, smem, stream, ...)            \
  do {                                                                          \
    const bool t__ = ::dad::g_timing.load(std::memory_order_relaxed);           \
    if (t__) ::dad::timing_mark(tag, stream, true);                             \
    kernel<<<grid, block, smem, stream>>>(__VA_ARGS__);                         \
    cudaError_t e__ = cudaGetLastError();                                       \
    if (t__) ::dad::timing_mark(tag, stream, false);                            \
    ::dad::g_launches.fetch_add(1, std::memory_order_relaxed);                  \
    if ((err) == cudaSuccess) (err) = e__;                                      \
  } while (0)

// True the first time it is asked on each device (per object): for per-function set-up such as the opt-in to
// large dynamic shared memory, which need not be repeated at every launch.
struct FirstUse {
  std::atomic<uint64_t> seen{0};
  int last = -1;
  bool on_this_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev > 63) return true;
    last = dev;
    const uint64_t bit = 1ull << dev;
    return (seen.fetch_or(bit, std::memory_order_relaxed) & bit) == 0;
  }
  void forget() {
    if (last >= 0) seen.fetch_and(~(1ull << last), std::memory_order_relaxed);
  }
};

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }

// ---- geometry shared by launchers and the workspace carve --------------------------------
constexpr int kColsAccThreads = 128;  // columns per CTA of the column-slab product
constexpr int kGramChunk = 64;        // columns per CTA of the Gram kernel

// Row splits of the column-slab product Z = Y^T X, chosen from the shape alone so that the
// launch fills the GPU; identical for workspace sizing and launching.
int cols_acc_splits(int S, int64_t N, int64_t h);

// Workspace of dad_rank_compress; all offsets in bytes from the (256-aligned) base.
struct CompressWs {
  size_t status;        // int32 status word (+ padding)
  size_t counters;      // uint32 arrival counters of the split reductions
  size_t n_counters;
  size_t n_pair_counters;  // of those: chunk counters of the one-launch pairs (before the last S, the Gram kernel's)
  size_t G;             // S*r*h_out accumulator-type iterate (fp64 pipeline only)
  size_t Y;             // S*N*r
  size_t Z;             // S*r*h_in
  size_t partial;       // S*splits*r*max(h) partial column slabs
  size_t gram_partial;  // S*chunks*r*r doubles
  size_t gram;          // S*r*r doubles (Cholesky factor after the Gram kernel)
  size_t tratio;        // S*r doubles: R_jj / ||column|| after the first pass
  size_t dead;          // S*r bytes, then S ints: whether the site needs the second pass
  // tensor-core pipeline: bf16 two-term (hi + lo) splits of the small fp32 operands
  size_t Fq;            // S*2*rp*h_out bf16: planes of the iterate G (operand of D G^T)
  size_t Fz;            // S*2*rp*h_in  bf16: planes of Z (operand of A Z^T)
  size_t Yt;            // S*2*rp*Npad  bf16: planes of Y^T (operand of Y^T A and W^T D)
  int64_t Npad;
  size_t tc_partial;    // split partial tiles of the tensor-core column products
  // one-launch compress: per-CTA partial sums S*C*r*max(h) of the accumulator type, slice lengths S*C*r doubles
  size_t fused_part, fused_sig;
  size_t total;
};
// f64: fp64 pipeline (fp32 inputs); tc: tensor-core pipeline (bf16 inputs, 16-byte-aligned layout);
// fused_c: cluster size of the one-launch compress (0: not used for this shape)
CompressWs compress_ws_layout(const dad_layer& L, int r, bool f64, bool tc, int fused_c);

// One-launch compress of small sites (fused_site.cu): a cluster of `C` CTAs per site runs the whole structured
// power iteration.  fused_cluster_size gives C for a shape, or 0 when the multi-launch pipelines take it.
int fused_cluster_size(const dad_layer& L, int r, int iters);
// The on-chip form of it (fused_dsm.cu): factor, Y and the rows of A and D in shared memory, every exchange over
// distributed shared memory; preferred where its buffers fit.
bool fused_dsm_fits(const dad_layer& L, int r, int C, bool* x_resident);
cudaError_t fused_dsm_compress(const dad_layer& L, const void* A, const void* D, int r, int iters, const float* Q0, float* P,
                               float* Q, float* sigma, int* status, int C, cudaStream_t st);
cudaError_t fused_compress(const dad_layer& L, const void* A, const void* D, int r, int iters, const float* Q0, float* P,
                           float* Q, float* sigma, void* FG, void* FZ, void* part, double* sig_part, int* status, int C,
                           cudaStream_t st);

// Workspace of dad_full_grad and of dad_reconstruct on the tensor cores.
struct GemmWs {
  size_t status, counters, n_counters, partial, Xb, Yb, total;  // Xb/Yb: bf16 copies of fp32 operands
};
GemmWs gemm_ws_layout(int64_t hx, int64_t hy, int S, int64_t N, bool convert_operands, int batch = 1, int products = 1);

// Whether the tensor-core kernels take this layer: bf16, all extents and strides multiples of 8
// elements (TMA wants 16-byte strides), and the driver's tensor-map encoder is available.
bool tc_eligible(const dad_layer& L);

// ---- launchers (all asynchronous on `st`; return the first CUDA error) ------------------------
// Y[s][n][j] = sum_c X[s][n][c] * F[s][j][c]      X: N x h (ld, site stride), F: r x h, Y: N x r
template <typename TAcc>
cudaError_t rows_dot(dad_dtype dt, const void* X, int64_t ld, int64_t stride, int S, int64_t N, int64_t h,
                     const TAcc* F, int r, TAcc* Y, cudaStream_t st);

// Z[s][j][c] = sum_n Y[s][n][j] * X[s][n][c]      Z: r x h; also written as fp32 to out32 if given
template <typename TAcc>
cudaError_t cols_acc(dad_dtype dt, const void* X, int64_t ld, int64_t stride, int S, int64_t N, int64_t h,
                     const TAcc* Y, int r, TAcc* Z, float* out32, TAcc* partial, unsigned* counters,
                     cudaStream_t st);

// One Cholesky-QR pass on the rows of G (S x r x h, in place): Gram -> factor -> triangular solve.
// pass = 0: first pass (records R_jj/||g_j||); pass = 1: second pass, zeroes rows whose total
// remainder is <= tol of their length.  out32 (optional) receives an fp32 copy of the result.
template <typename T>
cudaError_t cholqr_pass(T* G, int S, int r, int64_t h, int pass, double tol, double* gram_partial,
                        double* gram, double* tratio, unsigned char* dead, int* need2, unsigned* counters,
                        int* status, float* out32, __nv_bfloat16* planes, int plane_rows, cudaStream_t st);

// The same orthonormalisation (both passes, second one decided on the device) in one launch, for
// fp32 or fp64 storage (T): a thread-block cluster per site keeps the vectors in shared memory throughout.
bool orth_cluster_fits(int r, int64_t h, size_t elem_bytes = 4);
template <typename T>
cudaError_t orth_cluster(T* G, int S, int r, int64_t h, double tol, int* status, float* out32,
                         __nv_bfloat16* planes, int plane_rows, cudaStream_t st);
// fp32 storage with the Gram and substitution phases on the fp64 matrix-multiply unit (orth_mma.cu).
bool orth_mma_fits(int r, int64_t h);
cudaError_t orth_mma(float* G, int S, int r, int64_t h, double tol, int* status, float* out32, __nv_bfloat16* planes,
                     int plane_rows, cudaStream_t st);
// The same phases as two launches per pass, the factorisation once per site; preferred for many sites at r >= 32.
// Scratch as for cholqr_pass (gram_partial, gram, tratio, dead, need2, counters), which is large enough when preferred.
bool orth_split_preferred(int r, int64_t h, int S);
cudaError_t orth_split(float* G, int S, int r, int64_t h, double tol, double* gram_partial, double* gram, double* tratio,
                       unsigned char* dead, int* need2, unsigned* counters, int* status, float* out32,
                       __nv_bfloat16* planes, int plane_rows, cudaStream_t st);

// C[a][b] = sum_{s,n} X[s][n][a] * Y[s][n][b]  (fp32 FMA), C: hx x hy fp32 contiguous
cudaError_t gemm_tn_simt(dad_dtype dt, const void* X, int64_t ldX, int64_t strideX, const void* Y,
                         int64_t ldY, int64_t strideY, int S, int64_t N, int64_t hx, int64_t hy, float* C,
                         cudaStream_t st);

cudaError_t copy_two(const float* a, float* a_out, size_t na, const float* b, float* b_out, size_t nb,
                     cudaStream_t st);
cudaError_t widen_f32_to_f64(const float* in, double* out, size_t n, cudaStream_t st);
template <typename T>
cudaError_t row_norms(const T* M, int64_t rows, int64_t h, float* out, cudaStream_t st);
// planes[s][0/1][j][c] = hi / lo bf16 terms of in[s][j][c]  (j < r; plane_rows >= r rows per plane)
cudaError_t split_planes(const float* in, int S, int r, int64_t h, __nv_bfloat16* planes, int plane_rows,
                         cudaStream_t st);
// bf16 operand stacks of `batch` reconstructions, three-term (terms = 3) or hi terms only (terms = 1): P is
// batch x (nP elements), X3 is batch x terms x nP, same for Q.
cudaError_t stack_split3(const float* P, size_t nP, __nv_bfloat16* X3, const float* Q, size_t nQ, __nv_bfloat16* Y3,
                         int batch, int terms, cudaStream_t st);

// ---- tensor-core launchers (umma_gemm.cu) -------------------------------------------------------
bool tmap_encoder_available();
bool make_tmap_bf16_3d(CUtensorMap* map, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t s1_bytes,
                       uint64_t s2_bytes, uint32_t box0, uint32_t box1);
int umma_rank_pad(int r);
int umma_cols_acc_splits(int S, int64_t N, int64_t h);
// Geometry of the dense product C = X^T Y (hx x hy, contraction over S sites of N rows): tile bm x bn, stages of
// bk contraction rows (the row count of the operands' TMA boxes), `splits` CTAs share a tile's contraction.
struct GemmPlan {
  int bm, bn, bk, splits, batch;
  int products;                          // 256 x 256 tiles: products of S sites each that share the launch (tiles counts all)
  int rem_ctas;                          // 256 x 256 tiles: CTAs that take the tail of every tile's contraction
  int64_t tiles, k_blocks, kb_per_site;  // tiles: per batch entry
  int64_t kb_per_split;                  // blocks of each of the `splits` equal parts
};
// batch > 1: that many independent products of one site each (S must be 1) in one launch.
GemmPlan umma_gemm_plan(int64_t hx, int64_t hy, int S, int64_t N, int batch, int products = 1);
cudaError_t umma_rows_dot(const CUtensorMap& tmX, const CUtensorMap& tmF, int S, int64_t N, int64_t h, int r,
                          __nv_bfloat16* yt_planes, int64_t ld_planes, int* status, cudaStream_t st);
cudaError_t umma_cols_acc(const CUtensorMap& tmX, const CUtensorMap& tmYt, int S, int64_t N, int64_t h, int r, float* out,
                          float* out2, __nv_bfloat16* planes, int64_t ld_planes, float* partial, unsigned* counters,
                          int* status, cudaStream_t st);
// One launch for the pair Z = (X1 F^T)^T X2 (umma_pair.cu): whether it takes a shape, the partial blocks it needs, launch.
bool umma_pair_fits(int S, int64_t N, int64_t h2, int r);
size_t umma_pair_partial_bytes(int S, int64_t N, int64_t h2, int r);
cudaError_t umma_pair(const CUtensorMap& tmX1, const CUtensorMap& tmF, const CUtensorMap& tmX2, int S, int64_t N, int64_t h1,
                      int64_t h2, int r, float* out, float* out2, __nv_bfloat16* planes, int64_t ld_planes, float* partial,
                      unsigned* counters, int* status, cudaStream_t st);
cudaError_t umma_selftest_timeout(char* area, int* status, cudaStream_t st);
cudaError_t umma_gemm_tn(const CUtensorMap& tmX, const CUtensorMap& tmY, const GemmPlan& plan, int64_t hx, int64_t hy,
                         float* C, float* partial, unsigned* counters, int* status, cudaStream_t st);

}  // namespace dad

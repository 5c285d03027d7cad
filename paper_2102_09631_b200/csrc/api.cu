// C ABI entry points of libdad: argument validation, workspace carving, byte accounting and
// the launch sequence of each call.  Every step of the path runs in the kernels of this
// library; there is no host fallback.
#include <cstring>

#include "common.cuh"

namespace dad {

std::atomic<uint64_t> g_launches{0};

static bool layer_ok(const dad_layer* L) {
  if (!L) return false;
  if (L->S < 1 || L->N < 1 || L->h_in < 1 || L->h_out < 1) return false;
  if (L->S > 65535) return false;
  return true;
}

static dad_status validate_layer(const dad_layer* L) {
  if (!L) return DAD_ERR_NULL;
  if (L->dtype != DAD_F32 && L->dtype != DAD_BF16) return DAD_ERR_DTYPE;
  if (!layer_ok(L)) return DAD_ERR_SHAPE;
  if (L->ldA < L->h_in || L->ldD < L->h_out) return DAD_ERR_SHAPE;
  if (L->S > 1 && (L->strideA < L->N * L->ldA || L->strideD < L->N * L->ldD)) return DAD_ERR_SHAPE;
  // 63-bit element counts
  const double big = 9.0e18;
  if ((double)L->S * (double)L->N * (double)(L->ldA > L->ldD ? L->ldA : L->ldD) * 8.0 > big) return DAD_ERR_SHAPE;
  return DAD_OK;
}

static bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

CompressWs compress_ws_layout(const dad_layer& L, int r, bool f64) {
  CompressWs w;
  memset(&w, 0, sizeof(w));
  const size_t acc = f64 ? 8 : 4;
  const size_t S = (size_t)L.S, N = (size_t)L.N, hi = (size_t)L.h_in, ho = (size_t)L.h_out, rr = (size_t)r;
  const size_t hmax = hi > ho ? hi : ho;
  size_t off = 0;
  w.status = off;
  off += 256;
  w.n_counters = S * (size_t)ceil_div((int64_t)hmax, kColsAccThreads) + S;
  w.counters = off;
  off = align_up(off + w.n_counters * sizeof(unsigned), 256);
  w.G = off;
  off = align_up(off + (f64 ? S * rr * ho * acc : 0), 256);
  w.Y = off;
  off = align_up(off + S * N * rr * acc, 256);
  w.Z = off;
  off = align_up(off + S * rr * hi * acc, 256);
  const int s_in = cols_acc_splits(L.S, L.N, L.h_in), s_out = cols_acc_splits(L.S, L.N, L.h_out);
  size_t part = 0;
  if (s_in > 1) part = S * (size_t)s_in * rr * hi * acc;
  if (s_out > 1 && S * (size_t)s_out * rr * ho * acc > part) part = S * (size_t)s_out * rr * ho * acc;
  w.partial = off;
  off = align_up(off + part, 256);
  w.gram_partial = off;
  off = align_up(off + S * (size_t)ceil_div((int64_t)ho, kGramChunk) * rr * rr * 8, 256);
  w.gram = off;
  off = align_up(off + S * rr * rr * 8, 256);
  w.tratio = off;
  off = align_up(off + S * rr * 8, 256);
  w.dead = off;
  off = align_up(off + S * rr, 256);
  w.Fsplit = off;
  w.Ysplit = off;
  w.total = off;
  return w;
}

template <typename TAcc>
static cudaError_t run_compress(const dad_layer& L, const void* A, const void* D, int r, int iters, const float* Q0,
                                float* P, float* Q, float* sigma, char* ws, const CompressWs& w, cudaStream_t st) {
  constexpr bool f64 = sizeof(TAcc) == 8;
  const int S = L.S;
  const int64_t N = L.N, hi = L.h_in, ho = L.h_out;
  cudaError_t err = cudaMemsetAsync(ws + w.status, 0, w.counters + w.n_counters * sizeof(unsigned) - w.status, st);
  if (err != cudaSuccess) return err;
  int* status = reinterpret_cast<int*>(ws + w.status);
  unsigned* ctr_cols = reinterpret_cast<unsigned*>(ws + w.counters);
  unsigned* ctr_gram = ctr_cols + (w.n_counters - (size_t)S);
  TAcc* Y = reinterpret_cast<TAcc*>(ws + w.Y);
  TAcc* Z = reinterpret_cast<TAcc*>(ws + w.Z);
  TAcc* part = reinterpret_cast<TAcc*>(ws + w.partial);
  double* gram_partial = reinterpret_cast<double*>(ws + w.gram_partial);
  double* gram = reinterpret_cast<double*>(ws + w.gram);
  double* tratio = reinterpret_cast<double*>(ws + w.tratio);
  unsigned char* dead = reinterpret_cast<unsigned char*>(ws + w.dead);
  const double tol = f64 ? 1e-12 : 1e-6;
  TAcc* G;
  if constexpr (f64) {
    G = reinterpret_cast<TAcc*>(ws + w.G);
    err = widen_f32_to_f64(Q0, G, (size_t)S * r * ho, st);
    if (err == cudaSuccess && iters == 0 && Q != Q0)
      err = cudaMemcpyAsync(Q, Q0, sizeof(float) * (size_t)S * r * ho, cudaMemcpyDeviceToDevice, st);
  } else {
    G = reinterpret_cast<TAcc*>(Q);
    if (Q != Q0) err = cudaMemcpyAsync(Q, Q0, sizeof(float) * (size_t)S * r * ho, cudaMemcpyDeviceToDevice, st);
  }
  if (err != cudaSuccess) return err;
#define DAD_STEP(call)          \
  do {                          \
    err = (call);               \
    if (err != cudaSuccess) return err; \
  } while (0)
  for (int k = 0; k < iters; ++k) {
    DAD_STEP(rows_dot<TAcc>(L.dtype, D, L.ldD, L.strideD, S, N, ho, G, r, Y, st));                        // Y = D G^T
    DAD_STEP(cols_acc<TAcc>(L.dtype, A, L.ldA, L.strideA, S, N, hi, Y, r, Z, nullptr, part, ctr_cols, st));  // Z = Y^T A
    DAD_STEP(rows_dot<TAcc>(L.dtype, A, L.ldA, L.strideA, S, N, hi, Z, r, Y, st));                        // W = A Z^T
    DAD_STEP(cols_acc<TAcc>(L.dtype, D, L.ldD, L.strideD, S, N, ho, Y, r, G, nullptr, part, ctr_cols, st));  // Gt = W^T D
    DAD_STEP(cholqr_pass<TAcc>(G, S, r, ho, 0, tol, gram_partial, gram, tratio, dead, ctr_gram, status, nullptr, st));
    float* q32 = (f64 && k == iters - 1) ? Q : nullptr;
    DAD_STEP(cholqr_pass<TAcc>(G, S, r, ho, 1, tol, gram_partial, gram, tratio, dead, ctr_gram, status, q32, st));
  }
  DAD_STEP(rows_dot<TAcc>(L.dtype, D, L.ldD, L.strideD, S, N, ho, G, r, Y, st));
  DAD_STEP(cols_acc<TAcc>(L.dtype, A, L.ldA, L.strideA, S, N, hi, Y, r, Z, P, part, ctr_cols, st));
  if (sigma) DAD_STEP(row_norms<TAcc>(Z, (int64_t)S * r, hi, sigma, st));
#undef DAD_STEP
  return cudaSuccess;
}

}  // namespace dad

using namespace dad;

extern "C" {

uint64_t dad_bytes_dad(const dad_layer* L) {
  if (!layer_ok(L) || (L->dtype != DAD_F32 && L->dtype != DAD_BF16)) return 0;
  const uint64_t e = L->dtype == DAD_F32 ? 4u : 2u;
  return (uint64_t)L->N * (uint64_t)(L->h_in + L->h_out) * e;
}

uint64_t dad_bytes_rank(const dad_layer* L, int r) {
  if (!layer_ok(L) || r < 1) return 0;
  return (uint64_t)r * (uint64_t)(L->h_in + L->h_out) * 4u;
}

uint64_t dad_bytes_dsgd(const dad_layer* L) {
  if (!layer_ok(L)) return 0;
  return (uint64_t)L->h_in * (uint64_t)L->h_out * 4u;
}

static dad_status validate_rank(const dad_layer* L, int r) {
  if (r < 1 || r > DAD_MAX_RANK || r > L->h_in || r > L->h_out) return DAD_ERR_RANK;
  return DAD_OK;
}

size_t dad_workspace_bytes(const dad_layer* L, int r, int iters) {
  if (validate_layer(L) != DAD_OK || validate_rank(L, r) != DAD_OK || iters < 0) return 0;
  return compress_ws_layout(*L, r, L->dtype == DAD_F32).total;
}

dad_status dad_full_grad(const dad_layer* L, const void* A, const void* D, float* grad, uint64_t* bytes_tx,
                         void* ws, size_t ws_bytes, void* cuda_stream) {
  dad_status vs = validate_layer(L);
  if (vs != DAD_OK) return vs;
  if (!A || !D || !grad) return DAD_ERR_NULL;
  if (!aligned(A, 16) || !aligned(D, 16) || !aligned(grad, 16)) return DAD_ERR_ALIGN;
  (void)ws;
  (void)ws_bytes;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  cudaError_t err = gemm_tn_simt(L->dtype, A, L->ldA, L->strideA, D, L->ldD, L->strideD, L->S, L->N, L->h_in,
                                 L->h_out, grad, st);
  if (err != cudaSuccess) return DAD_ERR_CUDA;
  if (bytes_tx)
    for (int s = 0; s < L->S; ++s) bytes_tx[s] = dad_bytes_dad(L);
  return DAD_OK;
}

dad_status dad_rank_compress(const dad_layer* L, const void* A, const void* D, int r, int iters, const float* Q0,
                             float* P, float* Q, float* sigma, void* ws, size_t ws_bytes, void* cuda_stream) {
  dad_status vs = validate_layer(L);
  if (vs != DAD_OK) return vs;
  if (!A || !D || !Q0 || !P || !Q || !ws) return DAD_ERR_NULL;
  vs = validate_rank(L, r);
  if (vs != DAD_OK) return vs;
  if (iters < 0 || iters > 1000000) return DAD_ERR_SHAPE;
  if (!aligned(A, 16) || !aligned(D, 16) || !aligned(Q0, 16) || !aligned(P, 16) || !aligned(Q, 16) ||
      !aligned(ws, 256) || (sigma && !aligned(sigma, 4)))
    return DAD_ERR_ALIGN;
  const bool f64 = L->dtype == DAD_F32;
  const CompressWs w = compress_ws_layout(*L, r, f64);
  if (ws_bytes < w.total) return DAD_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  cudaError_t err = f64 ? run_compress<double>(*L, A, D, r, iters, Q0, P, Q, sigma, (char*)ws, w, st)
                        : run_compress<float>(*L, A, D, r, iters, Q0, P, Q, sigma, (char*)ws, w, st);
  return err == cudaSuccess ? DAD_OK : DAD_ERR_CUDA;
}

dad_status dad_gather_factors(const dad_layer* L, int r, const float* P, const float* Q, float* Pcat, float* Qcat,
                              uint64_t* bytes_tx, void* cuda_stream) {
  if (!L) return DAD_ERR_NULL;
  if (!layer_ok(L)) return DAD_ERR_SHAPE;
  if (r < 1 || r > DAD_MAX_RANK) return DAD_ERR_RANK;
  if (!P || !Q || !Pcat || !Qcat) return DAD_ERR_NULL;
  if (!aligned(P, 4) || !aligned(Q, 4) || !aligned(Pcat, 4) || !aligned(Qcat, 4)) return DAD_ERR_ALIGN;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (P != Pcat || Q != Qcat) {
    cudaError_t err = copy_two(P, Pcat, (size_t)L->S * r * L->h_in, Q, Qcat, (size_t)L->S * r * L->h_out, st);
    if (err != cudaSuccess) return DAD_ERR_CUDA;
  }
  if (bytes_tx)
    for (int s = 0; s < L->S; ++s) bytes_tx[s] = dad_bytes_rank(L, r);
  return DAD_OK;
}

size_t dad_reconstruct_workspace_bytes(int64_t h_in, int64_t h_out, int64_t K, dad_dtype math) {
  (void)h_in;
  (void)h_out;
  (void)K;
  (void)math;
  return 0;
}

dad_status dad_reconstruct(int64_t h_in, int64_t h_out, int64_t K, const float* Pcat, const float* Qcat, float* grad,
                           dad_dtype math, void* ws, size_t ws_bytes, void* cuda_stream) {
  if (h_in < 1 || h_out < 1 || K < 1) return DAD_ERR_SHAPE;
  if (math != DAD_F32 && math != DAD_BF16) return DAD_ERR_DTYPE;
  if (!Pcat || !Qcat || !grad) return DAD_ERR_NULL;
  if (!aligned(Pcat, 16) || !aligned(Qcat, 16) || !aligned(grad, 16)) return DAD_ERR_ALIGN;
  if (ws_bytes < dad_reconstruct_workspace_bytes(h_in, h_out, K, math)) return DAD_ERR_WORKSPACE;
  (void)ws;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  cudaError_t err = gemm_tn_simt(DAD_F32, Pcat, h_in, 0, Qcat, h_out, 0, 1, K, h_in, h_out, grad, st);
  return err == cudaSuccess ? DAD_OK : DAD_ERR_CUDA;
}

dad_status dad_check(const void* ws, void* cuda_stream) {
  if (!ws) return DAD_ERR_NULL;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  int status = 0;
  if (cudaMemcpyAsync(&status, ws, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return DAD_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return DAD_ERR_CUDA;
  if (status == (int)DAD_ERR_TIMEOUT || status == (int)DAD_ERR_NUMERIC) return (dad_status)status;
  return DAD_OK;
}

uint64_t dad_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* dad_status_string(dad_status s) {
  switch (s) {
    case DAD_OK: return "ok";
    case DAD_ERR_NULL: return "a required pointer is NULL";
    case DAD_ERR_SHAPE: return "shape or stride out of range";
    case DAD_ERR_DTYPE: return "unsupported dtype";
    case DAD_ERR_RANK: return "rank r out of range";
    case DAD_ERR_WORKSPACE: return "workspace too small";
    case DAD_ERR_ALIGN: return "pointer or stride misaligned";
    case DAD_ERR_CUDA: return "CUDA runtime error";
    case DAD_ERR_TIMEOUT: return "bounded device-side wait ran out";
    case DAD_ERR_NUMERIC: return "non-finite value reached the orthonormalisation";
  }
  return "unknown status";
}

}  // extern "C"

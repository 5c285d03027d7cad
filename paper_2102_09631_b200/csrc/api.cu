// C ABI entry points of libdad: argument validation, workspace carving, byte accounting and
// the launch sequence of each call.  Every step of the path runs in the kernels of this
// library; there is no host fallback.
#include <cstring>

#include "bounds.cuh"
#include "common.cuh"

namespace dad {

std::atomic<uint64_t> g_launches{0};
static std::atomic<bool> g_fused_on{true};
static std::atomic<bool> g_pair_on{false};

static bool layer_ok(const dad_layer* L) {
  if (!L) return false;
  if (L->S < 1 || L->N < 1 || L->h_in < 1 || L->h_out < 1) return false;
  if (L->S > 65535) return false;
  if (L->N > 0x7fffffff || L->h_in > 0x7fffffff || L->h_out > 0x7fffffff) return false;
  return true;
}

static dad_status validate_layer(const dad_layer* L) {
  if (!L) return DAD_ERR_NULL;
  if (L->dtype != DAD_F32 && L->dtype != DAD_BF16) return DAD_ERR_DTYPE;
  if (!layer_ok(L)) return DAD_ERR_SHAPE;
  if (L->ldA < L->h_in || L->ldD < L->h_out) return DAD_ERR_SHAPE;
  if (L->S > 1 && (L->strideA < L->N * L->ldA || L->strideD < L->N * L->ldD)) return DAD_ERR_SHAPE;
  const double big = 9.0e18;  // element counts must fit 63 bits
  if ((double)L->S * (double)L->N * (double)(L->ldA > L->ldD ? L->ldA : L->ldD) * 8.0 > big) return DAD_ERR_SHAPE;
  return DAD_OK;
}

// Bytes from the base of A (or D) to the end of its last element.
static size_t operand_bytes(const dad_layer& L, bool isA) {
  const size_t e = L.dtype == DAD_F32 ? 4 : 2;
  const int64_t ld = isA ? L.ldA : L.ldD, stride = isA ? L.strideA : L.strideD, h = isA ? L.h_in : L.h_out;
  return e * (size_t)((int64_t)(L.S - 1) * stride + (L.N - 1) * ld + h);
}

static bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// With one site the header leaves the site strides unspecified; every internal user gets N * ld instead.
static dad_layer normalised(const dad_layer& in) {
  dad_layer L = in;
  if (L.S == 1) {
    L.strideA = L.N * L.ldA;
    L.strideD = L.N * L.ldD;
  }
  return L;
}

bool tc_eligible(const dad_layer& L) {
  if (L.dtype != DAD_BF16) return false;
  if ((L.h_in | L.h_out | L.ldA | L.ldD) % 8 != 0) return false;
  if (L.S > 1 && ((L.strideA | L.strideD) % 8 != 0)) return false;
  if ((double)L.strideA * 2.0 >= 1.0e12 || (double)L.strideD * 2.0 >= 1.0e12) return false;  // TMA strides < 2^40 bytes
  return tmap_encoder_available();
}

CompressWs compress_ws_layout(const dad_layer& L, int r, bool f64, bool tc, int fused_c) {
  CompressWs w;
  memset(&w, 0, sizeof(w));
  const size_t acc = f64 ? 8 : 4;
  const size_t S = (size_t)L.S, N = (size_t)L.N, hi = (size_t)L.h_in, ho = (size_t)L.h_out, rr = (size_t)r;
  const size_t hmax = hi > ho ? hi : ho;
  size_t off = 0;
  w.status = off;
  off += 256;
  // arrival counters: column tiles of the split products | chunks of the one-launch pairs | sites (Gram kernel)
  const bool pair_in = tc && umma_pair_fits(L.S, L.N, L.h_in, r), pair_out = tc && umma_pair_fits(L.S, L.N, L.h_out, r);
  w.n_pair_counters = (pair_in || pair_out) ? S * 16 : 0;
  w.n_counters = S * (size_t)ceil_div((int64_t)hmax, kColsAccThreads) + w.n_pair_counters + S;
  w.counters = off;
  off = align_up(off + w.n_counters * sizeof(unsigned), 256);
  w.G = off;
  off = align_up(off + ((f64 || fused_c > 0) ? S * rr * ho * acc : 0), 256);
  w.Y = off;
  off = align_up(off + (tc ? 0 : S * N * rr * acc), 256);
  w.Z = off;
  off = align_up(off + ((tc && fused_c == 0) ? 0 : S * rr * hi * acc), 256);
  size_t part = 0;
  if (!tc) {
    const int s_in = cols_acc_splits(L.S, L.N, L.h_in), s_out = cols_acc_splits(L.S, L.N, L.h_out);
    if (s_in > 1) part = S * (size_t)s_in * rr * hi * acc;
    if (s_out > 1 && S * (size_t)s_out * rr * ho * acc > part) part = S * (size_t)s_out * rr * ho * acc;
  }
  w.partial = off;
  off = align_up(off + part, 256);
  w.gram_partial = off;
  off = align_up(off + S * (size_t)ceil_div((int64_t)ho, kGramChunk) * rr * rr * 8, 256);
  w.gram = off;
  off = align_up(off + S * rr * rr * 8, 256);
  w.tratio = off;
  off = align_up(off + S * rr * 8, 256);
  w.dead = off;
  off = align_up(off + align_up(S * rr, 16) + S * sizeof(int), 256);
  w.Fq = w.Fz = w.Yt = w.tc_partial = off;
  if (tc) {
    const size_t rp = (size_t)umma_rank_pad(r);
    w.Npad = (int64_t)align_up(N, 8);
    w.Fq = off;
    off = align_up(off + S * 2 * rp * ho * 2, 256);
    w.Fz = off;
    off = align_up(off + S * 2 * rp * hi * 2, 256);
    w.Yt = off;
    off = align_up(off + S * 2 * rp * (size_t)w.Npad * 2, 256);
    const size_t p_in = (size_t)umma_cols_acc_splits(L.S, L.N, L.h_in) * (size_t)ceil_div(L.h_in, 128);
    const size_t p_out = (size_t)umma_cols_acc_splits(L.S, L.N, L.h_out) * (size_t)ceil_div(L.h_out, 128);
    w.tc_partial = off;
    size_t part_bytes = S * (p_in > p_out ? p_in : p_out) * 128 * rp * 4;
    if (pair_in && umma_pair_partial_bytes(L.S, L.N, L.h_in, r) > part_bytes) part_bytes = umma_pair_partial_bytes(L.S, L.N, L.h_in, r);
    if (pair_out && umma_pair_partial_bytes(L.S, L.N, L.h_out, r) > part_bytes) part_bytes = umma_pair_partial_bytes(L.S, L.N, L.h_out, r);
    off = align_up(off + part_bytes, 256);
  }
  w.fused_part = w.fused_sig = off;
  if (fused_c > 0) {
    w.fused_part = off;
    off = align_up(off + S * (size_t)fused_c * rr * hmax * acc, 256);
    w.fused_sig = off;
    off = align_up(off + S * (size_t)fused_c * rr * 8, 256);
  }
  w.total = off;
  return w;
}

GemmWs gemm_ws_layout(int64_t hx, int64_t hy, int S, int64_t N, bool convert_operands, int batch, int products) {
  GemmWs w;
  memset(&w, 0, sizeof(w));
  size_t off = 0;
  w.status = off;
  off += 256;
  const GemmPlan g = umma_gemm_plan(hx, hy, S, N, batch, products);
  const size_t tiles = (size_t)g.tiles * (size_t)batch;
  w.n_counters = tiles;
  w.counters = off;
  off = align_up(off + tiles * sizeof(unsigned), 256);
  w.partial = off;
  const size_t slots = (size_t)g.splits + (g.rem_ctas > 0 ? 1 : 0);  // partial tiles per output tile
  off = align_up(off + (slots > 1 ? tiles * slots * (size_t)g.bm * (size_t)g.bn * 4 : 0), 256);
  w.Xb = w.Yb = off;
  if (convert_operands) {
    w.Xb = off;
    off = align_up(off + (size_t)batch * S * N * hx * 2, 256);
    w.Yb = off;
    off = align_up(off + (size_t)batch * S * N * hy * 2, 256);
  }
  w.total = off;
  return w;
}

#define DAD_STEP(call)                  \
  do {                                  \
    err = (call);                       \
    if (err != cudaSuccess) return err; \
  } while (0)

// General pipeline: fp32 inputs with fp64 accumulation (TAcc = double), or bf16 inputs in a layout
// the tensor-core kernels do not take, with fp32 accumulation (TAcc = float).
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
  int* need2 = reinterpret_cast<int*>(ws + w.dead + align_up((size_t)S * r, 16));
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
  for (int k = 0; k < iters; ++k) {
    DAD_STEP(rows_dot<TAcc>(L.dtype, D, L.ldD, L.strideD, S, N, ho, G, r, Y, st));                           // Y = D G^T
    DAD_STEP(cols_acc<TAcc>(L.dtype, A, L.ldA, L.strideA, S, N, hi, Y, r, Z, nullptr, part, ctr_cols, st));  // Z = Y^T A
    DAD_STEP(rows_dot<TAcc>(L.dtype, A, L.ldA, L.strideA, S, N, hi, Z, r, Y, st));                           // W = A Z^T
    DAD_STEP(cols_acc<TAcc>(L.dtype, D, L.ldD, L.strideD, S, N, ho, Y, r, G, nullptr, part, ctr_cols, st));  // Gt = W^T D
    // the second pass returns at once for sites whose first pass was well conditioned, so both write the outputs
    float* q32 = (f64 && k == iters - 1) ? Q : nullptr;
    if (orth_cluster_fits(r, ho, sizeof(TAcc))) {
      DAD_STEP(orth_cluster<TAcc>(G, S, r, ho, tol, status, q32, nullptr, 0, st));
      continue;
    }
    DAD_STEP(cholqr_pass<TAcc>(G, S, r, ho, 0, tol, gram_partial, gram, tratio, dead, need2, ctr_gram, status, q32,
                               nullptr, 0, st));
    DAD_STEP(cholqr_pass<TAcc>(G, S, r, ho, 1, tol, gram_partial, gram, tratio, dead, need2, ctr_gram, status, q32,
                               nullptr, 0, st));
  }
  DAD_STEP(rows_dot<TAcc>(L.dtype, D, L.ldD, L.strideD, S, N, ho, G, r, Y, st));
  DAD_STEP(cols_acc<TAcc>(L.dtype, A, L.ldA, L.strideA, S, N, hi, Y, r, Z, P, part, ctr_cols, st));
  if (sigma) DAD_STEP(row_norms<TAcc>(Z, (int64_t)S * r, hi, sigma, st));
  return cudaSuccess;
}

// Tensor-core pipeline for bf16 inputs: every product runs as tcgen05 MMAs with fp32 accumulation;
// the small fp32 operand of each product (G, Y, Z, W) is handed on as two bf16 planes (hi + lo).
static cudaError_t run_compress_tc(const dad_layer& L, const void* A, const void* D, int r, int iters, const float* Q0,
                                   float* P, float* Q, float* sigma, char* ws, const CompressWs& w, cudaStream_t st) {
  const int S = L.S;
  const int64_t N = L.N, hi = L.h_in, ho = L.h_out;
  const int rp = umma_rank_pad(r);
  cudaError_t err = cudaMemsetAsync(ws + w.status, 0, w.counters + w.n_counters * sizeof(unsigned) - w.status, st);
  if (err != cudaSuccess) return err;
  int* status = reinterpret_cast<int*>(ws + w.status);
  unsigned* ctr_cols = reinterpret_cast<unsigned*>(ws + w.counters);
  unsigned* ctr_gram = ctr_cols + (w.n_counters - (size_t)S);
  unsigned* ctr_pair = ctr_gram - w.n_pair_counters;
  double* gram_partial = reinterpret_cast<double*>(ws + w.gram_partial);
  double* gram = reinterpret_cast<double*>(ws + w.gram);
  double* tratio = reinterpret_cast<double*>(ws + w.tratio);
  unsigned char* dead = reinterpret_cast<unsigned char*>(ws + w.dead);
  int* need2 = reinterpret_cast<int*>(ws + w.dead + align_up((size_t)S * r, 16));
  __nv_bfloat16* Fq = reinterpret_cast<__nv_bfloat16*>(ws + w.Fq);
  __nv_bfloat16* Fz = reinterpret_cast<__nv_bfloat16*>(ws + w.Fz);
  __nv_bfloat16* Yt = reinterpret_cast<__nv_bfloat16*>(ws + w.Yt);
  float* part = reinterpret_cast<float*>(ws + w.tc_partial);
  const double tol = 1e-6;

  // tensor maps: X row tiles (rows_dot), X column tiles (cols_acc), and the three plane buffers
  CUtensorMap tmA_rows, tmA_cols, tmD_rows, tmD_cols, tmFq, tmFz, tmYt;
  const uint64_t sA = (uint64_t)L.strideA * 2, sD = (uint64_t)L.strideD * 2;
  bool ok = make_tmap_bf16_3d(&tmA_rows, A, hi, N, S, (uint64_t)L.ldA * 2, sA, 64, 128) &&
            make_tmap_bf16_3d(&tmA_cols, A, hi, N, S, (uint64_t)L.ldA * 2, sA, 64, 64) &&
            make_tmap_bf16_3d(&tmD_rows, D, ho, N, S, (uint64_t)L.ldD * 2, sD, 64, 128) &&
            make_tmap_bf16_3d(&tmD_cols, D, ho, N, S, (uint64_t)L.ldD * 2, sD, 64, 64) &&
            make_tmap_bf16_3d(&tmFq, Fq, ho, rp, (uint64_t)S * 2, (uint64_t)ho * 2, (uint64_t)rp * ho * 2, 64, rp) &&
            make_tmap_bf16_3d(&tmFz, Fz, hi, rp, (uint64_t)S * 2, (uint64_t)hi * 2, (uint64_t)rp * hi * 2, 64, rp) &&
            make_tmap_bf16_3d(&tmYt, Yt, N, rp, (uint64_t)S * 2, (uint64_t)w.Npad * 2, (uint64_t)rp * w.Npad * 2, 64, rp);
  if (!ok) return cudaErrorInvalidValue;

  // Small calls take each half of the operator (Y = D G^T, Z = Y^T A; W = A Z^T, G~ = W^T D) as ONE launch in which Y
  // (or W) stays on the SM; large ones as the two streaming kernels with Y^T handed on through the workspace.
  const bool pair_on = g_pair_on.load(std::memory_order_relaxed);
  const bool pair_in = pair_on && umma_pair_fits(S, N, hi, r), pair_out = pair_on && umma_pair_fits(S, N, ho, r);
  auto half_in = [&](float* out32, __nv_bfloat16* planes) -> cudaError_t {  // (D G^T)^T A from the planes Fq
    if (pair_in) return umma_pair(tmD_rows, tmFq, tmA_cols, S, N, ho, hi, r, out32, nullptr, planes, hi, part, ctr_pair, status, st);
    cudaError_t e = umma_rows_dot(tmD_rows, tmFq, S, N, ho, r, Yt, w.Npad, status, st);
    if (e != cudaSuccess) return e;
    return umma_cols_acc(tmA_cols, tmYt, S, N, hi, r, out32, nullptr, planes, hi, part, ctr_cols, status, st);
  };
  auto half_out = [&]() -> cudaError_t {  // (A Z^T)^T D from the planes Fz, into Q
    if (pair_out) return umma_pair(tmA_rows, tmFz, tmD_cols, S, N, hi, ho, r, Q, nullptr, nullptr, 0, part, ctr_pair, status, st);
    cudaError_t e = umma_rows_dot(tmA_rows, tmFz, S, N, hi, r, Yt, w.Npad, status, st);
    if (e != cudaSuccess) return e;
    return umma_cols_acc(tmD_cols, tmYt, S, N, ho, r, Q, nullptr, nullptr, 0, part, ctr_cols, status, st);
  };

  if (Q != Q0) DAD_STEP(cudaMemcpyAsync(Q, Q0, sizeof(float) * (size_t)S * r * ho, cudaMemcpyDeviceToDevice, st));
  DAD_STEP(split_planes(Q0, S, r, ho, Fq, rp, st));
  for (int k = 0; k < iters; ++k) {
    DAD_STEP(half_in(nullptr, Fz));
    DAD_STEP(half_out());
    if (orth_split_preferred(r, ho, S)) {
      DAD_STEP(orth_split(Q, S, r, ho, tol, gram_partial, gram, tratio, dead, need2, ctr_gram, status, nullptr, Fq, rp, st));
    } else if (orth_mma_fits(r, ho)) {
      DAD_STEP(orth_mma(Q, S, r, ho, tol, status, nullptr, Fq, rp, st));
    } else if (orth_cluster_fits(r, ho)) {
      DAD_STEP(orth_cluster(Q, S, r, ho, tol, status, nullptr, Fq, rp, st));
    } else {
      DAD_STEP(cholqr_pass<float>(Q, S, r, ho, 0, tol, gram_partial, gram, tratio, dead, need2, ctr_gram, status,
                                  nullptr, Fq, rp, st));
      DAD_STEP(cholqr_pass<float>(Q, S, r, ho, 1, tol, gram_partial, gram, tratio, dead, need2, ctr_gram, status,
                                  nullptr, Fq, rp, st));
    }
  }
  DAD_STEP(half_in(P, nullptr));
  if (sigma) DAD_STEP(row_norms<float>(P, (int64_t)S * r, hi, sigma, st));
  return cudaSuccess;
}

static cudaError_t run_gemm_tc(const void* X, int64_t ldX, int64_t strideX, const void* Y, int64_t ldY, int64_t strideY,
                               int S, int64_t N, int64_t hx, int64_t hy, float* C, char* ws, const GemmWs& w,
                               cudaStream_t st, int batch = 1, int products = 1) {
  // the second status slot (byte 4) belongs to the dense products; the first keeps what a compress call reported
  cudaError_t err = cudaMemsetAsync(ws + w.status + 4, 0, w.counters + w.n_counters * sizeof(unsigned) - w.status - 4, st);
  if (err != cudaSuccess) return err;
  CUtensorMap tmX, tmY;
  const GemmPlan g = umma_gemm_plan(hx, hy, S, N, batch, products);
  // third dimension: the sites of one product (of `products` products of S sites each), or one-site products
  const uint64_t d2 = batch > 1 ? (uint64_t)batch : (uint64_t)S * (uint64_t)products;
  if (!make_tmap_bf16_3d(&tmX, X, hx, N, d2, (uint64_t)ldX * 2, (uint64_t)strideX * 2, 64, (uint32_t)g.bk) ||
      !make_tmap_bf16_3d(&tmY, Y, hy, N, d2, (uint64_t)ldY * 2, (uint64_t)strideY * 2, 64, (uint32_t)g.bk))
    return cudaErrorInvalidValue;
  return umma_gemm_tn(tmX, tmY, g, hx, hy, C, reinterpret_cast<float*>(ws + w.partial),
                      reinterpret_cast<unsigned*>(ws + w.counters), reinterpret_cast<int*>(ws + w.status + 4), st);
}

#undef DAD_STEP

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

size_t dad_workspace_bytes(const dad_layer* layer, int r, int iters) {
  if (validate_layer(layer) != DAD_OK || validate_rank(layer, r) != DAD_OK || iters < 0) return 0;
  const dad_layer Ln = normalised(*layer);
  const dad_layer* L = &Ln;
  const bool tc = tc_eligible(*L);
  const size_t a = compress_ws_layout(*L, r, L->dtype == DAD_F32, tc, fused_cluster_size(*L, r, iters)).total;
  const size_t b = tc ? gemm_ws_layout(L->h_in, L->h_out, L->S, L->N, false).total : 256;
  return a > b ? a : b;
}

dad_status dad_full_grad(const dad_layer* layer, const void* A, const void* D, float* grad, uint64_t* bytes_tx,
                         void* ws, size_t ws_bytes, void* cuda_stream) {
  dad_status vs = validate_layer(layer);
  if (vs != DAD_OK) return vs;
  const dad_layer Ln = normalised(*layer);
  const dad_layer* L = &Ln;
  if (!A || !D || !grad) return DAD_ERR_NULL;
  if (!aligned(A, 16) || !aligned(D, 16) || !aligned(grad, 16)) return DAD_ERR_ALIGN;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  cudaError_t err;
  {
    const BoundsRange ranges[] = {{A, operand_bytes(*L, true)}, {D, operand_bytes(*L, false)},
                                  {grad, sizeof(float) * (size_t)L->h_in * L->h_out}, {ws, ws_bytes}};
    if (bounds_register(ranges, 4, st) != cudaSuccess) return DAD_ERR_CUDA;
  }
  if (tc_eligible(*L)) {
    const GemmWs w = gemm_ws_layout(L->h_in, L->h_out, L->S, L->N, false);
    if (!ws) return DAD_ERR_NULL;
    if (!aligned(ws, 256)) return DAD_ERR_ALIGN;
    if (ws_bytes < w.total) return DAD_ERR_WORKSPACE;
    err = run_gemm_tc(A, L->ldA, L->strideA, D, L->ldD, L->strideD, L->S, L->N, L->h_in, L->h_out, grad, (char*)ws, w, st);
  } else {
    err = gemm_tn_simt(L->dtype, A, L->ldA, L->strideA, D, L->ldD, L->strideD, L->S, L->N, L->h_in, L->h_out, grad, st);
  }
  if (err != cudaSuccess) return DAD_ERR_CUDA;
  if (bytes_tx)
    for (int s = 0; s < L->S; ++s) bytes_tx[s] = dad_bytes_dad(L);
  return DAD_OK;
}

// Whether `groups` gradients of this shape run as one launch of the 256 x 256 kernel (else one call per layer).
static bool full_grad_grouped_tc(const dad_layer& L, int groups) {
  if (!tc_eligible(L)) return false;
  const GemmPlan g = umma_gemm_plan(L.h_in, L.h_out, L.S / groups, L.N, 1, groups);
  return g.bm == 256;
}

size_t dad_full_grad_grouped_workspace_bytes(const dad_layer* layer, int groups) {
  if (validate_layer(layer) != DAD_OK || groups < 1 || layer->S % groups != 0) return 0;
  const dad_layer L = normalised(*layer);
  if (full_grad_grouped_tc(L, groups)) return gemm_ws_layout(L.h_in, L.h_out, L.S / groups, L.N, false, 1, groups).total;
  dad_layer one = L;
  one.S = L.S / groups;
  return dad_workspace_bytes(&one, 1, 0);
}

dad_status dad_full_grad_grouped(const dad_layer* layer, int groups, const void* A, const void* D, float* grads,
                                 uint64_t* bytes_tx, void* ws, size_t ws_bytes, void* cuda_stream) {
  dad_status vs = validate_layer(layer);
  if (vs != DAD_OK) return vs;
  if (groups < 1 || layer->S % groups != 0) return DAD_ERR_SHAPE;
  const dad_layer L = normalised(*layer);
  if (!A || !D || !grads) return DAD_ERR_NULL;
  if (!aligned(A, 16) || !aligned(D, 16) || !aligned(grads, 16)) return DAD_ERR_ALIGN;
  const int Sg = L.S / groups;
  if (groups > 1 && full_grad_grouped_tc(L, groups)) {
    const GemmWs w = gemm_ws_layout(L.h_in, L.h_out, Sg, L.N, false, 1, groups);
    if (!ws) return DAD_ERR_NULL;
    if (!aligned(ws, 256)) return DAD_ERR_ALIGN;
    if (ws_bytes < w.total) return DAD_ERR_WORKSPACE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    const BoundsRange ranges[] = {{A, operand_bytes(L, true)}, {D, operand_bytes(L, false)},
                                  {grads, sizeof(float) * (size_t)groups * L.h_in * L.h_out}, {ws, ws_bytes}};
    if (bounds_register(ranges, 4, st) != cudaSuccess) return DAD_ERR_CUDA;
    const cudaError_t err = run_gemm_tc(A, L.ldA, L.strideA, D, L.ldD, L.strideD, Sg, L.N, L.h_in, L.h_out, grads, (char*)ws, w,
                                        st, 1, groups);
    if (err != cudaSuccess) return DAD_ERR_CUDA;
  } else {
    dad_layer one = L;  // one call per layer: its sites are slices g * Sg ... of the stacked buffers
    one.S = Sg;
    const size_t e = L.dtype == DAD_F32 ? 4 : 2;
    for (int g = 0; g < groups; ++g) {
      const dad_status st1 = dad_full_grad(&one, (const char*)A + e * (size_t)g * Sg * L.strideA,
                                           (const char*)D + e * (size_t)g * Sg * L.strideD,
                                           grads + (size_t)g * L.h_in * L.h_out, nullptr, ws, ws_bytes, cuda_stream);
      if (st1 != DAD_OK) return st1;
    }
  }
  if (bytes_tx)
    for (int s = 0; s < L.S; ++s) bytes_tx[s] = dad_bytes_dad(&L);
  return DAD_OK;
}

dad_status dad_rank_compress(const dad_layer* layer, const void* A, const void* D, int r, int iters, const float* Q0,
                             float* P, float* Q, float* sigma, void* ws, size_t ws_bytes, void* cuda_stream) {
  dad_status vs = validate_layer(layer);
  if (vs != DAD_OK) return vs;
  const dad_layer Ln = normalised(*layer);
  const dad_layer* L = &Ln;
  if (!A || !D || !Q0 || !P || !Q || !ws) return DAD_ERR_NULL;
  vs = validate_rank(L, r);
  if (vs != DAD_OK) return vs;
  if (iters < 0 || iters > 1000000) return DAD_ERR_SHAPE;
  if (!aligned(A, 16) || !aligned(D, 16) || !aligned(Q0, 16) || !aligned(P, 16) || !aligned(Q, 16) ||
      !aligned(ws, 256) || (sigma && !aligned(sigma, 4)))
    return DAD_ERR_ALIGN;
  const bool f64 = L->dtype == DAD_F32;
  const bool tc = tc_eligible(*L);
  const int fused_c = fused_cluster_size(*L, r, iters);
  const CompressWs w = compress_ws_layout(*L, r, f64, tc, fused_c);
  if (ws_bytes < w.total) return DAD_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  cudaError_t err;
  {
    const size_t nP = sizeof(float) * (size_t)L->S * r * L->h_in, nQ = sizeof(float) * (size_t)L->S * r * L->h_out;
    const BoundsRange ranges[] = {{A, operand_bytes(*L, true)}, {D, operand_bytes(*L, false)}, {Q0, nQ}, {P, nP}, {Q, nQ},
                                  {sigma, sizeof(float) * (size_t)L->S * r}, {ws, ws_bytes}};
    if (bounds_register(ranges, 7, st) != cudaSuccess) return DAD_ERR_CUDA;
  }
  if (fused_c > 0 && g_fused_on.load(std::memory_order_relaxed)) {
    char* base = static_cast<char*>(ws);
    err = cudaMemsetAsync(base + w.status, 0, 4, st);
    if (err == cudaSuccess && fused_dsm_fits(*L, r, fused_c, nullptr))
      err = fused_dsm_compress(*L, A, D, r, iters, Q0, P, Q, sigma, reinterpret_cast<int*>(base + w.status), fused_c, st);
    else if (err == cudaSuccess)
      err = fused_compress(*L, A, D, r, iters, Q0, P, Q, sigma, base + w.G, base + w.Z, base + w.fused_part,
                           reinterpret_cast<double*>(base + w.fused_sig), reinterpret_cast<int*>(base + w.status), fused_c, st);
  } else if (tc)
    err = run_compress_tc(*L, A, D, r, iters, Q0, P, Q, sigma, (char*)ws, w, st);
  else if (f64)
    err = run_compress<double>(*L, A, D, r, iters, Q0, P, Q, sigma, (char*)ws, w, st);
  else
    err = run_compress<float>(*L, A, D, r, iters, Q0, P, Q, sigma, (char*)ws, w, st);
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
    const size_t nP = sizeof(float) * (size_t)L->S * r * L->h_in, nQ = sizeof(float) * (size_t)L->S * r * L->h_out;
    const BoundsRange ranges[] = {{P, nP}, {Q, nQ}, {Pcat, nP}, {Qcat, nQ}};
    if (bounds_register(ranges, 4, st) != cudaSuccess) return DAD_ERR_CUDA;
    cudaError_t err = copy_two(P, Pcat, (size_t)L->S * r * L->h_in, Q, Qcat, (size_t)L->S * r * L->h_out, st);
    if (err != cudaSuccess) return DAD_ERR_CUDA;
  }
  if (bytes_tx)
    for (int s = 0; s < L->S; ++s) bytes_tx[s] = dad_bytes_rank(L, r);
  return DAD_OK;
}

// bf16 products of the tensor-core reconstruction for this problem: 3 (two-term splits), 1 (hi terms only), or 0
// when the fp32 kernel takes it.
static int reconstruct_terms(int64_t h_in, int64_t h_out, int64_t K, dad_dtype math) {
  if (math != DAD_BF16 && math != DAD_BF16_1TERM) return 0;
  if (h_in % 8 != 0 || h_out % 8 != 0 || 3 * K > 0x7fffffff || !tmap_encoder_available()) return 0;
  return math == DAD_BF16 ? 3 : 1;
}
static bool math_ok(dad_dtype math) { return math == DAD_F32 || math == DAD_BF16 || math == DAD_BF16_1TERM; }

size_t dad_reconstruct_batched_workspace_bytes(int64_t h_in, int64_t h_out, int64_t K, int batch, dad_dtype math) {
  if (h_in < 1 || h_out < 1 || K < 1 || batch < 1) return 0;
  const int terms = reconstruct_terms(h_in, h_out, K, math);
  if (terms == 0) return 0;
  return gemm_ws_layout(h_in, h_out, 1, terms * K, true, batch).total;
}

size_t dad_reconstruct_workspace_bytes(int64_t h_in, int64_t h_out, int64_t K, dad_dtype math) {
  return dad_reconstruct_batched_workspace_bytes(h_in, h_out, K, 1, math);
}

dad_status dad_reconstruct_batched(int64_t h_in, int64_t h_out, int64_t K, int batch, const float* Pcat,
                                   const float* Qcat, float* grad, dad_dtype math, void* ws, size_t ws_bytes,
                                   void* cuda_stream) {
  if (h_in < 1 || h_out < 1 || K < 1 || h_in > 0x7fffffff || h_out > 0x7fffffff || batch < 1 || batch > 65535)
    return DAD_ERR_SHAPE;
  if (!math_ok(math)) return DAD_ERR_DTYPE;
  if (!Pcat || !Qcat || !grad) return DAD_ERR_NULL;
  if (!aligned(Pcat, 16) || !aligned(Qcat, 16) || !aligned(grad, 16)) return DAD_ERR_ALIGN;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  cudaError_t err = cudaSuccess;
  {
    const BoundsRange ranges[] = {{Pcat, sizeof(float) * (size_t)batch * K * h_in}, {Qcat, sizeof(float) * (size_t)batch * K * h_out},
                                  {grad, sizeof(float) * (size_t)batch * h_in * h_out}, {ws, ws_bytes}};
    if (bounds_register(ranges, 4, st) != cudaSuccess) return DAD_ERR_CUDA;
  }
  if (const int terms = reconstruct_terms(h_in, h_out, K, math)) {
    const GemmWs w = gemm_ws_layout(h_in, h_out, 1, terms * K, true, batch);  // `terms` bf16 products, one contraction
    if (!ws) return DAD_ERR_NULL;
    if (!aligned(ws, 256)) return DAD_ERR_ALIGN;
    if (ws_bytes < w.total) return DAD_ERR_WORKSPACE;
    __nv_bfloat16* Xb = reinterpret_cast<__nv_bfloat16*>((char*)ws + w.Xb);
    __nv_bfloat16* Yb = reinterpret_cast<__nv_bfloat16*>((char*)ws + w.Yb);
    err = stack_split3(Pcat, (size_t)K * h_in, Xb, Qcat, (size_t)K * h_out, Yb, batch, terms, st);
    if (err == cudaSuccess)
      err = run_gemm_tc(Xb, h_in, terms * K * h_in, Yb, h_out, terms * K * h_out, 1, terms * K, h_in, h_out, grad, (char*)ws,
                        w, st, batch);
  } else {
    for (int b = 0; b < batch && err == cudaSuccess; ++b)
      err = gemm_tn_simt(DAD_F32, Pcat + (size_t)b * K * h_in, h_in, 0, Qcat + (size_t)b * K * h_out, h_out, 0, 1, K, h_in,
                         h_out, grad + (size_t)b * h_in * h_out, st);
  }
  return err == cudaSuccess ? DAD_OK : DAD_ERR_CUDA;
}

dad_status dad_reconstruct(int64_t h_in, int64_t h_out, int64_t K, const float* Pcat, const float* Qcat, float* grad,
                           dad_dtype math, void* ws, size_t ws_bytes, void* cuda_stream) {
  return dad_reconstruct_batched(h_in, h_out, K, 1, Pcat, Qcat, grad, math, ws, ws_bytes, cuda_stream);
}

dad_status dad_check(const void* ws, void* cuda_stream) {
  if (!ws) return DAD_ERR_NULL;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  int status[2] = {0, 0};  // [0]: last dad_rank_compress on ws, [1]: last dense product on ws
  if (cudaMemcpyAsync(status, ws, sizeof(status), cudaMemcpyDeviceToHost, st) != cudaSuccess) return DAD_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return DAD_ERR_CUDA;
  for (int i = 0; i < 2; ++i)
    if (status[i] == (int)DAD_ERR_TIMEOUT || status[i] == (int)DAD_ERR_NUMERIC) return (dad_status)status[i];
  return DAD_OK;
}

int dad_compress_path(const dad_layer* layer, int r, int iters, int* cluster_size) {
  if (cluster_size) *cluster_size = 0;
  if (validate_layer(layer) != DAD_OK || validate_rank(layer, r) != DAD_OK || iters < 0) return -1;
  const dad_layer L = normalised(*layer);
  const int c = g_fused_on.load(std::memory_order_relaxed) ? fused_cluster_size(L, r, iters) : 0;
  if (c > 0) {
    if (cluster_size) *cluster_size = c;
    return fused_dsm_fits(L, r, c, nullptr) ? DAD_PATH_FUSED : DAD_PATH_FUSED_L2;
  }
  if (!tc_eligible(L)) return DAD_PATH_GENERAL;
  const bool paired = g_pair_on.load(std::memory_order_relaxed) &&
                      (umma_pair_fits(L.S, L.N, L.h_in, r) || umma_pair_fits(L.S, L.N, L.h_out, r));
  return paired ? DAD_PATH_TENSOR_PAIRED : DAD_PATH_TENSOR;
}

void dad_fused_enable(int on) { g_fused_on.store(on != 0, std::memory_order_relaxed); }
void dad_pair_enable(int on) { g_pair_on.store(on != 0, std::memory_order_relaxed); }

dad_status dad_selftest_bounded_wait(void* ws, size_t ws_bytes, void* cuda_stream) {
  if (!ws) return DAD_ERR_NULL;
  if (!aligned(ws, 256)) return DAD_ERR_ALIGN;
  if (ws_bytes < DAD_SELFTEST_BYTES) return DAD_ERR_WORKSPACE;
  if (!tmap_encoder_available()) return DAD_ERR_CUDA;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  char* base = static_cast<char*>(ws);
  if (cudaMemsetAsync(base, 0, DAD_SELFTEST_BYTES, st) != cudaSuccess) return DAD_ERR_CUDA;
  return umma_selftest_timeout(base + 1024, reinterpret_cast<int*>(base), st) == cudaSuccess ? DAD_OK : DAD_ERR_CUDA;
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

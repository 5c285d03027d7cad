// dad_rank_dad_host: the whole per-layer path for callers whose activations and errors live in host
// memory.  Copies A, D and the start vectors to the device, runs compress -> gather -> reconstruct
// there (Algorithm 1 with the direct sum of outer products at the aggregator), and copies the
// gradient back -- all queued on one stream, nothing allocated: the device staging area is the
// caller's.
#include "common.cuh"

namespace {

struct HostScratch {
  size_t A, D, Q0, P, Q, grad, ws, ws_bytes, total;
};

dad_layer device_layer(const dad_layer& host) {
  dad_layer L = host;  // same shape, densely packed on the device
  L.ldA = host.h_in;
  L.ldD = host.h_out;
  L.strideA = host.N * host.h_in;
  L.strideD = host.N * host.h_out;
  return L;
}

bool carve(const dad_layer& host, int r, int iters, dad_dtype math, HostScratch* out) {
  const dad_layer L = device_layer(host);
  const size_t need = dad_workspace_bytes(&L, r, iters);
  if (need == 0) return false;
  const size_t e = host.dtype == DAD_F32 ? 4 : 2;
  const size_t S = (size_t)host.S, N = (size_t)host.N, hi = (size_t)host.h_in, ho = (size_t)host.h_out, rr = (size_t)r;
  const size_t rec = dad_reconstruct_workspace_bytes(host.h_in, host.h_out, (int64_t)(S * rr), math);
  size_t off = 0;
  auto take = [&off](size_t bytes) {
    const size_t at = off;
    off = dad::align_up(off + bytes, 256);
    return at;
  };
  out->A = take(S * N * hi * e);
  out->D = take(S * N * ho * e);
  out->Q0 = take(S * rr * ho * 4);
  out->P = take(S * rr * hi * 4);
  out->Q = take(S * rr * ho * 4);
  out->grad = take(hi * ho * 4);
  out->ws_bytes = need > rec ? need : rec;
  out->ws = take(out->ws_bytes);
  out->total = off;
  return true;
}

// rows of `width` elements, `ld` apart on the host, packed on the device
cudaError_t copy_in(void* dst, const void* src, size_t elem, int64_t rows, int64_t width, int64_t ld, cudaStream_t st) {
  if (ld == width) return cudaMemcpyAsync(dst, src, elem * (size_t)rows * width, cudaMemcpyHostToDevice, st);
  return cudaMemcpy2DAsync(dst, elem * (size_t)width, src, elem * (size_t)ld, elem * (size_t)width, (size_t)rows,
                           cudaMemcpyHostToDevice, st);
}

}  // namespace

extern "C" {

size_t dad_rank_dad_host_scratch_bytes(const dad_layer* layer, int r, int iters, dad_dtype math) {
  HostScratch sc;
  if (!layer || (math != DAD_F32 && math != DAD_BF16 && math != DAD_BF16_1TERM) || !carve(*layer, r, iters, math, &sc)) return 0;
  return sc.total;
}

dad_status dad_rank_dad_host(const dad_layer* layer, const void* A_host, const void* D_host, const float* Q0_host, int r,
                             int iters, dad_dtype math, float* grad_host, uint64_t* bytes_tx, void* dev_scratch,
                             size_t dev_scratch_bytes, void* cuda_stream) {
  if (!layer || !A_host || !D_host || !Q0_host || !grad_host || !dev_scratch) return DAD_ERR_NULL;
  if (math != DAD_F32 && math != DAD_BF16 && math != DAD_BF16_1TERM) return DAD_ERR_DTYPE;
  if (reinterpret_cast<uintptr_t>(dev_scratch) % 256) return DAD_ERR_ALIGN;
  // the caller's own strides feed the copies: rows must not overlap, sites must not overlap (before anything is queued)
  if (layer->S >= 1 && layer->N >= 1 && layer->h_in >= 1 && layer->h_out >= 1) {
    if (layer->ldA < layer->h_in || layer->ldD < layer->h_out) return DAD_ERR_SHAPE;
    if (layer->S > 1 && (layer->strideA < layer->N * layer->ldA || layer->strideD < layer->N * layer->ldD)) return DAD_ERR_SHAPE;
  }
  HostScratch sc;
  if (!carve(*layer, r, iters, math, &sc)) {
    // let the device entry point name the reason (shape, dtype, rank) without touching memory
    const dad_layer L = device_layer(*layer);
    if (L.dtype != DAD_F32 && L.dtype != DAD_BF16) return DAD_ERR_DTYPE;
    if (r < 1 || r > DAD_MAX_RANK || r > L.h_in || r > L.h_out) return DAD_ERR_RANK;
    return DAD_ERR_SHAPE;
  }
  if (dev_scratch_bytes < sc.total) return DAD_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  char* base = static_cast<char*>(dev_scratch);
  const dad_layer L = device_layer(*layer);
  const size_t e = layer->dtype == DAD_F32 ? 4 : 2;
  const int S = layer->S;
  const size_t rr = (size_t)r;
  const bool dense = layer->ldA == layer->h_in && layer->ldD == layer->h_out &&
                     (S == 1 || (layer->strideA == L.strideA && layer->strideD == L.strideD));
  if (dense) {  // one copy per operand
    if (cudaMemcpyAsync(base + sc.A, A_host, e * (size_t)S * L.strideA, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(base + sc.D, D_host, e * (size_t)S * L.strideD, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return DAD_ERR_CUDA;
  } else {      // strided rows or sites: one (2-D) copy per site and operand
    for (int s = 0; s < S; ++s) {
      const char* a = static_cast<const char*>(A_host) + e * (size_t)s * layer->strideA;
      const char* d = static_cast<const char*>(D_host) + e * (size_t)s * layer->strideD;
      if (copy_in(base + sc.A + e * (size_t)s * L.strideA, a, e, layer->N, layer->h_in, layer->ldA, st) != cudaSuccess ||
          copy_in(base + sc.D + e * (size_t)s * L.strideD, d, e, layer->N, layer->h_out, layer->ldD, st) != cudaSuccess)
        return DAD_ERR_CUDA;
    }
  }
  if (cudaMemcpyAsync(base + sc.Q0, Q0_host, (size_t)S * rr * layer->h_out * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return DAD_ERR_CUDA;
  // the status words of a workspace must start out clear
  if (cudaMemsetAsync(base + sc.ws, 0, 256, st) != cudaSuccess) return DAD_ERR_CUDA;
  float* P = reinterpret_cast<float*>(base + sc.P);
  float* Q = reinterpret_cast<float*>(base + sc.Q);
  float* grad = reinterpret_cast<float*>(base + sc.grad);
  dad_status rc = dad_rank_compress(&L, base + sc.A, base + sc.D, r, iters, reinterpret_cast<const float*>(base + sc.Q0), P, Q,
                                    nullptr, base + sc.ws, sc.ws_bytes, cuda_stream);
  if (rc != DAD_OK) return rc;
  rc = dad_gather_factors(&L, r, P, Q, P, Q, bytes_tx, cuda_stream);  // the stacks are the factor buffers themselves
  if (rc != DAD_OK) return rc;
  rc = dad_reconstruct(L.h_in, L.h_out, (int64_t)S * r, P, Q, grad, math, base + sc.ws, sc.ws_bytes, cuda_stream);
  if (rc != DAD_OK) return rc;
  if (cudaMemcpyAsync(grad_host, grad, (size_t)L.h_in * L.h_out * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return DAD_ERR_CUDA;
  return DAD_OK;
}

}  // extern "C"

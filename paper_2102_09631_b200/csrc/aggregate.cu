// Aggregator-side steps of rank-dAD that follow the gather:
//   - the second structured power iteration on the stacked factors (Algorithm 1: "SPI(Q_i, G_i)" at the
//     aggregator, whose r-row result is what gets broadcast back), and
//   - the effective rank of a site's factors (Sec. 3.3.1, last paragraph; Algorithm 2's early stop):
//     the leading components are kept while sigma_j > theta * sigma_1; the rest are not transmitted.
#include "common.cuh"

namespace dad {

// r_eff[s] = number of leading components kept; rows j >= r_eff[s] of P_s and Q_s are set to zero.
__global__ void __launch_bounds__(256)
effective_rank_kernel(const float* __restrict__ sigma, int r, float theta, int32_t* __restrict__ r_eff,
                      float* __restrict__ P, int64_t h_in, float* __restrict__ Q, int64_t h_out) {
  __shared__ int keep_s;
  const int s = blockIdx.x;
  if (threadIdx.x == 0) {
    const float* sg = sigma + (int64_t)s * r;
    const float bar = theta * sg[0];  // fp32 product, fp32 comparison
    int keep = 0;
    while (keep < r && sg[keep] > bar) ++keep;
    keep_s = keep;
    r_eff[s] = keep;
  }
  __syncthreads();
  const int keep = keep_s;
  if (P) {
    float* Ps = P + ((int64_t)s * r + keep) * h_in;
    for (int64_t i = threadIdx.x; i < (int64_t)(r - keep) * h_in; i += blockDim.x) Ps[i] = 0.f;
  }
  if (Q) {
    float* Qs = Q + ((int64_t)s * r + keep) * h_out;
    for (int64_t i = threadIdx.x; i < (int64_t)(r - keep) * h_out; i += blockDim.x) Qs[i] = 0.f;
  }
}

cudaError_t effective_rank(const float* sigma, int S, int r, float theta, int32_t* r_eff, float* P, int64_t h_in,
                           float* Q, int64_t h_out, cudaStream_t st) {
  cudaError_t err = cudaSuccess;
  DAD_LAUNCH(err, "effective_rank", effective_rank_kernel, (unsigned)S, 256, 0, st, sigma, r, theta, r_eff, P, h_in, Q,
             h_out);
  return err;
}

}  // namespace dad

using namespace dad;

static dad_layer stack_layer(int64_t h_in, int64_t h_out, int64_t K) {
  dad_layer L;
  L.S = 1;
  L.N = K;
  L.h_in = h_in;
  L.h_out = h_out;
  L.dtype = DAD_F32;
  L.ldA = h_in;
  L.ldD = h_out;
  L.strideA = K * h_in;
  L.strideD = K * h_out;
  return L;
}

extern "C" {

size_t dad_aggregate_workspace_bytes(int64_t h_in, int64_t h_out, int64_t K, int r, int iters) {
  if (h_in < 1 || h_out < 1 || K < 1) return 0;
  const dad_layer L = stack_layer(h_in, h_out, K);
  return dad_workspace_bytes(&L, r, iters);
}

dad_status dad_aggregate_compress(int64_t h_in, int64_t h_out, int64_t K, const float* Pcat, const float* Qcat, int r,
                                  int iters, const float* Q0, float* Phat, float* Qhat, float* sigma, void* ws,
                                  size_t ws_bytes, void* cuda_stream) {
  if (h_in < 1 || h_out < 1 || K < 1) return DAD_ERR_SHAPE;
  // The stacks play the parts of the component matrices: Pcat^T Qcat is "A^T D" with A = Pcat, D = Qcat.
  const dad_layer L = stack_layer(h_in, h_out, K);
  return dad_rank_compress(&L, Pcat, Qcat, r, iters, Q0, Phat, Qhat, sigma, ws, ws_bytes, cuda_stream);
}

dad_status dad_effective_rank(const dad_layer* layer, int r, float theta, const float* sigma, int32_t* r_eff, float* P,
                              float* Q, void* cuda_stream) {
  if (!layer || !sigma || !r_eff) return DAD_ERR_NULL;
  if (layer->S < 1 || layer->S > 65535 || layer->h_in < 1 || layer->h_out < 1) return DAD_ERR_SHAPE;
  if (r < 1 || r > DAD_MAX_RANK) return DAD_ERR_RANK;
  if (!(theta >= 0.f) || theta > 1.f) return DAD_ERR_SHAPE;
  cudaError_t err = effective_rank(sigma, layer->S, r, theta, r_eff, P, layer->h_in, Q, layer->h_out,
                                   reinterpret_cast<cudaStream_t>(cuda_stream));
  return err == cudaSuccess ? DAD_OK : DAD_ERR_CUDA;
}

}  // extern "C"

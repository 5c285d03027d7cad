// The table of address ranges and the record of violations of the -DDAD_BOUNDS_CHECK build (see bounds.cuh), and
// the entry points that read the record.
#include <cstdlib>

#include "bounds.cuh"
#include "common.cuh"

namespace dad {

#ifdef DAD_BOUNDS_CHECK
__device__ BoundsTable g_bounds;
__device__ unsigned long long g_bounds_trip[4];

cudaError_t bounds_register(const BoundsRange* ranges, int n, cudaStream_t st) {
  // DAD_BOUNDS_SHRINK=<bytes> cuts that much off the end of every range: a way to see the checker fire (on accesses
  // that are in fact legitimate) without handing any kernel a bad index.
  static const size_t shrink = [] {
    const char* v = getenv("DAD_BOUNDS_SHRINK");
    return v ? (size_t)strtoull(v, nullptr, 10) : (size_t)0;
  }();
  BoundsTable t{};
  for (int i = 0; i < n && t.n < kMaxBoundsRanges; ++i) {
    if (!ranges[i].p || ranges[i].bytes == 0) continue;
    t.lo[t.n] = reinterpret_cast<unsigned long long>(ranges[i].p);
    t.hi[t.n] = t.lo[t.n] + (ranges[i].bytes > shrink ? ranges[i].bytes - shrink : 0);
    ++t.n;
  }
  // pageable source: the runtime stages the copy before returning, and the copy itself is ordered on the stream
  return cudaMemcpyToSymbolAsync(g_bounds, &t, sizeof(t), 0, cudaMemcpyHostToDevice, st);
}
#else
cudaError_t bounds_register(const BoundsRange*, int, cudaStream_t) { return cudaSuccess; }
#endif

}  // namespace dad

extern "C" {

int dad_bounds_check_build(void) {
#ifdef DAD_BOUNDS_CHECK
  return 1;
#else
  return 0;
#endif
}

dad_status dad_bounds_report(uint64_t out[4], int reset, void* cuda_stream) {
  if (!out) return DAD_ERR_NULL;
  out[0] = out[1] = out[2] = out[3] = 0;
#ifdef DAD_BOUNDS_CHECK
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  unsigned long long h[4] = {0, 0, 0, 0};
  if (cudaStreamSynchronize(st) != cudaSuccess) return DAD_ERR_CUDA;
  if (cudaMemcpyFromSymbol(h, dad::g_bounds_trip, sizeof(h)) != cudaSuccess) return DAD_ERR_CUDA;
  for (int i = 0; i < 4; ++i) out[i] = h[i];
  if (reset) {
    const unsigned long long z[4] = {0, 0, 0, 0};
    if (cudaMemcpyToSymbol(dad::g_bounds_trip, z, sizeof(z)) != cudaSuccess) return DAD_ERR_CUDA;
  }
#else
  (void)reset;
  (void)cuda_stream;
#endif
  return DAD_OK;
}

}  // extern "C"

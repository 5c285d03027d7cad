// Checked global-memory accesses for the -DDAD_BOUNDS_CHECK build of the library (a stand-in for a memory checker
// where none can be run): every entry point registers the address ranges of the buffers it was given, and the
// kernels that compute their own indices go through DAD_LD / DAD_ST, which test the address against those ranges.
// An access outside every range is NOT made -- a load gives zero, a store is dropped -- and is recorded (count,
// first address, size, source line) for dad_bounds_report; nothing traps.  In the ordinary build the macros are
// plain loads and stores and cost nothing.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace dad {

constexpr int kMaxBoundsRanges = 16;
struct BoundsTable {
  unsigned long long lo[kMaxBoundsRanges], hi[kMaxBoundsRanges];  // [lo, hi) in bytes
  int n;
};

// Host side (both builds; a no-op without DAD_BOUNDS_CHECK): make `ranges` the table the kernels queued on `st`
// after this call check against.
struct BoundsRange {
  const void* p;
  size_t bytes;
};
cudaError_t bounds_register(const BoundsRange* ranges, int n, cudaStream_t st);

#ifdef DAD_BOUNDS_CHECK
extern __device__ BoundsTable g_bounds;
extern __device__ unsigned long long g_bounds_trip[4];  // count, first address, size, line

__device__ __forceinline__ bool bounds_ok(const void* p, size_t bytes, int line) {
  if (!__isGlobal(p)) return true;  // shared memory reached through a generic pointer is not this table's business
  const unsigned long long a = reinterpret_cast<unsigned long long>(p);
  const int n = g_bounds.n;
  for (int i = 0; i < n; ++i)
    if (a >= g_bounds.lo[i] && a + bytes <= g_bounds.hi[i]) return true;
  if (atomicAdd(&g_bounds_trip[0], 1ull) == 0ull) {
    g_bounds_trip[1] = a;
    g_bounds_trip[2] = bytes;
    g_bounds_trip[3] = (unsigned long long)line;
  }
  return false;
}
template <typename T>
__device__ __forceinline__ T checked_load(const T* p, int line) {
  if (bounds_ok(p, sizeof(T), line)) return *p;
  T zero{};
  return zero;
}
template <typename T, typename V>
__device__ __forceinline__ void checked_store(T* p, V v, int line) {
  if (bounds_ok(p, sizeof(T), line)) *p = (T)v;
}
template <typename T>
__device__ __forceinline__ T checked_ldcg(const T* p, int line) {
  if (bounds_ok(p, sizeof(T), line)) return __ldcg(p);
  T zero{};
  return zero;
}
#define DAD_RANGE_OK(ptr, bytes) ::dad::bounds_ok((ptr), (bytes), __LINE__)
#define DAD_LDCG(ptr) ::dad::checked_ldcg((ptr), __LINE__)
#define DAD_LD(ptr) ::dad::checked_load((ptr), __LINE__)
#define DAD_ST(ptr, value) ::dad::checked_store((ptr), (value), __LINE__)
#else
#define DAD_RANGE_OK(ptr, bytes) true
#define DAD_LDCG(ptr) __ldcg(ptr)
#define DAD_LD(ptr) (*(ptr))
#define DAD_ST(ptr, value) (*(ptr) = (value))
#endif

}  // namespace dad

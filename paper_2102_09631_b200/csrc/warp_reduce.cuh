// Deterministic warp-wide sums of many values per lane (fixed exchange tree).
#pragma once

namespace dad {

// Sum of v[i] over the 32 lanes for NV values per lane with NV - 2 exchanges in all instead of 5 * NV: at every
// step a lane hands half of its values to the partner lane and keeps the other half, so the value count halves
// while the lane distance does.  On return v[0 .. NV/32 - 1] of lane l hold the complete sums of the original
// indices (l's bits, highest distance first, select the half kept) -- see reduced_index().  Fixed tree: deterministic.
template <typename T, int NV>
__device__ __forceinline__ void warp_reduce_scatter(T (&v)[NV], int lane) {
  static_assert(NV % 32 == 0, "one exchange step per lane bit");
#pragma unroll
  for (int o = 16, n = NV; o >= 1; o >>= 1, n >>= 1) {
    const bool upper = (lane & o) != 0;
#pragma unroll
    for (int i = 0; i < n / 2; ++i) {
      const T send = upper ? v[i] : v[i + n / 2];
      const T keep = upper ? v[i + n / 2] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
    }
  }
}
// Original index of v[i] after warp_reduce_scatter<T, NV> in lane `lane`.
template <int NV>
__device__ __forceinline__ int reduced_index(int lane, int i) {
  int idx = 0, n = NV;
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) {
    n >>= 1;
    if (lane & o) idx += n;
  }
  return idx + i;
}

}  // namespace dad

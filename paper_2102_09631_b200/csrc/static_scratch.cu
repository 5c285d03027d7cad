// dad_reconstruct_static: reconstruction from stacked factors for callers that cannot hand the
// library any scratch memory of their own.
//
// Some hosts of this library run where device allocation is off the table: a plug-in inside a
// serving process whose memory pool belongs to the framework, a step that executes under a fixed
// device-memory budget, or code that must not trigger the implicit device synchronisation an
// allocation brings.  dad_reconstruct on the tensor cores needs scratch (bf16 copies of the two
// factor stacks, split partial tiles, counters); here that scratch is a fixed array that lives in
// the library's device image, so the call allocates nothing -- at the price of 32 MiB held on every
// GPU that loads the library, for as long as the process lives.  (The first call on a device makes the
// runtime load the module that holds the array, which is when those 32 MiB are taken; later calls
// change nothing in the device's memory.)
#include <mutex>

#include "common.cuh"

namespace {

// Scratch shared by every call of dad_reconstruct_static on this device.  In host code this name is
// only a handle for cudaGetSymbolAddress; the device address it yields is what the kernels get.
static __device__ __align__(256) unsigned char g_static_scratch[DAD_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device, resolved once per device.
// The first call on a device is also where the CUDA runtime loads this translation unit's module, which is when the
// array's 32 MiB are reserved on that device; a __device__ array starts out zeroed, so the status words at its head
// need no clearing.
cudaError_t scratch_for_current_device(void** out) {
  int dev = -1;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lk(g_mu);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    err = cudaGetSymbolAddress(&p, g_static_scratch);
    if (err != cudaSuccess) return err;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" dad_status dad_reconstruct_static(int64_t h_in, int64_t h_out, int64_t K, const float* Pcat,
                                             const float* Qcat, float* grad, dad_dtype math, void* cuda_stream) {
  if (h_in < 1 || h_out < 1 || K < 1) return DAD_ERR_SHAPE;
  if (math != DAD_F32 && math != DAD_BF16 && math != DAD_BF16_1TERM) return DAD_ERR_DTYPE;
  const size_t need = dad_reconstruct_workspace_bytes(h_in, h_out, K, math);
  if (need > (size_t)DAD_STATIC_SCRATCH_BYTES) return DAD_ERR_WORKSPACE;  // larger problems: dad_reconstruct with caller scratch
  void* scratch = nullptr;
  if (need > 0) {
    if (scratch_for_current_device(&scratch) != cudaSuccess)
      return DAD_ERR_CUDA;
  }
  return dad_reconstruct(h_in, h_out, K, Pcat, Qcat, grad, math, scratch, need > 0 ? (size_t)DAD_STATIC_SCRATCH_BYTES : 0,
                         cuda_stream);
}

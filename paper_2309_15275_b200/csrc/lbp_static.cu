// lbp_backward_static: Algorithm 1 with the scratch memory taken from a
// fixed-size array that is part of the library image, for callers that are not
// able to allocate device memory themselves.
//
// Why it exists.  lbp_backward needs scratch for x_hat, g_y_hat and the status
// block, and leaves its allocation to the caller.  Some callers cannot provide
// it: code that runs under a memory budget fixed at start-up (a server that has
// handed all device memory to its own pool and forbids cudaMalloc afterwards),
// plug-ins that are only given input and output buffers by their host
// framework, and code on a path where an allocation would synchronise the
// device or is simply not permitted.  For them the library holds one scratch
// array per GPU, reserved when the library is loaded on that GPU and kept until
// the process exits.
//
// The array name below is a host-side handle in host code, not a device
// address; the device address is looked up once per device with
// cudaGetSymbolAddress while that device is current, and that address is what
// the kernels receive.
#include <cuda_runtime.h>

#include <atomic>

#include "lbp.h"
#include "lbp_internal.h"

namespace {

// 32 MiB on every GPU that loads the library.
constexpr size_t kStaticScratchBytes = LBP_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::atomic<void*> g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch array on the current device (looked up on the
// first call per device; a query, not an allocation).
int static_scratch_address(void** out) {
  int dev = 0;
  LBP_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return LBP_ERR_ARCH;
  void* ptr = g_scratch_addr[dev].load(std::memory_order_acquire);
  if (ptr == nullptr) {
    // two threads may both look it up: they get the same address
    LBP_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
    g_scratch_addr[dev].store(ptr, std::memory_order_release);
  }
  *out = ptr;
  return LBP_OK;
}

}  // namespace

extern "C" int lbp_backward_static(const void* x, const void* g_y, const void* W, void* g_x,
                                   void* g_W, const lbp_layer* layer, const lbp_basis* set, int r,
                                   void* stream) {
  if (layer == nullptr) return LBP_ERR_NULL;
  // 0 means an invalid layer or rank: the validation below names the exact error
  const size_t need = lbp_workspace_bytes(layer, r);
  if (need > kStaticScratchBytes) return LBP_ERR_WORKSPACE;  // beyond the built-in scratch
  if (int e = lbp::check_device_arch()) return e;
  void* scratch = nullptr;
  if (int e = static_scratch_address(&scratch)) return e;
  // every argument check of lbp_backward, before anything is enqueued
  if (int e = lbp::validate_backward_call(x, g_y, W, g_x, g_W, layer, set, r, scratch,
                                          kStaticScratchBytes))
    return e;
  // The array keeps what the previous call left in it.  Only the status block
  // must start clean (a stale report would be read as this call's); x_hat,
  // g_y_hat and the partial sums are fully rewritten before they are read.
  LBP_CUDA_TRY(cudaMemsetAsync(scratch, 0, lbp_status_bytes(), static_cast<cudaStream_t>(stream)));
  return lbp_backward(x, g_y, W, g_x, g_W, layer, set, r, scratch, kStaticScratchBytes, stream);
}

// sq_linear_static: the whole layer with the library's own, statically reserved scratch.
//
// Some callers of this library cannot allocate device memory at the point where they need a
// layer evaluated: an inference server whose request loop must never enter cudaMalloc (it
// synchronises the device and can fail under memory pressure), a plugin that runs inside a host
// framework which hands it input and output tensors but no allocator, code that has already
// carved the GPU's memory into fixed pools.  sq_linear wants a caller-made workspace for the
// packed activations and their steps; this variant keeps that workspace in a fixed array that is
// part of the loaded library image, so the call path contains no allocation of any kind.
#include <atomic>

#include "sq_internal.h"

namespace {

// The scratch itself.  Every GPU that loads the library holds these bytes until the process
// exits.  In host code this name is only a handle for the symbol, not a device address: the
// address is fetched with cudaGetSymbolAddress below and that pointer is what the kernels get.
static __device__ __align__(256) unsigned char g_static_scratch[SQ_LINEAR_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::atomic<void*> g_scratch_ptr[kMaxDevices];

// Device address of the scratch on the current device; looked up once per device, with that
// device current.  Returns nullptr when the lookup fails.
void* static_scratch_ptr() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  void* p = g_scratch_ptr[dev].load(std::memory_order_acquire);
  if (p != nullptr) return p;
  if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
    cudaGetLastError();
    return nullptr;
  }
  g_scratch_ptr[dev].store(p, std::memory_order_release);
  return p;
}

}  // namespace

extern "C" sq_status_t sq_linear_static(const sq_rotation_t* rot, const void* X, int64_t M, const void* Wq,
                                        const void* sw, int64_t N, int64_t K, void* Y, void* stream) {
  if (!rot || M < 0 || N < 0 || K < 2) return SQ_ERR_INVALID_ARG;
  if (M == 0 || N == 0) return SQ_OK;
  const size_t need = sq_linear_workspace_bytes(M, K);
  if (need > static_cast<size_t>(SQ_LINEAR_STATIC_SCRATCH_BYTES)) return SQ_ERR_UNSUPPORTED;
  void* scratch = static_scratch_ptr();
  if (scratch == nullptr) return SQ_ERR_CUDA;
  // Nothing in the scratch has to start at zero: steps 1+2 overwrite every byte of the packed
  // rows and steps that step 3 reads, so what an earlier call left behind is never seen.
  return sq_linear(rot, X, M, Wq, sw, N, K, scratch, static_cast<size_t>(SQ_LINEAR_STATIC_SCRATCH_BYTES), Y, stream);
}

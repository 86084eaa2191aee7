// surgeon_prune_compact_static: surgeon_prune_compact for callers that have no device scratch
// to hand over and no way to get any.
//
// Some code that wants to prune an activation runs where device memory cannot be allocated: a
// forward hook called while a framework's caching allocator is locked or its pool is frozen
// (for instance while a stream is being captured), a plug-in behind a host API that forbids
// cudaMalloc, or a process whose memory budget was handed out in full at start-up.  Such a
// caller already owns the input and the output buffers of the store, but the select and the
// compaction also need a bit over a megabyte of scratch.  This entry point keeps that
// scratch inside the library image, so nothing is allocated by anybody.
#include <mutex>

#include "surgeon_internal.cuh"

namespace surgeon {
namespace {

// fp32 needs the larger scratch of the two dtypes
constexpr size_t kStaticScratchBytes = prune_workspace_bytes(SURGEON_STATIC_MAX_N, 0);
static_assert(kStaticScratchBytes >= prune_workspace_bytes(SURGEON_STATIC_MAX_N, 1), "scratch");

// The scratch itself: part of the module's global data, present once on every device that
// loads the library, for the life of the process.  In host code this name is only a handle for
// the symbol; the device address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of g_static_scratch on the current device; resolved once per device.
cudaError_t static_scratch(void** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    if (p == nullptr || (reinterpret_cast<uintptr_t>(p) & 255u) != 0) return cudaErrorInvalidValue;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace
}  // namespace surgeon

using namespace surgeon;

extern "C" surgeon_status surgeon_prune_compact_static(const void* x, int64_t n, surgeon_dtype dt,
                                                       double ratio, surgeon_compressed* out,
                                                       void* cuda_stream) {
  if (n > SURGEON_STATIC_MAX_N) return SURGEON_ERR_UNSUPPORTED;  // built-in scratch is too small
  void* scratch = nullptr;
  if (static_scratch(&scratch) != cudaSuccess) return SURGEON_ERR_CUDA;
  // Same checks and the same kernels as the ordinary call; they clear the part of the scratch
  // that has to start at zero, so whatever an earlier call left behind does no harm.
  return surgeon_prune_compact(x, n, dt, ratio, out, scratch, kStaticScratchBytes, cuda_stream);
}

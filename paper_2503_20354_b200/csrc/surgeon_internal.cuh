// Internal declarations shared by the translation units of libsurgeon (CUDA side only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "surgeon.h"

namespace surgeon {

// Storage type and magnitude-key mask per dtype.  The key is the bit pattern with the sign
// bit cleared, compared as an unsigned integer (Algorithm 1: prune step prunes by magnitude).
template <int DT> struct Elem;
template <> struct Elem<0> {
  using type = uint32_t;
  static constexpr uint32_t kKeyMask = 0x7FFFFFFFu;
  static constexpr uint32_t kSentinel = 0xFFFFFFFFu;
  static constexpr int kKeyBits = 31;
};
template <> struct Elem<1> {
  using type = uint16_t;
  static constexpr uint32_t kKeyMask = 0x7FFFu;
  static constexpr uint32_t kSentinel = 0xFFFFu;
  static constexpr int kKeyBits = 15;
};

constexpr int kTileBlocks = 8;                         // offset blocks per compaction tile
constexpr int kTileElems = kTileBlocks * SURGEON_BLOCK;  // 8192 elements per CTA tile

// Scratch layout of surgeon_prune_compact (offsets in bytes from the workspace base).
struct SelectState {
  uint32_t prefix;        // key bits fixed so far (lower bits zero)
  uint32_t compact_ticket;
  long long k_remaining;  // rank still to find inside the current prefix bucket
  long long n_greater;    // keys known to be strictly above the bucket
  uint32_t pass_ticket[4];
  uint32_t pad[2];
};
static_assert(sizeof(SelectState) == 48, "SelectState layout");
constexpr size_t kWsStateBytes = 256;
constexpr int kMaxBins = 2048;
constexpr size_t kWsHistBytes = 3 * kMaxBins * sizeof(uint32_t);  // one histogram per pass

constexpr size_t prune_workspace_bytes(int64_t n) {
  const int64_t tiles = (n + kTileElems - 1) / kTileElems;
  size_t b = kWsStateBytes + kWsHistBytes + static_cast<size_t>(tiles) * 8;
  return (b + 255) & ~static_cast<size_t>(255);
}

// Host launchers (each enqueues on `stream` and returns the last CUDA error).
cudaError_t launch_prune_compact(const void* x, int64_t n, int dt, int64_t k,
                                 const surgeon_compressed& out, void* workspace,
                                 cudaStream_t stream);
cudaError_t launch_decompress(const surgeon_compressed& act, void* x_out, cudaStream_t stream);

size_t weight_grad_fp32_workspace(const surgeon_layer_desc& d);
cudaError_t launch_weight_grad_fp32(const surgeon_compressed& act, const surgeon_layer_desc& d,
                                    const float* grad_out, float* dw, int accumulate,
                                    void* workspace, cudaStream_t stream);

size_t weight_grad_tc_workspace(const surgeon_layer_desc& d);
cudaError_t launch_weight_grad_tc(const surgeon_compressed& act, const surgeon_layer_desc& d,
                                  const float* grad_out, float* dw, int accumulate,
                                  void* workspace, cudaStream_t stream);

// Number of SMs of the current device (cached per device id).
int sm_count();
// Adds to the process-wide kernel-launch counter behind surgeon_launch_count().
void note_launches(int n);

__device__ __forceinline__ uint32_t lane_id() { return threadIdx.x & 31; }
__device__ __forceinline__ uint32_t lanemask_lt() {
  uint32_t m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}
__device__ __forceinline__ uint32_t warp_sum(uint32_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}
// Exclusive prefix sum over the lanes of a warp.
__device__ __forceinline__ uint32_t warp_excl_scan(uint32_t v) {
  uint32_t s = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t t = __shfl_up_sync(0xFFFFFFFFu, s, o);
    if (lane_id() >= static_cast<uint32_t>(o)) s += t;
  }
  return s - v;
}

}  // namespace surgeon

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

constexpr int kBlockShift = 7;                       // log2(SURGEON_BLOCK)
constexpr int kBlockWords = SURGEON_BLOCK / 32;      // bitmap words per offset block
static_assert((1 << kBlockShift) == SURGEON_BLOCK, "SURGEON_BLOCK must be 128");

// ---- scratch of surgeon_prune_compact ---------------------------------------------------------
// Compaction tile ("chunk") = 4 KB of input = 256 16-byte vectors: the unit one warp emits and
// the unit of the exclusive scan that places it.
constexpr int kTileVecs = 256;
constexpr int64_t compact_tile_elems(int dt) { return dt == 0 ? 1024 : 2048; }
constexpr int kBuckets = 32768;        // histogram bins of the select pass (top 15 key bits)
constexpr int kLowBins = 65536;        // bins of the fp32 refinement (low 16 key bits)
constexpr int64_t kSampleMinN = 65536; // tensors up to this size list every non-zero element

struct SelectState {
  uint32_t ticket_sample, ticket_hist, ticket_refine, ticket_count;
  uint32_t blo, bhi;             // bucket bracket around the threshold, predicted from the sample
  uint32_t list_count, list_overflow;
  uint32_t b1, mode;             // bucket of the threshold; 0 = candidate list usable, 1 = re-read x
  uint32_t k1, above;            // rank of the threshold inside bucket b1; keys in buckets above b1
  uint32_t zero_count;           // elements whose key is exactly 0
  uint32_t error;                // surgeon_status raised by a bounded wait of the select kernels
  uint32_t pad[2];
};
static_assert(sizeof(SelectState) == 64, "SelectState layout");
constexpr size_t kWsStateBytes = 256;

// Byte offsets of the parts of the scratch buffer; everything in [0, zero_bytes) must be zero
// when the first kernel starts.  Per compaction tile: cnt_gt / cnt_zero are filled by the
// histogram pass (keys above the bracket, exact zeros), cnt_gt / cnt_eq are completed from the
// candidate list once the threshold is known; full_gt / full_eq are used instead when the
// tensor had to be re-read; prefix holds the exclusive scan the compaction kernel starts from.
struct PruneLayout {
  size_t hist1, hist_s, hist2, cnt_gt, cnt_eq, cnt_zero, full_gt, full_eq, prefix, zero_bytes,
      list, total;
  int64_t tiles, list_cap;
};
constexpr PruneLayout prune_layout(int64_t n, int dt) {
  PruneLayout L{};
  L.tiles = (n + compact_tile_elems(dt) - 1) / compact_tile_elems(dt);
  const size_t per_tile = static_cast<size_t>(L.tiles) * 4;
  size_t off = kWsStateBytes;
  L.hist1 = off; off += static_cast<size_t>(kBuckets) * 4;
  L.hist_s = off; off += static_cast<size_t>(kBuckets) * 4;
  L.hist2 = off; if (dt == 0) off += static_cast<size_t>(kLowBins) * 4;
  L.cnt_gt = off; off += per_tile;
  L.cnt_eq = off; off += per_tile;
  L.cnt_zero = off; off += per_tile;
  L.full_gt = off; off += per_tile;
  L.full_eq = off; off += per_tile;
  off = (off + 15) & ~static_cast<size_t>(15);
  L.prefix = off; off += per_tile * 2 + 8;   // tiles + 1 entries
  off = (off + 255) & ~static_cast<size_t>(255);
  L.zero_bytes = off;
  L.list = off;
  L.list_cap = n <= kSampleMinN ? n : n / 32 + kSampleMinN;
  off += static_cast<size_t>(L.list_cap) * 8;
  L.total = (off + 255) & ~static_cast<size_t>(255);
  return L;
}
constexpr size_t prune_workspace_bytes(int64_t n, int dt) { return prune_layout(n, dt).total; }

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

// The driver's cuTensorMapEncodeTiled, looked up through the runtime (the library carries no
// link-time dependency on the driver library); nullptr if unavailable.
void* tensor_map_encode_fn();
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

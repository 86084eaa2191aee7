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
constexpr int kBuckets = 32768;        // bins of the sample histogram (top 15 key bits)
constexpr int kBinsA = 512;            // level A of the select among candidates: the top bits of
                                       // (key - lo_key), shifted so that the bracket fits
constexpr int kBinsB = 4096;           // up to two further levels of 2048 bins each
constexpr int kFbBins = 2048;          // digit histogram of the fall-back radix select
// Tensors below this size go straight to the fall-back select: its passes over a tensor that
// stays in L2 finish sooner than the four dependent kernels of the sampled path.  Alone on the
// GPU that holds up to 16-32 MB; next to other streams' kernels the fall-back's cooperative
// grid (one CTA per 32 chunks) has to wait for them, and 4 MB is where both cases gain.
constexpr int64_t kStreamMinBytes = 4 << 20;
// Candidate slots: per chunk, room for 1/16 of its elements (fp32: 32-bit keys, bf16: 16-bit).
constexpr int slot_entries(int dt) { return dt == 0 ? 64 : 128; }
constexpr int slot_entry_bytes(int dt) { return dt == 0 ? 4 : 2; }

struct SelectState {
  uint32_t ticket_sample, ticket_classify, barrier_count, error;
  uint32_t blo, bhi;             // bucket bracket around the threshold, predicted from the sample
  uint32_t lo_key, hi_key;       // the same bracket as an inclusive key range (lo_key >= 1)
  uint32_t mode;                 // 0 = threshold among the candidates, level B pending (fp32);
                                 // 1 = bracket unusable, fall back to a radix select over x;
                                 // 2 = threshold already final in the header;
                                 // 4 = likewise, and every key inside the bracket equals it
  uint32_t list_overflow;
  uint32_t above_total, cand_total;   // keys above hi_key / inside [lo_key, hi_key]
  uint32_t shiftA;               // level A bin of a key = (key - lo_key) >> shiftA
  uint32_t binA, rankA, aboveA;  // level A: bin of the threshold, its rank inside, candidates above
  uint32_t fb_prefix, fb_rank, fb_above;   // fall-back select: key bits fixed so far, rank, count above
  uint32_t reserved0;            // (unused)
  uint32_t cand_key_max, cand_keyinv_max;   // extremes of the keys inside the bracket: max key, max ~key
  uint32_t pad[10];
};
static_assert(sizeof(SelectState) == 128, "SelectState layout");
constexpr size_t kWsStateBytes = 256;

// Byte offsets of the parts of the scratch buffer; everything in [0, zero_bytes) must be zero
// when the first kernel starts.  Per chunk: cnt_gt = keys above the bracket, cand_cnt = keys
// inside it (both written by the classify pass), val = (kept for sure << 31 | ties) once the
// threshold is known, prefix = exclusive scan of val (chunks + 1 entries), slots = the keys
// inside the bracket.  partial: one scan carry per CTA of the count kernel.
struct PruneLayout {
  size_t hist_s, hist_a, hist_b, hist_fb, zero_bytes, cnt_gt, cand_cnt, val, prefix, partial,
      slots, total;
  int64_t tiles;
};
constexpr size_t kMaxCountCtas = 1024;
constexpr PruneLayout prune_layout(int64_t n, int dt) {
  PruneLayout L{};
  L.tiles = (n + compact_tile_elems(dt) - 1) / compact_tile_elems(dt);
  const size_t t = static_cast<size_t>(L.tiles);
  size_t off = kWsStateBytes;
  L.hist_s = off; off += static_cast<size_t>(kBuckets) * 4;
  L.hist_a = off; off += static_cast<size_t>(kBinsA) * 4;
  L.hist_b = off; off += static_cast<size_t>(kBinsB) * 4;
  L.hist_fb = off; off += static_cast<size_t>(3 * kFbBins) * 4;
  L.zero_bytes = off;
  L.cnt_gt = off; off += t * 4;
  L.cand_cnt = off; off += t * 4;
  off = (off + 15) & ~static_cast<size_t>(15);
  L.val = off; off += t * 8;
  L.prefix = off; off += (t + 1) * 8;
  L.partial = off; off += kMaxCountCtas * 8;
  off = (off + 255) & ~static_cast<size_t>(255);
  L.slots = off;
  off += t * static_cast<size_t>(slot_entries(dt)) * slot_entry_bytes(dt);
  L.total = (off + 255) & ~static_cast<size_t>(255);
  return L;
}
constexpr size_t prune_workspace_bytes(int64_t n, int dt) { return prune_layout(n, dt).total; }

// Host launchers (each enqueues on `stream` and returns the last CUDA error).
cudaError_t launch_prune_compact(const void* x, int64_t n, int dt, int64_t k,
                                 const surgeon_compressed& out, void* workspace,
                                 cudaStream_t stream, int drop_zeros = 0, int stall = 0);
cudaError_t launch_decompress(const surgeon_compressed& act, void* x_out, cudaStream_t stream);
// Eq. 4 on device: *gi_out = sqrt(sum dw^2 / n); workspace = SURGEON_GI_WORKSPACE_BYTES of scratch.
cudaError_t launch_gradient_importance(const float* dw, long long n, double* gi_out,
                                       void* workspace, cudaStream_t stream);

size_t weight_grad_fp32_workspace(const surgeon_layer_desc& d);
cudaError_t launch_weight_grad_fp32(const surgeon_compressed& act, const surgeon_layer_desc& d,
                                    const float* grad_out, float* dw, int accumulate,
                                    void* workspace, cudaStream_t stream);

size_t weight_grad_grouped_workspace(const surgeon_layer_desc& d);
cudaError_t launch_weight_grad_grouped(const surgeon_compressed& act, const surgeon_layer_desc& d,
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
// Lets `kernel` use `bytes` of dynamic shared memory; the attribute is set when a kernel first
// needs that much on a device, later calls only look it up.
cudaError_t allow_dynamic_smem(const void* kernel, int bytes);
// Adds to the process-wide kernel-launch counter behind surgeon_launch_count().
void note_launches(int n);

// Programmatic dependent launch.  A kernel launched with `dependent` set may start while the
// kernel before it on the stream is still running (once every CTA of that kernel has called
// pdl_trigger or has exited): its set-up then overlaps the predecessor's tail.  It must call
// pdl_wait before it touches anything the predecessor writes; pdl_wait returns when the
// predecessor has completed and its writes are visible.  Both calls do nothing in a kernel that
// was launched the ordinary way.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                 cudaStream_t stream, bool dependent, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = dependent ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Checked builds (-DSURGEON_BOUNDS, the library's stand-in for a memory checker): every guarded
// global store tests its index against the size the host computed for the buffer; an index
// outside records SURGEON_ERR_INTERNAL in `status_word` and the store is skipped.  In the
// ordinary build the test compiles away.
#ifdef SURGEON_BOUNDS
#define SURGEON_IN_BOUNDS(idx, limit, status_word)                                              \
  ((static_cast<unsigned long long>(idx) < static_cast<unsigned long long>(limit)) ||           \
   (atomicMax((status_word), static_cast<uint32_t>(SURGEON_ERR_INTERNAL)), false))
#else
#define SURGEON_IN_BOUNDS(idx, limit, status_word) true
#endif

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

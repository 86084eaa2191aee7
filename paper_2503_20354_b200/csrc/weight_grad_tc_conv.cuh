// Plan and launcher of the fast stride-1 convolution kernel (weight_grad_tc_conv.cu).
#pragma once

#include <cuda.h>

#include "surgeon_internal.cuh"

#include <cstring>

namespace surgeon {

// Plans depend only on the layer geometry (and the device's SM count): a weight-gradient call
// looks its plan up in a small per-thread table instead of searching tilings and split counts
// again (the searches cost microseconds, as much as a kernel launch).  `Tag` separates the tables
// of the different planners.
template <typename Tag, typename P, typename F>
inline bool memo_plan(const surgeon_layer_desc& d, int extra, P* out, F compute) {
  struct Entry { surgeon_layer_desc d; int extra, dev; bool used, ok; P p; };
  constexpr int kEntries = 64;
  thread_local Entry table[kEntries] = {};
  thread_local int next = 0;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) dev = 0;
  for (int i = 0; i < kEntries; ++i) {
    const Entry& e = table[i];
    if (e.used && e.extra == extra && e.dev == dev && std::memcmp(&e.d, &d, sizeof(d)) == 0) {
      if (e.ok) *out = e.p;
      return e.ok;
    }
  }
  Entry& e = table[next];
  next = (next + 1) % kEntries;
  e.d = d; e.extra = extra; e.dev = dev; e.used = true;
  e.p = P{};
  e.ok = compute(&e.p);
  if (e.ok) *out = e.p;
  return e.ok;
}

struct FastParams {
  int mode;                 // 0 = 3x3 pad 1 through a shared-memory patch, 1 = 1x1 direct
  int stride;               // 1 or 2
  int B, C, H, W, O, OH, OW;
  int P;                    // output positions per image (= OH*OW)
  int n_gemm;               // C*KH*KW
  int acc_n, n_acc;         // columns per accumulator, accumulators per CTA (1 or 2)
  int n_tiles, m_tiles;
  int tiles_per_img, total_ktiles, ktiles_per_split, splits;
  int tmem_cols, stages, smem_bytes;
};

// False when the layer is not one the fast kernel handles.
bool plan_conv_fast(const surgeon_layer_desc& d, FastParams* out);

// Bytes of scratch for the bf16 copy of the output gradient.
size_t conv_fast_grad_bf16_bytes(const FastParams& p);

// Enqueues the bf16 conversion of grad_out into grad_bf16 and the kernel;
// partial = [splits][O][n_gemm] fp32, status = one zeroed word.
cudaError_t launch_conv_fast(const surgeon_compressed& act, const FastParams& p,
                             const float* grad_out, void* grad_bf16, float* partial,
                             uint32_t* status, cudaStream_t stream);

// fp32 -> bf16 (round to nearest even) copy of n elements, as one streaming kernel.
cudaError_t launch_grad_to_bf16(const float* g, long long n, void* out_bf16, cudaStream_t stream);
// The same for `rows` rows of `len` elements, written with a row pitch of `pitch` >= len
// elements (a multiple of 8); the padding is zero.
cudaError_t launch_grad_to_bf16_rows(const float* g, long long rows, int len, int pitch,
                                     void* out_bf16, cudaStream_t stream);

// ---- layers whose im2col operand is the activation itself (weight_grad_tc_direct.cu) ----------
struct DirectParams {
  int mode;                 // 0 = linear [T, C] (MN-major operands), 1 = conv 1x1 stride 1 (K-major),
                            // 2 = conv 1x1 stride 2 (K-major, sampled input)
  int ow, in_w, in_hw;      // mode 2: output row length, input row length, input plane size
  int taps;                 // 1, or kh*kw for a k x k stride-1 conv (mode 1 over shifted gradients)
  int kh, kw, pad, in_h, oh;  // taps > 1: kernel and map sizes (with ow, in_w)
  int o_real;               // output channels of the layer; O = taps * o_real
  int row_shift;            // taps > 1: only the kw column shifts are stored; rows shift by TMA offset
  int copies;               // stacked gradient copies: taps, or kw with row_shift
  int g_len;                // conv: elements per row of the gradient copy (T, or oh * in_w)
  int upt, n_units;         // conv: accumulator units per tap (of acc_n columns), units in all
  int C, O;                 // input channels / gradient channels (taps * output channels)
  int T;                    // linear: rows; conv: positions per image
  int pitch;                // elements per row of the bf16 gradient copy
  int imgs;                 // conv: batch; linear: 1
  int acc_n, n_acc, n_cols; // columns per accumulator, accumulators per CTA, their product
  int m_tiles, n_tiles, splits;
  int tiles_per_img, total_ktiles, ktiles_per_split;
  int rows_per_tile;        // channels per row tile (128, or fewer when C is spread evenly; a multiple of 16)
  int pair;                 // 1: CTA pairs (cta_group::2) over two row tiles; m_tiles is then even
  int a_stages, b_stages;   // depth of the activation-tile and gradient-tile rings
  int tmem_cols, smem_bytes;
  long long n_words;        // words of the bitmap (filled by the launcher)
  const long long* n_keep_ptr;  // device address of the store's count of packed values (launcher)
  unsigned partial_blk;     // index of the bitmap's last block if it is partial, else 0xFFFFFFFF
};
bool plan_direct(const surgeon_layer_desc& d, DirectParams* out);
size_t direct_grad_bf16_bytes(const DirectParams& p);
// partial = [splits][O][C] fp32 (O counts the stacked taps), status = one zeroed word.
cudaError_t launch_direct(const surgeon_compressed& act, const DirectParams& p,
                          const float* grad_out, void* grad_bf16, float* partial,
                          uint32_t* status, cudaStream_t stream);
// The pre-pass that writes the bf16 copy (or shifted copies) of the output gradient, and the
// tensor map over it (conv: boxes of 64 positions x box_rows rows; linear: 64 columns x 64 rows).
cudaError_t launch_direct_prepass(const DirectParams& p, const float* grad_out, void* grad_bf16,
                                  cudaStream_t stream);
cudaError_t encode_direct_grad_map(const DirectParams& p, void* grad_bf16, int box_rows, CUtensorMap* out);

// ---- the same layers on CTA pairs with the operand roles exchanged (weight_grad_tc_swap.cu) -----
struct SwapParams {
  DirectParams d;           // layer geometry and the layout of the bf16 gradient copy
  int nt, half;             // input channels per pair tile (MMA N, a multiple of 16) and per CTA
  int n_acc;                // accumulators per CTA: 128 gradient rows x nt channels each
  int lpr;                  // lanes (runs of 32 elements) per row of the activation tile: 2 or 4
  // conv: the stacked gradient rows (tap, output channel) are cut into units of 128 TMEM lanes.
  // Per tap a_units full units of 128 rows (one TMA box each; the last may be partly filled when
  // rem_box is 0); the o_real - 128 * a_full rows left over, if any, go `rpu` taps to a unit in
  // boxes of rem_box rows (a power of two below 128).
  int a_full, a_units, rem_box, rpu;
  int n_units;              // units in all (linear: groups of 128 gradient columns)
  int m_tiles, n_tiles, splits, ktiles_per_split;
  int gw, groups;           // warps per producer group, groups (one K-tile in flight per group)
  int a_stages, g_stages;   // depth of the activation-tile and gradient-tile rings
  int stage_bytes;          // staging area of packed values (fp32 activations), 0 if none
  int tmem_cols, smem_bytes;
  long long n_words;        // words of the bitmap (filled by the launcher)
  const long long* n_keep_ptr;
  unsigned partial_blk;     // index of the bitmap's last block if it is partial, else 0xFFFFFFFF
};
bool plan_swap(const surgeon_layer_desc& d, SwapParams* out);
int swap_resident_pairs();   // CTA pairs the device holds at once
size_t swap_partial_bytes(const SwapParams& p);
// partial = [splits][O][C] fp32 (O counts the stacked taps), status = one zeroed word.
cudaError_t launch_swap(const surgeon_compressed& act, const SwapParams& p, const float* grad_out,
                        void* grad_bf16, float* partial, uint32_t* status, cudaStream_t stream);

}  // namespace surgeon

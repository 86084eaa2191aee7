// Tensor-core path of surgeon_weight_grad (Algorithm 1: Reshape and gradient steps, Eq. 2) for sm_100a.
//
// Implicit GEMM on tcgen05:  D[nn, o] = sum_k Acol[nn, k] * G[o, k]
//   nn = (c, r, s)  im2col column of the activation  -> MMA M (128 rows per CTA tile, TMEM lanes)
//   o  = output channel                              -> MMA N (tile of <= 256, TMEM columns)
//   k  = (b, y, x) output position / row t           -> MMA K, 64 per pipeline stage
// Both operands are bf16, K-major, in the 128-byte-swizzled shared-memory layout that the UMMA
// descriptors name; accumulation is fp32 in tensor memory.
//
// Nothing dense comes from HBM: producer warps read the bitmap, the block offsets and the packed
// values, rebuild the rows of the pruned activation a K-tile needs in a shared-memory patch
// (Algorithm 1: Reshape step, "Reshape"), and write the im2col view of that patch into the operand
// tile.  The same warps convert the fp32 output gradient to bf16 on the way into its tile.  One
// elected thread issues the MMAs; tcgen05.commit hands stages back to the producers.
// The reduction is split over CTAs in contiguous K ranges; partial tiles go to scratch and are
// summed in a fixed order, so results are bitwise reproducible.
//
// Every wait on an mbarrier is bounded; when one gives up the CTA records SURGEON_ERR_TIMEOUT in
// the scratch status word, frees its tensor memory and returns.
#include <cuda.h>

#include "surgeon_internal.cuh"
#include "tc_common.cuh"
#include "weight_grad_tc_conv.cuh"

namespace surgeon {

namespace {

using namespace tc;

constexpr int kTileM = 128;          // im2col columns (nn) per CTA tile = TMEM lanes
constexpr int kTileK = 64;           // bf16 elements per stage row = one 128-byte swizzle row
constexpr int kProducerWarps = 8;
constexpr int kProducerThreads = kProducerWarps * 32;
constexpr int kThreads = 32 + kProducerThreads;  // warp 0 issues MMAs
constexpr int kPatchBytes = 32 * 1024;
constexpr int kPatchElems = kPatchBytes / 2;
constexpr int kMaxStages = 4;
constexpr size_t kStatusBytes = 256;  // scratch header in front of the partial tiles

struct TcParams {
  // layer
  int kind, B, C, H, W, O, KH, KW, stride, pad, OH, OW;
  int P;            // output positions per image (conv) or rows T (linear)
  int n_gemm;       // C*KH*KW
  int RS;           // KH*KW
  // tiling
  int tile_n;       // output channels per CTA tile (multiple of 16, <= 256)
  int m_tiles, n_tiles, splits;
  int tiles_per_img, total_ktiles, ktiles_per_split;
  int stages, tmem_cols;
  int group_ch;     // channels (conv) decompressed per patch pass
  int max_rows;     // input rows one K-tile can touch (conv)
  int dt;           // activation dtype
  int g_vec_ok;     // gradient rows can be read with 16-byte loads
  int ch_pitch;     // elements between the channels of the patch (conv), a multiple of 32
  long long n_words;  // words of the bitmap (filled by the launcher)
};

__device__ __forceinline__ void producer_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(kProducerThreads) : "memory");
}

// ---- decompression of one contiguous flat range into shared memory (one warp) ---------------
// dst[i] = bf16 of the pruned activation at flat index start + i, i < len  (Algorithm 1: Reshape step).
template <int DT>
__device__ __forceinline__ void decompress_range(const uint32_t* __restrict__ bitmap,
                                                 const void* __restrict__ values,
                                                 const uint32_t* __restrict__ offsets,
                                                 long long start, int len,
                                                 unsigned short* __restrict__ dst) {
  const uint32_t lane = lane_id();
  const uint32_t lt = lanemask_lt();
  const long long first_word = start >> 5;
  const long long last_word = (start + len - 1) >> 5;
  const long long blk = start >> kBlockShift;
  const long long blk_word0 = blk * kBlockWords;
  uint32_t w = 0;
  if (blk_word0 + lane < first_word) w = __ldg(bitmap + blk_word0 + lane);
  uint32_t rank0 = __ldg(offsets + blk) + warp_sum(__popc(w));    // kept before first_word
  // 32 bitmap words per round: every lane fetches one word, a warp scan ranks them, and the
  // value loads of the round do not depend on one another
  for (long long w0 = first_word; w0 <= last_word; w0 += 32) {
    const long long mine = w0 + lane;
    const uint32_t my_word = (mine <= last_word) ? __ldg(bitmap + mine) : 0u;
    const uint32_t my_cnt = __popc(my_word);
    const uint32_t my_excl = warp_excl_scan(my_cnt);
    const int n_here = static_cast<int>(last_word - w0 < 31 ? last_word - w0 + 1 : 32);
#pragma unroll 4
    for (int i = 0; i < n_here; ++i) {
      const uint32_t word = __shfl_sync(0xFFFFFFFFu, my_word, i);
      const uint32_t before = __shfl_sync(0xFFFFFFFFu, my_excl, i);
      const long long j = ((w0 + i) << 5) + lane;
      const bool in_range = (j >= start) && (j < start + len);
      unsigned short v = 0;
      if (in_range && ((word >> lane) & 1u)) {
        const uint32_t r = rank0 + before + __popc(word & lt);
        if (DT == 0) v = to_bf16_bits(__ldg(reinterpret_cast<const float*>(values) + r));
        else v = __ldg(reinterpret_cast<const unsigned short*>(values) + r);
      }
      if (in_range) dst[j - start] = v;
    }
    rank0 += __shfl_sync(0xFFFFFFFFu, my_excl + my_cnt, 31);
  }
}

// One thread rebuilds up to 32 consecutive elements: dst[0..31] (64 bytes, 16-byte aligned) =
// bf16 of the pruned activation at flat indices start .. start + len - 1, zeros after them.
// The work after the fixed part is one load and one store per kept element.
template <int DT>
__device__ __forceinline__ void decompress_run(const uint32_t* __restrict__ bitmap,
                                               const void* __restrict__ values,
                                               const uint32_t* __restrict__ offsets,
                                               long long n_words, long long start, int len,
                                               unsigned short* __restrict__ dst) {
  uint4* d4 = reinterpret_cast<uint4*>(dst);
  d4[0] = make_uint4(0, 0, 0, 0); d4[1] = make_uint4(0, 0, 0, 0);
  d4[2] = make_uint4(0, 0, 0, 0); d4[3] = make_uint4(0, 0, 0, 0);
  const long long blk = start >> kBlockShift;
  const long long wi = start >> 5;
  uint32_t rank = __ldg(offsets + blk);
  for (long long w = blk * kBlockWords; w < wi; ++w) rank += __popc(__ldg(bitmap + w));
  const uint32_t w0 = __ldg(bitmap + wi);
  const uint32_t w1 = (wi + 1 < n_words) ? __ldg(bitmap + wi + 1) : 0u;
  const uint32_t sh = static_cast<uint32_t>(start & 31);
  rank += __popc(w0 & ((1u << sh) - 1u));
  uint32_t bits = __funnelshift_r(w0, w1, sh);
  if (len < 32) bits &= (1u << len) - 1u;
  const uint32_t count = __popc(bits);
  for (uint32_t g = 0; g < count; g += 8) {      // eight independent loads in flight per round
    uint32_t v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = ld_packed<DT>(values, rank + g + i, g + i < count);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (g + i < count) {
        const int b = __ffs(bits) - 1;
        bits &= bits - 1;
        dst[b] = (DT == 0) ? to_bf16_bits(__uint_as_float(v[i])) : static_cast<unsigned short>(v[i]);
      }
    }
  }
}

struct RowInfo {   // one im2col row (nn) of the CTA's M tile
  short c;         // input channel, -1 when nn is past the end
  signed char r, s;
};

template <int DT>
__global__ void __launch_bounds__(kThreads, 1)
dw_tc_kernel(const uint32_t* __restrict__ bitmap, const void* __restrict__ values,
             const uint32_t* __restrict__ offsets, const float* __restrict__ grad,
             float* __restrict__ partial, uint32_t* __restrict__ status, TcParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  // carve: [stages][A 16 KB | B tile_n*128] | patch | barriers | row table
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int b_bytes = p.tile_n * 128;
  const int stage_bytes = kTileM * 128 + b_bytes;
  unsigned short* patch = reinterpret_cast<unsigned short*>(smem + p.stages * stage_bytes);
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(
      smem + p.stages * stage_bytes + kPatchBytes);
  RowInfo* rows = reinterpret_cast<RowInfo*>(bars + 2 * kMaxStages + 2);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(rows + kTileM);
  volatile uint32_t* fail = tmem_slot + 1;

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const uint32_t lane = lane_id();
  const int m_tile = blockIdx.x, n_tile = blockIdx.y, split = blockIdx.z;
  const int nn0 = m_tile * kTileM;
  const int o0 = n_tile * p.tile_n;
  const int kt_begin = split * p.ktiles_per_split;
  const int kt_end = min(kt_begin + p.ktiles_per_split, p.total_ktiles);
  const int n_kt = kt_end - kt_begin;

  const uint32_t full_bar = smem_u32(bars);
  const uint32_t empty_bar = smem_u32(bars + kMaxStages);
  const uint32_t acc_bar = smem_u32(bars + 2 * kMaxStages);

  if (tid == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(full_bar + 8 * s, kProducerWarps);
      mbar_init(empty_bar + 8 * s, 1);
    }
    mbar_init(acc_bar, 1);
    *fail = 0;
    fence_barrier_init();
  }
  for (int i = tid; i < kTileM; i += kThreads) {
    const int nn = nn0 + i;
    RowInfo ri;
    if (nn < p.n_gemm) {
      const int c = nn / p.RS;
      const int rs = nn - c * p.RS;
      ri.c = static_cast<short>(c);
      ri.r = static_cast<signed char>(rs / p.KW);
      ri.s = static_cast<signed char>(rs - (rs / p.KW) * p.KW);
    } else {
      ri.c = -1; ri.r = 0; ri.s = 0;
    }
    rows[i] = ri;
  }
  if (warp == 0) tmem_alloc(smem_u32(tmem_slot), p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ================= MMA issuer =================
    if (lane == 0) {
      const uint32_t idesc = make_idesc(kTileM, p.tile_n);
      const uint32_t smem0 = smem_u32(smem);
      const uint64_t a_base = make_desc(smem0);
      const uint64_t b_base = make_desc(smem0 + kTileM * 128);
      const uint64_t stage_inc = static_cast<uint64_t>(stage_bytes >> 4);
      uint64_t da = a_base, db = b_base;
      uint32_t parity = 0, accum = 0;
      int s = 0;
      bool ok = true;
      for (int it = 0; it < n_kt; ++it) {
        ok = mbar_wait(full_bar + 8 * s, parity);
        if (!ok) break;
        tc_fence_after();
        umma_ktile<1, 2>(tmem_base, p.tile_n, da, db, 0, idesc, accum);
        umma_commit(empty_bar + 8 * s);   // stage is free once these MMAs have read it
        accum = 1;
        if (++s == p.stages) { s = 0; parity ^= 1; da = a_base; db = b_base; }
        else { da += stage_inc; db += stage_inc; }
      }
      if (!ok) { *fail = 1; atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT)); }
      umma_commit(acc_bar);               // accumulator complete (or abandoned)
    }
    __syncwarp();
  } else {
    // ================= producers =================
    const int ptid = tid - 32;
    const int pwarp = warp - 1;
    const int first_c = rows[0].c;       // M tiles never start past the end
    int last_c = first_c;
    for (int i = kTileM - 1; i >= 0; --i) {
      if (rows[i].c >= 0) { last_c = rows[i].c; break; }
    }
    bool ok = true;
    for (int it = 0; it < n_kt; ++it) {
      const int s = it % p.stages;
      if (it >= p.stages && ptid == 0) {     // one thread polls; the rest wait at the barrier below
        const uint32_t parity = ((it / p.stages) - 1) & 1;
        if (!mbar_wait(empty_bar + 8 * s, parity, 32)) {
          *fail = 1;
          atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
        }
      }
      producer_sync();            // after it, every producer reads the same value of *fail
      if (*fail) { ok = false; break; }
      unsigned char* a_tile = smem + s * stage_bytes;
      unsigned char* b_tile = a_tile + kTileM * 128;
      const int kt = kt_begin + it;
      const int img = kt / p.tiles_per_img;
      const int p0 = (kt - img * p.tiles_per_img) * kTileK;

      // ---- gradient tile: fp32 -> bf16, rows = output channels, K contiguous ----
      if (p.kind == 1) {
        const int tasks = p.tile_n * 8;
        for (int t = ptid; t < tasks; t += kProducerThreads) {
          const int row = t >> 3, chunk = t & 7;
          const int o = o0 + row;
          const int pp = p0 + chunk * 8;
          uint4 out = make_uint4(0, 0, 0, 0);
          if (o < p.O && pp < p.P) {
            const float* src = grad + (static_cast<long long>(img) * p.O + o) * p.P + pp;
            if (p.g_vec_ok && pp + 8 <= p.P) {
              const float4 a = __ldg(reinterpret_cast<const float4*>(src));
              const float4 b = __ldg(reinterpret_cast<const float4*>(src) + 1);
              out.x = pack_bf16x2(a.x, a.y); out.y = pack_bf16x2(a.z, a.w);
              out.z = pack_bf16x2(b.x, b.y); out.w = pack_bf16x2(b.z, b.w);
            } else {
              float v[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) v[e] = (pp + e < p.P) ? __ldg(src + e) : 0.0f;
              out.x = pack_bf16x2(v[0], v[1]); out.y = pack_bf16x2(v[2], v[3]);
              out.z = pack_bf16x2(v[4], v[5]); out.w = pack_bf16x2(v[6], v[7]);
            }
          }
          *reinterpret_cast<uint4*>(b_tile + tile_off(row, chunk)) = out;
        }
      } else {
        // linear: grad is [T, O]; lanes take consecutive output channels
        const int tasks = p.tile_n * 8;
        for (int t = ptid; t < tasks; t += kProducerThreads) {
          const int chunk = t / p.tile_n, row = t - chunk * p.tile_n;
          const int o = o0 + row;
          const int pp = p0 + chunk * 8;
          float v[8];
#pragma unroll
          for (int e = 0; e < 8; ++e)
            v[e] = (o < p.O && pp + e < p.P)
                       ? __ldg(grad + static_cast<long long>(pp + e) * p.O + o) : 0.0f;
          uint4 out;
          out.x = pack_bf16x2(v[0], v[1]); out.y = pack_bf16x2(v[2], v[3]);
          out.z = pack_bf16x2(v[4], v[5]); out.w = pack_bf16x2(v[6], v[7]);
          *reinterpret_cast<uint4*>(b_tile + tile_off(row, chunk)) = out;
        }
      }

      // ---- activation tile: decompress a patch, then write its im2col view ----
      if (p.kind == 1) {
        const int k_valid = min(kTileK, p.P - p0);
        const int y_first = p0 / p.OW;
        const int y_last = (p0 + k_valid - 1) / p.OW;
        int iy_lo = y_first * p.stride - p.pad;
        int iy_hi = y_last * p.stride + p.KH - 1 - p.pad;
        if (iy_lo < 0) iy_lo = 0;
        if (iy_hi > p.H - 1) iy_hi = p.H - 1;
        const int range_len = (iy_hi - iy_lo + 1) * p.W;
        for (int cg = first_c; cg <= last_c; cg += p.group_ch) {
          const int cg_end = min(cg + p.group_ch, last_c + 1);
          // one task = 32 consecutive elements of one channel's rows
          const int runs = (range_len + 31) >> 5;
          const int n_tasks = (cg_end - cg) * runs;
          for (int t = ptid; t < n_tasks; t += kProducerThreads) {
            const int ci = t / runs, run = t - ci * runs;
            const long long start =
                ((static_cast<long long>(img) * p.C + cg + ci) * p.H + iy_lo) * p.W + 32 * run;
            decompress_run<DT>(bitmap, values, offsets, p.n_words, start,
                               min(32, range_len - 32 * run), patch + ci * p.ch_pitch + 32 * run);
          }
          producer_sync();
          // rows of this channel group: nn in [cg*RS, cg_end*RS)
          int row_lo = cg * p.RS - nn0;
          int row_hi = cg_end * p.RS - nn0;
          if (row_lo < 0) row_lo = 0;
          if (row_hi > kTileM || cg_end > last_c) row_hi = kTileM;   // last group also zeroes pad rows
          const int tasks = (row_hi - row_lo) * 8;
          for (int t = ptid; t < tasks; t += kProducerThreads) {
            const int row = row_lo + (t >> 3), chunk = t & 7;
            const RowInfo ri = rows[row];
            uint32_t h[8];
            if (ri.c < 0) {
#pragma unroll
              for (int e = 0; e < 8; ++e) h[e] = 0;
            } else {
              const unsigned short* src = patch + (ri.c - cg) * p.ch_pitch;
              int pp = p0 + chunk * 8;
              int y = pp / p.OW;
              int x = pp - y * p.OW;
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const int iy = y * p.stride + ri.r - p.pad;
                const int ix = x * p.stride + ri.s - p.pad;
                uint32_t v = 0;
                if (pp < p.P && iy >= iy_lo && iy <= iy_hi && ix >= 0 && ix < p.W)
                  v = src[(iy - iy_lo) * p.W + ix];
                h[e] = v;
                ++pp; ++x;
                if (x == p.OW) { x = 0; ++y; }
              }
            }
            uint4 out;
            out.x = h[0] | (h[1] << 16); out.y = h[2] | (h[3] << 16);
            out.z = h[4] | (h[5] << 16); out.w = h[6] | (h[7] << 16);
            *reinterpret_cast<uint4*>(a_tile + tile_off(row, chunk)) = out;
          }
          producer_sync();   // the patch is overwritten by the next group / stage
        }
      } else {
        // linear: activation [T, C]; patch[k][i] = A[p0 + k, nn0 + i]
        const int k_valid = min(kTileK, p.P - p0);
        const int c_valid = min(kTileM, p.n_gemm - nn0);
        for (int k = pwarp; k < k_valid; k += kProducerWarps) {
          decompress_range<DT>(bitmap, values, offsets,
                               static_cast<long long>(p0 + k) * p.C + nn0, c_valid,
                               patch + k * kTileM);
        }
        producer_sync();
        for (int t = ptid; t < kTileM * 8; t += kProducerThreads) {
          const int chunk = t >> 7, row = t & (kTileM - 1);
          uint32_t h[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const int k = chunk * 8 + e;
            h[e] = (row < c_valid && k < k_valid) ? patch[k * kTileM + row] : 0u;
          }
          uint4 out;
          out.x = h[0] | (h[1] << 16); out.y = h[2] | (h[3] << 16);
          out.z = h[4] | (h[5] << 16); out.w = h[6] | (h[7] << 16);
          *reinterpret_cast<uint4*>(a_tile + tile_off(row, chunk)) = out;
        }
        producer_sync();
      }
      fence_proxy_async();   // generic-proxy writes -> visible to the tensor core's reads
      __syncwarp();
      if (lane == 0) mbar_arrive(full_bar + 8 * s);
    }
    (void)ok;
  }

  // ================= epilogue: TMEM -> scratch partial tile =================
  if (warp >= 1) {
    // 8 warps: a warp may read the 32 TMEM lanes of its quarter (warp % 4); the two warps of a
    // quarter take alternate groups of 16 columns
    const bool done = mbar_wait(acc_bar, 0, 64);
    tc_fence_after();
    if (done && !*fail) {
      const int lane_grp = warp & 3;              // TMEM lanes this warp may read
      const int row = lane_grp * 32 + static_cast<int>(lane);
      const int nn = nn0 + row;
      float* out = partial + static_cast<long long>(split) * p.O * p.n_gemm;
      for (int col = 16 * ((warp - 1) >> 2); col < p.tile_n; col += 32) {
        uint32_t r[16];
        tmem_ld16(tmem_base + (static_cast<uint32_t>(lane_grp * 32) << 16) + col, r);
        if (nn < p.n_gemm) {
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const int o = o0 + col + e;
            if (o < p.O && SURGEON_IN_BOUNDS(static_cast<long long>(split) * p.O * p.n_gemm +
                                                 static_cast<long long>(o) * p.n_gemm + nn,
                                             static_cast<long long>(p.splits) * p.O * p.n_gemm, status))
              out[static_cast<long long>(o) * p.n_gemm + nn] = __uint_as_float(r[e]);
          }
        }
      }
    } else if (!done && lane == 0) {
      atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, p.tmem_cols);
}

// ---- conv layers: the same GEMM with two producer groups and the gradient by TMA ---------------
// Group g (8 warps) fills the K-tiles g, g + 2, ... of the CTA's range, each group with its own
// patch, so the load latency of one group's decompression hides behind the other group's gather.
// The output gradient is a bf16 copy written by a pre-pass ([B][O][pitch]); one thread of the
// group starts its TMA load when the stage is free.  The gather copies 8 output positions per
// task; when they lie in one output row and inside the map it is 8 strided shared-memory reads
// without per-element tests.
constexpr int kGGroups = 2;
constexpr int kGGroupWarps = 8;
constexpr int kGGroupThreads = kGGroupWarps * 32;
constexpr int kGThreads = 32 + kGGroups * kGGroupThreads;
constexpr int kGPatchBytes = 24 * 1024;      // per group
constexpr int kGPatchElems = kGPatchBytes / 2;

__device__ __forceinline__ void ggroup_sync(int g) {
  asm volatile("bar.sync %0, %1;" ::"r"(g + 1), "n"(kGGroupThreads) : "memory");
}

template <int DT>
__global__ void __launch_bounds__(kGThreads, 1)
dw_conv_im2col_kernel(const uint32_t* __restrict__ bitmap, const void* __restrict__ values,
                      const uint32_t* __restrict__ offsets,
                      const __grid_constant__ CUtensorMap grad_map, float* __restrict__ partial,
                      uint32_t* __restrict__ status, TcParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int b_bytes = p.tile_n * 128;
  const int stage_bytes = kTileM * 128 + b_bytes;
  unsigned char* patch_base = smem + p.stages * stage_bytes;
  __shared__ __align__(8) unsigned long long bars[2 * kMaxStages + 1];
  __shared__ RowInfo rows[kTileM];
  __shared__ int2 chunk_yx[kGGroups][8];      // output (y, x) of the first position of each chunk
  __shared__ uint32_t tmem_slot;
  __shared__ volatile uint32_t fail;

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const uint32_t lane = lane_id();
  const int m_tile = blockIdx.x, n_tile = blockIdx.y, split = blockIdx.z;
  const int nn0 = m_tile * kTileM;
  const int o0 = n_tile * p.tile_n;
  const int kt_begin = split * p.ktiles_per_split;
  const int kt_end = min(kt_begin + p.ktiles_per_split, p.total_ktiles);
  const int n_kt = kt_end - kt_begin;

  const uint32_t full_bar = smem_u32(bars);
  const uint32_t empty_bar = smem_u32(bars + kMaxStages);
  const uint32_t acc_bar = smem_u32(bars + 2 * kMaxStages);
  if (tid == 0) {
    tma_prefetch_desc(&grad_map);
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(full_bar + 8 * s, kGGroupWarps + 1);   // the group's warps + the thread that starts the TMA
      mbar_init(empty_bar + 8 * s, 1);
    }
    mbar_init(acc_bar, 1);
    fail = 0;
    fence_barrier_init();
  }
  for (int i = tid; i < kTileM; i += kGThreads) {
    const int nn = nn0 + i;
    RowInfo ri;
    if (nn < p.n_gemm) {
      const int c = nn / p.RS;
      const int rs = nn - c * p.RS;
      ri.c = static_cast<short>(c);
      ri.r = static_cast<signed char>(rs / p.KW);
      ri.s = static_cast<signed char>(rs - (rs / p.KW) * p.KW);
    } else {
      ri.c = -1; ri.r = 0; ri.s = 0;
    }
    rows[i] = ri;
  }
  if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;

  if (warp == 0) {
    // ================= MMA issuer =================
    if (lane == 0) {
      const uint32_t idesc = make_idesc(kTileM, p.tile_n);
      const uint32_t smem0 = smem_u32(smem);
      const uint64_t a_base = make_desc(smem0);
      const uint64_t b_base = make_desc(smem0 + kTileM * 128);
      const uint64_t stage_inc = static_cast<uint64_t>(stage_bytes >> 4);
      uint64_t da = a_base, db = b_base;
      uint32_t parity = 0, accum = 0;
      int s = 0;
      bool ok = true;
      for (int it = 0; it < n_kt; ++it) {
        ok = mbar_wait_suspend(full_bar + 8 * s, parity);
        if (!ok) break;
        tc_fence_after();
        umma_ktile<1, 2>(tmem_base, p.tile_n, da, db, 0, idesc, accum);
        umma_commit(empty_bar + 8 * s);
        accum = 1;
        if (++s == p.stages) { s = 0; parity ^= 1; da = a_base; db = b_base; }
        else { da += stage_inc; db += stage_inc; }
      }
      if (!ok) { fail = 1; atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT)); }
      umma_commit(acc_bar);
    }
    __syncwarp();
  } else {
    // ================= producers =================
    const int g = (warp - 1) / kGGroupWarps;
    const int gtid = tid - 32 - g * kGGroupThreads;
    unsigned short* patch = reinterpret_cast<unsigned short*>(patch_base + g * kGPatchBytes);
    const int first_c = rows[0].c;       // M tiles never start past the end
    int last_c = first_c;
    for (int i = kTileM - 1; i >= 0; --i) {
      if (rows[i].c >= 0) { last_c = rows[i].c; break; }
    }
    int s = g % p.stages;
    uint32_t round = g / p.stages;
    for (int it = g; it < n_kt; it += kGGroups) {
      if (round > 0 && gtid == 0 && !mbar_wait_suspend(empty_bar + 8 * s, (round - 1) & 1)) {
        fail = 1;
        atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
      }
      const int kt = kt_begin + it;
      const int img = kt / p.tiles_per_img;
      const int p0 = (kt - img * p.tiles_per_img) * kTileK;
      if (gtid < 8) {                    // where each 8-position chunk of the tile starts
        const int pp = p0 + 8 * gtid;
        const int y = pp / p.OW;
        chunk_yx[g][gtid] = make_int2(y, pp - y * p.OW);
      }
      ggroup_sync(g);                    // after it, every thread of the group reads the same `fail`
      if (fail) break;
      unsigned char* a_tile = smem + s * stage_bytes;
      if (gtid == 0) {
        mbar_arrive_expect_tx(full_bar + 8 * s, static_cast<uint32_t>(b_bytes));
        tma_load_3d(smem_u32(a_tile) + kTileM * 128, &grad_map, p0, o0, img, full_bar + 8 * s);
      }
      const int k_valid = min(kTileK, p.P - p0);
      const int y_first = p0 / p.OW;
      const int y_last = (p0 + k_valid - 1) / p.OW;
      int iy_lo = y_first * p.stride - p.pad;
      int iy_hi = y_last * p.stride + p.KH - 1 - p.pad;
      if (iy_lo < 0) iy_lo = 0;
      if (iy_hi > p.H - 1) iy_hi = p.H - 1;
      const int range_len = (iy_hi - iy_lo + 1) * p.W;
      const int runs = (range_len + 31) >> 5;
      for (int cg = first_c; cg <= last_c; cg += p.group_ch) {
        const int cg_end = min(cg + p.group_ch, last_c + 1);
        const int n_tasks = (cg_end - cg) * runs;       // one task = 32 consecutive elements
        for (int t = gtid; t < n_tasks; t += kGGroupThreads) {
          const int ci = t / runs, run = t - ci * runs;
          const long long start =
              ((static_cast<long long>(img) * p.C + cg + ci) * p.H + iy_lo) * p.W + 32 * run;
          decompress_run<DT>(bitmap, values, offsets, p.n_words, start,
                             min(32, range_len - 32 * run), patch + ci * p.ch_pitch + 32 * run);
        }
        ggroup_sync(g);
        int row_lo = cg * p.RS - nn0;
        int row_hi = cg_end * p.RS - nn0;
        if (row_lo < 0) row_lo = 0;
        if (row_hi > kTileM || cg_end > last_c) row_hi = kTileM;   // last group also zeroes pad rows
        const int tasks = (row_hi - row_lo) * 8;
        for (int t = gtid; t < tasks; t += kGGroupThreads) {
          const int row = row_lo + (t >> 3), chunk = t & 7;
          const RowInfo ri = rows[row];
          uint32_t h[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) h[e] = 0;
          const int pp0 = p0 + chunk * 8;
          if (ri.c >= 0 && pp0 < p.P) {
            const unsigned short* src = patch + (ri.c - cg) * p.ch_pitch;
            const int2 yx = chunk_yx[g][chunk];
            const int iy = yx.x * p.stride + ri.r - p.pad;
            const int ix0 = yx.y * p.stride + ri.s - p.pad;
            if (yx.y + 7 < p.OW && pp0 + 7 < p.P) {
              // the 8 positions lie in one output row
              if (iy >= iy_lo && iy <= iy_hi) {
                const unsigned short* rowp = src + (iy - iy_lo) * p.W;
                if (ix0 >= 0 && ix0 + 7 * p.stride < p.W) {
#pragma unroll
                  for (int e = 0; e < 8; ++e) h[e] = rowp[ix0 + e * p.stride];
                } else {
#pragma unroll
                  for (int e = 0; e < 8; ++e) {
                    const int ix = ix0 + e * p.stride;
                    if (ix >= 0 && ix < p.W) h[e] = rowp[ix];
                  }
                }
              }
            } else {
              int pp = pp0, y = yx.x, x = yx.y;
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const int iy2 = y * p.stride + ri.r - p.pad;
                const int ix = x * p.stride + ri.s - p.pad;
                if (pp < p.P && iy2 >= iy_lo && iy2 <= iy_hi && ix >= 0 && ix < p.W)
                  h[e] = src[(iy2 - iy_lo) * p.W + ix];
                ++pp; ++x;
                if (x == p.OW) { x = 0; ++y; }
              }
            }
          }
          uint4 out;
          out.x = h[0] | (h[1] << 16); out.y = h[2] | (h[3] << 16);
          out.z = h[4] | (h[5] << 16); out.w = h[6] | (h[7] << 16);
          *reinterpret_cast<uint4*>(a_tile + tile_off(row, chunk)) = out;
        }
        ggroup_sync(g);   // the patch is overwritten by the next channel group / tile
      }
      fence_proxy_async();   // generic-proxy writes -> visible to the tensor core's reads
      __syncwarp();
      if (lane == 0) mbar_arrive(full_bar + 8 * s);
      s += kGGroups;
      while (s >= p.stages) { s -= p.stages; ++round; }
    }
  }

  // ================= epilogue: TMEM -> scratch partial tile =================
  if (warp >= 1) {
    const bool done = mbar_wait(acc_bar, 0, 64);
    tc_fence_after();
    if (done && !fail) {
      const int lane_grp = warp & 3;              // TMEM lanes this warp may read
      const int row = lane_grp * 32 + static_cast<int>(lane);
      const int nn = nn0 + row;
      float* out = partial + static_cast<long long>(split) * p.O * p.n_gemm;
      for (int col = 16 * ((warp - 1) >> 2); col < p.tile_n; col += 16 * (kGGroups * kGGroupWarps / 4)) {
        uint32_t r[16];
        tmem_ld16(tmem_base + (static_cast<uint32_t>(lane_grp * 32) << 16) + col, r);
        if (nn < p.n_gemm) {
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const int o = o0 + col + e;
            if (o < p.O && SURGEON_IN_BOUNDS(static_cast<long long>(split) * p.O * p.n_gemm +
                                                 static_cast<long long>(o) * p.n_gemm + nn,
                                             static_cast<long long>(p.splits) * p.O * p.n_gemm, status))
              out[static_cast<long long>(o) * p.n_gemm + nn] = __uint_as_float(r[e]);
          }
        }
      }
    } else if (!done && lane == 0) {
      atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, p.tmem_cols);
}

// Sums the split partials in order and writes (or adds to) dw; copies the device status into
// the activation's header when a wait timed out.
__global__ void __launch_bounds__(256)
reduce_splits_kernel(const float* __restrict__ partial, long long mn, int splits,
                     float* __restrict__ dw, int accumulate, const uint32_t* __restrict__ status,
                     surgeon_header* __restrict__ hdr) {
  pdl_wait();                            // the partial tiles are complete
  const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i == 0 && *status != 0 && hdr) atomicMax(&hdr->status, *status);
  if (i >= mn) return;
  float s = partial[i];
  for (int z = 1; z < splits; ++z) s += partial[z * mn + i];
  dw[i] = accumulate ? dw[i] + s : s;
}

// Four elements per thread (mn a multiple of 4, 16-byte aligned pointers).
__global__ void __launch_bounds__(256)
reduce_splits4_kernel(const float* __restrict__ partial, long long mn, int splits,
                      float* __restrict__ dw, int accumulate, const uint32_t* __restrict__ status,
                      surgeon_header* __restrict__ hdr) {
  pdl_wait();                            // the partial tiles are complete
  const long long i = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) * 4;
  if (i == 0 && *status != 0 && hdr) atomicMax(&hdr->status, *status);
  if (i >= mn) return;
  float4 s = *reinterpret_cast<const float4*>(partial + i);
#pragma unroll 4
  for (int z = 1; z < splits; ++z) {
    const float4 v = *reinterpret_cast<const float4*>(partial + z * mn + i);
    s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
  }
  if (accumulate) {
    const float4 d = *reinterpret_cast<const float4*>(dw + i);
    s.x += d.x; s.y += d.y; s.z += d.z; s.w += d.w;
  }
  *reinterpret_cast<float4*>(dw + i) = s;
}

static void launch_reduce_splits(const float* partial, long long mn, int splits, float* dw,
                                 int accumulate, const uint32_t* status, surgeon_header* hdr,
                                 cudaStream_t stream) {
  const bool vec = (mn & 3) == 0 && ((reinterpret_cast<uintptr_t>(partial) | reinterpret_cast<uintptr_t>(dw)) & 15) == 0;
  // launched as a programmatic dependent of the kernel that writes the partial tiles: it is
  // resident (or queued) when that kernel ends and starts at once
  if (vec)
    launch_kernel(reduce_splits4_kernel, dim3(static_cast<unsigned>((mn / 4 + 255) / 256)), dim3(256), 0, stream,
                  true, partial, mn, splits, dw, accumulate, status, hdr);
  else
    launch_kernel(reduce_splits_kernel, dim3(static_cast<unsigned>((mn + 255) / 256)), dim3(256), 0, stream,
                  true, partial, mn, splits, dw, accumulate, status, hdr);
}

// The same for a tap-stacked partial [splits][taps * O][C]: dw[o][c][tap] gets row tap * O + o.
// One block sums `chunk` input channels of one output channel for all taps: the reads
// run along c (contiguous in the partial, a kilobyte per warp), the writes along (c, tap)
// (contiguous in dw), transposed through shared memory.  taps <= 49.
__global__ void __launch_bounds__(256)
reduce_splits_taps_kernel(const float* __restrict__ partial, int o_real, int c_in, int taps,
                          int chunk, int splits, float* __restrict__ dw, int accumulate,
                          const uint32_t* __restrict__ status, surgeon_header* __restrict__ hdr) {
  extern __shared__ __align__(16) float tile[];    // [n_c][taps]
  pdl_wait();                                      // the partial tiles are complete
  const int c0 = blockIdx.x * chunk;
  const int o = blockIdx.y;
  if (blockIdx.x == 0 && o == 0 && threadIdx.x == 0 && *status != 0 && hdr)
    atomicMax(&hdr->status, *status);
  const long long mn = static_cast<long long>(o_real) * c_in * taps;
  const int n_c = min(chunk, c_in - c0);
  float* out = dw + (static_cast<long long>(o) * c_in + c0) * taps;
  if ((c_in & 3) == 0) {
    // four channels per thread: 16-byte reads of the partials, 16-byte writes of dw (c0 is a
    // multiple of 32 and n_c of 4, so both stay aligned); the split sums keep their order
    const int n_c4 = n_c >> 2;
    for (int idx = threadIdx.x; idx < n_c4 * taps; idx += 256) {
      const int tap = idx / n_c4, cl = (idx - tap * n_c4) * 4;
      const float* src = partial + (static_cast<long long>(tap) * o_real + o) * c_in + c0 + cl;
      float4 s = *reinterpret_cast<const float4*>(src);
#pragma unroll 4
      for (int z = 1; z < splits; ++z) {
        const float4 v = *reinterpret_cast<const float4*>(src + z * mn);
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
      }
      tile[cl * taps + tap] = s.x;
      tile[(cl + 1) * taps + tap] = s.y;
      tile[(cl + 2) * taps + tap] = s.z;
      tile[(cl + 3) * taps + tap] = s.w;
    }
    __syncthreads();
    const int n4 = (n_c * taps) >> 2;                  // n_c is a multiple of 4
    for (int idx = threadIdx.x; idx < n4; idx += 256) {
      float4 v = *reinterpret_cast<const float4*>(tile + 4 * idx);
      if (accumulate) {
        const float4 d = *reinterpret_cast<const float4*>(out + 4 * idx);
        v.x += d.x; v.y += d.y; v.z += d.z; v.w += d.w;
      }
      *reinterpret_cast<float4*>(out + 4 * idx) = v;
    }
    return;
  }
  for (int idx = threadIdx.x; idx < n_c * taps; idx += 256) {
    const int tap = idx / n_c, cl = idx - tap * n_c;     // consecutive threads, consecutive channels
    const float* src = partial + (static_cast<long long>(tap) * o_real + o) * c_in + c0 + cl;
    float s = src[0];
    for (int z = 1; z < splits; ++z) s += src[z * mn];
    tile[cl * taps + tap] = s;
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < n_c * taps; idx += 256)
    out[idx] = accumulate ? out[idx] + tile[idx] : tile[idx];
}

bool plan(const surgeon_layer_desc& d, int dt, TcParams* out) {
  TcParams p{};
  p.kind = d.kind; p.B = d.batch; p.C = d.c_in; p.H = d.h; p.W = d.w; p.O = d.c_out;
  p.KH = d.kh; p.KW = d.kw; p.stride = d.stride; p.pad = d.pad;
  p.OH = (d.h + 2 * d.pad - d.kh) / d.stride + 1;
  p.OW = (d.w + 2 * d.pad - d.kw) / d.stride + 1;
  p.RS = d.kh * d.kw;
  p.n_gemm = d.c_in * p.RS;
  p.dt = dt;
  int imgs;
  if (d.kind == 1) { p.P = p.OH * p.OW; imgs = d.batch; }
  else { p.P = d.batch; imgs = 1; }
  if (d.kh > 127 || d.kw > 127 || d.c_in > 32767) return false;
  const int nt = (p.O + 255) / 256;
  p.n_tiles = nt;
  p.tile_n = ((p.O + nt - 1) / nt + 15) / 16 * 16;
  p.m_tiles = (p.n_gemm + kTileM - 1) / kTileM;
  p.tiles_per_img = (p.P + kTileK - 1) / kTileK;
  const long long total = static_cast<long long>(imgs) * p.tiles_per_img;
  if (total > 2147483647LL) return false;
  p.total_ktiles = static_cast<int>(total);
  const int sms = sm_count();
  const long long tiles_mn = static_cast<long long>(p.m_tiles) * p.n_tiles;
  int splits = static_cast<int>(tiles_mn >= sms ? 1 : sms / tiles_mn);
  const int max_by_work = (p.total_ktiles + 3) / 4;   // at least 4 K-tiles per split
  if (splits > max_by_work) splits = max_by_work;
  if (splits < 1) splits = 1;
  if (splits > 65535) splits = 65535;
  p.ktiles_per_split = (p.total_ktiles + splits - 1) / splits;
  p.splits = (p.total_ktiles + p.ktiles_per_split - 1) / p.ktiles_per_split;
  // patch: rows one K-tile can touch
  if (d.kind == 1) {
    const int out_rows = (kTileK + p.OW - 2) / p.OW + 1;           // rows spanned by 64 positions
    int in_rows = (out_rows - 1) * p.stride + p.KH;
    if (in_rows > p.H) in_rows = p.H;
    p.max_rows = in_rows;
    const long long per_ch = (static_cast<long long>(in_rows) * p.W + 31) / 32 * 32;
    if (per_ch > kPatchElems) return false;
    p.ch_pitch = static_cast<int>(per_ch);
    p.group_ch = static_cast<int>(kPatchElems / per_ch);
  } else {
    p.max_rows = 1;
    p.group_ch = 1;
  }
  p.g_vec_ok = (d.kind == 1 && (p.P % 4) == 0) ? 1 : 0;
  p.tmem_cols = 32;
  while (p.tmem_cols < p.tile_n) p.tmem_cols *= 2;
  const int stage_bytes = kTileM * 128 + p.tile_n * 128;
  const int fixed = kPatchBytes + 1024 /*align*/ + 1024 /*barriers, row table*/;
  int stages = (227 * 1024 - fixed) / stage_bytes;
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < 2) return false;
  p.stages = stages;
  *out = p;
  return true;
}

size_t smem_bytes(const TcParams& p) {
  return static_cast<size_t>(p.stages) * (kTileM * 128 + p.tile_n * 128) + kPatchBytes + 2048;
}

// Plan of dw_conv_im2col_kernel: the tiling of `plan`, two patches of kGPatchBytes, and the
// bf16 gradient copy (rows padded to a multiple of 8 elements for the tensor map).
bool plan_im2col(const surgeon_layer_desc& d, int dt, TcParams* out, int* pitch) {
  if (d.kind != 1) return false;
  TcParams p;
  if (!plan(d, dt, &p)) return false;
  const long long per_ch = (static_cast<long long>(p.max_rows) * p.W + 31) / 32 * 32;
  if (per_ch > kGPatchElems) return false;
  p.ch_pitch = static_cast<int>(per_ch);
  p.group_ch = static_cast<int>(kGPatchElems / per_ch);
  const int stage_bytes = kTileM * 128 + p.tile_n * 128;
  int stages = (224 * 1024 - kGGroups * kGPatchBytes - 1024) / stage_bytes;
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < 2) return false;
  p.stages = stages;
  *pitch = (p.P + 7) / 8 * 8;
  *out = p;
  return true;
}

size_t im2col_smem_bytes(const TcParams& p) {
  return static_cast<size_t>(p.stages) * (kTileM * 128 + p.tile_n * 128) + kGGroups * kGPatchBytes + 1024;
}

size_t im2col_grad_bytes(const TcParams& p, int pitch) {
  const size_t b = static_cast<size_t>(p.B) * p.O * pitch * 2;
  return (b + 255) & ~static_cast<size_t>(255);
}

}  // namespace

static size_t fast_partial_bytes(const FastParams& f) {
  const size_t b = static_cast<size_t>(f.splits) * f.O * f.n_gemm * sizeof(float);
  return (b + 255) & ~static_cast<size_t>(255);
}

static size_t direct_partial_bytes(const DirectParams& p) {
  const size_t b = static_cast<size_t>(p.splits) * p.O * p.C * sizeof(float);
  return (b + 255) & ~static_cast<size_t>(255);
}

size_t weight_grad_tc_workspace(const surgeon_layer_desc& d) {
  SwapParams sp;
  if (plan_swap(d, &sp)) return kStatusBytes + swap_partial_bytes(sp) + direct_grad_bf16_bytes(sp.d);
  DirectParams dp;
  if (plan_direct(d, &dp)) return kStatusBytes + direct_partial_bytes(dp) + direct_grad_bf16_bytes(dp);
  FastParams f;
  if (plan_conv_fast(d, &f))
    return kStatusBytes + fast_partial_bytes(f) + conv_fast_grad_bf16_bytes(f);
  TcParams p;
  int pitch = 0;
  if (plan_im2col(d, 0, &p, &pitch))
    return kStatusBytes + ((static_cast<size_t>(p.splits) * p.O * p.n_gemm * sizeof(float) + 255) & ~size_t(255)) +
           im2col_grad_bytes(p, pitch);
  if (!plan(d, 0, &p)) return 0;
  return kStatusBytes + static_cast<size_t>(p.splits) * p.O * p.n_gemm * sizeof(float);
}

cudaError_t launch_weight_grad_tc(const surgeon_compressed& act, const surgeon_layer_desc& d,
                                  const float* grad_out, float* dw, int accumulate,
                                  void* workspace, cudaStream_t stream) {
  // No geometry plan fits: say so before anything touches the workspace (its size query gave 0).
  if (weight_grad_tc_workspace(d) == 0 || workspace == nullptr) return cudaErrorNotSupported;
  uint32_t* status = static_cast<uint32_t*>(workspace);
  float* partial = reinterpret_cast<float*>(static_cast<char*>(workspace) + kStatusBytes);
  cudaError_t e = cudaMemsetAsync(status, 0, kStatusBytes, stream);
  if (e != cudaSuccess) return e;
#ifdef SURGEON_DW_STATS
  cudaMemsetAsync(reinterpret_cast<char*>(status) + 14 * 8, 0xFF, 8, stream);
#endif
  DirectParams dp;
  SwapParams sp;
  const bool swapped = plan_swap(d, &sp);
  if (swapped || plan_direct(d, &dp)) {
    if (swapped) {
      dp = sp.d;
      dp.splits = sp.splits;
      void* grad_bf16 = reinterpret_cast<char*>(partial) + swap_partial_bytes(sp);
      e = launch_swap(act, sp, grad_out, grad_bf16, partial, status, stream);
    } else {
      void* grad_bf16 = reinterpret_cast<char*>(partial) + direct_partial_bytes(dp);
      e = launch_direct(act, dp, grad_out, grad_bf16, partial, status, stream);
    }
    if (e != cudaSuccess) return e;
    const long long mn = static_cast<long long>(dp.O) * dp.C;
    if (dp.taps > 1)
    {
      // the widest chunk of channels (coalescing) that still gives four blocks per SM
      int chunk = 256;
      while (chunk > 32 && (static_cast<long long>(dp.o_real) * ((dp.C + chunk - 1) / chunk) < 4LL * sm_count() ||
                            chunk * dp.taps * 4 > 48 * 1024))
        chunk >>= 1;
      launch_kernel(reduce_splits_taps_kernel, dim3((dp.C + chunk - 1) / chunk, dp.o_real), dim3(256),
                    static_cast<size_t>(chunk) * dp.taps * sizeof(float), stream, true,
                    static_cast<const float*>(partial), dp.o_real, dp.C, dp.taps, chunk, dp.splits, dw, accumulate,
                    static_cast<const uint32_t*>(status), act.header);
    }

    else
      launch_reduce_splits(partial, mn, dp.splits, dw, accumulate, status, act.header, stream);
    note_launches(1);
    return cudaGetLastError();
  }
  FastParams f;
  if (plan_conv_fast(d, &f)) {
    void* grad_bf16 = reinterpret_cast<char*>(partial) + fast_partial_bytes(f);
    e = launch_conv_fast(act, f, grad_out, grad_bf16, partial, status, stream);
    if (e != cudaSuccess) return e;
    const long long fmn = static_cast<long long>(f.O) * f.n_gemm;
    launch_reduce_splits(partial, fmn, f.splits, dw, accumulate, status, act.header, stream);
    note_launches(1);
    return cudaGetLastError();
  }
  TcParams p;
  int pitch = 0;
  if (plan_im2col(d, act.dt, &p, &pitch)) {
    p.n_words = (act.n + 31) / 32;
    const size_t pbytes = (static_cast<size_t>(p.splits) * p.O * p.n_gemm * sizeof(float) + 255) & ~size_t(255);
    void* grad_bf16 = reinterpret_cast<char*>(partial) + pbytes;
    if (pitch != p.P)
      e = launch_grad_to_bf16_rows(grad_out, static_cast<long long>(p.B) * p.O, p.P, pitch, grad_bf16, stream);
    else
      e = launch_grad_to_bf16(grad_out, static_cast<long long>(p.B) * p.O * p.P, grad_bf16, stream);
    if (e != cudaSuccess) return e;
    using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);
    const EncodeFn encode = reinterpret_cast<EncodeFn>(tensor_map_encode_fn());
    if (!encode) return cudaErrorNotSupported;
    CUtensorMap map;
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(p.P), static_cast<cuuint64_t>(p.O),
                                static_cast<cuuint64_t>(p.B)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(pitch) * 2,
                                   static_cast<cuuint64_t>(pitch) * p.O * 2};
    const cuuint32_t box[3] = {static_cast<cuuint32_t>(kTileK), static_cast<cuuint32_t>(p.tile_n), 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    if (encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, grad_bf16, dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
    const size_t smem = im2col_smem_bytes(p);
    dim3 grid(p.m_tiles, p.n_tiles, p.splits);
    if (act.dt == 0) {
      e = allow_dynamic_smem(reinterpret_cast<const void*>(dw_conv_im2col_kernel<0>), static_cast<int>(smem));
      if (e != cudaSuccess) return e;
      dw_conv_im2col_kernel<0><<<grid, kGThreads, smem, stream>>>(act.bitmap, act.values, act.block_offsets,
                                                                 map, partial, status, p);
    } else {
      e = allow_dynamic_smem(reinterpret_cast<const void*>(dw_conv_im2col_kernel<1>), static_cast<int>(smem));
      if (e != cudaSuccess) return e;
      dw_conv_im2col_kernel<1><<<grid, kGThreads, smem, stream>>>(act.bitmap, act.values, act.block_offsets,
                                                                 map, partial, status, p);
    }
    const long long mn = static_cast<long long>(p.O) * p.n_gemm;
    launch_reduce_splits(partial, mn, p.splits, dw, accumulate, status, act.header, stream);
    note_launches(2);
    return cudaGetLastError();
  }
  if (!plan(d, act.dt, &p)) return cudaErrorNotSupported;
  p.n_words = (act.n + 31) / 32;
  const size_t smem = smem_bytes(p);
  const uint32_t* offs = act.block_offsets;
  dim3 grid(p.m_tiles, p.n_tiles, p.splits);
  if (act.dt == 0) {
    e = allow_dynamic_smem(reinterpret_cast<const void*>(dw_tc_kernel<0>), static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    dw_tc_kernel<0><<<grid, kThreads, smem, stream>>>(act.bitmap, act.values, offs, grad_out,
                                                      partial, status, p);
  } else {
    e = allow_dynamic_smem(reinterpret_cast<const void*>(dw_tc_kernel<1>), static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    dw_tc_kernel<1><<<grid, kThreads, smem, stream>>>(act.bitmap, act.values, offs, grad_out,
                                                      partial, status, p);
  }
  const long long mn = static_cast<long long>(p.O) * p.n_gemm;
  launch_reduce_splits(partial, mn, p.splits, dw, accumulate, status, act.header, stream);
  note_launches(2);
  return cudaGetLastError();
}

}  // namespace surgeon

// Fast tensor-core weight-gradient kernel for 3x3 / pad 1 ("patch" mode) and 1x1 / pad 0
// ("direct" mode) convolutions of stride 1 or 2 whose rows are a multiple of 8 (stride 1) or
// 16 (stride 2) elements wide.  Algorithm 1: Reshape and gradient steps with Eq. 2; same GEMM view as
// weight_grad_tc.cu:  D[nn, o] = sum_k Acol[nn, k] * G[o, k],  nn = (c, r, s),  k = (b, y, x).
//
// What differs from the general kernel:
//   * the output gradient is converted to bf16 once by a streaming pre-pass into scratch and
//     then arrives in the swizzled operand tile by TMA, several stages ahead of the MMAs;
//   * two producer groups of 8 warps rebuild activation tiles for alternate pipeline stages,
//     so the load latency of one group hides behind the other group's arithmetic;
//   * per K-tile, the bitmap bits a group needs and the rank of their first kept element are
//     staged in shared memory one tile ahead; decompression then works on units of 8 output
//     elements with eight independent loads of packed values per thread;
//   * patch mode copies the im2col view with 16-byte loads and funnel shifts for the s = 0 / 2
//     columns (stride 2 keeps even and odd input columns in separate planes of the patch);
//     direct mode decompresses straight into the swizzled operand tile;
//   * one or two accumulators (<= 512 TMEM columns) share each activation tile.
#include <cuda.h>

#include "surgeon_internal.cuh"
#include "tc_common.cuh"
#include "weight_grad_tc_conv.cuh"

namespace surgeon {

namespace {

using namespace tc;

constexpr int kTileM = 128;
constexpr int kTileK = 64;
constexpr int kGroups = 2;
constexpr int kGroupWarps = 8;
constexpr int kGroupThreads = kGroupWarps * 32;
constexpr int kThreads = 32 + kGroups * kGroupThreads;
constexpr int kPatchBytes = 16 * 1024;       // per group
constexpr int kMetaWords = 1024;             // staged bitmap words / chunk bits per group
constexpr int kMaxStages = 4;

__device__ __forceinline__ void group_sync(int g) {
  asm volatile("bar.sync %0, %1;" ::"r"(g + 1), "n"(kGroupThreads) : "memory");
}

// Eight elements selected by `bits` (bit e*step set = element e kept); the packed vector holds
// the kept elements of these bit positions consecutively from index r0.  Returns 8 packed bf16.
template <int DT>
__device__ __forceinline__ uint4 gather8(uint32_t bits, uint32_t r0, int step,
                                         const void* __restrict__ values) {
  uint4 out = make_uint4(0, 0, 0, 0);
  if (bits == 0) return out;
  if (DT == 0) {
    const float* v = reinterpret_cast<const float*>(values);
    float f[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int b = e * step;
      const bool on = (bits >> b) & 1u;
      f[e] = on ? __ldg(v + r0 + __popc(bits & ((1u << b) - 1u))) : 0.0f;
    }
    out.x = pack_bf16x2(f[0], f[1]); out.y = pack_bf16x2(f[2], f[3]);
    out.z = pack_bf16x2(f[4], f[5]); out.w = pack_bf16x2(f[6], f[7]);
  } else {
    const unsigned short* v = reinterpret_cast<const unsigned short*>(values);
    uint32_t h[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int b = e * step;
      const bool on = (bits >> b) & 1u;
      h[e] = on ? static_cast<uint32_t>(__ldg(v + r0 + __popc(bits & ((1u << b) - 1u)))) : 0u;
    }
    out.x = h[0] | (h[1] << 16); out.y = h[2] | (h[3] << 16);
    out.z = h[4] | (h[5] << 16); out.w = h[6] | (h[7] << 16);
  }
  return out;
}

template <int DT>
__global__ void __launch_bounds__(kThreads, 1)
dw_conv_fast_kernel(const uint32_t* __restrict__ bitmap, const void* __restrict__ values,
                    const uint32_t* __restrict__ offsets,
                    const __grid_constant__ CUtensorMap grad_map, float* __restrict__ partial,
                    uint32_t* __restrict__ status, FastParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int n_cols = p.n_acc * p.acc_n;               // gradient rows (output channels) per CTA
  const int stage_bytes = kTileM * 128 + n_cols * 128;
  unsigned char* patch_base = smem + p.stages * stage_bytes;
  uint32_t* meta_base = reinterpret_cast<uint32_t*>(patch_base + kGroups * kPatchBytes);
  unsigned long long* bars =
      reinterpret_cast<unsigned long long*>(meta_base + kGroups * 2 * kMetaWords);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kMaxStages + 2);
  volatile uint32_t* fail = tmem_slot + 1;

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const uint32_t lane = lane_id();
  const int m_tile = blockIdx.x, n_tile = blockIdx.y, split = blockIdx.z;
  const int nn0 = m_tile * kTileM;
  const int o0 = n_tile * n_cols;
  const int kt_begin = split * p.ktiles_per_split;
  const int kt_end = min(kt_begin + p.ktiles_per_split, p.total_ktiles);
  const int n_kt = kt_end - kt_begin;
  const int rows_valid = min(kTileM, p.n_gemm - nn0);

  const uint32_t full_bar = smem_u32(bars);
  const uint32_t empty_bar = smem_u32(bars + kMaxStages);
  const uint32_t acc_bar = smem_u32(bars + 2 * kMaxStages);

  if (tid == 0) {
    tma_prefetch_desc(&grad_map);
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(full_bar + 8 * s, kGroupWarps + 1);   // 8 warps + the thread that starts the TMA
      mbar_init(empty_bar + 8 * s, 1);
    }
    mbar_init(acc_bar, 1);
    *fail = 0;
    fence_barrier_init();
  }
  // rows of the activation tile past the end of the im2col matrix stay zero for the whole kernel
  if (rows_valid < kTileM) {
    const int pad_chunks = (kTileM - rows_valid) * 8;
    for (int s = 0; s < p.stages; ++s)
      for (int t = tid; t < pad_chunks; t += kThreads) {
        const int row = rows_valid + (t >> 3);
        *reinterpret_cast<uint4*>(smem + s * stage_bytes + tile_off(row, t & 7)) =
            make_uint4(0, 0, 0, 0);
      }
    fence_proxy_async();
  }
  if (warp == 0) tmem_alloc(smem_u32(tmem_slot), p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ================= MMA issuer =================
    if (lane == 0) {
      const uint32_t idesc = make_idesc(kTileM, p.acc_n);
      const uint32_t smem0 = smem_u32(smem);
      const uint64_t a_base = make_desc(smem0);
      const uint64_t b_base = make_desc(smem0 + kTileM * 128);
      const uint64_t stage_inc = static_cast<uint64_t>(stage_bytes >> 4);
      const uint64_t acc_inc = static_cast<uint64_t>((p.acc_n * 128) >> 4);
      uint64_t da = a_base, db = b_base;
      uint32_t parity = 0, accum = 0;
      int s = 0;
      bool ok = true;
      for (int it = 0; it < n_kt; ++it) {
        ok = mbar_wait(full_bar + 8 * s, parity);
        if (!ok) break;
        tc_fence_after();
        if (p.n_acc == 1) umma_ktile<1, 2>(tmem_base, p.acc_n, da, db, acc_inc, idesc, accum);
        else umma_ktile<2, 2>(tmem_base, p.acc_n, da, db, acc_inc, idesc, accum);
        umma_commit(empty_bar + 8 * s);
        accum = 1;
        if (++s == p.stages) { s = 0; parity ^= 1; da = a_base; db = b_base; }
        else { da += stage_inc; db += stage_inc; }
      }
      if (!ok) { *fail = 1; atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT)); }
      umma_commit(acc_bar);
    }
    __syncwarp();
  } else {
    // ================= producers: group g fills K-tiles it = g, g + 2, ... =================
    const int g = (warp - 1) / kGroupWarps;
    const int gtid = tid - 32 - g * kGroupThreads;
    const int gwarp = gtid >> 5;
    unsigned short* patch = reinterpret_cast<unsigned short*>(patch_base + g * kPatchBytes);
    uint32_t* m_words = meta_base + g * 2 * kMetaWords;
    uint32_t* m_rank = m_words + kMetaWords;
    const int first_c = (p.mode == 0) ? nn0 / 9 : nn0;
    const int last_c = (p.mode == 0) ? (nn0 + rows_valid - 1) / 9 : nn0 + rows_valid - 1;
    const int n_ch = last_c - first_c + 1;   // mode 0: <= 16, mode 1: <= 128
    const int HW = p.H * p.W;
    const int half_w = p.W >> 1;

    struct Tile { int img, p0, k_valid, iy_lo, range_len; };
    auto tile_of = [&](int it) {
      Tile t;
      const int kt = kt_begin + it;
      t.img = kt / p.tiles_per_img;
      t.p0 = (kt - t.img * p.tiles_per_img) * kTileK;
      t.k_valid = min(kTileK, p.P - t.p0);
      t.iy_lo = 0;
      t.range_len = 0;
      if (p.mode == 0) {
        const int y_first = t.p0 / p.OW;
        const int y_last = (t.p0 + t.k_valid - 1) / p.OW;
        t.iy_lo = max(y_first * p.stride - 1, 0);
        const int iy_hi = min(y_last * p.stride + 1, p.H - 1);
        t.range_len = (iy_hi - t.iy_lo + 1) * p.W;
      }
      return t;
    };
    auto plane_of = [&](const Tile& t, int ri) -> long long {
      return (static_cast<long long>(t.img) * p.C + first_c + ri) * HW;
    };
    // Stage what the decompression of a tile needs.
    //  patch mode : per channel range, its bitmap words and the rank of each word's first bit;
    //  direct mode: per (channel, chunk of 8 outputs), the 8*stride bitmap bits and their rank.
    auto stage_meta = [&](const Tile& t) {
      if (p.mode == 0) {
        for (int ri = gwarp; ri < n_ch; ri += kGroupWarps) {
          const long long start = plane_of(t, ri) + static_cast<long long>(t.iy_lo) * p.W;
          const long long first_word = start >> 5;
          const long long blk = start >> kBlockShift;
          const long long blk_word0 = blk * kBlockWords;
          uint32_t wb = 0;
          if (blk_word0 + lane < first_word) wb = __ldg(bitmap + blk_word0 + lane);
          const int nwords = static_cast<int>(((start + t.range_len - 1) >> 5) - first_word) + 1;
          uint32_t w = 0;
          if (static_cast<int>(lane) < nwords) w = __ldg(bitmap + first_word + lane);
          const uint32_t base = static_cast<uint32_t>(__ldg(offsets + blk)) + warp_sum(__popc(wb));
          const uint32_t ex = warp_excl_scan(__popc(w));
          m_words[ri * 32 + lane] = w;
          m_rank[ri * 32 + lane] = base + ex;
        }
      } else {
        const int nbits = 8 * p.stride;
        const uint32_t bmask = (nbits == 8) ? 0xFFu : 0xFFFFu;
        for (int ri = gtid; ri < n_ch; ri += kGroupThreads) {
          const long long plane = plane_of(t, ri);
          // cursor = (flat position, kept elements before it)
          const int y0 = t.p0 / p.OW;
          const int x00 = t.p0 - y0 * p.OW;
          long long pos = plane + static_cast<long long>(y0 * p.stride) * p.W + x00 * p.stride;
          const long long blk = pos >> kBlockShift;
          uint32_t rank = static_cast<uint32_t>(__ldg(offsets + blk));
          {
            const long long blk_word0 = blk * kBlockWords;
            const int before = static_cast<int>((pos >> 5) - blk_word0);
#pragma unroll
            for (int w = 0; w < kBlockWords - 1; ++w)
              if (w < before) rank += __popc(__ldg(bitmap + blk_word0 + w));
            const uint32_t w0 = __ldg(bitmap + (pos >> 5));
            rank += __popc(w0 & ((1u << (pos & 31)) - 1u));
          }
          int y = y0, x = x00;
          for (int chunk = 0; chunk < 8; ++chunk) {
            uint32_t bits = 0;
            if (chunk * 8 < t.k_valid) {
              const long long want = plane + static_cast<long long>(y * p.stride) * p.W + x * p.stride;
              while (pos < want) {       // skipped input (odd rows of a stride-2 layer)
                const int lo = static_cast<int>(pos & 31);
                const long long left = want - pos;
                const int take = (left < 32 - lo) ? static_cast<int>(left) : 32 - lo;
                const uint32_t m = (take == 32) ? 0xFFFFFFFFu : (((1u << take) - 1u) << lo);
                rank += __popc(__ldg(bitmap + (pos >> 5)) & m);
                pos += take;
              }
              bits = (__ldg(bitmap + (pos >> 5)) >> (pos & 31)) & bmask;
            }
            m_words[ri * 8 + chunk] = bits;
            m_rank[ri * 8 + chunk] = rank;
            rank += __popc(bits);
            pos += nbits;
            x += 8;
            if (x >= p.OW) { x = 0; ++y; }
          }
        }
      }
    };

    if (g < n_kt) stage_meta(tile_of(g));
    for (int it = g; it < n_kt; it += kGroups) {
      const int s = it % p.stages;
      if (it >= p.stages && gtid == 0) {     // one thread polls; the rest wait at the barrier below
        if (!mbar_wait(empty_bar + 8 * s, ((it / p.stages) - 1) & 1, 32)) {
          *fail = 1;
          atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
        }
      }
      group_sync(g);    // staged metadata visible; every thread of the group sees the same *fail
      if (*fail) break;
      unsigned char* a_tile = smem + s * stage_bytes;
      const Tile t = tile_of(it);

      // gradient tile(s): bf16 rows [o0, o0 + n_cols) x 64 positions of image t.img, by TMA
      if (gtid == 0) {
        mbar_arrive_expect_tx(full_bar + 8 * s, static_cast<uint32_t>(n_cols) * 128u);
        const uint32_t b_addr = smem_u32(a_tile) + kTileM * 128;
        for (int a = 0; a < p.n_acc; ++a)
          tma_load_3d(b_addr + a * p.acc_n * 128, &grad_map, t.p0, o0 + a * p.acc_n, t.img,
                      full_bar + 8 * s);
      }

      if (p.mode == 0) {
        // ---- decompress the channel ranges into the patch, 8 input elements per thread ----
        const int units_per_range = t.range_len >> 3;
        const int units = n_ch * units_per_range;
        for (int u = gtid; u < units; u += kGroupThreads) {
          const int ri = u / units_per_range;
          const int uu = u - ri * units_per_range;
          const long long start = plane_of(t, ri) + static_cast<long long>(t.iy_lo) * p.W;
          const int rel = static_cast<int>(start & 31) + uu * 8;
          const uint32_t word = m_words[ri * 32 + (rel >> 5)];
          const int sh = rel & 31;
          const uint32_t r0 = m_rank[ri * 32 + (rel >> 5)] + __popc(word & ((1u << sh) - 1u));
          const uint4 v = gather8<DT>((word >> sh) & 0xFFu, r0, 1, values);
          unsigned short* dst = patch + ri * t.range_len;
          if (p.stride == 1) {
            *reinterpret_cast<uint4*>(dst + uu * 8) = v;
          } else {
            // even input columns to the first half of the row, odd ones to the second half
            const int e0 = uu * 8;
            const int row = e0 / p.W;
            const int xin = e0 - row * p.W;
            uint2 ev, od;
            ev.x = __byte_perm(v.x, v.y, 0x5410); ev.y = __byte_perm(v.z, v.w, 0x5410);
            od.x = __byte_perm(v.x, v.y, 0x7632); od.y = __byte_perm(v.z, v.w, 0x7632);
            *reinterpret_cast<uint2*>(dst + row * p.W + (xin >> 1)) = ev;
            *reinterpret_cast<uint2*>(dst + row * p.W + half_w + (xin >> 1)) = od;
          }
        }
        group_sync(g);
        // ---- im2col view: one task = (channel, filter row r, chunk) -> columns s = 0, 1, 2 ----
        const int tasks = n_ch * 24;
        for (int q = gtid; q < tasks; q += kGroupThreads) {
          const int ci = q / 24;
          const int rem = q - ci * 24;
          const int r = rem >> 3, chunk = rem & 7;
          const int pp = t.p0 + chunk * 8;
          const int y = pp / p.OW;
          const int x0 = pp - y * p.OW;
          const int iy = y * p.stride + r - 1;
          uint4 s0 = make_uint4(0, 0, 0, 0), s1 = s0, s2 = s0;
          if (pp < p.P && iy >= 0 && iy < p.H) {
            const unsigned short* rowp = patch + ci * t.range_len + (iy - t.iy_lo) * p.W;
            if (p.stride == 1) {
              const unsigned short* src = rowp + x0;
              const uint4 c4 = *reinterpret_cast<const uint4*>(src);
              const uint32_t left = (x0 > 0) ? src[-1] : 0u;
              const uint32_t right = (x0 + 8 < p.W) ? src[8] : 0u;
              s1 = c4;
              s0.x = (c4.x << 16) | left;
              s0.y = __funnelshift_l(c4.x, c4.y, 16);
              s0.z = __funnelshift_l(c4.y, c4.z, 16);
              s0.w = __funnelshift_l(c4.z, c4.w, 16);
              s2.x = __funnelshift_r(c4.x, c4.y, 16);
              s2.y = __funnelshift_r(c4.y, c4.z, 16);
              s2.z = __funnelshift_r(c4.z, c4.w, 16);
              s2.w = (c4.w >> 16) | (right << 16);
            } else {
              // input column 2x + s - 1: s = 1 -> even plane[x], s = 2 -> odd plane[x],
              // s = 0 -> odd plane[x - 1]
              s1 = *reinterpret_cast<const uint4*>(rowp + x0);
              const unsigned short* odd = rowp + half_w + x0;
              s2 = *reinterpret_cast<const uint4*>(odd);
              const uint32_t left = (x0 > 0) ? odd[-1] : 0u;
              s0.x = (s2.x << 16) | left;
              s0.y = __funnelshift_l(s2.x, s2.y, 16);
              s0.z = __funnelshift_l(s2.y, s2.z, 16);
              s0.w = __funnelshift_l(s2.z, s2.w, 16);
            }
          }
          const int row0 = (first_c + ci) * 9 + r * 3 - nn0;
          if (row0 >= 0 && row0 < rows_valid)
            *reinterpret_cast<uint4*>(a_tile + tile_off(row0, chunk)) = s0;
          if (row0 + 1 >= 0 && row0 + 1 < rows_valid)
            *reinterpret_cast<uint4*>(a_tile + tile_off(row0 + 1, chunk)) = s1;
          if (row0 + 2 >= 0 && row0 + 2 < rows_valid)
            *reinterpret_cast<uint4*>(a_tile + tile_off(row0 + 2, chunk)) = s2;
        }
      } else {
        // ---- 1x1: decompress straight into the operand tile; row = channel, chunk = 8 outputs
        const int units = rows_valid * 8;
        for (int u = gtid; u < units; u += kGroupThreads) {
          const int ri = u >> 3, chunk = u & 7;
          const uint4 v = gather8<DT>(m_words[u], m_rank[u], p.stride, values);
          *reinterpret_cast<uint4*>(a_tile + tile_off(ri, chunk)) = v;
        }
        group_sync(g);    // everyone is done with this tile's metadata
      }
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(full_bar + 8 * s);
      if (it + kGroups < n_kt) stage_meta(tile_of(it + kGroups));
    }
  }

  // ================= epilogue: TMEM -> scratch partial tile =================
  if (warp >= 1) {
    // 16 warps: a warp may read the 32 TMEM lanes of its quarter (warp % 4); the four warps of a
    // quarter take every fourth group of 16 columns
    const bool done = mbar_wait(acc_bar, 0, 64);
    tc_fence_after();
    if (done && !*fail) {
      const int lane_grp = warp & 3;
      const int row = lane_grp * 32 + static_cast<int>(lane);
      const int nn = nn0 + row;
      float* out = partial + static_cast<long long>(split) * p.O * p.n_gemm;
      for (int col = 16 * ((warp - 1) >> 2); col < n_cols; col += 64) {
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

// fp32 -> bf16 (round to nearest even), 8 elements per thread.
__global__ void __launch_bounds__(256)
grad_to_bf16_kernel(const float* __restrict__ g, long long n, unsigned short* __restrict__ out) {
  pdl_trigger();
  const long long n8 = n >> 3;
  const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < n8;
       i += stride) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(g) + 2 * i);
    const float4 b = __ldg(reinterpret_cast<const float4*>(g) + 2 * i + 1);
    uint4 o;
    o.x = pack_bf16x2(a.x, a.y); o.y = pack_bf16x2(a.z, a.w);
    o.z = pack_bf16x2(b.x, b.y); o.w = pack_bf16x2(b.z, b.w);
    reinterpret_cast<uint4*>(out)[i] = o;
  }
  if (blockIdx.x == 0)
    for (long long j = (n8 << 3) + threadIdx.x; j < n; j += blockDim.x)
      out[j] = static_cast<unsigned short>(pack_bf16x2(g[j], 0.0f) & 0xFFFFu);
}

// rows of `len` floats -> rows of `pitch` bf16 (pitch a multiple of 8, padding zero)
__global__ void __launch_bounds__(256)
grad_to_bf16_rows_kernel(const float* __restrict__ g, long long rows, int len, int pitch,
                         unsigned short* __restrict__ out) {
  pdl_trigger();
  const int per_row = pitch >> 3;
  const long long total = rows * per_row;
  const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
       i += stride) {
    const long long r = i / per_row;
    const int c0 = static_cast<int>(i - r * per_row) * 8;
    const float* src = g + r * len + c0;
    float v[8];
    if ((len & 3) == 0 && c0 + 8 <= len) {         // rows start on 16-byte boundaries
      const float4 a = __ldg(reinterpret_cast<const float4*>(src));
      const float4 b = __ldg(reinterpret_cast<const float4*>(src) + 1);
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
      v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = (c0 + e < len) ? __ldg(src + e) : 0.0f;
    }
    uint4 o;
    o.x = pack_bf16x2(v[0], v[1]); o.y = pack_bf16x2(v[2], v[3]);
    o.z = pack_bf16x2(v[4], v[5]); o.w = pack_bf16x2(v[6], v[7]);
    reinterpret_cast<uint4*>(out)[i] = o;
  }
}

using TensorMapEncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                       const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                       const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                       CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
TensorMapEncodeFn tensor_map_encoder() {
  return reinterpret_cast<TensorMapEncodeFn>(tensor_map_encode_fn());
}

}  // namespace

static bool compute_plan_conv_fast(const surgeon_layer_desc& d, FastParams* out) {
  if (d.kind != 1 || (d.stride != 1 && d.stride != 2)) return false;
  int mode;
  if (d.kh == 3 && d.kw == 3 && d.pad == 1) mode = 0;
  else if (d.kh == 1 && d.kw == 1 && d.pad == 0) mode = 1;
  else return false;
  FastParams p{};
  p.mode = mode;
  p.stride = d.stride;
  p.B = d.batch; p.C = d.c_in; p.H = d.h; p.W = d.w; p.O = d.c_out;
  p.OH = (d.h + 2 * d.pad - d.kh) / d.stride + 1;
  p.OW = (d.w + 2 * d.pad - d.kw) / d.stride + 1;
  p.P = p.OH * p.OW;
  p.n_gemm = d.c_in * d.kh * d.kw;
  if (mode == 0) {
    if (d.w % (8 * d.stride) != 0 || p.OW % 8 != 0) return false;
  } else if (d.stride == 1) {
    if ((d.h * d.w) % 8 != 0) return false;      // chunks of 8 never straddle an image
  } else {
    if (d.w % 16 != 0 || p.OW % 8 != 0) return false;
  }
  if (p.P % 8 != 0) return false;                 // TMA row pitch of the bf16 gradient: 16 bytes
  // accumulator width: the widest multiple of 16 up to 256 that divides O, else 256 with padding
  int acc_n = 0;
  for (int c = 256; c >= 128; c -= 16)
    if (p.O % c == 0) { acc_n = c; break; }
  if (acc_n == 0) acc_n = (p.O <= 256) ? (p.O + 15) / 16 * 16 : 256;
  const int acc_total = (p.O + acc_n - 1) / acc_n;
  p.acc_n = acc_n;
  p.n_acc = acc_total >= 2 ? 2 : 1;
  p.n_tiles = (acc_total + p.n_acc - 1) / p.n_acc;
  p.m_tiles = (p.n_gemm + kTileM - 1) / kTileM;
  p.tiles_per_img = (p.P + kTileK - 1) / kTileK;
  const long long total = static_cast<long long>(d.batch) * p.tiles_per_img;
  if (total > 2147483647LL) return false;
  p.total_ktiles = static_cast<int>(total);
  if (mode == 0) {
    const int out_rows = (kTileK + p.OW - 2) / p.OW + 1;
    int in_rows = (out_rows - 1) * d.stride + 3;
    if (in_rows > p.H) in_rows = p.H;
    const int range_len = in_rows * p.W;
    if (range_len + 31 > 32 * 32) return false;
    if (16 * range_len * 2 > kPatchBytes) return false;
  }
  // split K so that the CTA count fills whole waves of SMs
  const int sms = sm_count();
  const long long tiles_mn = static_cast<long long>(p.m_tiles) * p.n_tiles;
  const int max_splits = (p.total_ktiles + 7) / 8 < 1 ? 1 : (p.total_ktiles + 7) / 8;
  int best = 1;
  double best_cost = 1e30;
  for (int s = 1; s <= max_splits && s <= 64; ++s) {
    const long long ctas = tiles_mn * s;
    const long long waves = (ctas + sms - 1) / sms;
    const int kts = (p.total_ktiles + s - 1) / s;
    // time ~ waves * (K-tiles per CTA + fixed prologue/epilogue), plus the split reduction
    const double cost = static_cast<double>(waves) * (kts + 12) + 0.02 * s * tiles_mn / sms;
    if (cost < best_cost - 1e-9) { best_cost = cost; best = s; }
  }
  p.ktiles_per_split = (p.total_ktiles + best - 1) / best;
  p.splits = (p.total_ktiles + p.ktiles_per_split - 1) / p.ktiles_per_split;
  p.tmem_cols = 32;
  while (p.tmem_cols < p.n_acc * p.acc_n) p.tmem_cols *= 2;
  const int stage_bytes = kTileM * 128 + p.n_acc * p.acc_n * 128;
  const int fixed = kGroups * kPatchBytes + kGroups * 2 * kMetaWords * 4 + 1024 + 256;
  int stages = (227 * 1024 - fixed) / stage_bytes;
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < 2) return false;
  p.stages = stages;
  p.smem_bytes = stages * stage_bytes + fixed;
  *out = p;
  return true;
}

bool plan_conv_fast(const surgeon_layer_desc& d, FastParams* out) {
  struct Tag {};
  return memo_plan<Tag>(d, 0, out, [&](FastParams* p) { return compute_plan_conv_fast(d, p); });
}

cudaError_t launch_grad_to_bf16(const float* g, long long n, void* out_bf16, cudaStream_t stream) {
  const long long want = (n / 8 + 255) / 256;
  const long long cap = 16LL * sm_count();
  const int grid = static_cast<int>(want < 1 ? 1 : (want > cap ? cap : want));
  grad_to_bf16_kernel<<<grid, 256, 0, stream>>>(g, n, static_cast<unsigned short*>(out_bf16));
  note_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_grad_to_bf16_rows(const float* g, long long rows, int len, int pitch,
                                     void* out_bf16, cudaStream_t stream) {
  const long long want = (rows * (pitch >> 3) + 255) / 256;
  const long long cap = 16LL * sm_count();
  const int grid = static_cast<int>(want < 1 ? 1 : (want > cap ? cap : want));
  grad_to_bf16_rows_kernel<<<grid, 256, 0, stream>>>(g, rows, len, pitch,
                                                     static_cast<unsigned short*>(out_bf16));
  note_launches(1);
  return cudaGetLastError();
}

size_t conv_fast_grad_bf16_bytes(const FastParams& p) {
  const size_t b = static_cast<size_t>(p.B) * p.O * p.P * 2;
  return (b + 255) & ~static_cast<size_t>(255);
}

cudaError_t launch_conv_fast(const surgeon_compressed& act, const FastParams& p,
                             const float* grad_out, void* grad_bf16, float* partial,
                             uint32_t* status, cudaStream_t stream) {
  // 1. gradient fp32 -> bf16 (scratch), then a 3-D tensor map over [B][O][P] for the TMA loads
  const long long gn = static_cast<long long>(p.B) * p.O * p.P;
  {
    const long long want = (gn / 8 + 255) / 256;
    const long long cap = 16LL * sm_count();
    const int grid = static_cast<int>(want < 1 ? 1 : (want > cap ? cap : want));
    grad_to_bf16_kernel<<<grid, 256, 0, stream>>>(grad_out, gn,
                                                  static_cast<unsigned short*>(grad_bf16));
  }
  CUtensorMap map;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(p.P), static_cast<cuuint64_t>(p.O),
                              static_cast<cuuint64_t>(p.B)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(p.P) * 2,
                                 static_cast<cuuint64_t>(p.P) * p.O * 2};
  const cuuint32_t box[3] = {static_cast<cuuint32_t>(kTileK), static_cast<cuuint32_t>(p.acc_n), 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const TensorMapEncodeFn encode = tensor_map_encoder();
  if (!encode) return cudaErrorNotSupported;
  const CUresult r = encode(
      &map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, grad_bf16, dims, strides, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;

  const uint32_t* offs = act.block_offsets;
  dim3 grid(p.m_tiles, p.n_tiles, p.splits);
  cudaError_t e;
  if (act.dt == 0) {
    e = allow_dynamic_smem(reinterpret_cast<const void*>(dw_conv_fast_kernel<0>), p.smem_bytes);
    if (e != cudaSuccess) return e;
    dw_conv_fast_kernel<0><<<grid, kThreads, p.smem_bytes, stream>>>(
        act.bitmap, act.values, offs, map, partial, status, p);
  } else {
    e = allow_dynamic_smem(reinterpret_cast<const void*>(dw_conv_fast_kernel<1>), p.smem_bytes);
    if (e != cudaSuccess) return e;
    dw_conv_fast_kernel<1><<<grid, kThreads, p.smem_bytes, stream>>>(
        act.bitmap, act.values, offs, map, partial, status, p);
  }
  note_launches(2);
  return cudaGetLastError();
}

}  // namespace surgeon

// Fast tensor-core weight-gradient kernel for stride-1 convolutions whose rows are a multiple of
// 8 elements wide: 3x3 / pad 1 ("patch" mode) and 1x1 / pad 0 ("direct" mode).
// Algorithm 1 lines 11-12 with Eq. 2; same GEMM view as weight_grad_tc.cu:
//   D[nn, o] = sum_k Acol[nn, k] * G[o, k],  nn = (c, r, s),  k = (b, y, x).
//
// What differs from the general kernel:
//   * two producer groups of 8 warps fill alternate pipeline stages, so the global-load latency
//     of one group hides behind the other group's arithmetic and the MMAs;
//   * per K-tile, the bitmap words of every channel range and the rank of each word's first
//     bit are staged in shared memory one tile ahead; decompression then works on units of
//     8 elements (one bitmap byte) with eight independent loads of packed values per thread;
//   * patch mode copies the im2col view with one 16-byte load per (channel, filter row, chunk)
//     and funnel shifts for the s = 0 / s = 2 columns; direct mode (1x1) decompresses straight
//     into the swizzled operand tile;
//   * one or two accumulators (<= 512 TMEM columns) share each activation tile.
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
constexpr int kMetaWords = 512;              // bitmap words staged per group and K-tile
constexpr int kMaxStages = 4;
constexpr int kGBatch = 4;                   // gradient chunks a thread keeps in flight

__device__ __forceinline__ void group_sync(int g) {
  asm volatile("bar.sync %0, %1;" ::"r"(g + 1), "n"(kGroupThreads) : "memory");
}

// Unit = 8 consecutive elements (one bitmap byte).  words/wrank: staged bitmap words of the
// range and the rank of each word's first bit; rel = bit offset of the unit from the first
// staged word.  Returns the 8 elements as packed bf16 (Algorithm 1 line 11).
template <int DT>
__device__ __forceinline__ uint4 decompress_unit(const uint32_t* __restrict__ words,
                                                 const uint32_t* __restrict__ wrank, int rel,
                                                 const void* __restrict__ values) {
  const int wi = rel >> 5, sh = rel & 31;
  const uint32_t word = words[wi];
  const uint32_t byte = (word >> sh) & 0xFFu;
  uint32_t r = wrank[wi] + __popc(word & ((1u << sh) - 1u));
  uint4 out = make_uint4(0, 0, 0, 0);
  if (byte == 0) return out;
  if (DT == 0) {
    const float* v = reinterpret_cast<const float*>(values);
    float f[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const bool on = (byte >> e) & 1u;
      f[e] = on ? __ldg(v + r) : 0.0f;
      r += on ? 1u : 0u;
    }
    out.x = pack_bf16x2(f[0], f[1]); out.y = pack_bf16x2(f[2], f[3]);
    out.z = pack_bf16x2(f[4], f[5]); out.w = pack_bf16x2(f[6], f[7]);
  } else {
    const unsigned short* v = reinterpret_cast<const unsigned short*>(values);
    uint32_t h[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const bool on = (byte >> e) & 1u;
      h[e] = on ? static_cast<uint32_t>(__ldg(v + r)) : 0u;
      r += on ? 1u : 0u;
    }
    out.x = h[0] | (h[1] << 16); out.y = h[2] | (h[3] << 16);
    out.z = h[4] | (h[5] << 16); out.w = h[6] | (h[7] << 16);
  }
  return out;
}

template <int DT>
__global__ void __launch_bounds__(kThreads, 1)
dw_conv_fast_kernel(const uint32_t* __restrict__ bitmap, const void* __restrict__ values,
                    const unsigned long long* __restrict__ offsets, const float* __restrict__ grad,
                    float* __restrict__ partial, uint32_t* __restrict__ status, FastParams p) {
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
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(full_bar + 8 * s, kGroupWarps);
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
      bool ok = true;
      for (int it = 0; it < n_kt; ++it) {
        const int s = it % p.stages;
        ok = mbar_wait(full_bar + 8 * s, (it / p.stages) & 1);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_addr = smem_u32(smem + s * stage_bytes);
        const uint32_t b_addr = a_addr + kTileM * 128;
#pragma unroll
        for (int kk = 0; kk < kTileK / 16; ++kk) {
          const uint64_t da = make_desc(a_addr + kk * 32);
          for (int a = 0; a < p.n_acc; ++a)
            umma_bf16(tmem_base + a * p.acc_n, da, make_desc(b_addr + a * p.acc_n * 128 + kk * 32),
                      idesc, (it > 0 || kk > 0) ? 1u : 0u);
        }
        umma_commit(empty_bar + 8 * s);
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
    const int range_words = (p.mode == 0) ? 32 : 4;

    // Geometry of K-tile `it` of this CTA.
    struct Tile { int img, p0, k_valid, iy_lo, range_len; };
    auto tile_of = [&](int it) {
      Tile t;
      const int kt = kt_begin + it;
      t.img = kt / p.tiles_per_img;
      t.p0 = (kt - t.img * p.tiles_per_img) * kTileK;
      t.k_valid = min(kTileK, p.P - t.p0);
      if (p.mode == 0) {
        const int y_first = t.p0 / p.W;
        const int y_last = (t.p0 + t.k_valid - 1) / p.W;
        t.iy_lo = max(y_first - 1, 0);
        const int iy_hi = min(y_last + 1, p.H - 1);
        t.range_len = (iy_hi - t.iy_lo + 1) * p.W;
      } else {
        t.iy_lo = 0;
        t.range_len = t.k_valid;
      }
      return t;
    };
    // First flat index of range `ri` (channel first_c + ri) of a tile.
    auto range_start = [&](const Tile& t, int ri) -> long long {
      const long long plane = (static_cast<long long>(t.img) * p.C + first_c + ri) * p.P;
      return (p.mode == 0) ? plane + static_cast<long long>(t.iy_lo) * p.W : plane + t.p0;
    };
    // Stage the bitmap words and per-word ranks of every range of a tile.
    auto stage_meta = [&](const Tile& t) {
      if (p.mode == 0) {
        for (int ri = gwarp; ri < n_ch; ri += kGroupWarps) {
          const long long start = range_start(t, ri);
          const long long first_word = start >> 5;
          const long long blk = start >> 10;
          const long long blk_word0 = blk << 5;
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
        for (int ri = gtid; ri < n_ch; ri += kGroupThreads) {
          const long long start = range_start(t, ri);
          const long long first_word = start >> 5;
          const long long blk = start >> 10;
          const long long blk_word0 = blk << 5;
          uint32_t base = static_cast<uint32_t>(__ldg(offsets + blk));
          const int before = static_cast<int>(first_word - blk_word0);
#pragma unroll 8
          for (int w = 0; w < 31; ++w)
            if (w < before) base += __popc(__ldg(bitmap + blk_word0 + w));
          const int nwords = static_cast<int>(((start + t.range_len - 1) >> 5) - first_word) + 1;
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            const uint32_t word = (w < nwords) ? __ldg(bitmap + first_word + w) : 0u;
            m_words[ri * 4 + w] = word;
            m_rank[ri * 4 + w] = base;
            base += __popc(word);
          }
        }
      }
    };

    if (g < n_kt) stage_meta(tile_of(g));
    for (int it = g; it < n_kt; it += kGroups) {
      const int s = it % p.stages;
      if (it >= p.stages) {
        if (!mbar_wait(empty_bar + 8 * s, ((it / p.stages) - 1) & 1)) {
          *fail = 1;
          atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
        }
      }
      group_sync(g);    // staged metadata visible; every thread of the group sees the same *fail
      if (*fail) break;
      unsigned char* a_tile = smem + s * stage_bytes;
      unsigned char* b_tile = a_tile + kTileM * 128;
      const Tile t = tile_of(it);

      // gradient chunks travel through registers in batches, loads issued early
      const int g_tasks = n_cols * 8;
      const int g_batches = (g_tasks + kGroupThreads * kGBatch - 1) / (kGroupThreads * kGBatch);
      float4 gr[kGBatch][2];
      auto g_issue = [&](int batch) {
#pragma unroll
        for (int i = 0; i < kGBatch; ++i) {
          const int task = (batch * kGBatch + i) * kGroupThreads + gtid;
          const int row = task >> 3, chunk = task & 7;
          const int o = o0 + row;
          const int pp = t.p0 + chunk * 8;
          gr[i][0] = make_float4(0.f, 0.f, 0.f, 0.f);
          gr[i][1] = gr[i][0];
          if (task < g_tasks && o < p.O && pp < p.P) {
            const float4* src = reinterpret_cast<const float4*>(
                grad + (static_cast<long long>(t.img) * p.O + o) * p.P + pp);
            gr[i][0] = __ldg(src);
            gr[i][1] = __ldg(src + 1);
          }
        }
      };
      auto g_store = [&](int batch) {
#pragma unroll
        for (int i = 0; i < kGBatch; ++i) {
          const int task = (batch * kGBatch + i) * kGroupThreads + gtid;
          if (task < g_tasks) {
            uint4 out;
            out.x = pack_bf16x2(gr[i][0].x, gr[i][0].y); out.y = pack_bf16x2(gr[i][0].z, gr[i][0].w);
            out.z = pack_bf16x2(gr[i][1].x, gr[i][1].y); out.w = pack_bf16x2(gr[i][1].z, gr[i][1].w);
            *reinterpret_cast<uint4*>(b_tile + tile_off(task >> 3, task & 7)) = out;
          }
        }
      };
      g_issue(0);

      if (p.mode == 0) {
        // ---- decompress the channel ranges into the patch, 8 elements per thread ----
        const int units_per_range = t.range_len >> 3;
        const int units = n_ch * units_per_range;
        for (int u = gtid; u < units; u += kGroupThreads) {
          const int ri = u / units_per_range;
          const int uu = u - ri * units_per_range;
          const int bit0 = static_cast<int>(range_start(t, ri) & 31);
          const uint4 v = decompress_unit<DT>(m_words + ri * 32, m_rank + ri * 32, bit0 + uu * 8,
                                              values);
          *reinterpret_cast<uint4*>(patch + ri * t.range_len + uu * 8) = v;
        }
        group_sync(g);
        g_store(0);
        if (g_batches > 1) g_issue(1);
        // ---- im2col view: one task = (channel, filter row r, chunk) -> columns s = 0, 1, 2 ----
        const int tasks = n_ch * 24;
        for (int q = gtid; q < tasks; q += kGroupThreads) {
          const int ci = q / 24;
          const int rem = q - ci * 24;
          const int r = rem >> 3, chunk = rem & 7;
          const int pp = t.p0 + chunk * 8;
          const int y = pp / p.W;
          const int x0 = pp - y * p.W;
          const int iy = y + r - 1;
          uint4 c4 = make_uint4(0, 0, 0, 0);
          uint32_t left = 0, right = 0;
          if (pp < p.P && iy >= 0 && iy < p.H) {
            const unsigned short* src = patch + ci * t.range_len + (iy - t.iy_lo) * p.W + x0;
            c4 = *reinterpret_cast<const uint4*>(src);
            if (x0 > 0) left = src[-1];
            if (x0 + 8 < p.W) right = src[8];
          }
          const int row0 = (first_c + ci) * 9 + r * 3 - nn0;
          uint4 lo4, hi4;   // shifted by -1 (s = 0) and by +1 (s = 2)
          lo4.x = (c4.x << 16) | left;
          lo4.y = __funnelshift_l(c4.x, c4.y, 16);
          lo4.z = __funnelshift_l(c4.y, c4.z, 16);
          lo4.w = __funnelshift_l(c4.z, c4.w, 16);
          hi4.x = __funnelshift_r(c4.x, c4.y, 16);
          hi4.y = __funnelshift_r(c4.y, c4.z, 16);
          hi4.z = __funnelshift_r(c4.z, c4.w, 16);
          hi4.w = (c4.w >> 16) | (right << 16);
          if (row0 >= 0 && row0 < rows_valid)
            *reinterpret_cast<uint4*>(a_tile + tile_off(row0, chunk)) = lo4;
          if (row0 + 1 >= 0 && row0 + 1 < rows_valid)
            *reinterpret_cast<uint4*>(a_tile + tile_off(row0 + 1, chunk)) = c4;
          if (row0 + 2 >= 0 && row0 + 2 < rows_valid)
            *reinterpret_cast<uint4*>(a_tile + tile_off(row0 + 2, chunk)) = hi4;
        }
      } else {
        // ---- 1x1: decompress straight into the operand tile; row = channel, chunk = unit ----
        const int units = rows_valid * 8;
        for (int u = gtid; u < units; u += kGroupThreads) {
          const int ri = u >> 3, chunk = u & 7;
          uint4 v = make_uint4(0, 0, 0, 0);
          if (chunk * 8 < t.k_valid) {
            const int bit0 = static_cast<int>(range_start(t, ri) & 31);
            v = decompress_unit<DT>(m_words + ri * 4, m_rank + ri * 4, bit0 + chunk * 8, values);
          }
          *reinterpret_cast<uint4*>(a_tile + tile_off(ri, chunk)) = v;
        }
        g_store(0);
        if (g_batches > 1) g_issue(1);
      }
      for (int b = 1; b < g_batches; ++b) {
        g_store(b);
        if (b + 1 < g_batches) g_issue(b + 1);
      }
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(full_bar + 8 * s);
      // metadata of this group's next tile (the group_sync at the top of the loop publishes it;
      // the one after the decompression above guarantees nobody still reads the old one)
      if (p.mode == 1) group_sync(g);
      if (it + kGroups < n_kt) stage_meta(tile_of(it + kGroups));
    }
  }

  // ================= epilogue: TMEM -> scratch partial tile =================
  if (warp >= 1 && warp <= 4) {
    const bool done = mbar_wait(acc_bar, 0, 256);
    tc_fence_after();
    if (done && !*fail) {
      const int lane_grp = warp & 3;
      const int row = lane_grp * 32 + static_cast<int>(lane);
      const int nn = nn0 + row;
      float* out = partial + static_cast<long long>(split) * p.O * p.n_gemm;
      for (int col = 0; col < n_cols; col += 16) {
        uint32_t r[16];
        tmem_ld16(tmem_base + (static_cast<uint32_t>(lane_grp * 32) << 16) + col, r);
        if (nn < p.n_gemm) {
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const int o = o0 + col + e;
            if (o < p.O) out[static_cast<long long>(o) * p.n_gemm + nn] = __uint_as_float(r[e]);
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

}  // namespace

bool plan_conv_fast(const surgeon_layer_desc& d, FastParams* out) {
  if (d.kind != 1 || d.stride != 1) return false;
  int mode;
  if (d.kh == 3 && d.kw == 3 && d.pad == 1) mode = 0;
  else if (d.kh == 1 && d.kw == 1 && d.pad == 0) mode = 1;
  else return false;
  if (d.w % 8 != 0) return false;
  FastParams p{};
  p.mode = mode;
  p.B = d.batch; p.C = d.c_in; p.H = d.h; p.W = d.w; p.O = d.c_out;
  p.P = d.h * d.w;
  p.n_gemm = d.c_in * d.kh * d.kw;
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
    const int out_rows = (kTileK + p.W - 2) / p.W + 1;
    int in_rows = out_rows + 2;
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

cudaError_t launch_conv_fast(const surgeon_compressed& act, const FastParams& p,
                             const float* grad_out, float* partial, uint32_t* status,
                             cudaStream_t stream) {
  const unsigned long long* offs = reinterpret_cast<const unsigned long long*>(act.block_offsets);
  dim3 grid(p.m_tiles, p.n_tiles, p.splits);
  cudaError_t e;
  if (act.dt == 0) {
    e = cudaFuncSetAttribute(dw_conv_fast_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             p.smem_bytes);
    if (e != cudaSuccess) return e;
    dw_conv_fast_kernel<0><<<grid, kThreads, p.smem_bytes, stream>>>(
        act.bitmap, act.values, offs, grad_out, partial, status, p);
  } else {
    e = cudaFuncSetAttribute(dw_conv_fast_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             p.smem_bytes);
    if (e != cudaSuccess) return e;
    dw_conv_fast_kernel<1><<<grid, kThreads, p.smem_bytes, stream>>>(
        act.bitmap, act.values, offs, grad_out, partial, status, p);
  }
  return cudaGetLastError();
}

}  // namespace surgeon

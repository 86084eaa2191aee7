// Weight gradient of a GROUPED convolution from the compressed store (Algorithm 1: Reshape and
// gradient steps with Eq. 2, for the layer type of ResNeXt's 3x3 convolutions and of depthwise
// convolutions; the paper adapts ResNeXt-29, Section 5.1).
//
//   dw[o, c', r, s] = sum_{b, y, x} g[b, o, y, x] * A[b, grp*(C/G) + c', y*stride + r - pad,
//                                                      x*stride + s - pad],   grp = o / (O/G)
//
// Every group is its own small problem: O/G x (C/G * kh * kw) outputs (4 x 36 ... 16 x 144 for
// ResNeXt-29 32x4d, 1 x 9 for a depthwise 3x3) over a long reduction.  That is far below one MMA
// tile per group and the layer is bound by the one read of the fp32 gradient, so both values of
// surgeon_layer_desc::path run this CUDA-core kernel (fp32 products, sums kept in double across
// images).  A CTA takes one group and one band of output rows: per image it rebuilds the band's
// input rows of the group's channels from the store into shared memory (zero padding
// materialised, so the inner loop has no bounds tests), copies the band of the group's gradient
// planes beside them, and every thread accumulates up to 8 output channels of a few (c', r, s)
// columns.  Partial sums per (band, image chunk) are added in a fixed order by a second kernel:
// results are bitwise reproducible.
#include <type_traits>

#include "surgeon_internal.cuh"

namespace surgeon {

namespace {

constexpr int kThreads = 256;
constexpr int kRO = 8;        // most output channels per thread and column (the block size n_ob counts in)
constexpr int kUMax = 4;      // (output block, column) units per thread
constexpr int kSmemBudget = 160 * 1024;

struct GroupedParams {
  int B, C, H, W, O, KH, KW, stride, pad, OH, OW, G, Cg, Og;
  int band, n_bands;          // output rows per band, bands per image
  int in_rows, Wp;            // input rows of a band (padding rows included), padded row length
  int ncol, n_ob, n_units;    // columns (c', r, s), blocks of kRO output channels, their product
  int S;                      // position splits: threads [s * n_units, (s + 1) * n_units) take positions s, s + S, ...
  int chunks, imgs_per_chunk; // image chunks (grid.z)
  int a_floats, g_floats;     // shared-memory floats of one image's activation band / gradient band
  int nb;                     // images per round (both tiles hold that many)
  long long n_words;          // words of the bitmap (filled by the launcher)
  unsigned partial_blk;       // index of the bitmap's last block if it is partial, else 0xFFFFFFFF
};

// Where element j of the pruned activation lives: fetched in two steps so that the loads of many
// elements are in flight together (the metadata first, then the one value).
struct ActRef { uint4 words; uint32_t base; };
__device__ __forceinline__ ActRef act_meta(const uint32_t* __restrict__ bitmap, const uint32_t* __restrict__ offsets,
                                           long long j, long long n_words, unsigned partial_blk) {
  ActRef r;
  const long long blk = j >> kBlockShift;
  r.base = __ldg(offsets + blk);
  if (static_cast<unsigned long long>(blk) != partial_blk) {
    r.words = __ldg(reinterpret_cast<const uint4*>(bitmap) + blk);
  } else {                                     // the last, partial block of the bitmap
    const long long w0 = blk * kBlockWords;
    r.words.x = __ldg(bitmap + w0);
    r.words.y = (w0 + 1 < n_words) ? __ldg(bitmap + w0 + 1) : 0u;
    r.words.z = (w0 + 2 < n_words) ? __ldg(bitmap + w0 + 2) : 0u;
    r.words.w = (w0 + 3 < n_words) ? __ldg(bitmap + w0 + 3) : 0u;
  }
  return r;
}
// Index of element j in the packed vector, or -1 when it was pruned.
__device__ __forceinline__ long long act_rank(const ActRef& r, long long j) {
  const uint32_t wq = (static_cast<uint32_t>(j) >> 5) & 3u, bit = static_cast<uint32_t>(j) & 31u;
  const uint32_t w = wq == 0 ? r.words.x : (wq == 1 ? r.words.y : (wq == 2 ? r.words.z : r.words.w));
  if (!((w >> bit) & 1u)) return -1;
  uint32_t k = r.base + __popc(w & ((1u << bit) - 1u));
  k += wq > 0 ? __popc(r.words.x) : 0u;
  k += wq > 1 ? __popc(r.words.y) : 0u;
  k += wq > 2 ? __popc(r.words.z) : 0u;
  return static_cast<long long>(k);
}
template <int DT>
__device__ __forceinline__ float act_value(const void* __restrict__ values, long long k) {
  if (k < 0) return 0.0f;
  if (DT == 0) return __ldg(reinterpret_cast<const float*>(values) + k);
  const uint32_t h = __ldg(reinterpret_cast<const unsigned short*>(values) + k);
  return __uint_as_float(h << 16);
}

// RO: output channels a thread really accumulates per unit (1, 2, 4 or 8: the smallest that covers
// min(Og, 8)); PV: output positions per step (4 when the output rows are a multiple of 4 wide: the
// gradient then comes as 16-byte shared-memory loads, else 1).
// UM: units a thread may own (1, 2 or 4; more than one only when a group has more than 256 units).
template <int DT, int RO, int PV, int UM>
__global__ void __launch_bounds__(kThreads, 2)
dw_grouped_kernel(const uint32_t* __restrict__ bitmap, const void* __restrict__ values,
                  const uint32_t* __restrict__ offsets, const float* __restrict__ grad,
                  double* __restrict__ partial, GroupedParams p) {
  extern __shared__ __align__(16) float sm[];
  float* As = sm;                       // [Cg][in_rows][Wp], zero where the input has padding
  float* Gs = sm + p.nb * p.a_floats;   // [n_ob * kRO][band * OW], zero rows past Og; both tiles hold nb images
  const int tid = threadIdx.x;
  const int grp = blockIdx.x, band = blockIdx.y, chunk = blockIdx.z;
  const int y0 = band * p.band;
  const int rows = min(p.band, p.OH - y0);          // output rows of this band
  const int npos = rows * p.OW;
  const int iy0 = y0 * p.stride - p.pad;            // input row of As row 0
  const int b_begin = chunk * p.imgs_per_chunk;
  const int b_end = min(b_begin + p.imgs_per_chunk, p.B);
  const int RS = p.KH * p.KW;
  const int gpitch = p.band * p.OW;

  // this thread's units and position split
  const int total_threads_used = p.n_units * p.S;
  double acc[UM][RO];
#pragma unroll
  for (int u = 0; u < UM; ++u)
#pragma unroll
    for (int e = 0; e < RO; ++e) acc[u][e] = 0.0;

  // nb images per round: the loads of a round (gradient planes, then three dependent levels of
  // the store) are latency, not bandwidth, so several images' worth are kept in flight together
  for (int b0 = b_begin; b0 < b_end; b0 += p.nb) {
    const int nb_here = min(p.nb, b_end - b0);
    __syncthreads();                                 // the previous round's tiles are no longer read
    // ---- the band of the group's gradient planes ----
    for (int i = tid; i < nb_here * p.g_floats; i += kThreads) {
      const int bi = i / p.g_floats, ii = i - bi * p.g_floats;
      const int ol = ii / gpitch, pos = ii - ol * gpitch;
      float v = 0.0f;
      if (ol < p.Og && pos < npos)
        v = __ldg(grad + (static_cast<long long>(b0 + bi) * p.O + grp * p.Og + ol) * (p.OH * p.OW) + y0 * p.OW + pos);
      Gs[i] = v;
    }
    // ---- the band's input rows of the group's channels, rebuilt from the store, four elements
    // per thread at a time with their loads in flight together ----
    const int a_total = nb_here * p.a_floats;
    for (int i0 = tid; i0 < a_total; i0 += 4 * kThreads) {
      long long jj[4];
      ActRef ref[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int ia = i0 + q * kThreads;
        jj[q] = -1;
        if (ia < a_total) {
          const int bi = ia / p.a_floats, i = ia - bi * p.a_floats;
          const int b = b0 + bi;
          const int cl = i / (p.in_rows * p.Wp);
          const int rem = i - cl * (p.in_rows * p.Wp);
          const int ry = rem / p.Wp, rx = rem - ry * p.Wp;
          const int iy = iy0 + ry, ix = rx - p.pad;
          if (cl < p.Cg && iy >= 0 && iy < p.H && ix >= 0 && ix < p.W)      // (a_floats is padded to a multiple of 4)
            jj[q] = ((static_cast<long long>(b) * p.C + grp * p.Cg + cl) * p.H + iy) * p.W + ix;
        }
        if (jj[q] >= 0) ref[q] = act_meta(bitmap, offsets, jj[q], p.n_words, p.partial_blk);
      }
      long long kk[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) kk[q] = jj[q] >= 0 ? act_rank(ref[q], jj[q]) : -1;
      float vv[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) vv[q] = act_value<DT>(values, kk[q]);
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (i0 + q * kThreads < a_total) As[i0 + q * kThreads] = vv[q];
    }
    __syncthreads();
    // ---- products: thread = (split s, unit u0 + 256 * k); unit = (output block, column) ----
#pragma unroll
    for (int k = 0; k < UM; ++k) {
      const int t = tid + k * kThreads;
      if (t >= total_threads_used) break;
      const int s = t / p.n_units, unit = t - s * p.n_units;
      const int ob = unit / p.ncol, col = unit - ob * p.ncol;
      const int cl = col / RS, rs = col - cl * RS;
      const int r = rs / p.KW, sx = rs - r * p.KW;
      const float* a_base0 = As + (cl * p.in_rows + r) * p.Wp + sx;
      const float* g_base0 = Gs + ob * kRO * gpitch;
      float f[RO];
#pragma unroll
      for (int e = 0; e < RO; ++e) f[e] = 0.0f;
      // steps of PV positions s, s + S, ...; (y, x) follow without a division per step
      const int steps_per_row = p.OW / PV;
      const int dy = p.S / steps_per_row, dx = p.S - dy * steps_per_row;
      for (int bi = 0; bi < nb_here; ++bi) {
      const float* a_base = a_base0 + bi * p.a_floats;
      const float* g_base = g_base0 + bi * p.g_floats;
      int y = s / steps_per_row, xs = s - y * steps_per_row;
      for (; y < rows;) {
        const int x = xs * PV;
        const float* ap = a_base + y * p.stride * p.Wp + x * p.stride;
        const float* gp = g_base + y * p.OW + x;
        if (PV == 4) {
          const float a0 = ap[0], a1 = ap[p.stride], a2 = ap[2 * p.stride], a3 = ap[3 * p.stride];
#pragma unroll
          for (int e = 0; e < RO; ++e) {
            const float4 g4 = *reinterpret_cast<const float4*>(gp + e * gpitch);
            f[e] = fmaf(g4.x, a0, f[e]); f[e] = fmaf(g4.y, a1, f[e]);
            f[e] = fmaf(g4.z, a2, f[e]); f[e] = fmaf(g4.w, a3, f[e]);
          }
        } else {
          const float a = ap[0];
#pragma unroll
          for (int e = 0; e < RO; ++e) f[e] = fmaf(gp[e * gpitch], a, f[e]);
        }
        y += dy; xs += dx;
        if (xs >= steps_per_row) { xs -= steps_per_row; ++y; }
      }
      }
#pragma unroll
      for (int e = 0; e < RO; ++e) acc[k][e] += static_cast<double>(f[e]);
    }
  }
  // ---- sum the position splits (fixed order) and write this CTA's partial tile ----
  __syncthreads();
  double* red = reinterpret_cast<double*>(sm);       // [S][n_units][kRO], fits: checked by the planner
#pragma unroll
  for (int k = 0; k < UM; ++k) {
    const int t = tid + k * kThreads;
    if (t < total_threads_used) {
#pragma unroll
      for (int e = 0; e < kRO; ++e) red[static_cast<long long>(t) * kRO + e] = e < RO ? acc[k][e < RO ? e : 0] : 0.0;
    }
  }
  __syncthreads();
  // partial[(chunk * n_bands + band)][o][col], o over all O output channels
  double* out = partial + static_cast<long long>(chunk * p.n_bands + band) * p.O * p.ncol;
  for (int i = tid; i < p.n_units * kRO; i += kThreads) {
    const int unit = i / kRO, e = i - unit * kRO;
    const int ob = unit / p.ncol, col = unit - ob * p.ncol;
    const int ol = ob * kRO + e;
    if (ol >= p.Og) continue;
    double s = 0.0;
    for (int sp = 0; sp < p.S; ++sp) s += red[(static_cast<long long>(sp) * p.n_units + unit) * kRO + e];
    out[static_cast<long long>(grp * p.Og + ol) * p.ncol + col] = s;
  }
}

// ---- 3x3, padding 1, stride 1 or 2, output rows a multiple of 8 wide (ResNeXt's grouped layers) ----
// Register tiles instead of one column per thread: a thread owns TO output channels x TC input
// channels x 9 taps of accumulators and walks strips of 8 consecutive output positions.  Per strip
// and (channel, kernel row) it loads the 10 (stride 2: 17) input values the three taps need as
// aligned 16-byte vectors and reuses them for all TO channels and all 3 column taps, so a
// shared-memory load feeds 13-26 FMAs instead of 2.  The band's input rows are rebuilt word by
// word of the bitmap into a zeroed tile (see the loop), with no index division per element.  Sums stay in fp32 inside a thread (at most kTermsPerThread terms, the planner cuts the
// images into chunks accordingly), the threads' tiles are added in double in a fixed order.
struct Grouped3Params {
  int B, C, H, W, O, OH, OW, G, Cg, Og;
  int band, n_bands, in_rows, Wp;
  int units, n_cb, S;          // (output block, channel block) units; channel blocks; strip splits
  int chunks, imgs_per_chunk, nb;
  int a_floats, g_floats;      // per image
  int dt;
  uint32_t rcp_cg, rcp_spr, rcp_w;    // 2^32 / d rounded up: __umulhi(n, rcp) = n / d while n * d < 2^32
  long long n_words, n, n_blocks;
  unsigned partial_blk;
};
constexpr int kTermsPerThread = 4096;
// n / d by one multiplication: rcp = floor((2^32 - 1) / d) + 1, exact while n * d < 2^32 (d = 1: rcp
// wraps to 0 and the quotient is n itself).
__host__ __device__ __forceinline__ uint32_t div_magic(int d) { return 0xFFFFFFFFu / static_cast<uint32_t>(d) + 1u; }
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst))),
               "l"(gsrc));
}
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ int fast_div(int n, uint32_t rcp) {
  return rcp ? static_cast<int>(__umulhi(static_cast<uint32_t>(n), rcp)) : n;
}
// Three CTAs share an SM: rebuilding a tile is two dependent global loads per element, so what
// hides that latency is the other CTAs' work.  That leaves a CTA 85 registers per thread (tiles of
// at most 4 channel pairs: 36 accumulators) and about 74 KB of shared memory.
constexpr int kG3CtasPerSm = 2;
constexpr int kG3Smem = 110 * 1024;
constexpr int kG3MaxTile = 8;

template <int TO, int TC, int ST>
__global__ void __launch_bounds__(kThreads, kG3CtasPerSm)
dw_grouped3_kernel(const uint32_t* __restrict__ bitmap, const void* __restrict__ values,
                   const uint32_t* __restrict__ offsets, const float* __restrict__ grad,
                   double* __restrict__ partial, Grouped3Params p) {
  constexpr int ACC = TO * TC * 9;
  constexpr int AW = ST == 1 ? 12 : 20;              // input values loaded per (channel, kernel row)
  extern __shared__ __align__(16) float sm[];
  float* As = sm;                                     // [nb][Cg][in_rows][Wp], column 0 = input column -1
  float* Gs = sm + p.nb * p.a_floats;                 // [nb][Og][band * OW]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int grp = blockIdx.x, band = blockIdx.y, chunk = blockIdx.z;
  const int y0 = band * p.band;
  const int rows = min(p.band, p.OH - y0);
  const int npos = rows * p.OW;
  const int iy0 = y0 * ST - 1;                        // input row of As row 0
  const int iy_lo = max(iy0, 0), iy_hi = min(iy0 + (rows - 1) * ST + 3, p.H);   // valid input rows [lo, hi)
  const int n_valid = iy_hi - iy_lo;
  const int b_begin = chunk * p.imgs_per_chunk;
  const int b_end = min(b_begin + p.imgs_per_chunk, p.B);
  const int gpitch = p.band * p.OW;
  const int spr = p.OW >> 3;                          // strips per output row
  const int n_strips = rows * spr;
  const uint32_t rcp_strips = div_magic(n_strips);

  float acc[ACC];
#pragma unroll
  for (int i = 0; i < ACC; ++i) acc[i] = 0.0f;

  // more than 55 % of the tensor kept (the last block offset is the kept count): the rebuild walks
  // the bitmap words with a lane per bit instead of a lane per word
  const bool dense = static_cast<double>(__ldg(offsets + p.n_blocks)) > 0.55 * static_cast<double>(p.n);
  // this thread's unit and strip split
  const int unit = tid / p.S, sidx = tid - unit * p.S;
  const bool worker = unit < p.units;
  const int ob = unit / p.n_cb, cb = unit - ob * p.n_cb;

  // rebuilding: a lane takes one bitmap word of a channel plane's valid rows and scatters its kept
  // values (the tiles are zeroed every round, so pruned elements cost nothing)
  const int plane_len = n_valid * p.W;
  const int wpp = (plane_len + 31) / 32 + 1;          // words a plane's range can touch
  const uint32_t rcp_wpp_k = div_magic(wpp);

  auto plane_range = [&](int b, int cl, long long& e_lo, long long& e_hi) {
    e_lo = (static_cast<long long>(b) * p.C + grp * p.Cg + cl) * (p.H * p.W) + iy_lo * p.W;
    e_hi = e_lo + plane_len;
  };
  for (int b0 = b_begin; b0 < b_end; b0 += p.nb) {
    const int nb_here = min(p.nb, b_end - b0);
    __syncthreads();                                  // the previous round's tiles are no longer read
    // ---- gradient planes of the group, rows of the band: asynchronous 16-byte copies, a warp per
    // plane; all of a thread's copies are in flight together and are waited for once ----
    {
      const int q4 = npos >> 2;                       // vectors per plane
      for (int pl = warp; pl < nb_here * p.Og; pl += kThreads / 32) {
        const int bi = pl / p.Og, o = pl - bi * p.Og;
        const float4* src = reinterpret_cast<const float4*>(
            grad + (static_cast<long long>(b0 + bi) * p.O + grp * p.Og + o) * (p.OH * p.OW) + y0 * p.OW);
        float4* dst = reinterpret_cast<float4*>(Gs + bi * p.g_floats + o * gpitch);
        for (int v = lane; v < q4; v += 32) cp_async16(dst + v, src + v);
      }
    }
    for (int i = tid; i < (nb_here * p.a_floats) >> 2; i += kThreads)
      reinterpret_cast<float4*>(As)[i] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    // ---- the band's input rows of the group's channels from the store ----
    // A lane takes one bitmap word at a time (two per pass): it fetches the word's block (bitmap
    // words and offset, independent loads), ranks the word's first kept element and scatters the
    // word's kept values into the zeroed tile, eight loads in flight at a time.  The metadata of the
    // first pass is requested before the barrier that ends the zeroing, so its latency and that of
    // the gradient copies overlap.  The work is per kept element, which is what wins on sparse
    // stores (ResNeXt stage 1 at the rule's ratios: 108 us against 158 us for the lane-per-bit walk
    // below); on mostly kept stores it loses (a lane's loads each touch their own cache line: 149
    // against 128 us on a stage-2 layer), hence the two paths.
    {
      struct WordRef { uint32_t bits, kfirst; int lo, col0, pos; };   // pos: tile index of bit `lo`
      const int total = nb_here * p.Cg * wpp;
      auto fetch = [&](int wi) {
        WordRef r{0u, 0u, 0, 0, 0};
        if (wi >= total) return r;
        const int plane = fast_div(wi, rcp_wpp_k), k = wi - plane * wpp;
        const int bi = fast_div(plane, p.rcp_cg), cl = plane - bi * p.Cg;
        long long e_lo, e_hi;
        plane_range(b0 + bi, cl, e_lo, e_hi);
        const long long w = (e_lo >> 5) + k;          // this lane's word
        const long long j0 = w << 5;
        if (j0 >= e_hi) return r;
        const ActRef m = act_meta(bitmap, offsets, j0, p.n_words, p.partial_blk);
        const uint32_t wq = static_cast<uint32_t>(w) & 3u;
        const uint32_t full = wq == 0 ? m.words.x : (wq == 1 ? m.words.y : (wq == 2 ? m.words.z : m.words.w));
        int lo = j0 < e_lo ? static_cast<int>(e_lo - j0) : 0;                 // first bit inside the range
        uint32_t bits = full & (0xFFFFFFFFu << lo);
        if (e_hi - j0 < 32) bits &= (1u << static_cast<int>(e_hi - j0)) - 1u;
        if (!bits) return r;
        lo = __ffs(bits) - 1;                         // the word's first kept bit inside the range
        uint32_t kfirst = m.base + __popc(full & ~(0xFFFFFFFFu << lo));
        kfirst += wq > 0 ? __popc(m.words.x) : 0u;
        kfirst += wq > 1 ? __popc(m.words.y) : 0u;
        kfirst += wq > 2 ? __popc(m.words.z) : 0u;
        const int rel = static_cast<int>(j0 + lo - e_lo);
        const int row0 = fast_div(rel, p.rcp_w);
        r.bits = bits; r.kfirst = kfirst; r.lo = lo; r.col0 = rel - row0 * p.W;
        r.pos = bi * p.a_floats + (cl * p.in_rows + (iy_lo - iy0) + row0) * p.Wp + 1 + r.col0;
        return r;
      };
      auto emit = [&](const WordRef& r) {
        uint32_t bits = r.bits;
        const int cnt = __popc(bits);
        for (int i = 0; i < cnt; i += 8) {
          float v[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            v[q] = 0.0f;
            if (i + q < cnt) {
              const long long kk = static_cast<long long>(r.kfirst) + i + q;
              v[q] = p.dt == 0 ? __ldg(reinterpret_cast<const float*>(values) + kk)
                               : __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(values) + kk)) << 16);
            }
          }
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            if (i + q < cnt) {
              const int e = __ffs(bits) - 1;
              bits &= bits - 1;
              // the tile's rows are 4 places longer than the input's: every wrap past the end of an
              // input row skips those
              const int d = e - r.lo;
              As[r.pos + d + 4 * fast_div(r.col0 + d, p.rcp_w)] = v[q];
            }
          }
        }
      };
      bool first = true;
      if (!dense) {
        for (int base = 0; base < total || first; base += 2 * kThreads) {
          const WordRef r0 = fetch(base + tid), r1 = fetch(base + kThreads + tid);
          if (first) {
            cp_async_wait_all();
            __syncthreads();                          // zeros in place, gradient planes landed
            first = false;
          }
          emit(r0);
          emit(r1);
        }
      } else {
        // Mostly kept words: a lane's 20-32 loads would each touch their own cache line.  Here lane j
        // fetches the metadata of word base + j and the warp then walks those 32 words with lane l
        // on bit l: one coalesced load per word, the words' loads independent of one another.
        const uint32_t lt = (1u << lane) - 1u;
        for (int base = warp * 32; base < total || first; base += kThreads) {
          const WordRef r = fetch(base + lane);
          if (first) {
            cp_async_wait_all();
            __syncthreads();
            first = false;
          }
          for (int i0 = 0; i0 < 32; i0 += 8) {        // eight words' loads in flight before the first store
            float v[8];
            int dst[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const uint32_t b = __shfl_sync(0xFFFFFFFFu, r.bits, i0 + q);
              const uint32_t k0 = __shfl_sync(0xFFFFFFFFu, r.kfirst, i0 + q);
              const int lo = __shfl_sync(0xFFFFFFFFu, r.lo, i0 + q);
              const int c0 = __shfl_sync(0xFFFFFFFFu, r.col0, i0 + q);
              const int ps = __shfl_sync(0xFFFFFFFFu, r.pos, i0 + q);
              dst[q] = -1;
              v[q] = 0.0f;
              if ((b >> lane) & 1u) {
                const long long kk = static_cast<long long>(k0) + __popc(b & lt);   // b starts at bit `lo`, whose rank is k0
                v[q] = p.dt == 0 ? __ldg(reinterpret_cast<const float*>(values) + kk)
                                 : __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(values) + kk)) << 16);
                const int d = static_cast<int>(lane) - lo;
                dst[q] = ps + d + 4 * fast_div(c0 + d, p.rcp_w);
              }
            }
#pragma unroll
            for (int q = 0; q < 8; ++q)
              if (dst[q] >= 0) As[dst[q]] = v[q];
          }
        }
      }
    }
    __syncthreads();
    // ---- products ----
    if (worker) {
      const int total = nb_here * n_strips;
      for (int fs = sidx; fs < total; fs += p.S) {
        const int bi = fast_div(fs, rcp_strips), st = fs - bi * n_strips;
        const int yl = fast_div(st, p.rcp_spr), x0 = (st - yl * spr) << 3;
        const float* gp = Gs + bi * p.g_floats + (ob * TO) * gpitch + yl * p.OW + x0;
        float g[TO][8];
#pragma unroll
        for (int o = 0; o < TO; ++o) {
          const float4 lo = *reinterpret_cast<const float4*>(gp + o * gpitch);
          const float4 hi = *reinterpret_cast<const float4*>(gp + o * gpitch + 4);
          g[o][0] = lo.x; g[o][1] = lo.y; g[o][2] = lo.z; g[o][3] = lo.w;
          g[o][4] = hi.x; g[o][5] = hi.y; g[o][6] = hi.z; g[o][7] = hi.w;
        }
        const float* abase = As + bi * p.a_floats + ((cb * TC) * p.in_rows + ST * yl) * p.Wp + ST * x0;
#pragma unroll
        for (int c = 0; c < TC; ++c) {
#pragma unroll
          for (int r = 0; r < 3; ++r) {
            const float* ap = abase + (c * p.in_rows + r) * p.Wp;
            float a[AW];
#pragma unroll
            for (int v = 0; v < AW / 4; ++v) {
              const float4 t = *reinterpret_cast<const float4*>(ap + 4 * v);
              a[4 * v] = t.x; a[4 * v + 1] = t.y; a[4 * v + 2] = t.z; a[4 * v + 3] = t.w;
            }
#pragma unroll
            for (int o = 0; o < TO; ++o)
#pragma unroll
              for (int s = 0; s < 3; ++s) {
                float f = acc[(o * TC + c) * 9 + r * 3 + s];
#pragma unroll
                for (int i = 0; i < 8; ++i) f = fmaf(g[o][i], a[ST * i + s], f);
                acc[(o * TC + c) * 9 + r * 3 + s] = f;
              }
          }
        }
      }
    }
  }
  // ---- add the strip splits of every unit in a fixed order, write this CTA's partial tile ----
  __syncthreads();
  float* red = sm;                                    // [thread][ACC]
  if (worker) {
#pragma unroll
    for (int i = 0; i < ACC; ++i) red[tid * ACC + i] = acc[i];
  }
  __syncthreads();
  const int ncol = p.Cg * 9;
  double* out = partial + static_cast<long long>(chunk * p.n_bands + band) * p.O * ncol;
  for (int i = tid; i < p.units * ACC; i += kThreads) {
    const int u = i / ACC, a = i - u * ACC;
    double s = 0.0;
    for (int sp = 0; sp < p.S; ++sp) s += static_cast<double>(red[(u * p.S + sp) * ACC + a]);
    const int uo = u / p.n_cb, uc = u - uo * p.n_cb;
    const int o = a / (TC * 9), rem = a - o * (TC * 9);
    const int c = rem / 9, rs = rem - c * 9;
    out[static_cast<long long>(grp * p.Og + uo * TO + o) * ncol + (uc * TC + c) * 9 + rs] = s;
  }
}

// dw[i] (= [o][c'][r][s] flattened, the layout of the partial tiles) = sum of the partial tiles in
// index order, in double.
__global__ void __launch_bounds__(256)
grouped_reduce_kernel(const double* __restrict__ partial, long long mn, int parts, float* __restrict__ dw,
                      int accumulate) {
  const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= mn) return;
  double s = 0.0;
  for (int z = 0; z < parts; ++z) s += partial[z * mn + i];
  dw[i] = accumulate ? dw[i] + static_cast<float>(s) : static_cast<float>(s);
}

bool plan_grouped(const surgeon_layer_desc& d, GroupedParams* out) {
  if (d.kind != 1 || d.groups <= 1 || d.c_in % d.groups || d.c_out % d.groups) return false;
  GroupedParams p{};
  p.B = d.batch; p.C = d.c_in; p.H = d.h; p.W = d.w; p.O = d.c_out;
  p.KH = d.kh; p.KW = d.kw; p.stride = d.stride; p.pad = d.pad;
  p.OH = (d.h + 2 * d.pad - d.kh) / d.stride + 1;
  p.OW = (d.w + 2 * d.pad - d.kw) / d.stride + 1;
  p.G = d.groups; p.Cg = d.c_in / d.groups; p.Og = d.c_out / d.groups;
  p.ncol = p.Cg * p.KH * p.KW;
  p.n_ob = (p.Og + kRO - 1) / kRO;
  p.n_units = p.n_ob * p.ncol;
  if (p.n_units > kUMax * kThreads) return false;
  // few units: the threads left over split the positions among them
  p.S = p.n_units >= kThreads ? 1 : kThreads / p.n_units;
  p.Wp = (p.OW - 1) * p.stride + p.KW;
  if (p.Wp < p.W + p.pad) p.Wp = p.W + p.pad;          // every input column has a place
  // the tallest band whose two tiles (and the final sum of the splits) fit the budget
  const long long red_bytes = static_cast<long long>(p.S) * p.n_units * kRO * 8;
  if (red_bytes > kSmemBudget) return false;
  int band = p.OH;
  for (;; --band) {
    if (band < 1) return false;
    const long long in_rows = static_cast<long long>(band - 1) * p.stride + p.KH;
    const long long a = (static_cast<long long>(p.Cg) * in_rows * p.Wp + 3) / 4 * 4;   // the gradient tile stays 16-byte aligned
    const long long g = static_cast<long long>(p.n_ob) * kRO * band * p.OW;
    if ((a + g) * 4 <= kSmemBudget) { p.in_rows = static_cast<int>(in_rows); p.a_floats = static_cast<int>(a); p.g_floats = static_cast<int>(g); break; }
  }
  p.band = band;
  p.n_bands = (p.OH + band - 1) / band;
  // images per round: as many as keep the tiles within 48 KB (several CTAs share an SM), up to 8
  p.nb = static_cast<int>((48 * 1024) / (static_cast<long long>(p.a_floats + p.g_floats) * 4));
  if (p.nb > 8) p.nb = 8;
  if (p.nb < 1) p.nb = 1;
  // image chunks: about four CTAs per SM in all
  const long long per_chunk0 = static_cast<long long>(p.G) * p.n_bands;
  long long chunks = (4LL * sm_count() + per_chunk0 - 1) / per_chunk0;
  if (chunks > p.B) chunks = p.B;
  if (chunks < 1) chunks = 1;
  if (chunks > 65535) chunks = 65535;
  p.imgs_per_chunk = static_cast<int>((p.B + chunks - 1) / chunks);
  p.chunks = (p.B + p.imgs_per_chunk - 1) / p.imgs_per_chunk;
  if (p.n_bands > 65535 || p.G > 2147483647) return false;
  *out = p;
  return true;
}

// The register-tiled kernel's launch: 3x3, padding 1, stride 1 or 2, even maps under stride 2, output
// rows a multiple of 8 wide.  TO / TC = the largest of 4, 2, 1 that divide the group's output /
// input channels with TO * TC <= 4.
struct Grouped3Tile { int to, tc; };
bool plan_grouped3(const surgeon_layer_desc& d, Grouped3Params* out, Grouped3Tile* tile) {
  if (d.kind != 1 || d.groups <= 1 || d.c_in % d.groups || d.c_out % d.groups) return false;
  if (d.kh != 3 || d.kw != 3 || d.pad != 1 || (d.stride != 1 && d.stride != 2)) return false;
  if (d.stride == 2 && ((d.h | d.w) & 1)) return false;
  Grouped3Params p{};
  p.B = d.batch; p.C = d.c_in; p.H = d.h; p.W = d.w; p.O = d.c_out;
  p.OH = (d.h + 2 - 3) / d.stride + 1;
  p.OW = (d.w + 2 - 3) / d.stride + 1;
  if (p.OW % 8 || p.OW < 8) return false;
  p.G = d.groups; p.Cg = d.c_in / d.groups; p.Og = d.c_out / d.groups;
  int to = p.Og % 4 == 0 ? 4 : (p.Og % 2 == 0 ? 2 : 1);
  int tc = p.Cg % 4 == 0 ? 4 : (p.Cg % 2 == 0 ? 2 : 1);
  while (to * tc > kG3MaxTile) { if (tc >= to) tc >>= 1; else to >>= 1; }
  p.n_cb = p.Cg / tc;
  p.units = (p.Og / to) * p.n_cb;
  if (p.units > kThreads) return false;
  p.S = kThreads / p.units;
  p.Wp = p.W + 4;                                   // column 0 = input column -1; 16-byte aligned rows
  const long long red_bytes = static_cast<long long>(kThreads) * to * tc * 9 * 4;
  int band = p.OH;
  for (;; --band) {
    if (band < 1) return false;
    const long long in_rows = static_cast<long long>(band - 1) * d.stride + 3;
    const long long a = static_cast<long long>(p.Cg) * in_rows * p.Wp;
    const long long g = static_cast<long long>(p.Og) * band * p.OW;
    if ((a + g) * 4 <= kG3Smem) { p.in_rows = static_cast<int>(in_rows); p.a_floats = static_cast<int>(a); p.g_floats = static_cast<int>(g); break; }
  }
  if (red_bytes > kG3Smem) return false;
  p.band = band;
  p.n_bands = (p.OH + band - 1) / band;
  p.nb = static_cast<int>(kG3Smem / (static_cast<long long>(p.a_floats + p.g_floats) * 4));
  if (p.nb > 8) p.nb = 8;
  // image chunks: one resident wave of CTAs, and no thread adds more than kTermsPerThread terms in fp32
  const long long per_chunk0 = static_cast<long long>(p.G) * p.n_bands;
  long long chunks = (static_cast<long long>(kG3CtasPerSm) * sm_count()) / per_chunk0;
  const long long strips = static_cast<long long>(band) * (p.OW / 8);
  const long long max_imgs = (static_cast<long long>(kTermsPerThread) / 8) * p.S / strips;   // strips per thread = imgs * strips / S
  if (max_imgs < 1) return false;
  if (chunks < (p.B + max_imgs - 1) / max_imgs) chunks = (p.B + max_imgs - 1) / max_imgs;
  if (chunks > p.B) chunks = p.B;
  if (chunks < 1) chunks = 1;
  if (chunks > 65535 || p.n_bands > 65535) return false;
  p.imgs_per_chunk = static_cast<int>((p.B + chunks - 1) / chunks);
  p.chunks = (p.B + p.imgs_per_chunk - 1) / p.imgs_per_chunk;
  if (p.nb > p.imgs_per_chunk) p.nb = p.imgs_per_chunk;
  p.rcp_cg = div_magic(p.Cg);
  p.rcp_spr = div_magic(p.OW / 8);
  p.rcp_w = div_magic(p.W);
  *out = p;
  tile->to = to; tile->tc = tc;
  return true;
}
size_t grouped3_smem(const Grouped3Params& p, const Grouped3Tile& t) {
  const size_t tiles = static_cast<size_t>(p.nb) * (p.a_floats + p.g_floats) * 4;
  const size_t red = static_cast<size_t>(kThreads) * t.to * t.tc * 9 * 4;
  return (tiles > red ? tiles : red) + 16;
}

size_t grouped_smem(const GroupedParams& p) {
  const size_t tiles = static_cast<size_t>(p.nb) * (p.a_floats + p.g_floats) * 4;
  const size_t red = static_cast<size_t>(p.S) * p.n_units * kRO * 8;
  return (tiles > red ? tiles : red) + 16;
}

}  // namespace

size_t weight_grad_grouped_workspace(const surgeon_layer_desc& d) {
  Grouped3Params p3;
  Grouped3Tile t3;
  if (plan_grouped3(d, &p3, &t3))
    return static_cast<size_t>(p3.chunks) * p3.n_bands * p3.O * p3.Cg * 9 * sizeof(double);
  GroupedParams p;
  if (!plan_grouped(d, &p)) return 0;
  return static_cast<size_t>(p.chunks) * p.n_bands * p.O * p.ncol * sizeof(double);
}

cudaError_t launch_weight_grad_grouped(const surgeon_compressed& act, const surgeon_layer_desc& d,
                                       const float* grad_out, float* dw, int accumulate,
                                       void* workspace, cudaStream_t stream) {
  double* partial = static_cast<double*>(workspace);
  Grouped3Params p3;
  Grouped3Tile t3;
  if (plan_grouped3(d, &p3, &t3)) {
    p3.dt = act.dt;
    p3.n_words = (act.n + 31) / 32;
    p3.n = act.n;
    p3.n_blocks = (act.n + SURGEON_BLOCK - 1) / SURGEON_BLOCK;
    p3.partial_blk = (act.n % SURGEON_BLOCK) ? static_cast<unsigned>(act.n / SURGEON_BLOCK) : 0xFFFFFFFFu;
    const size_t smem = grouped3_smem(p3, t3);
    const dim3 grid(p3.G, p3.n_bands, p3.chunks);
    cudaError_t e = cudaSuccess;
    auto launch = [&](auto kernel) {
      e = allow_dynamic_smem(reinterpret_cast<const void*>(kernel), static_cast<int>(smem));
      if (e == cudaSuccess)
        kernel<<<grid, kThreads, smem, stream>>>(act.bitmap, act.values, act.block_offsets, grad_out, partial, p3);
    };
    auto by_stride = [&](auto to, auto tc) {
      constexpr int TO = decltype(to)::value, TC = decltype(tc)::value;
      if (d.stride == 1) launch(dw_grouped3_kernel<TO, TC, 1>);
      else launch(dw_grouped3_kernel<TO, TC, 2>);
    };
    using I1 = std::integral_constant<int, 1>;
    using I2 = std::integral_constant<int, 2>;
    using I4 = std::integral_constant<int, 4>;
    if (t3.to == 4 && t3.tc == 2) by_stride(I4{}, I2{});
    else if (t3.to == 2 && t3.tc == 4) by_stride(I2{}, I4{});
    else if (t3.to == 4) by_stride(I4{}, I1{});
    else if (t3.to == 2 && t3.tc == 2) by_stride(I2{}, I2{});
    else if (t3.to == 2) by_stride(I2{}, I1{});
    else if (t3.tc == 4) by_stride(I1{}, I4{});
    else if (t3.tc == 2) by_stride(I1{}, I2{});
    else by_stride(I1{}, I1{});
    if (e != cudaSuccess) return e;
    const long long mn = static_cast<long long>(p3.O) * p3.Cg * 9;
    grouped_reduce_kernel<<<static_cast<unsigned>((mn + 255) / 256), 256, 0, stream>>>(partial, mn, p3.chunks * p3.n_bands,
                                                                                   dw, accumulate);
    note_launches(2);
    return cudaGetLastError();
  }
  GroupedParams p;
  if (!plan_grouped(d, &p)) return cudaErrorNotSupported;
  p.n_words = (act.n + 31) / 32;
  p.partial_blk = (act.n % SURGEON_BLOCK) ? static_cast<unsigned>(act.n / SURGEON_BLOCK) : 0xFFFFFFFFu;
  const size_t smem = grouped_smem(p);
  dim3 grid(p.G, p.n_bands, p.chunks);
  cudaError_t e = cudaSuccess;
  auto launch = [&](auto kernel) {
    e = allow_dynamic_smem(reinterpret_cast<const void*>(kernel), static_cast<int>(smem));
    if (e == cudaSuccess)
      kernel<<<grid, kThreads, smem, stream>>>(act.bitmap, act.values, act.block_offsets, grad_out, partial, p);
  };
  const int ro = p.Og > 4 ? 8 : (p.Og > 2 ? 4 : p.Og);       // 1, 2, 4 or 8 accumulators per unit
  const bool quad = (p.OW % 4) == 0;
  const int um = p.n_units <= kThreads ? 1 : (p.n_units <= 2 * kThreads ? 2 : 4);
  auto by_um = [&](auto dt, auto ro_c, auto pv) {
    constexpr int D = decltype(dt)::value, R = decltype(ro_c)::value, V = decltype(pv)::value;
    if (um == 1) launch(dw_grouped_kernel<D, R, V, 1>);
    else if (um == 2) launch(dw_grouped_kernel<D, R, V, 2>);
    else launch(dw_grouped_kernel<D, R, V, 4>);
  };
  auto by_pv = [&](auto dt, auto ro_c) {
    if (quad) by_um(dt, ro_c, std::integral_constant<int, 4>{});
    else by_um(dt, ro_c, std::integral_constant<int, 1>{});
  };
  auto by_ro = [&](auto dt) {
    if (ro == 1) by_pv(dt, std::integral_constant<int, 1>{});
    else if (ro == 2) by_pv(dt, std::integral_constant<int, 2>{});
    else if (ro == 4) by_pv(dt, std::integral_constant<int, 4>{});
    else by_pv(dt, std::integral_constant<int, 8>{});
  };
  if (act.dt == 0) by_ro(std::integral_constant<int, 0>{});
  else by_ro(std::integral_constant<int, 1>{});
  if (e != cudaSuccess) return e;
  const long long mn = static_cast<long long>(p.O) * p.ncol;
  grouped_reduce_kernel<<<static_cast<unsigned>((mn + 255) / 256), 256, 0, stream>>>(partial, mn, p.chunks * p.n_bands, dw,
                                                                                 accumulate);
  note_launches(2);
  return cudaGetLastError();
}

}  // namespace surgeon

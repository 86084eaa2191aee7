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

size_t grouped_smem(const GroupedParams& p) {
  const size_t tiles = static_cast<size_t>(p.nb) * (p.a_floats + p.g_floats) * 4;
  const size_t red = static_cast<size_t>(p.S) * p.n_units * kRO * 8;
  return (tiles > red ? tiles : red) + 16;
}

}  // namespace

size_t weight_grad_grouped_workspace(const surgeon_layer_desc& d) {
  GroupedParams p;
  if (!plan_grouped(d, &p)) return 0;
  return static_cast<size_t>(p.chunks) * p.n_bands * p.O * p.ncol * sizeof(double);
}

cudaError_t launch_weight_grad_grouped(const surgeon_compressed& act, const surgeon_layer_desc& d,
                                       const float* grad_out, float* dw, int accumulate,
                                       void* workspace, cudaStream_t stream) {
  GroupedParams p;
  if (!plan_grouped(d, &p)) return cudaErrorNotSupported;
  double* partial = static_cast<double*>(workspace);
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

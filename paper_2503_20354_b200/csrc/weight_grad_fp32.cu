// fp32 CUDA-core path of surgeon_weight_grad (Algorithm 1: Reshape and gradient steps, Eq. 2).
//
// Implicit GEMM  dW[m, nn] = sum_k G[k, m] * Acol[k, nn]  with m = output channel,
// nn = (c, r, s) and k = (b, y, x) (or the row t of a linear layer).  The im2col operand is
// rebuilt from the compressed store element by element (bitmap bit -> rank in the packed
// vector -> value), straight into shared memory; the dense activation never exists in global
// memory.  The reduction is cut into chunks of kChunk terms; every chunk is summed in fp32 in
// a fixed order, and the chunk sums are added in double in a fixed order by a second kernel, so
// the result is reproducible and stays within ~3e-6 relative error of exact arithmetic.
#include "surgeon_internal.cuh"

namespace surgeon {

namespace {

constexpr int TM = 64, TN = 64, TK = 16;
constexpr int kChunk = 2048;

struct Geom {
  int kind, B, C, H, W, O, KH, KW, stride, pad, OH, OW;
  long long M, N, K;  // GEMM extents
};

__host__ __device__ inline Geom make_geom(const surgeon_layer_desc& d) {
  Geom g;
  g.kind = d.kind; g.B = d.batch; g.C = d.c_in; g.H = d.h; g.W = d.w; g.O = d.c_out;
  g.KH = d.kh; g.KW = d.kw; g.stride = d.stride; g.pad = d.pad;
  g.OH = (d.h + 2 * d.pad - d.kh) / d.stride + 1;
  g.OW = (d.w + 2 * d.pad - d.kw) / d.stride + 1;
  g.M = d.c_out;
  g.N = static_cast<long long>(d.c_in) * d.kh * d.kw;
  g.K = static_cast<long long>(d.batch) * g.OH * g.OW;
  return g;
}

// Value of the pruned activation at flat index j, widened to fp32.
template <int DT>
__device__ __forceinline__ float fetch_act(const uint32_t* __restrict__ bitmap,
                                           const void* __restrict__ values,
                                           const uint32_t* __restrict__ offsets,
                                           long long j) {
  const long long wi = j >> 5;
  const uint32_t w = __ldg(bitmap + wi);
  const uint32_t bit = static_cast<uint32_t>(j) & 31u;
  if (!((w >> bit) & 1u)) return 0.0f;
  const long long blk = j >> kBlockShift;
  long long r = static_cast<long long>(__ldg(offsets + blk));
  for (long long t = blk * kBlockWords; t < wi; ++t) r += __popc(__ldg(bitmap + t));
  r += __popc(w & ((1u << bit) - 1u));
  if (DT == 0) return __ldg(reinterpret_cast<const float*>(values) + r);
  const uint32_t h = __ldg(reinterpret_cast<const unsigned short*>(values) + r);
  return __uint_as_float(h << 16);
}

template <int DT>
__global__ void __launch_bounds__(256)
dw_fp32_kernel(const uint32_t* __restrict__ bitmap, const void* __restrict__ values,
               const uint32_t* __restrict__ offsets, const float* __restrict__ grad,
               float* __restrict__ partial, Geom g) {
  __shared__ float Gs[TK][TM + 4];
  __shared__ float As[TK][TN + 4];
  const int tid = threadIdx.x;
  const long long m0 = static_cast<long long>(blockIdx.y) * TM;
  const long long n0 = static_cast<long long>(blockIdx.x) * TN;
  const long long k_begin = static_cast<long long>(blockIdx.z) * kChunk;
  const long long k_end = (k_begin + kChunk < g.K) ? k_begin + kChunk : g.K;
  const int P = g.OH * g.OW;
  const int RS = g.KH * g.KW;

  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.0f;

  const int ty = tid >> 4, tx = tid & 15;
  for (long long k0 = k_begin; k0 < k_end; k0 += TK) {
    // ---- stage the gradient tile ----
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int kk, mm;
      if (g.kind == 1) { kk = tid & 15; mm = (tid >> 4) + 16 * i; }   // k is contiguous (NCHW)
      else { mm = tid & 63; kk = (tid >> 6) + 4 * i; }                 // m is contiguous ([T,O])
      const long long k = k0 + kk, m = m0 + mm;
      float v = 0.0f;
      if (k < k_end && m < g.M) {
        if (g.kind == 1) {
          const long long b = k / P;
          const long long sp = k - b * P;
          v = __ldg(grad + (b * g.O + m) * P + sp);
        } else {
          v = __ldg(grad + k * g.O + m);
        }
      }
      Gs[kk][mm] = v;
    }
    // ---- rebuild the im2col tile from the compressed store ----
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int kk, nn;
      if (g.kind == 1) { kk = tid & 15; nn = (tid >> 4) + 16 * i; }
      else { nn = tid & 63; kk = (tid >> 6) + 4 * i; }
      const long long k = k0 + kk, col = n0 + nn;
      float v = 0.0f;
      if (k < k_end && col < g.N) {
        if (g.kind == 1) {
          const int c = static_cast<int>(col / RS);
          const int rs = static_cast<int>(col - static_cast<long long>(c) * RS);
          const int r = rs / g.KW, s = rs - r * g.KW;
          const long long b = k / P;
          const int sp = static_cast<int>(k - b * P);
          const int y = sp / g.OW, xo = sp - y * g.OW;
          const int iy = y * g.stride + r - g.pad;
          const int ix = xo * g.stride + s - g.pad;
          if (iy >= 0 && iy < g.H && ix >= 0 && ix < g.W)
            v = fetch_act<DT>(bitmap, values, offsets,
                              ((b * g.C + c) * g.H + iy) * g.W + ix);
        } else {
          v = fetch_act<DT>(bitmap, values, offsets, k * g.C + col);
        }
      }
      As[kk][nn] = v;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      const float4 gv = *reinterpret_cast<const float4*>(&Gs[kk][ty * 4]);
      const float4 av = *reinterpret_cast<const float4*>(&As[kk][tx * 4]);
      const float gr[4] = {gv.x, gv.y, gv.z, gv.w};
      const float ar[4] = {av.x, av.y, av.z, av.w};
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(gr[a], ar[b], acc[a][b]);
    }
    __syncthreads();
  }
  float* out = partial + static_cast<long long>(blockIdx.z) * g.M * g.N;
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    const long long m = m0 + ty * 4 + a;
    if (m >= g.M) continue;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const long long col = n0 + tx * 4 + b;
      if (col < g.N) out[m * g.N + col] = acc[a][b];
    }
  }
}

__global__ void __launch_bounds__(256)
reduce_chunks_kernel(const float* __restrict__ partial, long long mn, int chunks,
                     float* __restrict__ dw, int accumulate) {
  const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= mn) return;
  double s = 0.0;
  for (int z = 0; z < chunks; ++z) s += static_cast<double>(partial[z * mn + i]);
  dw[i] = accumulate ? static_cast<float>(static_cast<double>(dw[i]) + s) : static_cast<float>(s);
}

}  // namespace

size_t weight_grad_fp32_workspace(const surgeon_layer_desc& d) {
  const Geom g = make_geom(d);
  const long long chunks = (g.K + kChunk - 1) / kChunk;
  return static_cast<size_t>(chunks < 1 ? 1 : chunks) * g.M * g.N * sizeof(float);
}

cudaError_t launch_weight_grad_fp32(const surgeon_compressed& act, const surgeon_layer_desc& d,
                                    const float* grad_out, float* dw, int accumulate,
                                    void* workspace, cudaStream_t stream) {
  const Geom g = make_geom(d);
  const long long chunks = (g.K + kChunk - 1) / kChunk;
  float* partial = static_cast<float*>(workspace);
  const uint32_t* offs = act.block_offsets;
  if (chunks > 0) {
    dim3 grid(static_cast<unsigned>((g.N + TN - 1) / TN), static_cast<unsigned>((g.M + TM - 1) / TM),
              static_cast<unsigned>(chunks));
    if (act.dt == 0)
      dw_fp32_kernel<0><<<grid, 256, 0, stream>>>(act.bitmap, act.values, offs, grad_out, partial, g);
    else
      dw_fp32_kernel<1><<<grid, 256, 0, stream>>>(act.bitmap, act.values, offs, grad_out, partial, g);
    note_launches(1);
  }
  const long long mn = g.M * g.N;
  reduce_chunks_kernel<<<static_cast<unsigned>((mn + 255) / 256), 256, 0, stream>>>(
      partial, mn, static_cast<int>(chunks), dw, accumulate);
  note_launches(1);
  return cudaGetLastError();
}

}  // namespace surgeon

// Gradient Importance of one layer (Eq. 4): G = sqrt( sum_j (dw_j)^2 / N ).
//
// Two small kernels, both with a fixed summation order, so the result does not depend on
// scheduling.  The first cuts dw into at most kGiBlocks contiguous slices, one per CTA: a thread
// adds the squares of every 256th element of its slice in double (a product of two fp32 values is
// exact in double), the CTA adds its threads' sums in a fixed tree and writes one partial.  The
// second adds the partials in index order, divides by N and takes the root.
#include "surgeon_internal.cuh"

namespace surgeon {

namespace {

constexpr int kGiThreads = 256;
constexpr int kGiBlocks = 1024;       // partials fit SURGEON_GI_WORKSPACE_BYTES
static_assert(kGiBlocks * sizeof(double) <= SURGEON_GI_WORKSPACE_BYTES, "partials fit the scratch");

// Sum of the 256 threads' values in a fixed order: lanes by shuffle tree, warps in index order.
__device__ __forceinline__ double block_sum_fixed(double v, double* s_warp) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xFFFFFFFFu, v, o);
  if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = v;
  __syncthreads();
  double t = 0.0;
  if (threadIdx.x == 0) {
    for (int w = 0; w < kGiThreads / 32; ++w) t += s_warp[w];
  }
  return t;   // valid in thread 0
}

__global__ void __launch_bounds__(kGiThreads)
gi_partial_kernel(const float* __restrict__ dw, long long n, long long per_block,
                  double* __restrict__ partial) {
  __shared__ double s_warp[kGiThreads / 32];
  const long long begin = static_cast<long long>(blockIdx.x) * per_block;
  const long long end = begin + per_block < n ? begin + per_block : n;
  double acc = 0.0;
  for (long long j = begin + threadIdx.x; j < end; j += kGiThreads) {
    const double v = static_cast<double>(__ldg(dw + j));
    acc += v * v;
  }
  const double t = block_sum_fixed(acc, s_warp);
  if (threadIdx.x == 0) partial[blockIdx.x] = t;
}

__global__ void __launch_bounds__(kGiThreads)
gi_final_kernel(const double* __restrict__ partial, int n_partials, long long n,
                double* __restrict__ gi_out) {
  __shared__ double s_warp[kGiThreads / 32];
  // thread t adds the partials t, t + 256, ... in that order
  double acc = 0.0;
  for (int i = threadIdx.x; i < n_partials; i += kGiThreads) acc += partial[i];
  const double t = block_sum_fixed(acc, s_warp);
  if (threadIdx.x == 0) *gi_out = n > 0 ? sqrt(t / static_cast<double>(n)) : 0.0;
}

}  // namespace

cudaError_t launch_gradient_importance(const float* dw, long long n, double* gi_out,
                                       void* workspace, cudaStream_t stream) {
  double* partial = static_cast<double*>(workspace);
  int blocks = 0;
  if (n > 0) {
    // slices of whole multiples of 256 elements, at least 4096 each
    long long per_block = (n + kGiBlocks - 1) / kGiBlocks;
    if (per_block < 4096) per_block = 4096;
    per_block = (per_block + kGiThreads - 1) / kGiThreads * kGiThreads;
    blocks = static_cast<int>((n + per_block - 1) / per_block);
    gi_partial_kernel<<<blocks, kGiThreads, 0, stream>>>(dw, n, per_block, partial);
    note_launches(1);
  }
  gi_final_kernel<<<1, kGiThreads, 0, stream>>>(partial, blocks, n, gi_out);
  note_launches(1);
  return cudaGetLastError();
}

}  // namespace surgeon

// Threshold select and compaction kernels of surgeon_prune_compact, and surgeon_decompress.
//
// Algorithm 1: prune step: the kept set of a layer is its n_keep largest-magnitude elements, ties
// at the threshold broken by lowest flat index.  Its decompose step / Section 4.2: the pruned activation is
// cached as the vector of kept elements plus one index bit per element.
//
//   select  : radix select on the magnitude key.  Each pass histograms one digit of the keys
//             that still match the prefix found so far; the last CTA to finish a pass scans the
//             histogram from the top and fixes the next digit.  The result (threshold key,
//             count above it, tie quota) is exact and unique, so it is deterministic whatever
//             the atomics' order.
//   compact : one streaming pass.  A warp owns one SURGEON_BLOCK (1024 elements); ballots turn
//             the per-element decisions directly into bitmap words; an ordered exclusive scan
//             over tiles (decoupled look-back on one packed 64-bit word per tile) gives every
//             tile its position in the packed vector and its rank among the ties.
#include "surgeon_internal.cuh"

namespace surgeon {

namespace {

constexpr int kHistThreads = 512;

template <int DT, int SHIFT, int BITS, bool LAST>
__global__ void __launch_bounds__(kHistThreads)
radix_hist_kernel(const void* __restrict__ xv, long long n, long long k_total, int pass,
                  SelectState* __restrict__ st, uint32_t* __restrict__ ghist,
                  surgeon_header* __restrict__ hdr) {
  using E = typename Elem<DT>::type;
  constexpr uint32_t kMask = Elem<DT>::kKeyMask;
  constexpr int NB = 1 << BITS;
  constexpr int HI = SHIFT + BITS;  // bits above this position are the prefix
  __shared__ uint32_t hist[NB];
  __shared__ bool s_last;
  const int tid = threadIdx.x;
  for (int i = tid; i < NB; i += kHistThreads) hist[i] = 0;
  __syncthreads();

  const uint32_t prefix = st->prefix;
  const uint32_t want = (HI < 32) ? (prefix >> (HI & 31)) : 0u;
  uint32_t zero_cnt = 0;  // digit 0 is counted in a register: post-ReLU data is half zeros
  auto add = [&](uint32_t key) {
    const uint32_t hi = (HI < 32) ? (key >> (HI & 31)) : 0u;
    if (hi == want) {
      const uint32_t d = (key >> SHIFT) & (NB - 1);
      if (d == 0) ++zero_cnt;
      else atomicAdd(&hist[d], 1u);
    }
  };

  constexpr int VEC = 16 / sizeof(E);
  const long long nvec = n / VEC;
  const uint4* __restrict__ xq = reinterpret_cast<const uint4*>(xv);
  const long long stride = static_cast<long long>(gridDim.x) * kHistThreads;
  for (long long v = static_cast<long long>(blockIdx.x) * kHistThreads + tid; v < nvec;
       v += stride) {
    const uint4 q = __ldg(xq + v);
    if (DT == 0) {
      add(q.x & kMask); add(q.y & kMask); add(q.z & kMask); add(q.w & kMask);
    } else {
      add(q.x & kMask); add((q.x >> 16) & kMask);
      add(q.y & kMask); add((q.y >> 16) & kMask);
      add(q.z & kMask); add((q.z >> 16) & kMask);
      add(q.w & kMask); add((q.w >> 16) & kMask);
    }
  }
  if (blockIdx.x == 0) {
    const E* __restrict__ xe = reinterpret_cast<const E*>(xv);
    for (long long j = nvec * VEC + tid; j < n; j += kHistThreads)
      add(static_cast<uint32_t>(xe[j]) & kMask);
  }
  zero_cnt = warp_sum(zero_cnt);
  if (lane_id() == 0 && zero_cnt) atomicAdd(&hist[0], zero_cnt);
  __syncthreads();
  for (int i = tid; i < NB; i += kHistThreads)
    if (hist[i]) atomicAdd(&ghist[i], hist[i]);
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const uint32_t t = atomicAdd(&st->pass_ticket[pass], 1u);
    s_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (!s_last) return;

  // Last CTA of the pass: every other CTA's histogram is in ghist.
  __threadfence();
  for (int i = tid; i < NB; i += kHistThreads) hist[i] = __ldcg(ghist + i);
  __syncthreads();
  if (tid == 0) {
    const long long kr = (pass == 0) ? k_total : st->k_remaining;
    long long above = 0;
    int b = NB - 1;
    for (; b > 0; --b) {
      const long long c = hist[b];
      if (above + c >= kr) break;
      above += c;
    }
    const uint32_t new_prefix = prefix | (static_cast<uint32_t>(b) << SHIFT);
    const long long ng = ((pass == 0) ? 0 : st->n_greater) + above;
    st->prefix = new_prefix;
    st->k_remaining = kr - above;
    st->n_greater = ng;
    if (LAST) {
      hdr->threshold_key = new_prefix;
      hdr->n_keep = k_total;
      hdr->n_greater = ng;
      hdr->tie_quota = k_total - ng;
    }
    __threadfence();
  }
}

// n_keep == 0 (ratio 1, or an empty tensor): nothing to select.
__global__ void header_empty_kernel(surgeon_header* hdr, uint32_t sentinel) {
  hdr->threshold_key = sentinel;
  hdr->n_keep = 0;
  hdr->n_greater = 0;
  hdr->tie_quota = 0;
}

// ---- compaction -----------------------------------------------------------------------------

constexpr unsigned long long kStAggregate = 1ull << 62;
constexpr unsigned long long kStPrefix = 2ull << 62;
constexpr unsigned long long kCountMask = 0x7FFFFFFFull;
constexpr uint32_t kSpinCap = 1u << 22;  // bounded look-back wait (each poll sleeps ~50 ns)

__device__ __forceinline__ unsigned long long pack_counts(unsigned long long gt,
                                                          unsigned long long eq) {
  return (gt << 31) | eq;
}

// Keep only the lowest `allowed` set bits of `m`.
__device__ __forceinline__ uint32_t lowest_set_bits(uint32_t m, long long allowed) {
  if (allowed <= 0) return 0u;
  int extra = __popc(m) - static_cast<int>(allowed < 32 ? allowed : 32);
  while (extra > 0) {
    m &= ~(0x80000000u >> __clz(m));
    --extra;
  }
  return m;
}

template <int DT>
__global__ void __launch_bounds__(256)
compact_kernel(const void* __restrict__ xv, long long n, surgeon_header* __restrict__ hdr,
               uint32_t* __restrict__ bitmap, void* __restrict__ values_v,
               unsigned long long* __restrict__ offsets, uint32_t* __restrict__ ticket,
               unsigned long long* __restrict__ tile_state, int num_tiles) {
  using E = typename Elem<DT>::type;
  constexpr uint32_t kMask = Elem<DT>::kKeyMask;
  const E* __restrict__ x = reinterpret_cast<const E*>(xv);
  E* __restrict__ values = reinterpret_cast<E*>(values_v);
  __shared__ uint32_t s_gt[kTileBlocks], s_eq[kTileBlocks];
  __shared__ int s_tile;
  __shared__ unsigned long long s_excl;

  const uint32_t tau = hdr->threshold_key;
  const long long quota = hdr->tie_quota;
  const int tid = threadIdx.x;
  const uint32_t lane = lane_id();
  const int warp = tid >> 5;
  const long long n_blocks = (n + SURGEON_BLOCK - 1) / SURGEON_BLOCK;
  const long long n_words = (n + 31) / 32;

  while (true) {
    if (tid == 0) s_tile = static_cast<int>(atomicAdd(ticket, 1u));
    __syncthreads();
    const int tile = s_tile;
    if (tile >= num_tiles) break;

    const long long block = static_cast<long long>(tile) * kTileBlocks + warp;
    const long long base = block * SURGEON_BLOCK;
    E xs[32];
    uint32_t gt_word = 0, eq_word = 0;  // lane i ends up holding the masks of word i
    if (base < n) {
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const long long idx = base + i * 32 + lane;
        xs[i] = (idx < n) ? x[idx] : static_cast<E>(0);
      }
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const long long idx = base + i * 32 + lane;
        const uint32_t key = static_cast<uint32_t>(xs[i]) & kMask;
        const bool valid = idx < n;
        const uint32_t g = __ballot_sync(0xFFFFFFFFu, valid && key > tau);
        const uint32_t e = __ballot_sync(0xFFFFFFFFu, valid && key == tau);
        if (lane == static_cast<uint32_t>(i)) { gt_word = g; eq_word = e; }
      }
    }
    const uint32_t gt_warp = warp_sum(__popc(gt_word));
    const uint32_t eq_warp = warp_sum(__popc(eq_word));
    if (lane == 0) { s_gt[warp] = gt_warp; s_eq[warp] = eq_warp; }
    __syncthreads();

    if (tid == 0) {
      unsigned long long gt_tile = 0, eq_tile = 0;
#pragma unroll
      for (int w = 0; w < kTileBlocks; ++w) { gt_tile += s_gt[w]; eq_tile += s_eq[w]; }
      const unsigned long long mine = pack_counts(gt_tile, eq_tile);
      volatile unsigned long long* vs = tile_state;
      unsigned long long excl = 0;
      if (tile == 0) {
        vs[0] = kStPrefix | mine;
      } else {
        vs[tile] = kStAggregate | mine;
        int p = tile - 1;
        while (true) {
          unsigned long long v = vs[p];
          uint32_t spins = 0;
          while ((v >> 62) == 0 && spins < kSpinCap) {
            __nanosleep(50);
            v = vs[p];
            ++spins;
          }
          if ((v >> 62) == 0) {  // gave up: report, stop waiting, let successors pass
            atomicMax(&hdr->status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
            break;
          }
          excl += v & ~(3ull << 62);
          if ((v >> 62) == 2 || p == 0) break;
          --p;
        }
        vs[tile] = kStPrefix | (excl + mine);
      }
      s_excl = excl;
    }
    __syncthreads();

    const unsigned long long excl = s_excl;
    long long gt_before = static_cast<long long>(excl >> 31);
    long long eq_before = static_cast<long long>(excl & kCountMask);
#pragma unroll
    for (int w = 0; w < kTileBlocks; ++w) {
      if (w < warp) { gt_before += s_gt[w]; eq_before += s_eq[w]; }
    }
    // kept before this warp's block = all greater + the ties that fit the quota
    const long long kept_before = gt_before + (eq_before < quota ? eq_before : quota);

    if (base < n) {
      // rank of this word's first tie among all ties of the tensor
      const long long eq_word_before = eq_before + warp_excl_scan(__popc(eq_word));
      const uint32_t keep_word = gt_word | lowest_set_bits(eq_word, quota - eq_word_before);
      const uint32_t kc = __popc(keep_word);
      const uint32_t word_excl = warp_excl_scan(kc);
      const uint32_t kept_warp = warp_sum(kc);
      const long long w_idx = block * 32 + lane;
      if (w_idx < n_words) bitmap[w_idx] = keep_word;
      if (lane == 0) {
        offsets[block] = static_cast<unsigned long long>(kept_before);
        if (block == n_blocks - 1) {
          const long long total = kept_before + kept_warp;
          offsets[n_blocks] = static_cast<unsigned long long>(total);
          if (total != hdr->n_keep)
            atomicMax(&hdr->status, static_cast<uint32_t>(SURGEON_ERR_INTERNAL));
        }
      }
      const uint32_t lt = lanemask_lt();
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const uint32_t kw = __shfl_sync(0xFFFFFFFFu, keep_word, i);
        const uint32_t wb = __shfl_sync(0xFFFFFFFFu, word_excl, i);
        if ((kw >> lane) & 1u) values[kept_before + wb + __popc(kw & lt)] = xs[i];
      }
    }
    __syncthreads();  // s_tile / s_gt / s_eq are rewritten by the next iteration
  }
}

__global__ void offsets_empty_kernel(unsigned long long* offsets) { offsets[0] = 0ull; }

// ---- decompress -------------------------------------------------------------------------------

// Algorithm 1: Reshape step: one warp rebuilds one SURGEON_BLOCK of the dense tensor.
template <int DT>
__global__ void __launch_bounds__(256)
decompress_kernel(const uint32_t* __restrict__ bitmap, const void* __restrict__ values_v,
                  const unsigned long long* __restrict__ offsets, long long n,
                  void* __restrict__ out_v) {
  using E = typename Elem<DT>::type;
  const E* __restrict__ values = reinterpret_cast<const E*>(values_v);
  E* __restrict__ out = reinterpret_cast<E*>(out_v);
  const uint32_t lane = lane_id();
  const long long n_blocks = (n + SURGEON_BLOCK - 1) / SURGEON_BLOCK;
  const long long n_words = (n + 31) / 32;
  const long long warps = (static_cast<long long>(gridDim.x) * blockDim.x) >> 5;
  for (long long block = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
       block < n_blocks; block += warps) {
    const long long w_idx = block * 32 + lane;
    const uint32_t word = (w_idx < n_words) ? bitmap[w_idx] : 0u;
    const uint32_t word_excl = warp_excl_scan(__popc(word));
    const unsigned long long first = offsets[block];
    const uint32_t lt = lanemask_lt();
    const long long base = block * SURGEON_BLOCK;
#pragma unroll 4
    for (int i = 0; i < 32; ++i) {
      const uint32_t w = __shfl_sync(0xFFFFFFFFu, word, i);
      const uint32_t wb = __shfl_sync(0xFFFFFFFFu, word_excl, i);
      const long long idx = base + i * 32 + lane;
      if (idx < n) out[idx] = ((w >> lane) & 1u) ? values[first + wb + __popc(w & lt)]
                                                 : static_cast<E>(0);
    }
  }
}

template <int DT>
cudaError_t run_prune_compact(const void* x, long long n, long long k,
                              const surgeon_compressed& out, void* workspace,
                              cudaStream_t stream) {
  char* ws = static_cast<char*>(workspace);
  SelectState* st = reinterpret_cast<SelectState*>(ws);
  uint32_t* ghist = reinterpret_cast<uint32_t*>(ws + kWsStateBytes);
  unsigned long long* tile_state =
      reinterpret_cast<unsigned long long*>(ws + kWsStateBytes + kWsHistBytes);
  cudaError_t e = cudaMemsetAsync(workspace, 0, prune_workspace_bytes(n), stream);
  if (e != cudaSuccess) return e;
  e = cudaMemsetAsync(out.header, 0, sizeof(surgeon_header), stream);
  if (e != cudaSuccess) return e;

  if (k == 0) {
    header_empty_kernel<<<1, 1, 0, stream>>>(out.header, Elem<DT>::kSentinel);
    note_launches(1);
  } else {
    constexpr int VEC = 16 / static_cast<int>(sizeof(typename Elem<DT>::type));
    const long long nvec = n / VEC;
    long long want = (nvec + kHistThreads * 4 - 1) / (kHistThreads * 4);
    const int grid = static_cast<int>(want < 1 ? 1 : (want > 2LL * sm_count() ? 2LL * sm_count() : want));
    if (DT == 0) {
      radix_hist_kernel<0, 20, 11, false><<<grid, kHistThreads, 0, stream>>>(
          x, n, k, 0, st, ghist, out.header);
      radix_hist_kernel<0, 9, 11, false><<<grid, kHistThreads, 0, stream>>>(
          x, n, k, 1, st, ghist + kMaxBins, out.header);
      radix_hist_kernel<0, 0, 9, true><<<grid, kHistThreads, 0, stream>>>(
          x, n, k, 2, st, ghist + 2 * kMaxBins, out.header);
      note_launches(3);
    } else {
      radix_hist_kernel<1, 4, 11, false><<<grid, kHistThreads, 0, stream>>>(
          x, n, k, 0, st, ghist, out.header);
      radix_hist_kernel<1, 0, 4, true><<<grid, kHistThreads, 0, stream>>>(
          x, n, k, 1, st, ghist + kMaxBins, out.header);
      note_launches(2);
    }
  }
  if (n == 0) {
    offsets_empty_kernel<<<1, 1, 0, stream>>>(
        reinterpret_cast<unsigned long long*>(out.block_offsets));
    note_launches(1);
  } else {
    const long long tiles = (n + kTileElems - 1) / kTileElems;
    const long long cap = 8LL * sm_count();
    const int grid = static_cast<int>(tiles < cap ? tiles : cap);
    compact_kernel<DT><<<grid, 256, 0, stream>>>(
        x, n, out.header, out.bitmap, out.values,
        reinterpret_cast<unsigned long long*>(out.block_offsets), &st->compact_ticket, tile_state,
        static_cast<int>(tiles));
    note_launches(1);
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_prune_compact(const void* x, int64_t n, int dt, int64_t k,
                                 const surgeon_compressed& out, void* workspace,
                                 cudaStream_t stream) {
  return dt == 0 ? run_prune_compact<0>(x, n, k, out, workspace, stream)
                 : run_prune_compact<1>(x, n, k, out, workspace, stream);
}

cudaError_t launch_decompress(const surgeon_compressed& act, void* x_out, cudaStream_t stream) {
  if (act.n == 0) return cudaSuccess;
  const long long n_blocks = (act.n + SURGEON_BLOCK - 1) / SURGEON_BLOCK;
  const long long ctas = (n_blocks + 7) / 8;
  const long long cap = 16LL * sm_count();
  const int grid = static_cast<int>(ctas < cap ? ctas : cap);
  const unsigned long long* offs = reinterpret_cast<const unsigned long long*>(act.block_offsets);
  if (act.dt == 0)
    decompress_kernel<0><<<grid, 256, 0, stream>>>(act.bitmap, act.values, offs, act.n, x_out);
  else
    decompress_kernel<1><<<grid, 256, 0, stream>>>(act.bitmap, act.values, offs, act.n, x_out);
  note_launches(1);
  return cudaGetLastError();
}

}  // namespace surgeon

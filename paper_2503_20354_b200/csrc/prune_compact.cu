// Threshold select and compaction kernels of surgeon_prune_compact, and surgeon_decompress.
//
// Algorithm 1, prune step: the kept set of a layer is its n_keep largest-magnitude elements, ties
// at the threshold broken by lowest flat index.  Its decompose step / Section 4.2: the pruned
// activation is cached as the vector of kept elements plus one index bit per element.
//
// The tensor is read twice: once to find the threshold, once to emit the store.  No CTA of the
// emitting pass waits on another: everything it needs to place a chunk's output (how many
// elements before the chunk are kept, how many ties precede it) is counted during the first read.
// Both reads are persistent kernels fed by TMA into a shared-memory ring, in which every lane owns
// 128 consecutive bytes, so bitmap words are built without cross-lane traffic.
//
//   sample   : a strided sample (about 1/32 of the tensor) gives a bracket [lo_key, hi_key] of
//              keys that contains the threshold with overwhelming probability and holds 1-3 %
//              of the elements.
//   classify : the first read.  Per 4 KB chunk: the number of keys above the bracket, the number
//              inside, and the keys inside themselves (the chunk's slot).  Its last CTA decides
//              where the threshold lies and, for bf16, which key it is.
//   count    : fp32 resolves the threshold among the listed keys with two histogram levels;
//              then the listed keys above / equal to the threshold complete the per-chunk counts,
//              and an exclusive scan over chunks follows (cooperative launch, grid barriers).
//              The one chunk inside which the tie quota ends is emitted here, by the CTA that
//              finds it, with its ties ranked by flat index.
//   compact  : the second read.  A chunk's warp starts from its entry of the scan and skips
//              that one chunk.
//
// If the threshold falls outside the bracket, a slot overflows (massive ties at a non-zero
// value) or the tensor is below kStreamMinBytes, the count kernel runs an exact radix select
// over the tensor and counts the chunks from the tensor (a small tensor is then emitted by
// compact_small_kernel).  The result is exact and unique either way.
// Every count fits 32 bits because n <= SURGEON_MAX_N < 2^31.
#include <cuda.h>

#include "surgeon_internal.cuh"
#include "tc_common.cuh"

namespace surgeon {

namespace {

using tc::smem_u32;

constexpr int kSelThreads = 1024;
constexpr uint32_t kFull = 0xFFFFFFFFu;
constexpr int kHistWords = kBuckets + 32;   // + one private bin per lane that swallows zeros
__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}

// dst[0 .. kBuckets) = src[0 .. kBuckets) with all loads of a thread in flight together
// (1024 threads; src is global memory written by other CTAs, dst shared memory).
__device__ __forceinline__ void load_hist_to_smem(const uint32_t* __restrict__ src, uint32_t* dst) {
  constexpr int kPer = kBuckets / 4 / kSelThreads;   // 8 vectors per thread
  uint4 v[kPer];
#pragma unroll
  for (int i = 0; i < kPer; ++i)
    v[i] = __ldcg(reinterpret_cast<const uint4*>(src) + i * kSelThreads + threadIdx.x);
#pragma unroll
  for (int i = 0; i < kPer; ++i)
    reinterpret_cast<uint4*>(dst)[i * kSelThreads + threadIdx.x] = v[i];
}
__device__ __forceinline__ void zero_hist_smem(uint32_t* dst) {
#pragma unroll
  for (int i = 0; i < kBuckets / 4 / kSelThreads; ++i)
    reinterpret_cast<uint4*>(dst)[i * kSelThreads + threadIdx.x] = make_uint4(0, 0, 0, 0);
}
// Adds the non-zero bins of a CTA's shared-memory histogram to the global one.
__device__ __forceinline__ void flush_hist(const uint32_t* hist, uint32_t* __restrict__ ghist) {
#pragma unroll 4
  for (int i = 0; i < kBuckets / 4 / kSelThreads; ++i) {
    const int v = i * kSelThreads + threadIdx.x;
    const uint4 h = reinterpret_cast<const uint4*>(hist)[v];
    if (h.x) atomicAdd(&ghist[4 * v + 0], h.x);
    if (h.y) atomicAdd(&ghist[4 * v + 1], h.y);
    if (h.z) atomicAdd(&ghist[4 * v + 2], h.z);
    if (h.w) atomicAdd(&ghist[4 * v + 3], h.w);
  }
}

// Cooperative search from the top of a histogram of NB bins (NB a multiple of 1024) by a CTA of
// 1024 threads: finds the bin b with  #(bins above b) < rank <= #(bins >= b)  and writes
// res[0] = b, res[1] = count in the bins above b.  `ld(i)` returns bin i.  rank >= 1 and the
// histogram holds at least `rank` entries.  scratch: 32 words of shared memory.
template <int NB, typename Load>
__device__ void find_from_top(Load ld, uint32_t rank, uint32_t* scratch, uint32_t* res) {
  constexpr int PER_WARP = NB / 32;
  constexpr int PER_LANE = PER_WARP / 32;
  const int warp = threadIdx.x >> 5;
  const uint32_t lane = lane_id();
  // level 1: warp w owns the PER_WARP bins below NB - w*PER_WARP
  const int top = NB - warp * PER_WARP;   // exclusive upper end
  uint32_t s = 0;
#pragma unroll 8
  for (int i = lane; i < PER_WARP; i += 32) s += ld(top - 1 - i);
  s = warp_sum(s);
  if (lane == 0) scratch[warp] = s;
  __syncthreads();
  uint32_t acc = 0;
  int W = 0;
  for (; W < 31; ++W) {
    const uint32_t t = scratch[W];
    if (acc + t >= rank) break;
    acc += t;
  }
  if (warp == W) {
    // level 2: lane L owns the PER_LANE bins below top - L*PER_LANE
    const int ltop = top - static_cast<int>(lane) * PER_LANE;
    uint32_t ls = 0;
#pragma unroll 8
    for (int i = 0; i < PER_LANE; ++i) ls += ld(ltop - 1 - ((i + lane) % PER_LANE));
    const uint32_t excl = warp_excl_scan(ls);
    const uint32_t want = rank - acc;
    if (excl < want && want <= excl + ls) {
      uint32_t a = excl;
      int b = ltop - 1;
      for (int i = 0; i < PER_LANE - 1; ++i, --b) {
        const uint32_t c = ld(b);
        if (a + c >= want) break;
        a += c;
      }
      res[0] = static_cast<uint32_t>(b);
      res[1] = acc + a;
    }
  }
  __syncthreads();
}

__device__ __forceinline__ uint32_t hash_u32(uint32_t v) {
  v ^= v >> 16; v *= 0x7FEB352Du; v ^= v >> 15; v *= 0x846CA68Bu; v ^= v >> 16;
  return v;
}

// ---- bracket of buckets around the threshold, predicted from a strided sample ------------------
template <int DT>
__global__ void __launch_bounds__(kSelThreads, 1)
sample_kernel(const uint4* __restrict__ xq, long long n, uint32_t k, uint32_t n_seg,
              uint32_t seg_stride, SelectState* __restrict__ st, uint32_t* __restrict__ shist) {
  constexpr uint32_t kMask = Elem<DT>::kKeyMask;
  constexpr int EPV = (DT == 0) ? 4 : 8;
  extern __shared__ __align__(128) uint32_t hist[];   // kHistWords
  __shared__ uint32_t scratch[32];
  __shared__ uint32_t res[2];
  __shared__ bool s_last;
  const int tid = threadIdx.x;
  const uint32_t lane = lane_id();
  zero_hist_smem(hist);
  __syncthreads();
  uint32_t zero_cnt = 0;
#pragma unroll 4
  for (uint32_t seg = blockIdx.x * 32 + (tid >> 5); seg < n_seg; seg += gridDim.x * 32) {
    // one segment = 32 lanes x 16 bytes, at a hashed position inside its stride
    const unsigned long long pos =
        static_cast<unsigned long long>(seg) * seg_stride + hash_u32(seg) % seg_stride;
    const uint4 q = __ldg(xq + pos * 32 + lane);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int e = 0; e < EPV; ++e) {
      const uint32_t bits = (DT == 0) ? w[e % 4] : (w[e >> 1] >> (16 * (e & 1)));
      const uint32_t key = bits & kMask;
      const bool isz = key == 0;
      zero_cnt += isz ? 1u : 0u;
      // zeros (half of post-ReLU data) go to a bin private to the lane: no conflicts, no branch
      atomicAdd(&hist[isz ? kBuckets + lane : (DT == 0 ? key >> 16 : key)], 1u);
    }
  }
  zero_cnt = warp_sum(zero_cnt);
  if (lane == 0 && zero_cnt) atomicAdd(&hist[0], zero_cnt);
  __syncthreads();
  flush_hist(hist, shist);
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(&st->ticket_sample, 1u) == gridDim.x - 1);
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  load_hist_to_smem(shist, hist);
  __syncthreads();
  // rank of the threshold inside the sample, +- 5 standard deviations of a binomial count
  // (single precision, one thread: double-precision arithmetic is slow on this GPU)
  __shared__ uint32_t s_rank[2];
  if (tid == 0) {
    const float S = static_cast<float>(32 * EPV) * static_cast<float>(n_seg);
    const float q = static_cast<float>(static_cast<double>(k) / static_cast<double>(n));
    const float r = q * S;
    const float delta = 5.0f * sqrtf(S * q * (1.0f - q)) + 16.0f;
    s_rank[0] = (r - delta >= 1.0f) ? static_cast<uint32_t>(r - delta) : 0u;           // 0: none
    s_rank[1] = (r + delta <= S - 1.0f) ? static_cast<uint32_t>(r + delta) + 1u : 0u;  // 0: none
  }
  __syncthreads();
  uint32_t bhi = kBuckets - 1, blo = 0;
  auto ld = [&](int i) { return hist[i]; };
  if (s_rank[0]) {
    find_from_top<kBuckets>(ld, s_rank[0], scratch, res);
    bhi = res[0];
    __syncthreads();
  }
  if (s_rank[1]) {
    find_from_top<kBuckets>(ld, s_rank[1], scratch, res);
    blo = res[0];
  }
  if (tid == 0) {
    st->blo = blo;
    st->bhi = bhi;
    // the bracket as keys; key 0 (exact zeros) is never a candidate
    const uint32_t lo = (DT == 0) ? (blo << 16) : blo;
    st->lo_key = lo < 1u ? 1u : lo;
    const uint32_t hi = (DT == 0) ? ((bhi << 16) | 0xFFFFu) : bhi;
    st->hi_key = hi;                                            // hi < lo_key: the bracket is {0}
    const int range_bits = hi >= st->lo_key ? 32 - __clz(hi - st->lo_key) : 0;   // widest relative key
    st->shiftA = range_bits > 9 ? static_cast<uint32_t>(range_bits - 9) : 0u;
  }
}

// ---- geometry shared by the two streaming kernels -----------------------------------------------
// Persistent CTAs.  One producer thread keeps a ring of 32 KB stages full with 2-D TMA loads of
// [256 rows x 128 bytes] (128-byte swizzle, so that 32 lanes can each read their own row without
// bank conflicts).  Each of the 8 consumer warps owns one 4 KB chunk of a stage; each LANE owns
// one 128-byte row of it, i.e. 32 (fp32) or 64 (bf16) consecutive elements.
constexpr int kCsWarps = 8;
constexpr int kCsThreads = (kCsWarps + 1) * 32;
constexpr int kCsStageRows = kCsWarps * 32;
constexpr int kCsStageBytes = kCsStageRows * 128;
constexpr int kCsStages = 3;
// The ring starts on a 4 KB boundary: every warp's 4 KB part of a stage is then 4 KB-aligned, which
// the compaction's gather uses to swizzle full shared-memory addresses.
constexpr uintptr_t kCsAlign = 4096;
constexpr int kMinTilesPerCta = 4;
constexpr size_t kCsSmem = static_cast<size_t>(kCsStages) * kCsStageBytes + kCsAlign;
static_assert(kCsStageRows * 128 / 16 == kCsWarps * kTileVecs, "a warp's 32 rows are one chunk");

// This lane's row (8 vectors) out of the swizzled stage; the ragged last row of the tensor, which
// the tensor map does not cover, comes from global memory.  Returns the row's valid element count.
template <int DT>
__device__ __forceinline__ int load_row(const unsigned char* region, const typename Elem<DT>::type* x,
                                        long long n, long long n_rows_full, long long grow,
                                        uint4 (&q)[8]) {
  constexpr int EPR = 128 / sizeof(typename Elem<DT>::type);
  const uint32_t lane = lane_id();
  const unsigned char* row = region + lane * 128;
#pragma unroll
  for (int j = 0; j < 8; ++j)
    q[j] = *reinterpret_cast<const uint4*>(row + ((j ^ (lane & 7)) << 4));
  const long long e0 = grow * EPR;
  long long nv = n - e0;
  nv = nv < 0 ? 0 : (nv > EPR ? EPR : nv);
  if (grow >= n_rows_full && nv > 0) {
    uint32_t t[64];
#pragma unroll
    for (int i = 0; i < 64; ++i) t[i] = (i < EPR && i < nv) ? static_cast<uint32_t>(x[e0 + i]) : 0u;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (DT == 0) q[j] = make_uint4(t[4 * j], t[4 * j + 1], t[4 * j + 2], t[4 * j + 3]);
      else q[j] = make_uint4(t[8 * j] | (t[8 * j + 1] << 16), t[8 * j + 2] | (t[8 * j + 3] << 16),
                             t[8 * j + 4] | (t[8 * j + 5] << 16), t[8 * j + 6] | (t[8 * j + 7] << 16));
    }
  }
  return static_cast<int>(nv);
}
// bf16 keys are compared two at a time inside their 32-bit word: a key is at most 0x7FFF, so
// key + (0x8000 - t) carries into bit 15 of its half exactly when key >= t, and never into the
// other half.  The flag bits of the 16 words of a group of 32 elements are collected in one mask,
// word i shifted right by i: bit (15 - i) is element 2i, bit (31 - i) element 2i + 1.
__device__ __forceinline__ uint32_t ge_const(uint32_t t) {       // t in [0, 0x8000]
  return (0x8000u - t) * 0x10001u;
}
__device__ __forceinline__ uint32_t pair_flags(uint32_t keys2, uint32_t c, int i) {
  return ((keys2 + c) >> i) & (0x80008000u >> i);
}
// The same mask in element order (bit e = element e).
__device__ __forceinline__ uint32_t pairs_to_element_order(uint32_t m) {
  const uint32_t r = __brev(m);              // bit (16 + i): element 2i, bit i: element 2i + 1
  auto spread = [](uint32_t x) {             // bit i -> bit 2i, for x < 2^16
    x = (x | (x << 8)) & 0x00FF00FFu;
    x = (x | (x << 4)) & 0x0F0F0F0Fu;
    x = (x | (x << 2)) & 0x33333333u;
    x = (x | (x << 1)) & 0x55555555u;
    return x;
  };
  return spread(r >> 16) | (spread(r & 0xFFFFu) << 1);
}
__device__ __forceinline__ uint32_t valid_mask(int nv, int w) {
  const int left = nv - 32 * w;
  return left >= 32 ? 0xFFFFFFFFu : (left <= 0 ? 0u : ((1u << left) - 1u));
}

// The chunk's keys inside the bracket (flagged in cw0 / cw1, `c_tot` of them in the warp) if they
// all are one key, else 0 (no candidate key is 0).  Called for chunks whose slot overflows only,
// and kept out of line so that the classify kernel's registers are those of its common path; it
// reads the lane's row again, a piece at a time.
template <int DT>
__device__ __noinline__ uint32_t one_key_of_chunk(const unsigned char* region,
                                                  const typename Elem<DT>::type* x, long long n,
                                                  long long n_rows_full, long long grow,
                                                  uint32_t cw0, uint32_t cw1, uint32_t c_tot) {
  using E = typename Elem<DT>::type;
  constexpr uint32_t kMask = Elem<DT>::kKeyMask;
  constexpr int EPR = 128 / sizeof(E);
  const uint32_t lane = lane_id();
  const bool ragged = grow >= n_rows_full;
  const unsigned char* row = region + lane * 128;
  const int src = __ffs(__ballot_sync(kFull, (cw0 | cw1) != 0u)) - 1;
  uint32_t k0 = 0;
  if (static_cast<int>(lane) == src) {
    const int e = cw0 ? __ffs(cw0) - 1 : 32 + __ffs(cw1) - 1;      // (fp32: cw1 is cw0)
    if (ragged) {
      k0 = static_cast<uint32_t>(x[grow * EPR + e]) & kMask;
    } else {
      const int byte = e * static_cast<int>(sizeof(E));
      k0 = static_cast<uint32_t>(*reinterpret_cast<const E*>(row + (((byte >> 4) ^ (lane & 7)) << 4) + (byte & 15))) & kMask;
    }
  }
  k0 = __shfl_sync(kFull, k0, src);
  uint32_t eq = 0;
  if (ragged) {                                  // the tensor's last, partial row: element by element
    for (int e = 0; e < EPR; ++e)
      if (grow * EPR + e < n) eq += (static_cast<uint32_t>(x[grow * EPR + e]) & kMask) == k0 ? 1u : 0u;
  } else {
    const uint32_t c_ge = ge_const(k0 & 0x7FFFu), c_gt = ge_const((k0 & 0x7FFFu) + 1u);   // bf16: k0 <= 0x7FFF
#pragma unroll 1
    for (int j = 0; j < 8; ++j) {                // one 16-byte piece at a time: few registers
      const uint4 v = *reinterpret_cast<const uint4*>(row + ((j ^ (lane & 7)) << 4));
      const uint32_t c[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (DT == 0) {
          eq += (c[i] & kMask) == k0 ? 1u : 0u;
        } else {
          const uint32_t keys2 = c[i] & 0x7FFF7FFFu;
          eq += __popc(((keys2 + c_ge) & ~(keys2 + c_gt)) & 0x80008000u);
        }
      }
    }
  }
  // (a ragged row's fill is key 0, never a candidate)
  return __reduce_add_sync(kFull, eq) == c_tot ? k0 : 0u;
}

// ---- the select's read of the tensor ---------------------------------------------------------
// Per chunk: how many keys lie above the bracket, how many inside; the keys inside go to the
// chunk's slot.  A level-A histogram of the keys inside (relative to lo_key) is kept per CTA.
// The last CTA places the threshold: above the bracket or a full slot -> fall back; inside ->
// bin of level A (bf16: the threshold itself); below, with lo_key == 1 -> the threshold is 0.
template <int DT>
__global__ void __launch_bounds__(kCsThreads, 2)
classify_kernel(const __grid_constant__ CUtensorMap xmap, const void* __restrict__ xv, long long n,
                long long n_rows_full, uint32_t k, SelectState* __restrict__ st,
                uint32_t* __restrict__ hist_a, uint32_t* __restrict__ cnt_gt,
                uint32_t* __restrict__ cand_cnt, void* __restrict__ slots_v,
                surgeon_header* __restrict__ hdr, int n_chunks, int n_stage_tiles,
                int drop_zeros) {
  using E = typename Elem<DT>::type;
  constexpr uint32_t kMask = Elem<DT>::kKeyMask;
  constexpr int EPR = 128 / sizeof(E);
  constexpr int WPL = EPR / 32;
  constexpr int kSlot = (DT == 0) ? 64 : 128;
  extern __shared__ __align__(1024) unsigned char cs_smem_raw[];
  unsigned char* ring = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(cs_smem_raw) + kCsAlign - 1) & ~(kCsAlign - 1));
  __shared__ __align__(8) unsigned long long bars[2 * kCsStages];
  __shared__ uint32_t s_hist[kBinsA];
  __shared__ uint32_t s_tot[4];        // keys above / inside the bracket, largest key inside, largest ~key inside
  __shared__ bool s_last;
  const E* __restrict__ x = reinterpret_cast<const E*>(xv);
  E* __restrict__ slots = reinterpret_cast<E*>(slots_v);   // fp32: 32-bit keys, bf16: 16-bit keys
  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const uint32_t lane = lane_id();
  if (st->mode == 1u) return;          // the sample found no usable bracket
  const uint32_t lo_key = st->lo_key, hi_key = st->hi_key;
  const uint32_t shiftA = st->shiftA;
  // bf16: the two comparisons as additions on packed pairs of keys (hi_key <= 0x7FFF there)
  const uint32_t c_above = ge_const(hi_key >= 0x7FFFu ? 0x8000u : hi_key + 1u);
  const uint32_t c_lo = hi_key >= lo_key ? ge_const(lo_key > 0x8000u ? 0x8000u : lo_key) : 0u;
  const uint32_t full_bar = smem_u32(bars);
  const uint32_t empty_bar = smem_u32(bars + kCsStages);
  if (tid == 0) {
    tc::tma_prefetch_desc(&xmap);
    for (int s = 0; s < kCsStages; ++s) {
      tc::mbar_init(full_bar + 8 * s, 1);
      tc::mbar_init(empty_bar + 8 * s, kCsWarps);
    }
    tc::fence_barrier_init();
    s_tot[0] = 0;
    s_tot[1] = 0;
    s_tot[2] = 0;
    s_tot[3] = 0;
  }
  for (int i = tid; i < kBinsA; i += kCsThreads) s_hist[i] = 0;
  __syncthreads();
  const int first = blockIdx.x;
  const int n_it = first < n_stage_tiles ? (n_stage_tiles - 1 - first) / static_cast<int>(gridDim.x) + 1 : 0;

  if (warp == kCsWarps) {
    // ---- producer ----
    if (lane == 0) {
      for (int it = 0; it < n_it; ++it) {
        const int s = it % kCsStages;
        if (it >= kCsStages && !tc::mbar_wait(empty_bar + 8 * s, ((it / kCsStages) - 1) & 1, 20)) {
          atomicMax(&st->error, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
          break;
        }
        const int t = first + it * static_cast<int>(gridDim.x);
        tc::mbar_arrive_expect_tx(full_bar + 8 * s, kCsStageBytes);
        tc::tma_load_2d(smem_u32(ring + s * kCsStageBytes), &xmap, 0, t * kCsStageRows,
                        full_bar + 8 * s);
      }
    }
  } else {
    // ---- consumers ----
    uint32_t w_above = 0, w_cand = 0;
    uint32_t w_kmax = 0, w_kinv = 0;     // largest key inside the bracket seen by this lane, and largest ~key
    for (int it = 0; it < n_it; ++it) {
      const int s = it % kCsStages;
      const int chunk = (first + it * static_cast<int>(gridDim.x)) * kCsWarps + warp;
      if (!tc::mbar_wait(full_bar + 8 * s, (it / kCsStages) & 1, 20)) {
        if (lane == 0) atomicMax(&st->error, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
        break;
      }
      const unsigned char* region = ring + s * kCsStageBytes + warp * 4096;
      if (chunk < n_chunks) {
        uint4 q[8];
        const long long grow = static_cast<long long>(chunk) * 32 + lane;
        const int nv = load_row<DT>(region, x, n, n_rows_full, grow, q);
        uint32_t cw[WPL];
        uint32_t ac = 0, cc = 0;
        if (DT == 0) {
          // Keys are below 2^31, so the sign bit of (hi_key - key) says key > hi_key and that of
          // (key - lo) says key < lo; a funnel shift collects it: two instructions per element
          // and comparison.  Element e ends up in bit 31 - e, one bit reversal per word puts it back.
          uint32_t aw = 0, lw = 0;
          const uint32_t lo_cmp = hi_key >= lo_key ? lo_key : 0x7FFFFFFFu;   // bracket {0}: nothing is a candidate
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint32_t c[4] = {q[j].x, q[j].y, q[j].z, q[j].w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const uint32_t key = c[i] & kMask;
              aw = __funnelshift_l(hi_key - key, aw, 1);
              lw = __funnelshift_l(key - lo_cmp, lw, 1);
            }
          }
          const uint32_t vm = valid_mask(nv, 0);
          aw = __brev(aw) & vm;
          cw[0] = ~__brev(lw) & ~aw & vm;
          if (hi_key < lo_key) cw[0] = 0u;
          ac = __popc(aw);
        } else {
          // above: key >= hi_key + 1; inside the bracket: key >= lo_key and not above
          uint32_t ga[WPL], gl[WPL];
#pragma unroll
          for (int w = 0; w < WPL; ++w) { ga[w] = 0; gl[w] = 0; }
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint32_t c[4] = {q[j].x, q[j].y, q[j].z, q[j].w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int pw = 4 * j + i;           // packed word of the row: elements 2pw, 2pw + 1
              const uint32_t keys2 = c[i] & 0x7FFF7FFFu;
              ga[(pw >> 4) % WPL] |= pair_flags(keys2, c_above, pw & 15);
              gl[(pw >> 4) % WPL] |= pair_flags(keys2, c_lo, pw & 15);
            }
          }
#pragma unroll
          for (int w = 0; w < WPL; ++w) {
            ac += __popc(ga[w]);        // zeros that fill a ragged row are never above
            const uint32_t in = gl[w] & ~ga[w];
            cw[w] = in ? (pairs_to_element_order(in) & valid_mask(nv, w)) : 0u;
          }
        }
#pragma unroll
        for (int w = 0; w < WPL; ++w) cc += __popc(cw[w]);
        const uint32_t a_tot = __reduce_add_sync(kFull, ac);
        const uint32_t c_tot = __reduce_add_sync(kFull, cc);
        if (lane == 0) { cnt_gt[chunk] = a_tot; cand_cnt[chunk] = c_tot; }
        w_above += a_tot;
        w_cand += c_tot;
        const bool ragged = grow >= n_rows_full;
        const unsigned char* row = region + lane * 128;
        auto key_at = [&](int e) -> uint32_t {        // key of element e of this lane's row
          if (ragged) return static_cast<uint32_t>(x[grow * EPR + e]) & kMask;
          const int byte = e * static_cast<int>(sizeof(E));
          return static_cast<uint32_t>(*reinterpret_cast<const E*>(
                     row + (((byte >> 4) ^ (lane & 7)) << 4) + (byte & 15))) & kMask;
        };
        if (c_tot > static_cast<uint32_t>(kSlot)) {
          if (lane == 0) st->list_overflow = 1u;
          // Too many keys inside the bracket for the slot: massive ties.  If they all are one and the
          // same key - here and in every other chunk - that key is the threshold and the counts
          // above are all the count kernel needs; the last CTA checks that through the extremes.
          const uint32_t k1 = one_key_of_chunk<DT>(region, x, n, n_rows_full, grow, cw[0], cw[WPL - 1], c_tot);
          w_kmax = k1 ? max(w_kmax, k1) : 0xFFFFFFFFu;
          w_kinv = k1 ? max(w_kinv, ~k1) : 0xFFFFFFFFu;
        } else if (c_tot) {
          // keys inside the bracket -> the chunk's slot (order does not matter)
          uint32_t pos = warp_excl_scan(cc);
          E* slot = slots + static_cast<long long>(chunk) * kSlot;
#pragma unroll
          for (int w = 0; w < WPL; ++w) {
            uint32_t m = cw[w];
            while (m) {
              const int e = 32 * w + __ffs(m) - 1;
              m &= m - 1;
              const uint32_t key = key_at(e);
              slot[pos++] = static_cast<E>(key);
              atomicAdd(&s_hist[(key - lo_key) >> shiftA], 1u);
              w_kmax = max(w_kmax, key);
              w_kinv = max(w_kinv, ~key);
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(empty_bar + 8 * s);
    }
    w_kmax = __reduce_max_sync(kFull, w_kmax);
    w_kinv = __reduce_max_sync(kFull, w_kinv);
    if (lane == 0) {
      if (w_above) atomicAdd(&s_tot[0], w_above);
      if (w_cand) atomicAdd(&s_tot[1], w_cand);
      if (w_kmax) atomicMax(&s_tot[2], w_kmax);
      if (w_kinv) atomicMax(&s_tot[3], w_kinv);
    }
  }
  __syncthreads();
  for (int i = tid; i < kBinsA; i += kCsThreads)
    if (s_hist[i]) atomicAdd(&hist_a[i], s_hist[i]);
  if (tid == 0) {
    if (s_tot[0]) atomicAdd(&st->above_total, s_tot[0]);
    if (s_tot[1]) atomicAdd(&st->cand_total, s_tot[1]);
    if (s_tot[2]) atomicMax(&st->cand_key_max, s_tot[2]);
    if (s_tot[3]) atomicMax(&st->cand_keyinv_max, s_tot[3]);
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(&st->ticket_classify, 1u) == gridDim.x - 1);
  __syncthreads();
  if (!s_last || warp != 0) return;

  // ---- last CTA, one warp: where does the threshold lie? ----
  __threadfence();
  const uint32_t above_total = __ldcg(&st->above_total);
  const uint32_t n_cand = __ldcg(&st->cand_total);
  const bool overflow = __ldcg(&st->list_overflow) != 0;
  const long long r = static_cast<long long>(k) - above_total;     // rank among the rest
  const long long zeros = (lo_key == 1u) ? n - above_total - n_cand : 0;
  uint32_t mode, tau = 0, n_greater = 0;
  if (overflow && r >= 1 && r <= n_cand &&
      __ldcg(&st->cand_key_max) == ~__ldcg(&st->cand_keyinv_max)) {
    // every key inside the bracket is the same one: it is the threshold, all candidates are ties
    mode = 4;
    tau = __ldcg(&st->cand_key_max);
    n_greater = above_total;
  } else if (overflow || r < 1) {
    mode = 1;
  } else if (r <= n_cand) {
    // level A from the top: lane L owns bins [kBinsA - 16(L+1), kBinsA - 16L)
    constexpr int kPerLane = kBinsA / 32;
    const int ltop = kBinsA - static_cast<int>(lane) * kPerLane;
    uint32_t ls = 0;
#pragma unroll
    for (int i = 0; i < kPerLane; ++i) ls += __ldcg(hist_a + ltop - 1 - i);
    const uint32_t excl = warp_excl_scan(ls);
    const uint32_t want = static_cast<uint32_t>(r);
    uint32_t bin = 0, aboveA = 0;
    if (excl < want && want <= excl + ls) {
      uint32_t a = excl;
      int b = ltop - 1;
      for (int i = 0; i < kPerLane - 1; ++i, --b) {
        const uint32_t c = __ldcg(hist_a + b);
        if (a + c >= want) break;
        a += c;
      }
      bin = static_cast<uint32_t>(b);
      aboveA = a;
    }
    const uint32_t owner = __ffs(__ballot_sync(kFull, excl < want && want <= excl + ls)) - 1;
    bin = __shfl_sync(kFull, bin, owner);
    aboveA = __shfl_sync(kFull, aboveA, owner);
    if (lane == 0) {
      st->binA = bin;
      st->aboveA = aboveA;
      st->rankA = want - aboveA;
    }
    mode = shiftA ? 0u : 2u;
    tau = lo_key + bin;                       // shiftA == 0: level A is exact
    n_greater = above_total + aboveA;
  } else if (lo_key == 1u && r <= n_cand + zeros) {
    mode = 2;
    tau = 0;
    n_greater = above_total + n_cand;
  } else {
    mode = 1;
  }
  if (lane == 0) {
    if (mode == 2 || mode == 4) {
      // store variant without kept zeros: a threshold of key 0 keeps the non-zero elements only
      const bool nz = drop_zeros && tau == 0u;
      hdr->threshold_key = tau;
      hdr->status = __ldcg(&st->error);
      hdr->n_keep = nz ? static_cast<long long>(n_greater) : static_cast<long long>(k);
      hdr->n_greater = n_greater;
      hdr->tie_quota = nz ? 0 : static_cast<long long>(k) - n_greater;
    }
    st->mode = mode;
    __threadfence();
  }
}

// n_keep == 0 (ratio 1, or an empty tensor): nothing to select.
__global__ void header_empty_kernel(surgeon_header* hdr, uint32_t sentinel, uint32_t* offsets,
                                    long long n_blocks) {
  if (n_blocks > 0) offsets[n_blocks] = 0u;      // the sentinel entry of the block offsets
  hdr->threshold_key = sentinel;
  hdr->status = SURGEON_OK;
  hdr->n_keep = 0;
  hdr->n_greater = 0;
  hdr->tie_quota = 0;
}

constexpr unsigned long long kCountMask = 0x7FFFFFFFull;
constexpr int kRows = 4;                 // rows of 32 lanes x 16 bytes per warp
constexpr int kTileWarps = kTileVecs / (kRows * 32);   // warps of the generic per-tile kernels
static_assert(kTileWarps * kRows * 32 == kTileVecs, "compaction tile");
constexpr int kCompactThreads = kTileWarps * 32;

// Defined with the compaction kernels below; the count kernel emits the boundary tile itself.
template <int DT, bool SLOW>
__device__ __forceinline__ void compact_tile(const typename Elem<DT>::type* __restrict__ x,
                                             long long n, const uint4 (&q)[kRows], int tile,
                                             uint32_t tau, long long quota, bool ties,
                                             long long gt_tile_before, long long eq_tile_before,
                                             surgeon_header* __restrict__ hdr,
                                             uint32_t* __restrict__ bitmap,
                                             typename Elem<DT>::type* __restrict__ values,
                                             uint32_t* __restrict__ offsets);
template <int DT>
__device__ __forceinline__ void load_tile(const typename Elem<DT>::type* __restrict__ x,
                                          long long n, int tile, uint4 (&q)[kRows]);

// ---- threshold (where still open), per-chunk counts, exclusive scan ------------------------------
// Launched cooperatively (all CTAs resident), so that the steps can be separated by grid-wide
// barriers: a counter every CTA increments and then polls, with a bounded number of polls.
// Returns false when the wait gave up (uniform over the CTA); the caller then leaves the kernel.
// `stall` is the diagnostic of SURGEON_DEBUG_STALL_BARRIER: the arrival target is one more than
// the CTAs that exist and the poll cap is 1024, so the wait is certain to run out, quickly.
__device__ __forceinline__ bool grid_barrier(SelectState* st, uint32_t& epoch, bool stall = false) {
  __shared__ uint32_t s_ok;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(&st->barrier_count, 1u);
    ++epoch;
    const uint32_t target = epoch * gridDim.x + (stall ? 1u : 0u);
    const uint32_t cap = stall ? 1024u : (1u << 22);
    uint32_t spins = 0, ok = 1;
    while (*reinterpret_cast<volatile uint32_t*>(&st->barrier_count) < target) {
      if (++spins > cap) { atomicMax(&st->error, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT)); ok = 0; break; }
      __nanosleep(40);
    }
    __threadfence();
    s_ok = ok;
  }
  __syncthreads();
  return s_ok != 0u;
}

// Calls f(key) for the first `cc` keys of chunk c's slot; one thread, 16-byte loads, four in flight.
template <int DT, typename F>
__device__ __forceinline__ void for_slot_keys(const typename Elem<DT>::type* __restrict__ slots,
                                              int c, uint32_t cc, F f) {
  constexpr int kSlot = (DT == 0) ? 64 : 128;
  constexpr int EPV = (DT == 0) ? 4 : 8;
  const uint4* __restrict__ p = reinterpret_cast<const uint4*>(slots + static_cast<long long>(c) * kSlot);
  const int nv = static_cast<int>((cc + EPV - 1) / EPV);
  for (int v0 = 0; v0 < nv; v0 += 4) {
    uint4 q[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) q[u] = (v0 + u < nv) ? __ldg(p + v0 + u) : make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint32_t w[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
      for (int e = 0; e < EPV; ++e) {
        const uint32_t idx = static_cast<uint32_t>((v0 + u) * EPV + e);
        const uint32_t key = (DT == 0) ? w[e % 4] : ((w[e >> 1] >> (16 * (e & 1))) & 0xFFFFu);
        if (idx < cc) f(key);
      }
    }
  }
}

// prefix[c] = (elements kept for sure before chunk c) << 31 | (ties at the threshold before it),
// c = 0 .. chunks (the last entry holds the totals).
// The fp32 instance is held to 32 registers (a few spills), so that a CTA fits on an SM beside one
// CTA of another stream's streaming kernel instead of waiting for an empty SM (those kernels are
// memory-bound in fp32 and lose nothing to the neighbour).  The bf16 streaming kernels are bound
// by instruction issue: sharing their SM cost the ViT-shaped stack 6 % even with the spills moved
// out of the way, so that instance keeps a whole SM.
template <int DT>
__global__ void __launch_bounds__(kSelThreads, DT == 0 ? 2 : 1)
count_kernel(const void* __restrict__ xv, long long n, uint32_t k, SelectState* __restrict__ st,
             surgeon_header* __restrict__ hdr, uint32_t* __restrict__ hist_b,
             uint32_t* __restrict__ hist_fb, const uint32_t* __restrict__ cnt_gt,
             const uint32_t* __restrict__ cand_cnt, const void* __restrict__ slots_v,
             unsigned long long* __restrict__ val, unsigned long long* __restrict__ prefix,
             unsigned long long* __restrict__ partial, int tiles,
             uint32_t* __restrict__ bitmap, void* __restrict__ values_v,
             uint32_t* __restrict__ offsets, int drop_zeros, int stall) {
  using E = typename Elem<DT>::type;
  constexpr uint32_t kMask = Elem<DT>::kKeyMask;
  constexpr int EPV = 16 / sizeof(E);
  constexpr long long kChunkElems = static_cast<long long>(kTileVecs) * EPV;
  __shared__ uint32_t s_hist[kBinsB];          // level B / fall-back digit histogram
  __shared__ int s_bnd;                        // the chunk inside which the tie quota ends, if this CTA owns it
  __shared__ uint32_t s_err;                   // a bounded wait of this call has given up
  __shared__ unsigned long long s_bnd_prefix;
  __shared__ uint32_t scratch[32];
  __shared__ uint32_t res[2];
  __shared__ unsigned long long s_tot[32];
  const E* __restrict__ x = reinterpret_cast<const E*>(xv);
  const E* __restrict__ slots = reinterpret_cast<const E*>(slots_v);
  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const uint32_t lane = lane_id();
  uint32_t epoch = 0;
  const uint32_t mode = __ldcg(&st->mode);
  uint32_t tau = 0, n_greater = 0;
  if (tid == 0) s_bnd = -1;                    // read after several barriers below
  // A barrier that gave up: the CTA reports it and leaves before it stores anything to the
  // outputs (the CTAs still waiting for it run out of polls in turn).
  auto leave = [&]() { if (tid == 0) atomicMax(&hdr->status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT)); };

  if (mode == 1u) {
    // ---- fall-back: exact radix select over the tensor itself, one digit per round ----
    constexpr int kRounds = (DT == 0) ? 3 : 2;
    const int shifts[3] = {DT == 0 ? 20 : 7, DT == 0 ? 10 : 0, 0};
    const int bits[3] = {DT == 0 ? 11 : 8, DT == 0 ? 10 : 7, 10};
    uint32_t fixed = 0, rank = k, above = 0;
    const long long nvec = n / EPV;
    const uint4* __restrict__ xq = reinterpret_cast<const uint4*>(xv);
    for (int round = 0; round < kRounds; ++round) {
      const int sh = shifts[round], nb = 1 << bits[round], hi = sh + bits[round];
      for (int i = tid; i < kFbBins; i += kSelThreads) s_hist[i] = 0;
      __syncthreads();
      uint32_t zero_cnt = 0;     // digit 0 in a register (half of post-ReLU data)
      auto add = [&](uint32_t key) {
        const bool match = hi >= 31 || (key >> hi) == (fixed >> hi);
        if (match) {
          const uint32_t d = (key >> sh) & (nb - 1);
          if (d == 0) ++zero_cnt;
          else atomicAdd(&s_hist[d], 1u);
        }
      };
      for (long long v = static_cast<long long>(blockIdx.x) * kSelThreads + tid; v < nvec;
           v += static_cast<long long>(gridDim.x) * kSelThreads) {
        const uint4 q = __ldg(xq + v);
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int i = 0; i < EPV; ++i)
          add(((DT == 0) ? w[i % 4] : (w[i >> 1] >> (16 * (i & 1)))) & kMask);
      }
      if (blockIdx.x == 0)
        for (long long j = nvec * EPV + tid; j < n; j += kSelThreads)
          add(static_cast<uint32_t>(x[j]) & kMask);
      zero_cnt = warp_sum(zero_cnt);
      if (lane == 0 && zero_cnt) atomicAdd(&s_hist[0], zero_cnt);
      __syncthreads();
      uint32_t* gh = hist_fb + round * kFbBins;
      for (int i = tid; i < kFbBins; i += kSelThreads)
        if (s_hist[i]) atomicAdd(&gh[i], s_hist[i]);
      if (!grid_barrier(st, epoch, stall != 0)) { leave(); return; }
      for (int i = tid; i < kFbBins; i += kSelThreads) s_hist[i] = __ldcg(gh + i);
      __syncthreads();
      find_from_top<kFbBins>([&](int i) { return s_hist[i]; }, rank, scratch, res);
      fixed |= res[0] << sh;
      above += res[1];
      rank -= res[1];
      __syncthreads();
    }
    tau = fixed;
    n_greater = above;
  } else if (mode == 0u) {
    // ---- further levels of at most 11 bits over the candidates that match so far ----
    const uint32_t lo_key = __ldcg(&st->lo_key);
    uint32_t shift = __ldcg(&st->shiftA), pre = __ldcg(&st->binA), rank = __ldcg(&st->rankA);
    uint32_t above_c = __ldcg(&st->aboveA);
    for (int level = 0; shift > 0; ++level) {
      const uint32_t nb = shift < 11u ? shift : 11u, ns = shift - nb;
      uint32_t* gh = hist_b + level * kFbBins;
      for (int c = blockIdx.x * kSelThreads + tid; c < tiles; c += gridDim.x * kSelThreads) {
        for_slot_keys<DT>(slots, c, __ldg(cand_cnt + c), [&](uint32_t key) {
          const uint32_t rel = key - lo_key;
          if ((rel >> shift) == pre) atomicAdd(&gh[(rel >> ns) & ((1u << nb) - 1u)], 1u);
        });
      }
      if (!grid_barrier(st, epoch, stall != 0)) { leave(); return; }
      for (int i = tid; i < kFbBins; i += kSelThreads) s_hist[i] = __ldcg(gh + i);
      __syncthreads();
      find_from_top<kFbBins>([&](int i) { return s_hist[i]; }, rank, scratch, res);
      pre = (pre << nb) | res[0];
      above_c += res[1];
      rank -= res[1];
      shift = ns;
      __syncthreads();
    }
    tau = lo_key + pre;
    n_greater = __ldcg(&st->above_total) + above_c;
  } else {
    tau = hdr->threshold_key;
  }
  const bool nz = drop_zeros && tau == 0u;       // store variant without kept zeros (see classify_kernel)
  const bool hdr_final = mode == 2u || mode == 4u;   // the classify pass has written the header
  if (!hdr_final && blockIdx.x == 0 && tid == 0) {
    hdr->threshold_key = tau;
    hdr->status = __ldcg(&st->error);
    hdr->n_keep = nz ? static_cast<long long>(n_greater) : static_cast<long long>(k);
    hdr->n_greater = n_greater;
    hdr->tie_quota = nz ? 0 : static_cast<long long>(k) - n_greater;
  }

  const long long quota = hdr_final ? hdr->tie_quota : (nz ? 0 : static_cast<long long>(k) - n_greater);

  // ---- per-chunk values; CTA b owns the chunks [b*per, (b+1)*per) ----
  const int per = (tiles + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
  const int c_begin = blockIdx.x * per < tiles ? blockIdx.x * per : tiles;
  const int c_end = c_begin + per < tiles ? c_begin + per : tiles;
  unsigned long long acc = 0;
  if (mode == 4u) {
    // every key inside the bracket equals the threshold (the slots may have overflowed): the
    // classify pass's counts are the answer
    for (int c = c_begin + tid; c < c_end; c += kSelThreads) {
      const unsigned long long v = (static_cast<unsigned long long>(__ldg(cnt_gt + c)) << 31) | __ldg(cand_cnt + c);
      val[c] = v;
      acc += v;
    }
  } else if (mode != 1u) {
    // one thread per chunk: the listed keys above / equal to the threshold complete the counts
    for (int c = c_begin + tid; c < c_end; c += kSelThreads) {
      const uint32_t cc = __ldg(cand_cnt + c), cg = __ldg(cnt_gt + c);
      uint32_t g = cg, q = 0;
      for_slot_keys<DT>(slots, c, cc, [&](uint32_t key) {
        g += key > tau ? 1u : 0u;
        q += key == tau ? 1u : 0u;
      });
      if (tau == 0) {         // lo_key == 1: whatever is neither above nor inside the bracket is 0
        const long long left = n - static_cast<long long>(c) * kChunkElems;
        q += static_cast<uint32_t>(left < kChunkElems ? left : kChunkElems) - cg - cc;
      }
      const unsigned long long v = (static_cast<unsigned long long>(g) << 31) | q;
      val[c] = v;
      acc += v;
    }
  } else {
   for (int c = c_begin + warp; c < c_end; c += 32) {
    uint32_t g = 0, q = 0;
    {
#pragma unroll
      for (int u = 0; u < kTileVecs / 32; ++u) {
        const long long base = (static_cast<long long>(c) * kTileVecs + u * 32 + lane) * EPV;
        if (base + EPV <= n) {
          const uint4 v = __ldg(reinterpret_cast<const uint4*>(x + base));
          const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int i = 0; i < EPV; ++i) {
            const uint32_t key = ((DT == 0) ? w[i % 4] : (w[i >> 1] >> (16 * (i & 1)))) & kMask;
            g += key > tau ? 1u : 0u;
            q += key == tau ? 1u : 0u;
          }
        } else {
          for (int i = 0; i < EPV; ++i) {
            if (base + i < n) {
              const uint32_t key = static_cast<uint32_t>(x[base + i]) & kMask;
              g += key > tau ? 1u : 0u;
              q += key == tau ? 1u : 0u;
            }
          }
        }
      }
      g = __reduce_add_sync(kFull, g);
      q = __reduce_add_sync(kFull, q);
    }
    const unsigned long long v = (static_cast<unsigned long long>(g) << 31) | q;
    if (lane == 0) { val[c] = v; acc += v; }
   }
  }
  acc = warp_sum_u64(acc);
  if (lane == 0) s_tot[warp] = acc;
  __syncthreads();
  if (tid == 0) {
    unsigned long long t = 0;
    for (int w = 0; w < 32; ++w) t += s_tot[w];
    partial[blockIdx.x] = t;
  }
  if (!grid_barrier(st, epoch, stall != 0)) { leave(); return; }

  // ---- exclusive scan: carry from the CTAs before, then warp w scans a sub-range ----
  unsigned long long carry = 0;
  {
    unsigned long long p = 0;
    for (int b = tid; b < static_cast<int>(blockIdx.x); b += kSelThreads) p += __ldcg(partial + b);
    p = warp_sum_u64(p);
    if (lane == 0) s_tot[warp] = p;
    __syncthreads();
    for (int w = 0; w < 32; ++w) carry += s_tot[w];
    __syncthreads();
  }
  const int sub = ((per + 31) / 32 + 31) & ~31;
  const int begin = c_begin + warp * sub < c_end ? c_begin + warp * sub : c_end;
  const int end = begin + sub < c_end ? begin + sub : c_end;
  unsigned long long wsum = 0;
#pragma unroll 4
  for (int c = begin + lane; c < end; c += 32) wsum += __ldcg(val + c);
  wsum = warp_sum_u64(wsum);
  if (lane == 0) s_tot[warp] = wsum;
  __syncthreads();
  for (int w = 0; w < warp; ++w) carry += s_tot[w];
  for (int c0 = begin; c0 < end; c0 += 32) {
    const int c = c0 + lane;
    const unsigned long long v = c < end ? __ldcg(val + c) : 0ull;
    unsigned long long incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long up = __shfl_up_sync(kFull, incl, o);
      if (lane >= static_cast<uint32_t>(o)) incl += up;
    }
    if (c < end) {
      const unsigned long long ex = carry + incl - v;
      prefix[c] = ex;
      const long long eq_b = static_cast<long long>(ex & 0x7FFFFFFFull);
      const long long eq_e = static_cast<long long>((ex + v) & 0x7FFFFFFFull);
      if (eq_b < quota && eq_e > quota) { s_bnd = c; s_bnd_prefix = ex; }
    }
    carry += __shfl_sync(kFull, incl, 31);
  }
  // The chunk inside which the tie quota ends is emitted here, with its ties ranked by index, by
  // the first two warps of the CTA that owns it; the compaction kernels skip that chunk.
  // Nothing is stored to the outputs once a bounded wait has given up anywhere in this call (the
  // counts the offsets come from may then be incomplete).
  if (tid == 0) s_err = *reinterpret_cast<volatile uint32_t*>(&st->error);
  __syncthreads();
  if (s_err == 0u && s_bnd >= 0 && warp < kTileWarps) {
    const unsigned long long pb = s_bnd_prefix;
    uint4 q[kRows];
    load_tile<DT>(x, n, s_bnd, q);
    compact_tile<DT, true>(x, n, q, s_bnd, tau, quota, false, static_cast<long long>(pb >> 31),
                           static_cast<long long>(pb & kCountMask), hdr, bitmap,
                           reinterpret_cast<E*>(values_v), offsets);
  }
  if (c_end == tiles && c_begin < tiles) {
    // the CTA that owns the last chunk also writes the totals and checks them
    __syncthreads();
    if (tid == 0) {
      // the sentinel entry of the block offsets = the number of stored values
      offsets[(n + SURGEON_BLOCK - 1) >> kBlockShift] =
          nz ? static_cast<uint32_t>(hdr_final ? hdr->n_greater : n_greater) : k;
      unsigned long long total = 0;
      for (int b = 0; b <= static_cast<int>(blockIdx.x); ++b) total += __ldcg(partial + b);
      prefix[tiles] = total;
      const long long gt_all = static_cast<long long>(total >> 31);
      const long long eq_all = static_cast<long long>(total & 0x7FFFFFFFull);
      const long long ng = hdr_final ? hdr->n_greater : static_cast<long long>(n_greater);
      const long long want = nz ? ng : static_cast<long long>(k);
      const long long kept = gt_all + (eq_all < quota ? eq_all : quota);
      // every mode and every barrier of this kernel is behind us: whatever gave up shows now
      const uint32_t err = *reinterpret_cast<volatile uint32_t*>(&st->error);
      if (err) atomicMax(&hdr->status, err);
      else if (gt_all != ng || kept != want)
        atomicMax(&hdr->status, static_cast<uint32_t>(SURGEON_ERR_INTERNAL));
    }
  }
}

// ---- compaction -----------------------------------------------------------------------------

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

// Emits one tile.  SLOW = false: every tie of the tile is kept, or none is (`ties`), so one
// decision per element suffices.  SLOW = true: the tie quota ends inside this tile; ties are
// ranked by flat index.  Nothing is exchanged between CTAs.
template <int DT, bool SLOW>
__device__ __forceinline__ void compact_tile(const typename Elem<DT>::type* __restrict__ x,
                                             long long n, const uint4 (&q)[kRows], int tile,
                                             uint32_t tau, long long quota, bool ties,
                                             long long gt_tile_before, long long eq_tile_before,
                                             surgeon_header* __restrict__ hdr,
                                             uint32_t* __restrict__ bitmap,
                                             typename Elem<DT>::type* __restrict__ values,
                                             uint32_t* __restrict__ offsets) {
  using E = typename Elem<DT>::type;
  constexpr uint32_t kMask = Elem<DT>::kKeyMask;
  constexpr int EPV = 16 / sizeof(E);          // elements per lane and row: 4 (fp32) / 8 (bf16)
  constexpr int ROW = 32 * EPV;                // elements per row: 128 / 256
  constexpr int WPR = ROW / 32;                // bitmap words per row: 4 / 8
  constexpr int LPW = 32 / EPV;                // lanes per bitmap word: 8 / 4
  constexpr int BPR = ROW / SURGEON_BLOCK;     // offset blocks per row: 1 / 2
  constexpr uint32_t kEMask = (1u << EPV) - 1u;
  __shared__ uint32_t s_gt[kTileWarps], s_eq[kTileWarps];
  const uint32_t lane = lane_id();
  const int warp = threadIdx.x >> 5;
  const long long n_blocks = (n + SURGEON_BLOCK - 1) >> kBlockShift;
  const long long n_words = (n + 31) / 32;
  const int my_word = lane / LPW;
  const int my_shift = EPV * (lane % LPW);
  const long long row0 = (static_cast<long long>(tile) * kTileWarps + warp) * kRows;

  // per row and lane EPV decisions: g = kept for sure, e = tie at the threshold (SLOW only)
  uint32_t g_all = 0, e_all = 0;      // kRows fields of EPV bits
#pragma unroll
  for (int r = 0; r < kRows; ++r) {
    const long long base = (row0 + r) * ROW + static_cast<long long>(lane) * EPV;
    const uint32_t w[4] = {q[r].x, q[r].y, q[r].z, q[r].w};
    uint32_t g = 0, e = 0;
#pragma unroll
    for (int i = 0; i < EPV; ++i) {
      const uint32_t bits = (DT == 0) ? w[i % 4] : (w[i >> 1] >> (16 * (i & 1)));
      const uint32_t key = bits & kMask;
      const bool valid = base + i < n;
      if (SLOW) {
        g |= (valid && key > tau) ? (1u << i) : 0u;
        e |= (valid && key == tau) ? (1u << i) : 0u;
      } else {
        g |= (valid && (key > tau || (ties && key == tau))) ? (1u << i) : 0u;
      }
    }
    g_all |= g << (EPV * r);
    e_all |= e << (EPV * r);
  }
  const uint32_t gt_warp = __reduce_add_sync(kFull, __popc(g_all));
  const uint32_t eq_warp = SLOW ? __reduce_add_sync(kFull, __popc(e_all)) : 0u;
  if (lane == 0) { s_gt[warp] = gt_warp; s_eq[warp] = eq_warp; }
  asm volatile("bar.sync 1, %0;" ::"n"(kCompactThreads) : "memory");   // the tile's two warps only

  long long gt_before = gt_tile_before, eq_before = eq_tile_before;
#pragma unroll
  for (int w = 0; w < kTileWarps; ++w) {
    if (w < warp) { gt_before += s_gt[w]; eq_before += s_eq[w]; }
  }
  // kept before = all greater + the ties that fit the quota.  In the fast path the kept ties of
  // this tile are already inside the "greater" counts and eq_before stays the tile's value.
  long long kept_before = gt_before + (eq_before < quota ? eq_before : quota);

  uint32_t my_words[WPR];      // lane r keeps the bitmap words of row r
  uint32_t my_off[BPR];        // and the offsets of its blocks
  uint32_t my_cnt[BPR];
#pragma unroll
  for (int j = 0; j < WPR; ++j) my_words[j] = 0;
#pragma unroll
  for (int j = 0; j < BPR; ++j) { my_off[j] = 0; my_cnt[j] = 0; }

  if (row0 * ROW < n) {
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      uint32_t keep = (g_all >> (EPV * r)) & kEMask;
      if (SLOW) {
        const uint32_t e = (e_all >> (EPV * r)) & kEMask;
        const uint32_t ec = __popc(e);
        const uint32_t before = warp_excl_scan(ec);      // ties of this row in lower lanes
        keep |= lowest_set_bits(e, quota - eq_before - before);
        eq_before += warp_sum(ec);
      }
      // bitmap words of the row, known to every lane
      const uint32_t shifted = keep << my_shift;
      uint32_t words[WPR];
#pragma unroll
      for (int j = 0; j < WPR; ++j)
        words[j] = __reduce_or_sync(kFull, my_word == j ? shifted : 0u);
      uint32_t pre = 0, total = 0, half = 0;
#pragma unroll
      for (int j = 0; j < WPR; ++j) {
        const uint32_t pc = __popc(words[j]);
        if (j < my_word) pre += pc;
        if (j == my_word) pre += __popc(words[j] & ((1u << my_shift) - 1u));
        if (j < WPR / 2) half += pc;
        total += pc;
      }
      if (static_cast<int>(lane) == r) {
#pragma unroll
        for (int j = 0; j < WPR; ++j) my_words[j] = words[j];
        my_off[0] = static_cast<uint32_t>(kept_before);
        if (BPR == 2) {
          my_off[BPR - 1] = static_cast<uint32_t>(kept_before) + half;
          my_cnt[0] = half;
          my_cnt[BPR - 1] = total - half;
        } else {
          my_cnt[0] = total;
        }
      }
      // packed values: consecutive kept elements go to consecutive addresses
      E* dst = values + kept_before + pre;
      const uint32_t w[4] = {q[r].x, q[r].y, q[r].z, q[r].w};
#pragma unroll
      for (int i = 0; i < EPV; ++i) {
        if ((keep >> i) & 1u) {
          if (SURGEON_IN_BOUNDS(dst - values, hdr->n_keep, &hdr->status))
            *dst = (DT == 0) ? static_cast<E>(w[i % 4])
                             : static_cast<E>((w[i >> 1] >> (16 * (i & 1))) & 0xFFFFu);
          ++dst;
        }
      }
      kept_before += total;
    }
    // lanes 0..kRows-1 store the words and offsets of their rows: contiguous 16-byte pieces
    if (lane < kRows) {
      const long long row = row0 + lane;
      const long long w0 = row * WPR;
      if (w0 + WPR <= n_words) {
#pragma unroll
        for (int j = 0; j < WPR; j += 4)
          *reinterpret_cast<uint4*>(bitmap + w0 + j) =
              make_uint4(my_words[j], my_words[j + 1], my_words[j + 2], my_words[j + 3]);
      } else {
#pragma unroll
        for (int j = 0; j < WPR; ++j)
          if (w0 + j < n_words) bitmap[w0 + j] = my_words[j];
      }
#pragma unroll
      for (int j = 0; j < BPR; ++j) {
        const long long blk = row * BPR + j;
        if (blk < n_blocks) {
          offsets[blk] = my_off[j];
          if (blk == n_blocks - 1) {
            const long long total = static_cast<long long>(my_off[j]) + my_cnt[j];
            offsets[n_blocks] = static_cast<uint32_t>(total);
            if (total != hdr->n_keep)
              atomicMax(&hdr->status, static_cast<uint32_t>(SURGEON_ERR_INTERNAL));
          }
        }
      }
    }
  }
}

template <int DT>
__device__ __forceinline__ void load_tile(const typename Elem<DT>::type* __restrict__ x,
                                          long long n, int tile, uint4 (&q)[kRows]) {
  constexpr int EPV = 16 / sizeof(typename Elem<DT>::type);
  constexpr int ROW = 32 * EPV;
  const long long row0 = (static_cast<long long>(tile) * kTileWarps + (threadIdx.x >> 5)) * kRows;
#pragma unroll
  for (int r = 0; r < kRows; ++r) {
    const long long base = (row0 + r) * ROW + static_cast<long long>(lane_id()) * EPV;
    if (base + EPV <= n) {
      q[r] = __ldg(reinterpret_cast<const uint4*>(x + base));
    } else {
      uint32_t t[8];
#pragma unroll
      for (int i = 0; i < 8; ++i)
        t[i] = (i < EPV && base + i < n) ? static_cast<uint32_t>(x[base + i]) : 0u;
      if (DT == 0) q[r] = make_uint4(t[0], t[1], t[2], t[3]);
      else q[r] = make_uint4(t[0] | (t[1] << 16), t[2] | (t[3] << 16), t[4] | (t[5] << 16),
                             t[6] | (t[7] << 16));
    }
  }
}

// True when a bounded wait of the select gave up or a self-check failed (uniform over the CTA); the
// status reaches the header, and the caller stores nothing: offsets taken from incomplete counts
// could point past the end of `values`.
__device__ __forceinline__ bool gave_up(surgeon_header* __restrict__ hdr, const uint32_t* __restrict__ err) {
  const uint32_t e = __ldcg(err);
  const uint32_t s = *reinterpret_cast<volatile uint32_t*>(&hdr->status);
  if (e && threadIdx.x == 0) atomicMax(&hdr->status, e);
  return (e | s) != 0u;
}

// One small CTA per tile: used for tensors too small for the streaming kernel.  The one tile
// inside which the tie quota ends (if any) is left to the count kernel.
template <int DT>
__global__ void __launch_bounds__(kCompactThreads)
compact_small_kernel(const void* __restrict__ xv, long long n, surgeon_header* __restrict__ hdr,
               uint32_t* __restrict__ bitmap, void* __restrict__ values_v,
               uint32_t* __restrict__ offsets, const unsigned long long* __restrict__ prefix,
               const uint32_t* __restrict__ err) {
  using E = typename Elem<DT>::type;
  const E* __restrict__ x = reinterpret_cast<const E*>(xv);
  const int tile = blockIdx.x;
  uint4 q[kRows];
  load_tile<DT>(x, n, tile, q);     // in flight while the header and the scan entries arrive
  if (gave_up(hdr, err)) return;    // the scan may be incomplete: store nothing
  const uint32_t tau = hdr->threshold_key;
  const long long quota = hdr->tie_quota;
  const unsigned long long pb = prefix[tile], pe = prefix[tile + 1];
  const long long eq_b = static_cast<long long>(pb & kCountMask);
  const long long eq_e = static_cast<long long>(pe & kCountMask);
  if (eq_b < quota && eq_e > quota) return;            // boundary tile
  compact_tile<DT, false>(x, n, q, tile, tau, quota, /*ties=*/eq_e <= quota,
                          static_cast<long long>(pb >> 31), eq_b, hdr, bitmap,
                          reinterpret_cast<E*>(values_v), offsets);
}

// ---- streaming compaction ---------------------------------------------------------------------
// Same ring and lane-per-row layout as classify_kernel.  A lane builds the bitmap word(s) of its
// row with no cross-lane traffic; one warp scan places the lanes' kept values; they are gathered
// in the warp's part of the stage (in place) and leave as 16-byte vectors.
template <int DT>
__global__ void __launch_bounds__(kCsThreads, 2)
compact_stream_kernel(const __grid_constant__ CUtensorMap xmap, const void* __restrict__ xv,
                      long long n, long long n_rows_full, surgeon_header* __restrict__ hdr,
                      uint32_t* __restrict__ bitmap, void* __restrict__ values_v,
                      uint32_t* __restrict__ offsets, const unsigned long long* __restrict__ prefix,
                      const uint32_t* __restrict__ err, int n_chunks, int n_stage_tiles) {
  using E = typename Elem<DT>::type;
  constexpr uint32_t kMask = Elem<DT>::kKeyMask;
  constexpr int EPR = 128 / sizeof(E);         // elements per row (= per lane): 32 / 64
  constexpr int EPV = 16 / sizeof(E);          // elements per 16-byte vector: 4 / 8
  constexpr int WPL = EPR / 32;                // bitmap words per lane: 1 / 2
  constexpr int BPC = 32 * EPR / SURGEON_BLOCK;   // offset blocks per chunk: 8 / 16
  constexpr int LPB = 32 / BPC;                // lanes per offset block: 4 / 2
  extern __shared__ __align__(1024) unsigned char cs_smem_raw[];
  unsigned char* ring = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(cs_smem_raw) + kCsAlign - 1) & ~(kCsAlign - 1));
  __shared__ __align__(8) unsigned long long bars[2 * kCsStages];
  const E* __restrict__ x = reinterpret_cast<const E*>(xv);
  E* __restrict__ values = reinterpret_cast<E*>(values_v);
  const int warp = threadIdx.x >> 5;
  const uint32_t lane = lane_id();
  const uint32_t full_bar = smem_u32(bars);
  const uint32_t empty_bar = smem_u32(bars + kCsStages);
  if (gave_up(hdr, err)) return;   // before any load or store; the whole CTA takes the same way
  if (threadIdx.x == 0) {
    tc::tma_prefetch_desc(&xmap);
    for (int s = 0; s < kCsStages; ++s) {
      tc::mbar_init(full_bar + 8 * s, 1);
      tc::mbar_init(empty_bar + 8 * s, kCsWarps);
    }
    tc::fence_barrier_init();
  }
  __syncthreads();
  const int first = blockIdx.x;
  const int n_it = first < n_stage_tiles ? (n_stage_tiles - 1 - first) / static_cast<int>(gridDim.x) + 1 : 0;

  if (warp == kCsWarps) {
    // ---- producer ----
    if (lane == 0) {
      for (int it = 0; it < n_it; ++it) {
        const int s = it % kCsStages;
        if (it >= kCsStages && !tc::mbar_wait(empty_bar + 8 * s, ((it / kCsStages) - 1) & 1, 20)) {
          atomicMax(&hdr->status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
          break;
        }
        const int t = first + it * static_cast<int>(gridDim.x);
        tc::mbar_arrive_expect_tx(full_bar + 8 * s, kCsStageBytes);
        tc::tma_load_2d(smem_u32(ring + s * kCsStageBytes), &xmap, 0, t * kCsStageRows,
                        full_bar + 8 * s);
      }
    }
    return;
  }

  // ---- consumers ----
  const uint32_t tau = hdr->threshold_key;
  const long long quota = hdr->tie_quota;
  const bool none = hdr->n_keep == 0;
  const long long n_words = (n + 31) / 32;
  const long long n_blocks = (n + SURGEON_BLOCK - 1) >> kBlockShift;
  auto chunk_of = [&](int it) { return (first + it * static_cast<int>(gridDim.x)) * kCsWarps + warp; };
  unsigned long long pb = 0, pe = 0;    // scan entries of this iteration's chunk, fetched one ahead
  if (n_it > 0 && chunk_of(0) < n_chunks) { pb = prefix[chunk_of(0)]; pe = prefix[chunk_of(0) + 1]; }
  for (int it = 0; it < n_it; ++it) {
    const int s = it % kCsStages;
    const int chunk = chunk_of(it);
    unsigned long long pb_next = 0, pe_next = 0;
    if (it + 1 < n_it && chunk_of(it + 1) < n_chunks) {
      pb_next = prefix[chunk_of(it + 1)];
      pe_next = prefix[chunk_of(it + 1) + 1];
    }
    if (!tc::mbar_wait(full_bar + 8 * s, (it / kCsStages) & 1, 20)) {
      if (lane == 0) atomicMax(&hdr->status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
      break;
    }
    unsigned char* region = ring + s * kCsStageBytes + warp * 4096;   // this warp's 32 rows
    const long long eq_b = static_cast<long long>(pb & kCountMask);
    const long long eq_e = static_cast<long long>(pe & kCountMask);
    const bool boundary = eq_b < quota && eq_e > quota;   // left to the count kernel
    if (chunk < n_chunks && !boundary) {
      // ---- this lane's row: 8 vectors, un-swizzled ----
      uint4 q[8];
      const unsigned char* row = region + lane * 128;
#pragma unroll
      for (int j = 0; j < 8; ++j)
        q[j] = *reinterpret_cast<const uint4*>(row + ((j ^ (lane & 7)) << 4));
      const long long grow = static_cast<long long>(chunk) * 32 + lane;   // row index in the tensor
      const long long e0 = grow * EPR;
      long long nv = n - e0;                      // valid elements of the row
      nv = nv < 0 ? 0 : (nv > EPR ? EPR : nv);
      if (grow >= n_rows_full && nv > 0) {        // the ragged last row is not covered by the map
        uint32_t t[64];
#pragma unroll
        for (int i = 0; i < 64; ++i) t[i] = (i < EPR && i < nv) ? static_cast<uint32_t>(x[e0 + i]) : 0u;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (DT == 0) q[j] = make_uint4(t[4 * j], t[4 * j + 1], t[4 * j + 2], t[4 * j + 3]);
          else q[j] = make_uint4(t[8 * j] | (t[8 * j + 1] << 16), t[8 * j + 2] | (t[8 * j + 3] << 16),
                                 t[8 * j + 4] | (t[8 * j + 5] << 16), t[8 * j + 6] | (t[8 * j + 7] << 16));
        }
      }
      // ---- one decision per element: key >= thr ----
      const bool ties = eq_e <= quota;            // every tie of this chunk is kept (else none is)
      const uint32_t thr = ties ? tau : tau + 1u;
      uint32_t word[WPL];
#pragma unroll
      for (int w = 0; w < WPL; ++w) word[w] = 0;
      const uint32_t c_thr = ge_const(thr > 0x8000u ? 0x8000u : thr);   // bf16: packed pairs of keys
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t c[4] = {q[j].x, q[j].y, q[j].z, q[j].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (DT == 0) {
            // key < thr is the sign bit of key - thr (key < 2^31, thr <= 2^31); collected by a funnel
            // shift with element e in bit 31 - e, put back in order below
            word[0] = __funnelshift_l((c[i] & kMask) - thr, word[0], 1);
          } else {
            const int pw = 4 * j + i;             // packed word of the row: elements 2pw, 2pw + 1
            word[(pw >> 4) % WPL] |= pair_flags(c[i] & 0x7FFF7FFFu, c_thr, pw & 15);
          }
        }
      }
      if (DT != 0) {
#pragma unroll
        for (int w = 0; w < WPL; ++w) word[w] = pairs_to_element_order(word[w]);
      } else {
        word[0] = ~__brev(word[0]);
      }
#pragma unroll
      for (int w = 0; w < WPL; ++w) {
        const long long left = nv - 32 * w;
        const uint32_t vmask = left >= 32 ? 0xFFFFFFFFu : (left <= 0 ? 0u : ((1u << left) - 1u));
        word[w] = none ? 0u : (word[w] & vmask);
      }
      uint32_t cnt = 0;
#pragma unroll
      for (int w = 0; w < WPL; ++w) cnt += __popc(word[w]);
      uint32_t incl = cnt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t up = __shfl_up_sync(kFull, incl, o);
        if (lane >= static_cast<uint32_t>(o)) incl += up;
      }
      const uint32_t lane_pre = incl - cnt;
      const uint32_t total = __shfl_sync(kFull, incl, 31);
      const long long kept_before = static_cast<long long>(pb >> 31) + (eq_b < quota ? eq_b : quota);

      // ---- bitmap words and block offsets: coalesced ----
#pragma unroll
      for (int w = 0; w < WPL; ++w) {
        const long long wi = static_cast<long long>(chunk) * 32 * WPL + lane * WPL + w;
        if (wi < n_words) bitmap[wi] = word[w];
      }
      const uint32_t off = __shfl_sync(kFull, lane_pre, (lane * LPB) & 31);
      const long long blk = static_cast<long long>(chunk) * BPC + lane;
      if (lane < BPC && blk < n_blocks) offsets[blk] = static_cast<uint32_t>(kept_before) + off;

      // ---- kept values: gathered in place (packed order), then out as 16-byte vectors ----
      __syncwarp();                                // every lane has its row in registers
      E* outp = reinterpret_cast<E*>(region);
      // The byte at offset a of the packed sequence lives at a ^ ((a >> 5) & 0x7C): the 32-bit word
      // index is XORed with the index of its 128-byte row.  Without it, lanes that keep their
      // whole row (chunks before the end of a large tie quota, e.g. the zeros of post-ReLU data at
      // a low ratio) all start a multiple of 32 words apart and every store of the gather is a
      // 32-way bank conflict.  The region is 4 KB-aligned, so the same expression works on the
      // full shared-memory address.
      auto swz = [](uint32_t p) -> uint32_t {       // the same map on element indices
        return p ^ ((((p * static_cast<uint32_t>(sizeof(E))) >> 7) & 31u) << (DT == 0 ? 0 : 1));
      };
      // The sequence starts `mis` elements into the region when that fits, mis = the misalignment
      // of its destination in `values`: 16-byte vectors of the region and of `values` then line up.
      const uint32_t mis = static_cast<uint32_t>(kept_before % EPV);
      const bool lined_up = total + mis <= static_cast<uint32_t>(32 * EPR);
      const uint32_t shift = lined_up ? mis : 0u;
      const uint32_t rbase = smem_u32(region);
      uint32_t a = rbase + (lane_pre + shift) * static_cast<uint32_t>(sizeof(E));
      auto put = [&](uint32_t v) {
        const uint32_t pa = a ^ ((a >> 5) & 0x7Cu);
        if (DT == 0) asm volatile("st.shared.u32 [%0], %1;" ::"r"(pa), "r"(v) : "memory");
        else asm volatile("st.shared.u16 [%0], %1;" ::"r"(pa), "h"(static_cast<unsigned short>(v)) : "memory");
        a += static_cast<uint32_t>(sizeof(E));
      };
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t c[4] = {q[j].x, q[j].y, q[j].z, q[j].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (DT == 0) {
            if ((word[0] >> (4 * j + i)) & 1u) put(c[i]);
          } else {
            const int e = 8 * j + 2 * i;
            if ((word[(e >> 5) % WPL] >> (e & 31)) & 1u) put(c[i]);
            if ((word[(e >> 5) % WPL] >> ((e + 1) & 31)) & 1u) put(c[i] >> 16);
          }
        }
      }
      __syncwarp();
      if (lined_up) {
        // slots [mis, mis + total) of the region go to gbase[mis ...]; gbase is 16-byte aligned
        E* gbase = values + (kept_before - mis);
        const uint32_t end = mis + total;
        const uint32_t v_first = mis ? 1u : 0u;    // first whole vector
        const uint32_t v_end = end / EPV;          // one past the last whole vector
        if (mis) {
          const uint32_t sl = mis + lane;
          if (sl < static_cast<uint32_t>(EPV) && sl < end &&
              SURGEON_IN_BOUNDS(kept_before - mis + sl, hdr->n_keep, &hdr->status))
            gbase[sl] = outp[swz(sl)];
        }
        for (uint32_t g = v_first + lane; g < v_end; g += 32) {
          // the four words of a vector share their row: one 16-byte load, words permuted by the XOR
          const uint32_t la = g * 16u;
          const uint32_t xr = (la >> 5) & 0x7Cu;
          uint4 u = *reinterpret_cast<const uint4*>(region + (la ^ (xr & 0x70u)));
          if (xr & 4u) { uint32_t t = u.x; u.x = u.y; u.y = t; t = u.z; u.z = u.w; u.w = t; }
          if (xr & 8u) { uint32_t t = u.x; u.x = u.z; u.z = t; t = u.y; u.y = u.w; u.w = t; }
          if (SURGEON_IN_BOUNDS(kept_before - mis + g * EPV + EPV - 1, hdr->n_keep, &hdr->status))
            *reinterpret_cast<uint4*>(gbase + g * EPV) = u;
        }
        const uint32_t t0 = (v_end > v_first ? v_end : v_first) * EPV;
        if (t0 + lane < end && SURGEON_IN_BOUNDS(kept_before - mis + t0 + lane, hdr->n_keep, &hdr->status))
          gbase[t0 + lane] = outp[swz(t0 + lane)];
      } else {
        // a full chunk with a misaligned destination: no room for the shift, element-wise vectors
        E* dst = values + kept_before;
        uint32_t head = mis ? EPV - mis : 0;
        if (head > total) head = total;
        const uint32_t n_vec = (total - head) / EPV;
        if (lane < head && SURGEON_IN_BOUNDS(kept_before + lane, hdr->n_keep, &hdr->status))
          dst[lane] = outp[swz(lane)];
        for (uint32_t v = lane; v < n_vec; v += 32) {
          const uint32_t b = head + v * EPV;
          uint4 o;
          if (DT == 0) {
            o = make_uint4(outp[swz(b)], outp[swz(b + 1)], outp[swz(b + 2)], outp[swz(b + 3)]);
          } else {
            o = make_uint4(outp[swz(b)] | (static_cast<uint32_t>(outp[swz(b + 1)]) << 16),
                           outp[swz(b + 2)] | (static_cast<uint32_t>(outp[swz(b + 3)]) << 16),
                           outp[swz(b + 4 % EPV)] | (static_cast<uint32_t>(outp[swz(b + 5 % EPV)]) << 16),
                           outp[swz(b + 6 % EPV)] | (static_cast<uint32_t>(outp[swz(b + 7 % EPV)]) << 16));
          }
          if (SURGEON_IN_BOUNDS(kept_before + head + v * EPV + EPV - 1, hdr->n_keep, &hdr->status))
            *reinterpret_cast<uint4*>(dst + head + v * EPV) = o;
        }
        const uint32_t done = head + n_vec * EPV;
        if (lane < total - done && SURGEON_IN_BOUNDS(kept_before + done + lane, hdr->n_keep, &hdr->status))
          dst[done + lane] = outp[swz(done + lane)];
      }
    }
    tc::fence_proxy_async();     // this warp's writes to the stage precede the next TMA fill
    __syncwarp();
    if (lane == 0) tc::mbar_arrive(empty_bar + 8 * s);
    pb = pb_next;
    pe = pe_next;
  }
}

__global__ void offsets_empty_kernel(uint32_t* offsets) { offsets[0] = 0u; }

// ---- decompress -------------------------------------------------------------------------------

// Algorithm 1, Reshape step: one warp rebuilds 1024 elements (32 bitmap words) of the dense tensor.
template <int DT>
__global__ void __launch_bounds__(256)
decompress_kernel(const uint32_t* __restrict__ bitmap, const void* __restrict__ values_v,
                  const uint32_t* __restrict__ offsets, long long n, void* __restrict__ out_v) {
  using E = typename Elem<DT>::type;
  const E* __restrict__ values = reinterpret_cast<const E*>(values_v);
  E* __restrict__ out = reinterpret_cast<E*>(out_v);
  const uint32_t lane = lane_id();
  const long long n_chunks = (n + 1023) / 1024;
  const long long n_words = (n + 31) / 32;
  const long long warps = (static_cast<long long>(gridDim.x) * blockDim.x) >> 5;
  for (long long chunk = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
       chunk < n_chunks; chunk += warps) {
    const long long w_idx = chunk * 32 + lane;
    const uint32_t word = (w_idx < n_words) ? bitmap[w_idx] : 0u;
    const uint32_t word_excl = warp_excl_scan(__popc(word));
    const long long first = offsets[chunk * (1024 / SURGEON_BLOCK)];
    const uint32_t lt = lanemask_lt();
    const long long base = chunk * 1024;
#pragma unroll 4
    for (int i = 0; i < 32; ++i) {
      const uint32_t w = __shfl_sync(kFull, word, i);
      const uint32_t wb = __shfl_sync(kFull, word_excl, i);
      const long long idx = base + i * 32 + lane;
      if (idx < n) out[idx] = ((w >> lane) & 1u) ? values[first + wb + __popc(w & lt)]
                                                 : static_cast<E>(0);
    }
  }
}

using TmaEncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                 const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                 const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The tensor as rows of 128 bytes (32 words), box = one ring stage, 128-byte swizzle.
bool make_row_map(const void* x, long long n_rows_full, CUtensorMap* map) {
  const TmaEncodeFn encode = reinterpret_cast<TmaEncodeFn>(tensor_map_encode_fn());
  if (!encode) return false;
  const cuuint64_t dims[2] = {32, static_cast<cuuint64_t>(n_rows_full)};
  const cuuint64_t strides[1] = {128};
  const cuuint32_t box[2] = {32, static_cast<cuuint32_t>(kCsStageRows)};
  const cuuint32_t estr[2] = {1, 1};
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(x), dims, strides, box,
                estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int DT>
cudaError_t run_prune_compact(const void* x, long long n, long long k, int drop_zeros, int stall,
                              const surgeon_compressed& out, void* workspace,
                              cudaStream_t stream) {
  using E = typename Elem<DT>::type;
  constexpr int VEC = 16 / static_cast<int>(sizeof(E));
  const PruneLayout L = prune_layout(n, DT);
  char* ws = static_cast<char*>(workspace);
  SelectState* st = reinterpret_cast<SelectState*>(ws);
  uint32_t* hist_s = reinterpret_cast<uint32_t*>(ws + L.hist_s);
  uint32_t* hist_a = reinterpret_cast<uint32_t*>(ws + L.hist_a);
  uint32_t* hist_b = reinterpret_cast<uint32_t*>(ws + L.hist_b);
  uint32_t* hist_fb = reinterpret_cast<uint32_t*>(ws + L.hist_fb);
  uint32_t* cnt_gt = reinterpret_cast<uint32_t*>(ws + L.cnt_gt);
  uint32_t* cand_cnt = reinterpret_cast<uint32_t*>(ws + L.cand_cnt);
  unsigned long long* val = reinterpret_cast<unsigned long long*>(ws + L.val);
  unsigned long long* prefix = reinterpret_cast<unsigned long long*>(ws + L.prefix);
  unsigned long long* partial = reinterpret_cast<unsigned long long*>(ws + L.partial);
  void* slots = ws + L.slots;
  cudaError_t e = cudaMemsetAsync(workspace, 0, L.zero_bytes, stream);
  if (e != cudaSuccess) return e;
  const int sms = sm_count();
  static bool attrs_done_on[64] = {false};   // per device; a race only repeats idempotent calls
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
  if (!attrs_done_on[dev]) {
    e = cudaFuncSetAttribute(sample_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kHistWords * 4);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(classify_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(kCsSmem));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(compact_stream_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(kCsSmem));
    if (e != cudaSuccess) return e;
    attrs_done_on[dev] = true;
  }
  const long long n_rows_full = n * static_cast<long long>(sizeof(E)) / 128;
  const int n_chunks = static_cast<int>(L.tiles);
  const int n_stage_tiles = (n_chunks + kCsWarps - 1) / kCsWarps;
  // at least kMinTilesPerCta stages per CTA: a CTA's set-up and tail cost about two stages' time, and a
  // small tensor then leaves SM slots to the kernels of other streams
  const int want_ctas = (n_stage_tiles + kMinTilesPerCta - 1) / kMinTilesPerCta;
  const int stream_grid = want_ctas < 2 * sms ? want_ctas : 2 * sms;
  CUtensorMap map;
  const bool streamed = n * static_cast<long long>(sizeof(E)) >= kStreamMinBytes && make_row_map(x, n_rows_full, &map);

  if (k == 0) {
    header_empty_kernel<<<1, 1, 0, stream>>>(out.header, Elem<DT>::kSentinel, out.block_offsets,
                                             (n + SURGEON_BLOCK - 1) >> kBlockShift);
    note_launches(1);
    if (n > 0) {   // nothing is kept: the scan is all zeros
      e = cudaMemsetAsync(prefix, 0, static_cast<size_t>(L.tiles + 1) * 8, stream);
      if (e != cudaSuccess) return e;
    }
  } else {
    if (streamed) {
      // sample: segments of 32 vectors, about 1/32 of the tensor, at most 16384 segments
      const long long n_seg_all = (n / VEC) / 32;
      long long n_seg = n_seg_all / 32;
      if (n_seg < 256) n_seg = 256;
      if (n_seg > 16384) n_seg = 16384;
      const long long seg_stride = n_seg_all / n_seg;   // >= 1: a streamed tensor has at least 2^22 elements
      const long long want = (n_seg + 127) / 128;
      const int grid = static_cast<int>(want < sms ? want : sms);
      sample_kernel<DT><<<grid, kSelThreads, kHistWords * 4, stream>>>(
          reinterpret_cast<const uint4*>(x), n, static_cast<uint32_t>(k),
          static_cast<uint32_t>(n_seg), static_cast<uint32_t>(seg_stride), st, hist_s);
      classify_kernel<DT><<<stream_grid, kCsThreads, kCsSmem, stream>>>(
          map, x, n, n_rows_full, static_cast<uint32_t>(k), st, hist_a, cnt_gt, cand_cnt, slots,
          out.header, n_chunks, n_stage_tiles, drop_zeros);
      note_launches(2);
    } else {
      // small tensor: straight to the fall-back select (mode = 1; the state is little-endian)
      e = cudaMemsetAsync(&st->mode, 1, 1, stream);
      if (e != cudaSuccess) return e;
    }
    {
      // cooperative launch: every CTA must be resident for the grid-wide barriers
      // list path: one thread per chunk; fall-back (known for small tensors): all SMs read x
      const long long want = streamed ? (L.tiles + kSelThreads - 1) / kSelThreads : (L.tiles + 31) / 32;
      const int grid = static_cast<int>(want < 1 ? 1 : (want < sms ? want : sms));
      const void* xa = x;
      long long na = n;
      uint32_t ka = static_cast<uint32_t>(k);
      surgeon_header* hdr = out.header;
      const uint32_t* cg = cnt_gt;
      const uint32_t* cc = cand_cnt;
      const void* sl = slots;
      int tiles = n_chunks;
      uint32_t* bm = out.bitmap;
      void* vals = out.values;
      uint32_t* offs = out.block_offsets;
      void* args[] = {&xa, &na, &ka, &st, &hdr, &hist_b, &hist_fb, &cg, &cc, &sl, &val, &prefix,
                      &partial, &tiles, &bm, &vals, &offs, &drop_zeros, &stall};
      e = cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(count_kernel<DT>), dim3(grid),
                                      dim3(kSelThreads), args, 0, stream);
      if (e != cudaSuccess) return e;
      note_launches(1);
    }
  }
  if (n == 0) {
    offsets_empty_kernel<<<1, 1, 0, stream>>>(out.block_offsets);
    note_launches(1);
  } else {
    if (streamed)
      compact_stream_kernel<DT><<<stream_grid, kCsThreads, kCsSmem, stream>>>(
          map, x, n, n_rows_full, out.header, out.bitmap, out.values, out.block_offsets, prefix,
          &st->error, n_chunks, n_stage_tiles);
    else
      compact_small_kernel<DT><<<static_cast<unsigned>(L.tiles), kCompactThreads, 0, stream>>>(
          x, n, out.header, out.bitmap, out.values, out.block_offsets, prefix, &st->error);
    note_launches(1);
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_prune_compact(const void* x, int64_t n, int dt, int64_t k,
                                 const surgeon_compressed& out, void* workspace,
                                 cudaStream_t stream, int drop_zeros, int stall) {
  return dt == 0 ? run_prune_compact<0>(x, n, k, drop_zeros, stall, out, workspace, stream)
                 : run_prune_compact<1>(x, n, k, drop_zeros, stall, out, workspace, stream);
}

cudaError_t launch_decompress(const surgeon_compressed& act, void* x_out, cudaStream_t stream) {
  if (act.n == 0) return cudaSuccess;
  const long long n_chunks = (act.n + 1023) / 1024;
  const long long ctas = (n_chunks + 7) / 8;
  const long long cap = 16LL * sm_count();
  const int grid = static_cast<int>(ctas < cap ? ctas : cap);
  if (act.dt == 0)
    decompress_kernel<0><<<grid, 256, 0, stream>>>(act.bitmap, act.values, act.block_offsets, act.n,
                                                   x_out);
  else
    decompress_kernel<1><<<grid, 256, 0, stream>>>(act.bitmap, act.values, act.block_offsets, act.n,
                                                   x_out);
  note_launches(1);
  return cudaGetLastError();
}

}  // namespace surgeon

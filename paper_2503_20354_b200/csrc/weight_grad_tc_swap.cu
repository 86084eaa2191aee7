// Tensor-core weight gradient on CTA pairs with the operand roles exchanged (Algorithm 1, Reshape
// and gradient steps with Eq. 2), for the layers whose operand tile is the activation itself: linear
// layers, 1x1 stride-1 convolutions and k x k stride-1 convolutions through shifted gradient copies.
//
//   D[g, c] = sum_k G[g, k] * A[c, k]          one MMA of a CTA pair (tcgen05, cta_group::2):
//   g (output channel, per tap for a k x k convolution) -> MMA M = 256: 128 gradient rows per CTA,
//                       by TMA, one to four accumulators per CTA (TMEM lanes = gradient rows)
//   c (input channel)  -> MMA N = nt <= 256 (TMEM columns): the operand both CTAs of the pair read.
//                       Each CTA rebuilds HALF of its rows from the compressed store and the
//                       pair's MMAs read both halves, so a rebuilt activation element serves
//                       256 * n_acc gradient rows while each CTA rebuilds only nt / 2 rows per
//                       K-tile: half the producer work per flop of one CTA working alone.  Any
//                       multiple of 16 channels is a legal N, so layers of 160 or 320 channels
//                       carry no padded rows.
//   k (row t, or image b and position p) -> MMA K, 64 per pipeline stage
//
// The dense activation exists only as shared-memory tiles.  Linear layers use MN-major operands
// (A[t, c] and G[t, o] are contiguous along c / o), convolutions K-major ones (contiguous along the
// position).  The gradient arrives as bf16 (one streaming pre-pass): for convolutions in boxes of
// 128 rows of one tap (the bound on this operand is the number and size of the TMA boxes, so they
// are as large as the layout allows; the rows left over when the output channels are not a
// multiple of 128 are packed, several taps to an accumulator, in smaller boxes), for linear layers
// in 64-column slabs.  Producer warps work in groups, one K-tile in flight per group; a lane
// owns a run of 32 consecutive elements.  Split-K partial tiles are reduced in a fixed order by
// the caller.  Every wait is bounded and ends in SURGEON_ERR_TIMEOUT.
//
// No load uses cluster multicast; the only cluster-scope operations are mbarrier arrivals and the
// commit that frees a stage in both CTAs.
#include <cuda.h>

#include <cstddef>
#include <cstdlib>

#include "surgeon_internal.cuh"
#include "tc_common.cuh"
#include "weight_grad_tc_conv.cuh"

namespace surgeon {

namespace {

using namespace tc;

constexpr int kTileK = 64;
constexpr int kProdWarps = 16;
constexpr int kThreads = 64 + kProdWarps * 32;   // warp 0: MMA, warp 1: TMA, warps 2..17: producers
constexpr int kMaxAStages = 8;
constexpr int kMaxGStages = 4;
constexpr int kAccBytes = 128 * kTileK * 2;      // one accumulator's gradient tile per stage: 16 KB
constexpr int kStageBytesPerWarp = 16 * (64 + 16) * 2;   // staging of packed values: 16 rows per warp

__device__ __forceinline__ uint64_t make_desc_mn(uint32_t saddr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>((kTileK * 128) >> 4) << 16;   // leading byte offset: next 64-wide slab
  d |= static_cast<uint64_t>(1024 >> 4) << 32;             // stride byte offset: next 8 k-rows
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;                     // 128-byte swizzle
  return d;
}

struct RunMeta {
  uint32_t base;       // kept elements before the run's 128-element block
  uint32_t next;       // bitmap word after the one the run starts in
  uint4 words;         // the block's bitmap words
  uint32_t j;          // flat index of the run's first element
  uint32_t nvalid;     // elements of the run that exist (0: nothing to do)
};

// The gradient rows of accumulator unit u (conv).  Full units: 128 rows of one tap.  Remainder
// units: the rows of `rpu` consecutive taps beyond their last full unit, rem_box rows each.
struct UnitPiece { int tap, o_lo; };
__device__ __forceinline__ bool unit_is_full(const SwapParams& p, int u) { return u < p.d.taps * p.a_units; }

template <int DT, int MODE, int LPR>
__global__ void __launch_bounds__(kThreads, 1)
dw_swap_kernel(const uint32_t* __restrict__ bitmap, const void* __restrict__ values,
               const uint32_t* __restrict__ offsets, const __grid_constant__ CUtensorMap grad_map,
               const __grid_constant__ CUtensorMap rem_map,
               float* __restrict__ partial, uint32_t* __restrict__ status, SwapParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int a_tile_bytes = p.half * 128;                 // this CTA's half of the activation tile
  const int g_stage_bytes = p.n_acc * kAccBytes;
  unsigned char* g_ring = smem + p.a_stages * a_tile_bytes;
  __shared__ __align__(8) unsigned long long bars[2 * kMaxAStages + 2 * kMaxGStages + 1];
  __shared__ uint32_t tmem_slot;
  __shared__ volatile uint32_t fail;

#ifdef SURGEON_DW_STATS
  const long long st_kernel_begin = clock64();
  if (threadIdx.x == 0) {
    unsigned long long gt;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt));
    atomicMin(reinterpret_cast<unsigned long long*>(status) + 14, gt);
  }
#endif
  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const uint32_t lane = lane_id();
  const uint32_t cta_rank = cluster_ctarank();
  const int m_tile = blockIdx.x >> 1, n_tile = blockIdx.y, split = blockIdx.z;
  const int ct0 = m_tile * p.nt;                              // first channel of the pair's tile
  const int c_first = ct0 + static_cast<int>(cta_rank) * p.half;   // first channel this CTA rebuilds
  const int rows_here = max(0, min(p.half, p.d.C - c_first));
  const int kt_begin = split * p.ktiles_per_split;
  const int kt_end = min(kt_begin + p.ktiles_per_split, p.d.total_ktiles);
  const int n_kt = kt_end - kt_begin;
  // gradient rows of this CTA: accumulator a holds unit (n_tile * n_acc + a) * 2 + rank (conv) or
  // the 128 columns from that index times 128 on (linear)
  const int unit0 = n_tile * p.n_acc * 2;                     // first unit of the pair's tile

  const uint32_t full_a = smem_u32(bars);
  const uint32_t empty_a = smem_u32(bars + kMaxAStages);
  const uint32_t full_g = smem_u32(bars + 2 * kMaxAStages);
  const uint32_t empty_g = smem_u32(bars + 2 * kMaxAStages + kMaxGStages);
  const uint32_t acc_bar = smem_u32(bars + 2 * kMaxAStages + 2 * kMaxGStages);
  if (tid == 0) {
    tma_prefetch_desc(&grad_map);
    if (MODE != 0) tma_prefetch_desc(&rem_map);
    for (int s = 0; s < p.a_stages; ++s) {
      mbar_init(full_a + 8 * s, 2 * p.gw);         // the warps of one group in each CTA of the pair
      mbar_init(empty_a + 8 * s, 1);
    }
    for (int s = 0; s < p.g_stages; ++s) {
      mbar_init(full_g + 8 * s, 1);                // rank 0's TMA thread (+ the bytes of both CTAs)
      mbar_init(empty_g + 8 * s, 1);
    }
    mbar_init(acc_bar, 1);
    fail = 0;
    fence_barrier_init();
  }
  if (warp == 0) tmem_alloc_pair(smem_u32(&tmem_slot), p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                    // both CTAs' barriers exist before either is arrived on
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;

  if (warp == 0) {
    // ================= MMA issuer (rank 0 of the pair) =================
    if (lane == 0 && cta_rank == 0) {
      const uint32_t idesc = make_idesc(256, p.nt) | (MODE == 0 ? ((1u << 15) | (1u << 16)) : 0u);
      const uint64_t a_base = (MODE == 0) ? make_desc_mn(smem_u32(smem)) : make_desc(smem_u32(smem));
      const uint64_t g_base = (MODE == 0) ? make_desc_mn(smem_u32(g_ring)) : make_desc(smem_u32(g_ring));
      const uint64_t a_inc = static_cast<uint64_t>(a_tile_bytes >> 4);
      const uint64_t g_inc = static_cast<uint64_t>(g_stage_bytes >> 4);
      constexpr uint64_t acc_inc = static_cast<uint64_t>(kAccBytes >> 4);
      constexpr int kStep = (MODE == 0) ? 128 : 2;
      uint64_t da = a_base, dg = g_base;
      uint32_t pa = 0, pg = 0, accum = 0;
      int sa = 0, sg = 0;
      bool ok = true;
#ifdef SURGEON_DW_STATS
      long long st_g = 0, st_a = 0;
      const long long st_begin = clock64();
#endif
      for (int it = 0; it < n_kt; ++it) {
#ifdef SURGEON_DW_STATS
        const long long c0 = clock64();
        ok = mbar_wait_suspend(full_g + 8 * sg, pg);
        const long long c1 = clock64();
        ok = ok && mbar_wait_suspend_cluster(full_a + 8 * sa, pa);
        st_g += c1 - c0; st_a += clock64() - c1;
#else
        ok = mbar_wait_suspend(full_g + 8 * sg, pg) && mbar_wait_suspend_cluster(full_a + 8 * sa, pa);
#endif
        if (!ok) break;
        tc_fence_after();
        for (int a = 0; a < p.n_acc; ++a) {
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            umma_bf16_pair(tmem_base + a * p.nt, dg + a * acc_inc + static_cast<uint64_t>(kk * kStep),
                           da + static_cast<uint64_t>(kk * kStep), idesc, kk > 0 ? 1u : accum);
        }
        umma_commit_pair(empty_a + 8 * sa);
        umma_commit_pair(empty_g + 8 * sg);
        accum = 1;
        if (++sa == p.a_stages) { sa = 0; pa ^= 1; da = a_base; } else { da += a_inc; }
        if (++sg == p.g_stages) { sg = 0; pg ^= 1; dg = g_base; } else { dg += g_inc; }
      }
      if (!ok) { fail = 1; atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT)); }
#ifdef SURGEON_DW_STATS
      atomicAdd(reinterpret_cast<unsigned long long*>(status) + 4, static_cast<unsigned long long>(st_g));
      atomicAdd(reinterpret_cast<unsigned long long*>(status) + 5, static_cast<unsigned long long>(st_a));
      atomicAdd(reinterpret_cast<unsigned long long*>(status) + 6, static_cast<unsigned long long>(clock64() - st_begin));
      atomicAdd(reinterpret_cast<unsigned long long*>(status) + 7, static_cast<unsigned long long>(n_kt));
      atomicAdd(reinterpret_cast<unsigned long long*>(status) + 11, static_cast<unsigned long long>(st_begin - st_kernel_begin));
      atomicAdd(reinterpret_cast<unsigned long long*>(status) + 12, 1ull);
#endif
      umma_commit_pair(acc_bar);
    }
    __syncwarp();
  } else if (warp == 1) {
    // ================= gradient tiles by TMA (each CTA loads its own 128 rows per accumulator) ====
    if (lane == 0) {
      int sg = 0;
      uint32_t round = 0;
      int img = 0, kin = 0;
      if (MODE != 0) { img = kt_begin / p.d.tiles_per_img; kin = kt_begin - img * p.d.tiles_per_img; }
      // bytes of both CTAs' loads of one K-tile
      uint32_t tx_bytes = static_cast<uint32_t>(2 * p.n_acc * kAccBytes);
      if (MODE != 0) {
        tx_bytes = 0;
        for (int i = 0; i < 2 * p.n_acc; ++i) {
          const int u = unit0 + i;
          if (u >= p.n_units) break;
          if (unit_is_full(p, u)) tx_bytes += kAccBytes;
          else tx_bytes += static_cast<uint32_t>(min(p.rpu, p.d.taps - (u - p.d.taps * p.a_units) * p.rpu) * p.rem_box) * 128u;
        }
      }
#ifdef SURGEON_DW_STATS
      long long st_e = 0;
#endif
      for (int it = 0; it < n_kt; ++it) {
#ifdef SURGEON_DW_STATS
        const long long c0 = clock64();
#endif
        if (round > 0 && !mbar_wait_suspend(empty_g + 8 * sg, (round - 1) & 1)) {
          fail = 1;
          atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
          break;
        }
#ifdef SURGEON_DW_STATS
        st_e += clock64() - c0;
#endif
        const uint32_t g_addr = smem_u32(g_ring + sg * g_stage_bytes);
        if (cta_rank == 0) mbar_arrive_expect_tx(full_g + 8 * sg, tx_bytes);
        if (MODE == 0) {
          for (int a = 0; a < p.n_acc; ++a)
#pragma unroll
            for (int g = 0; g < 2; ++g)
              tma_load_2d_pair(g_addr + a * kAccBytes + g * (kTileK * 128), &grad_map,
                               (unit0 + a * 2 + static_cast<int>(cta_rank)) * 128 + g * 64,
                               (kt_begin + it) * kTileK, full_g + 8 * sg);
        } else {
          const int p0 = kin * kTileK;
          // a tap's box: the copy holding its column shift, its row shift as an offset along the
          // flattened map, its rows in the 2-D tensor [images * copies * O rows][positions]
          auto load_box = [&](const CUtensorMap* map, uint32_t dst, int tap, int o_lo) {
            int copy = tap, x = p0;
            if (p.d.row_shift) {
              const int r = tap / p.d.kw;
              copy = tap - r * p.d.kw;
              x = p0 + (p.d.pad - r) * p.d.in_w;
            }
            tma_load_2d_pair(dst, map, x, (img * p.d.copies + copy) * p.d.o_real + o_lo, full_g + 8 * sg);
          };
          for (int a = 0; a < p.n_acc; ++a) {
            const int u = unit0 + a * 2 + static_cast<int>(cta_rank);
            if (u >= p.n_units) break;
            if (unit_is_full(p, u)) {
              const int tap = u / p.a_units;
              load_box(&grad_map, g_addr + a * kAccBytes, tap, (u - tap * p.a_units) * 128);
            } else {
              const int j = u - p.d.taps * p.a_units;
              for (int q = 0; q < p.rpu; ++q) {
                const int tap = j * p.rpu + q;
                if (tap < p.d.taps)
                  load_box(&rem_map, g_addr + a * kAccBytes + q * (p.rem_box * 128), tap, p.a_full * 128);
              }
            }
          }
          if (++kin == p.d.tiles_per_img) { kin = 0; ++img; }
        }
        if (++sg == p.g_stages) { sg = 0; ++round; }
      }
#ifdef SURGEON_DW_STATS
      if (cta_rank == 0) atomicAdd(reinterpret_cast<unsigned long long*>(status) + 8, static_cast<unsigned long long>(st_e));
#endif
    }
    __syncwarp();
  } else if ((warp - 2) < p.groups * p.gw) {
    // ================= producers =================
    // Group g rebuilds the K-tiles g, g + groups, ... of this CTA's range.  A lane owns one run of
    // 32 consecutive elements per tile = 64 bytes of the operand tile.  LPR lanes share a tile row
    // (conv: a channel, two runs of 32 positions; linear: a row t of the K-tile, 2 or 4 runs of
    // 32 channels, 64 channels to a slab).
    const int pw = warp - 2;
    const int wg = pw / p.gw, wi = pw - wg * p.gw;
    const int row = (32 / LPR) * wi + static_cast<int>(lane) / LPR;
    const int part = lane & (LPR - 1);
    const bool in_tile = row < ((MODE == 0) ? kTileK : p.half);   // the row is part of the operand tile
    const uint32_t xr = row & 7;
    const uint32_t y = (part & 1) * 4;                // first 16-byte chunk of the run
    const uint32_t rowbase = (MODE == 0 ? (part >> 1) * (kTileK * 128) : 0) + row * 128;
    unsigned char* stg = g_ring + p.g_stages * g_stage_bytes + pw * kStageBytesPerWarp;
    const uint32_t n_keep = static_cast<uint32_t>(__ldg(p.n_keep_ptr));
    int sa = wg % p.a_stages;
    uint32_t round = wg / p.a_stages;
    auto wait_stage = [&]() -> bool {
      if (round > 0 && lane == 0 && !mbar_wait_suspend(empty_a + 8 * sa, (round - 1) & 1)) {
        fail = 1;
        atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
      }
      __syncwarp();
      return fail == 0;
    };
    auto next_stage = [&]() {
      sa += p.groups;
      while (sa >= p.a_stages) { sa -= p.a_stages; ++round; }
    };
    const int kt_first = kt_begin + wg;
    long long j_run;
    long long t_row = 0;
    int kin = 0;
    int n_run;
    if (MODE == 0) {
      const int c = c_first + 32 * part;
      n_run = in_tile ? max(0, min(32, p.d.C - c)) : 0;
      t_row = static_cast<long long>(kt_first) * kTileK + row;
      j_run = t_row * p.d.C + c;
    } else {
      const int img = kt_first / p.d.tiles_per_img;
      kin = kt_first - img * p.d.tiles_per_img;
      n_run = (in_tile && row < rows_here) ? 1 : 0;
      j_run = (static_cast<long long>(img) * p.d.C + (c_first + row)) * p.d.T;
    }
    const long long j_step = (MODE == 0) ? static_cast<long long>(p.groups) * kTileK * p.d.C
                                         : static_cast<long long>(p.d.C) * p.d.T;
    auto fetch = [&]() {
      RunMeta r;
      r.base = 0; r.next = 0; r.words = make_uint4(0, 0, 0, 0); r.j = 0; r.nvalid = 0;
      long long j;
      int nvalid;
      if (MODE == 0) {
        nvalid = (t_row < p.d.T) ? n_run : 0;
        j = j_run;
      } else {
        const int pp = kin * kTileK + 32 * part;
        nvalid = n_run ? max(0, min(32, p.d.T - pp)) : 0;
        j = j_run + pp;
      }
      if (nvalid > 0) {
        r.nvalid = static_cast<uint32_t>(nvalid);
        r.j = static_cast<uint32_t>(j);
        const long long blk = j >> kBlockShift;
        const long long wi2 = j >> 5;
        r.base = __ldg(offsets + blk);
        if (static_cast<unsigned long long>(blk) != p.partial_blk) {
          r.words = __ldg(reinterpret_cast<const uint4*>(bitmap) + blk);
        } else {
          const long long w0 = blk * kBlockWords;
          r.words.x = __ldg(bitmap + w0);
          r.words.y = (w0 + 1 < p.n_words) ? __ldg(bitmap + w0 + 1) : 0u;
          r.words.z = (w0 + 2 < p.n_words) ? __ldg(bitmap + w0 + 2) : 0u;
          r.words.w = (w0 + 3 < p.n_words) ? __ldg(bitmap + w0 + 3) : 0u;
        }
        if ((r.j & 31u) && wi2 + 1 < p.n_words) r.next = __ldg(bitmap + wi2 + 1);
      }
      return r;
    };
    auto advance = [&]() {
      if (MODE == 0) { t_row += p.groups * kTileK; j_run += j_step; }
      else {
        kin += p.groups;
        while (kin >= p.d.tiles_per_img) { kin -= p.d.tiles_per_img; j_run += j_step; }
      }
    };
    // bits of a run and the rank of its first kept element, from its fetched metadata
    auto locate = [&](const RunMeta& m, uint32_t& rank, uint32_t& bits) {
      const uint32_t wq = (m.j >> 5) & 3, sh = m.j & 31;
      rank = m.base;
      rank += wq > 0 ? __popc(m.words.x) : 0u;
      rank += wq > 1 ? __popc(m.words.y) : 0u;
      rank += wq > 2 ? __popc(m.words.z) : 0u;
      const uint32_t w0 = wq == 0 ? m.words.x : (wq == 1 ? m.words.y : (wq == 2 ? m.words.z : m.words.w));
      const uint32_t w1 = wq == 3 ? m.next : (wq == 0 ? m.words.y : (wq == 1 ? m.words.z : m.words.w));
      rank += __popc(w0 & ((1u << sh) - 1u));
      bits = __funnelshift_r(w0, w1, sh);
      bits = m.nvalid >= 32 ? bits : (bits & ((1u << m.nvalid) - 1u));
    };
    // The store is streamed (every packed value and bitmap word is read once), so the metadata is
    // fetched two of the group's tiles ahead.  The loop is software-pipelined around the proxy
    // fence that publishes a tile: with TMA loads and MMA operand reads in flight that fence
    // holds the warp for about a thousand clocks, so the value loads of the group's NEXT tile are
    // issued between the tile's stores and its fence and travel while the fence waits.
    constexpr int V = (DT == 0) ? 4 : 8;                  // packed values per 16-byte vector
    constexpr int RPW = 32 / LPR;                         // rows per warp
    constexpr int VMAX = (32 * LPR + V - 1) / V + 1;      // vectors a row's piece can span
    constexpr int ITER = (RPW * VMAX + 31) / 32;
    constexpr int kSlot = 32 * LPR + 16;                  // bf16 values per row slot
    uint32_t v[32];                                       // the run's elements as loaded (sparse path)
    uint32_t rank = 0, bits = 0;
    bool dense = false;
    // Sparse tiles: one predicated global load per element, all of a lane's loads independent.
    // Dense fp32 tiles (more than 55 % of the warp's 1024 elements kept) go through the staging
    // copy instead: the lane-per-run loads touch a cache line per lane and saturate the L1 there.
    auto issue = [&](const RunMeta& m) {
      locate(m, rank, bits);
      dense = DT == 0 && p.stage_bytes > 0 && __reduce_add_sync(0xFFFFFFFFu, __popc(bits)) > 560u;
      if (!dense) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint32_t byte = (bits >> (8 * q)) & 0xFFu;
          uint32_t idx = rank + (q == 0 ? 0u : __popc(bits & ((1u << (8 * q)) - 1u)));
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const uint32_t on = (byte >> e) & 1u;
            v[8 * q + e] = ld_packed<DT>(values, idx, on != 0);
            idx += on;
          }
        }
      }
    };
    RunMeta cur = {}, nxt = {};
    if (wg < n_kt) { cur = fetch(); advance(); }
    if (wg + p.groups < n_kt) { nxt = fetch(); advance(); }
    if (wg < n_kt) issue(cur);
#ifdef SURGEON_DW_STATS
    long long st_w = 0;
    const long long st_pb = clock64();
#endif
#ifdef SURGEON_DW_STATS
    long long ph[6] = {0, 0, 0, 0, 0, 0};
#define PH_STAMP(i) { const long long c_ = clock64(); ph[i] += c_ - ph_t; ph_t = c_; }
#else
#define PH_STAMP(i)
#endif
    for (int it = wg; it < n_kt; it += p.groups) {
#ifdef SURGEON_DW_STATS
      long long ph_t = clock64();
#endif
      RunMeta nxt2 = {};
      if (it + 2 * p.groups < n_kt) { nxt2 = fetch(); advance(); }
      PH_STAMP(0)
      uint4 chunk[4];
      if (dense) {
        // The LPR lanes of a row hold consecutive runs, so a row's kept values are one contiguous
        // piece of the packed vector: the warp copies every piece into its staging area with
        // aligned, coalesced 16-byte loads (converted to bf16 on the way) and expands from there.
        const uint32_t cnt = __popc(bits);
        uint32_t seg_len = cnt + __shfl_xor_sync(0xFFFFFFFFu, cnt, 1);
        if (LPR == 4) seg_len += __shfl_xor_sync(0xFFFFFFFFu, seg_len, 2);
        const uint32_t seg_start = __shfl_sync(0xFFFFFFFFu, rank, lane & ~static_cast<uint32_t>(LPR - 1));
        const uint32_t a0 = seg_start & ~static_cast<uint32_t>(V - 1);
        const uint32_t nvec = seg_len ? (seg_start + seg_len - a0 + V - 1) / V : 0u;
        __syncwarp();
#pragma unroll
        for (int i = 0; i < ITER; ++i) {
          const int t = static_cast<int>(lane) + 32 * i;
          const int r = min(t / VMAX, RPW - 1), v = t - (t / VMAX) * VMAX;
          const uint32_t a0_r = __shfl_sync(0xFFFFFFFFu, a0, r * LPR);
          const uint32_t nvec_r = __shfl_sync(0xFFFFFFFFu, nvec, r * LPR);
          if (t < RPW * VMAX && static_cast<uint32_t>(v) < nvec_r) {
            const uint32_t first = a0_r + static_cast<uint32_t>(v) * V;
            unsigned char* dst = stg + r * (kSlot * 2) + v * 16 / (DT == 0 ? 2 : 1);
            if (DT == 0) {
              const float* src = reinterpret_cast<const float*>(values) + first;
              float4 f;
              if (first + V <= n_keep) f = __ldg(reinterpret_cast<const float4*>(src));
              else {
                f.x = first < n_keep ? __ldg(src) : 0.0f;
                f.y = first + 1 < n_keep ? __ldg(src + 1) : 0.0f;
                f.z = first + 2 < n_keep ? __ldg(src + 2) : 0.0f;
                f.w = 0.0f;
              }
              *reinterpret_cast<uint2*>(dst) = make_uint2(pack_bf16x2(f.x, f.y), pack_bf16x2(f.z, f.w));
            } else {
              const unsigned short* src = reinterpret_cast<const unsigned short*>(values) + first;
              uint4 u;
              if (first + V <= n_keep) u = __ldg(reinterpret_cast<const uint4*>(src));
              else {
                uint32_t h[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) h[e] = first + e < n_keep ? static_cast<uint32_t>(__ldg(src + e)) : 0u;
                u = make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
              }
              *reinterpret_cast<uint4*>(dst) = u;
            }
          }
        }
        __syncwarp();
        const unsigned short* slot = reinterpret_cast<const unsigned short*>(
            stg + (lane / LPR) * (kSlot * 2)) + (rank - a0);
        uint32_t k = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t v[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const uint32_t on = (bits >> (8 * q + e)) & 1u;
            v[e] = on ? static_cast<uint32_t>(slot[k]) : 0u;
            k += on;
          }
          chunk[q].x = v[0] | (v[1] << 16); chunk[q].y = v[2] | (v[3] << 16);
          chunk[q].z = v[4] | (v[5] << 16); chunk[q].w = v[6] | (v[7] << 16);
        }
      } else {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if (DT == 0) {
            chunk[q].x = pack_bf16x2(__uint_as_float(v[8 * q]), __uint_as_float(v[8 * q + 1]));
            chunk[q].y = pack_bf16x2(__uint_as_float(v[8 * q + 2]), __uint_as_float(v[8 * q + 3]));
            chunk[q].z = pack_bf16x2(__uint_as_float(v[8 * q + 4]), __uint_as_float(v[8 * q + 5]));
            chunk[q].w = pack_bf16x2(__uint_as_float(v[8 * q + 6]), __uint_as_float(v[8 * q + 7]));
          } else {
            chunk[q].x = v[8 * q] | (v[8 * q + 1] << 16); chunk[q].y = v[8 * q + 2] | (v[8 * q + 3] << 16);
            chunk[q].z = v[8 * q + 4] | (v[8 * q + 5] << 16); chunk[q].w = v[8 * q + 6] | (v[8 * q + 7] << 16);
          }
        }
      }
      PH_STAMP(1)
#ifdef SURGEON_DW_STATS
      const long long cw0 = clock64();
#endif
      if (!wait_stage()) break;
#ifdef SURGEON_DW_STATS
      st_w += clock64() - cw0;
#endif
      PH_STAMP(2)
      if (in_tile) {
        unsigned char* dst_row = smem + sa * a_tile_bytes + rowbase;
#pragma unroll
        for (int q = 0; q < 4; ++q)
          *reinterpret_cast<uint4*>(dst_row + (((y + q) ^ xr) << 4)) = chunk[q];
      }
      PH_STAMP(3)
      if (it + p.groups < n_kt) issue(nxt);      // the next tile's loads leave before the fence
      PH_STAMP(4)
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive_rank0(full_a + 8 * sa);
      PH_STAMP(5)
      next_stage();
      cur = nxt;
      nxt = nxt2;
    }
#ifdef SURGEON_DW_STATS
    if (pw == 0 && lane == 0 && cta_rank == 0) {
      atomicAdd(reinterpret_cast<unsigned long long*>(status) + 9, static_cast<unsigned long long>(st_w));
      atomicAdd(reinterpret_cast<unsigned long long*>(status) + 10, static_cast<unsigned long long>(clock64() - st_pb));
      for (int i = 0; i < 6; ++i)
        atomicAdd(reinterpret_cast<unsigned long long*>(status) + 17 + i, static_cast<unsigned long long>(ph[i]));
    }
#endif
  }

  // ================= epilogue: TMEM -> scratch partial tile =================
  if (warp >= 2) {
    // A warp may read the 32 TMEM lanes of its quarter (warp % 4) = 32 gradient rows; the warps of a
    // quarter take the groups of 16 columns (channels) in turn.  A thread holds 16 channels of ONE
    // gradient row; the 32 x 16 block goes through shared memory (the rings are idle by now: every
    // MMA has completed) so that four lanes write 64 contiguous bytes of a row of the partial tile.
    const bool done = mbar_wait(acc_bar, 0, 64);
    tc_fence_after();
    if (done && !fail) {
      const int lane_grp = warp & 3;
      float* out = partial + static_cast<long long>(split) * p.d.O * p.d.C;
      const int cols = p.n_acc * p.nt;
      float* buf = reinterpret_cast<float*>(smem) + (warp - 2) * (32 * 20);   // 32 rows x (16 + 4) floats
      const int rsub = static_cast<int>(lane >> 2), quad = lane & 3;
      const bool vec4 = (p.d.C & 3) == 0;
      for (int col = 16 * ((warp - 2) >> 2); col < cols; col += 16 * (kProdWarps / 4)) {
        const int a = col / p.nt;
        const int c_lo = ct0 + (col - a * p.nt);             // channel of the first of the 16 columns
        const int u = unit0 + a * 2 + static_cast<int>(cta_rank);
        uint32_t r[16];
        tmem_ld16(tmem_base + (static_cast<uint32_t>(lane_grp * 32) << 16) + col, r);
        __syncwarp();                                        // the previous block has been read out
#pragma unroll
        for (int e = 0; e < 16; e += 4)
          *reinterpret_cast<uint4*>(buf + lane * 20 + e) = make_uint4(r[e], r[e + 1], r[e + 2], r[e + 3]);
        __syncwarp();
        if (c_lo >= p.d.C) continue;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int rr = rsub + 8 * i;                       // row of the block this lane writes now
          const int row_in_acc = lane_grp * 32 + rr;
          long long grow = -1;                               // its row of the partial tile
          if (MODE == 0) {
            const int o = u * 128 + row_in_acc;
            if (o < p.d.O) grow = o;
          } else if (u < p.n_units) {
            if (unit_is_full(p, u)) {
              const int tap = u / p.a_units;
              const int o = (u - tap * p.a_units) * 128 + row_in_acc;
              if (o < p.d.o_real) grow = static_cast<long long>(tap) * p.d.o_real + o;
            } else {
              const int q = row_in_acc / p.rem_box;
              const int tap = (u - p.d.taps * p.a_units) * p.rpu + q;
              const int o = p.a_full * 128 + (row_in_acc - q * p.rem_box);
              if (tap < p.d.taps && o < p.d.o_real) grow = static_cast<long long>(tap) * p.d.o_real + o;
            }
          }
          if (grow < 0) continue;
          const float4 v = *reinterpret_cast<const float4*>(buf + rr * 20 + quad * 4);
          const int c = c_lo + quad * 4;
          float* dst = out + grow * p.d.C + c;
          if (vec4 && c + 4 <= p.d.C) {
            *reinterpret_cast<float4*>(dst) = v;
          } else {
            if (c < p.d.C) dst[0] = v.x;
            if (c + 1 < p.d.C) dst[1] = v.y;
            if (c + 2 < p.d.C) dst[2] = v.z;
            if (c + 3 < p.d.C) dst[3] = v.w;
          }
        }
      }
    } else if (!done && lane == 0) {
      atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                    // neither CTA leaves while the pair's MMAs or arrivals may touch it
  if (warp == 0) tmem_dealloc_pair(tmem_base, p.tmem_cols);
#ifdef SURGEON_DW_STATS
  if (tid == 0 && cta_rank == 0)
    atomicAdd(reinterpret_cast<unsigned long long*>(status) + 13, static_cast<unsigned long long>(clock64() - st_kernel_begin));
  if (tid == 0) {
    unsigned long long gt;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt));
    atomicMax(reinterpret_cast<unsigned long long*>(status) + 15, gt);
    atomicMax(reinterpret_cast<unsigned long long*>(status) + 16, static_cast<unsigned long long>(clock64() - st_kernel_begin));
  }
#endif
}

bool swap_enabled() {
  static const bool on = [] {
    const char* e = std::getenv("SURGEON_DW_SWAP");
    return e && e[0] == '1';
  }();
  return on;
}

// Shared memory: activation ring, gradient ring, staging (fp32 activations only).
bool size_swap_rings(SwapParams* p, int stage_bytes) {
  const int budget = 224 * 1024 - 1024 - stage_bytes;
  const int a_bytes = p->half * 128;
  const int g_bytes = p->n_acc * kAccBytes;
  const int a_min = p->groups + 1;
  int g_stages = (budget - a_min * a_bytes) / g_bytes;
  if (g_stages > 3) g_stages = 3;
  if (g_stages < 2) return false;
  int a_stages = (budget - g_stages * g_bytes) / a_bytes;
  if (a_stages > kMaxAStages) a_stages = kMaxAStages;
  if (a_stages < a_min) return false;
  p->a_stages = a_stages; p->g_stages = g_stages; p->stage_bytes = stage_bytes;
  p->smem_bytes = a_stages * a_bytes + g_stages * g_bytes + stage_bytes + 1024;
  return true;
}

// CTA pairs that can be resident at once.  A pair needs two SMs of one cluster-capable group, so
// this is fewer than half the SMs when the SM count of a GPC is odd; asked of the runtime once
// per device for the largest configuration (whole shared memory).
int resident_pairs() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return sm_count() / 2;
  if (cached[dev] == 0) {
    int n = 0;
    const int smem = 224 * 1024;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * sm_count(), 1, 1);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (cudaFuncSetAttribute(dw_swap_kernel<1, 1, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
        cudaOccupancyMaxActiveClusters(&n, dw_swap_kernel<1, 1, 2>, &cfg) != cudaSuccess || n <= 0) {
      cudaGetLastError();
      n = sm_count() / 2;
    }
    cached[dev] = n;
  }
  return cached[dev];
}

}  // namespace

int swap_resident_pairs() { return resident_pairs(); }

static bool compute_plan_swap(const surgeon_layer_desc& d, SwapParams* out) {
  SwapParams best{};
  DirectParams dp;
  if (!plan_direct(d, &dp)) return false;
  if (dp.mode == 2 || dp.C < 32) return false;
  if (dp.mode == 0 && (dp.C % 128) != 0) return false;      // whole 64-channel slabs per CTA
  // a TMA box of 128 gradient rows must fit the tensor of all copies
  if (dp.mode != 0 && static_cast<long long>(dp.imgs) * dp.copies * dp.o_real < 128) return false;
  const int pairs_per_wave = resident_pairs();
  if (pairs_per_wave < 1) return false;
  // conv: the units of gradient rows (128 TMEM lanes each)
  int a_full = 0, a_units = 0, rem_box = 0, rpu = 0, n_units = 0;
  if (dp.mode != 0) {
    a_full = dp.o_real / 128;
    const int rem = dp.o_real - 128 * a_full;
    a_units = a_full;
    if (rem > 0) {
      rem_box = 16;
      while (rem_box < rem) rem_box *= 2;
      if (rem_box >= 128) { a_units = a_full + 1; rem_box = 0; }   // a last, partly filled full unit
    }
    rpu = rem_box ? 128 / rem_box : 0;
    n_units = dp.taps * a_units + (rem_box ? (dp.taps + rpu - 1) / rpu : 0);
  }
  double best_cost = 1e30;
  const int mt_lo = (dp.C + 255) / 256, mt_hi = (dp.C + 31) / 32;
  for (int m_tiles = mt_lo; m_tiles <= mt_hi; ++m_tiles) {
    const int nt = ((dp.C + m_tiles - 1) / m_tiles + 15) / 16 * 16;
    if (nt > 256 || nt < 32) continue;
    if ((m_tiles - 1) * nt >= dp.C) continue;               // an empty last tile
    if (dp.mode == 0 && nt != 128 && nt != 256) continue;   // one or two slabs per CTA
    if (dp.mode == 0 && dp.C % nt != 0) continue;
    const int max_acc = 512 / nt < 4 ? 512 / nt : 4;
    for (int n_acc = 1; n_acc <= max_acc; ++n_acc) {
      SwapParams p{};
      p.d = dp;
      p.nt = nt; p.half = nt / 2; p.n_acc = n_acc; p.m_tiles = m_tiles;
      p.a_full = a_full; p.a_units = a_units; p.rem_box = rem_box; p.rpu = rpu;
      p.lpr = (dp.mode == 0) ? p.half / 32 : 2;
      const int runs = (dp.mode == 0) ? kTileK * p.lpr : 2 * p.half;
      p.gw = (runs + 31) / 32;
      p.groups = kProdWarps / p.gw;
      if (p.groups < 1) continue;
      if (p.groups > 4) p.groups = 4;
      p.n_units = (dp.mode == 0) ? (dp.O + 127) / 128 : n_units;
      p.n_tiles = (p.n_units + 2 * n_acc - 1) / (2 * n_acc);
      if (!size_swap_rings(&p, kProdWarps * kStageBytesPerWarp)) continue;
      // Clocks of one K-tile on a CTA, as measured on B200 with clock stamps in this kernel: the
      // slowest of the MMAs (128 x nt x 16 in nt / 2 clocks), the gradient boxes (L2 delivers about
      // 30 bytes per clock to an SM while all SMs pull) and the producers (0.28 clocks per rebuilt
      // element: latency of the fence that publishes a tile, not instruction issue, so more
      // groups of fewer warps - smaller halves - do better).
      const double mma = n_acc * 4.0 * (nt / 2.0);
      const double l2 = n_acc * kAccBytes / 30.0;
      const double prod = p.half * 64.0 * 0.28;
      double kt_clk = mma > prod ? mma : prod;
      if (l2 > kt_clk) kt_clk = l2;
      if (p.g_stages < 3) kt_clk *= 1.1;
      kt_clk += 80.0;
      const long long pairs = static_cast<long long>(m_tiles) * p.n_tiles;
      const int max_splits = (dp.total_ktiles + 7) / 8 < 1 ? 1 : (dp.total_ktiles + 7) / 8;
      for (int s = 1; s <= max_splits && s <= 148; ++s) {
        const long long waves = (pairs * s + pairs_per_wave - 1) / pairs_per_wave;
        const int kts = (dp.total_ktiles + s - 1) / s;
        // a wave: the K loop, the prologue and the epilogue (the accumulators leave through L2)
        const double cost = static_cast<double>(waves) * (kts * kt_clk + 6000.0 + 16.0 * n_acc * nt) +
                            60.0 * s * static_cast<double>(pairs) / pairs_per_wave;
        if (cost < best_cost - 1e-9) {
          best_cost = cost;
          best = p;
          best.ktiles_per_split = kts;
          best.splits = (dp.total_ktiles + kts - 1) / kts;
        }
      }
    }
  }
  if (best_cost >= 1e30) return false;
  best.tmem_cols = 32;
  while (best.tmem_cols < best.n_acc * best.nt) best.tmem_cols *= 2;
  *out = best;
  return true;
}

bool plan_swap(const surgeon_layer_desc& d, SwapParams* out) {
  if (!swap_enabled()) return false;
  struct Tag {};
  return memo_plan<Tag>(d, 0, out, [&](SwapParams* p) { return compute_plan_swap(d, p); });
}

size_t swap_partial_bytes(const SwapParams& p) {
  const size_t b = static_cast<size_t>(p.splits) * p.d.O * p.d.C * sizeof(float);
  return (b + 255) & ~static_cast<size_t>(255);
}

cudaError_t launch_swap(const surgeon_compressed& act, const SwapParams& plan, const float* grad_out,
                        void* grad_bf16, float* partial, uint32_t* status, cudaStream_t stream) {
  SwapParams p = plan;
  const bool staged = act.dt == 0;
  if (!size_swap_rings(&p, staged ? kProdWarps * kStageBytesPerWarp : 0)) return cudaErrorInvalidValue;
  p.n_words = (act.n + 31) / 32;
  p.n_keep_ptr = reinterpret_cast<const long long*>(reinterpret_cast<const char*>(act.header) +
                                                    offsetof(surgeon_header, n_keep));
  p.partial_blk = (act.n % SURGEON_BLOCK) ? static_cast<unsigned>(act.n / SURGEON_BLOCK) : 0xFFFFFFFFu;
  cudaError_t e = launch_direct_prepass(p.d, grad_out, grad_bf16, stream);
  if (e != cudaSuccess) return e;
  CUtensorMap map;
  CUtensorMap rem_map;
  if (p.d.mode == 0) {
    e = encode_direct_grad_map(p.d, grad_bf16, 64, &map);
    rem_map = map;
  } else {
    // The copies of all images as one 2-D tensor [images * copies * O rows][g_len positions] (the
    // rows of consecutive images follow one another at the same pitch): boxes of 64 positions x
    // 128 rows, and x rem_box rows for the rows past a tap's last full unit.
    using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);
    const EncodeFn encode = reinterpret_cast<EncodeFn>(tensor_map_encode_fn());
    if (!encode) return cudaErrorNotSupported;
    const cuuint64_t rows = static_cast<cuuint64_t>(p.d.imgs) * p.d.copies * p.d.o_real;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(p.d.g_len), rows};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(p.d.pitch) * 2};
    const cuuint32_t estr[2] = {1, 1};
    auto make = [&](CUtensorMap* m, int box_rows) {
      const cuuint32_t box[2] = {static_cast<cuuint32_t>(kTileK), static_cast<cuuint32_t>(box_rows)};
      return encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, grad_bf16, dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    };
    bool ok = make(&map, 128);
    ok = ok && make(&rem_map, p.rem_box ? p.rem_box : 128);
    e = ok ? cudaSuccess : cudaErrorInvalidValue;
  }
  if (e != cudaSuccess) return e;
  dim3 grid(2 * p.m_tiles, p.n_tiles, p.splits);
  auto launch = [&](auto kernel) -> cudaError_t {
    cudaError_t err = allow_dynamic_smem(reinterpret_cast<const void*>(kernel), p.smem_bytes);
    if (err != cudaSuccess) return err;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = static_cast<size_t>(p.smem_bytes);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, act.bitmap, act.values, act.block_offsets, map, rem_map,
                              partial, status, p);
  };
  if (p.d.mode == 0) {
    if (p.lpr == 4) e = act.dt == 0 ? launch(dw_swap_kernel<0, 0, 4>) : launch(dw_swap_kernel<1, 0, 4>);
    else e = act.dt == 0 ? launch(dw_swap_kernel<0, 0, 2>) : launch(dw_swap_kernel<1, 0, 2>);
  } else {
    e = act.dt == 0 ? launch(dw_swap_kernel<0, 1, 2>) : launch(dw_swap_kernel<1, 1, 2>);
  }
  note_launches(1);
  return e;
}

}  // namespace surgeon

// Tensor-core weight gradient for layers whose im2col operand is the activation itself: linear
// layers ([T, C] activations), 1x1 / pad 0 convolutions of stride 1 or 2, and k x k stride-1
// convolutions through shifted copies of the output gradient (NCHW).  Algorithm 1,
// Reshape and gradient steps with Eq. 2:  D[c, o] = sum_k A[k, c] * G[k, o].
//
//   c (input channel)  -> MMA M, 128 per CTA (TMEM lanes)
//   o (output channel, per tap for a k x k convolution) -> MMA N, one to three accumulators of
//                         up to 256 columns, at most 512 in all
//   k (row t, or image b and position p) -> MMA K, 64 per pipeline stage
//
// Operand layouts follow the memory order of the tensors, so that neither needs a transpose:
//   linear : A[t, c] and G[t, o] are contiguous along c / o -> both operands MN-major
//            (rows of 64 channels = 128 bytes, one row per k, 128-byte swizzle);
//   conv   : A[b, c, p] and G[b, o, p] are contiguous along p -> both operands K-major.
// The output gradient is converted to bf16 once by a streaming pre-pass and arrives by TMA.
// The activation operand is rebuilt from the compressed store by 16 producer warps, 8 per K-tile,
// two tiles in flight: a lane owns a run of 32 consecutive elements (64 bytes of the swizzled
// tile), finds the rank of its first kept element from the block offset and the block's bitmap
// words, and rebuilds the run as four 16-byte chunks with one predicated load per element (all
// independent; fp32 tiles that are mostly kept go through a coalesced per-warp staging copy
// instead).  The metadata of a lane's next run is fetched while the current one is rebuilt.
// One thread issues the MMAs, one the TMA loads; split-K partial tiles are reduced in a fixed
// order by the caller.  Every wait is bounded and ends in SURGEON_ERR_TIMEOUT.
#include <cuda.h>

#include <cstddef>
#include <cstdlib>

#include "surgeon_internal.cuh"
#include "tc_common.cuh"
#include "weight_grad_tc_conv.cuh"

namespace surgeon {

namespace {

using namespace tc;

constexpr int kTileM = 128;
constexpr int kTileK = 64;
constexpr int kGroups = 2;                       // producer groups of 8 warps, one K-tile in flight each
constexpr int kProdWarps = 8 * kGroups;
constexpr int kProdThreads = kProdWarps * 32;
constexpr int kThreads = 64 + kProdThreads;     // warp 0: MMA, warp 1: TMA, warps 2..17: producers
// CTA pairs (cta_group::2) halve the gradient traffic per MMA.  They measured slower than single
// CTAs while the activation producers are the bound (a pair waits for the slower of its two
// tiles), so they are off unless the environment variable SURGEON_DW_PAIRS is set to 1.
static bool use_pairs() {
  static const bool on = [] {
    const char* e = std::getenv("SURGEON_DW_PAIRS");
    return e && e[0] == '1';
  }();
  return on;
}
constexpr int kMaxAStages = 8;
constexpr int kMaxBStages = 4;
constexpr int kATileBytes = kTileM * kTileK * 2;              // 16 KB
// staging of packed values: per warp 16 rows of 64 + 16 bf16 (conv) or 8 rows of 128 + 16 (linear)
constexpr int kStageBytesPerWarp = 16 * (64 + 16) * 2;
constexpr int kStageBytes = kProdWarps * kStageBytesPerWarp;  // 40 KB

// Shared-memory matrix descriptor of an MN-major operand with 128-byte swizzle: rows of 64
// elements (128 bytes) per k, 8 rows per 1024-byte group (stride byte offset), the next 64
// elements along M/N one slab of 64 k-rows further (leading byte offset).
__device__ __forceinline__ uint64_t make_desc_mn(uint32_t saddr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>((kTileK * 128) >> 4) << 16;   // leading byte offset: next 64-wide slab
  d |= static_cast<uint64_t>(1024 >> 4) << 32;             // stride byte offset: next 8 k-rows
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;                     // 128-byte swizzle
  return d;
}

// What a lane fetches for the 32 consecutive elements ("word") it rebuilds: the kept count before
// their 128-element block, the block's bitmap words, and the bitmap word after the one the run
// starts in (the run need not start on a word boundary).
struct WordRaw {
  uint32_t base;
  uint32_t next;
  uint4 words;
  uint32_t j;          // flat index of the run's first element
  uint32_t nvalid;     // elements of the run that exist (0: nothing to do)
};

template <int DT, int MODE, int PAIR>
__global__ void __launch_bounds__(kThreads, 1)
dw_direct_kernel(const uint32_t* __restrict__ bitmap, const void* __restrict__ values,
                 const uint32_t* __restrict__ offsets, const __grid_constant__ CUtensorMap grad_map,
                 float* __restrict__ partial, uint32_t* __restrict__ status, DirectParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  // Two rings: activation tiles (16 KB each, many) and gradient tiles (n_cols rows each, few).
  // The activation ring is deep because rebuilding a tile takes longer than its MMAs; the
  // gradient tiles arrive by TMA well ahead and need only be double- or triple-buffered.
  // In a CTA pair each CTA holds half of the gradient rows of every accumulator.
  const int b_stage_bytes = p.n_cols * (PAIR ? 64 : 128);
  const int acc_rows = PAIR ? p.acc_n / 2 : p.acc_n;     // gradient rows per accumulator in this CTA
  const uint32_t cta_rank = PAIR ? cluster_ctarank() : 0u;
  unsigned char* b_ring = smem + p.a_stages * kATileBytes;
  __shared__ __align__(8) unsigned long long bars[2 * kMaxAStages + 2 * kMaxBStages + 1];
  __shared__ uint32_t tmem_slot;
  __shared__ volatile uint32_t fail;

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const uint32_t lane = lane_id();
  const int m_tile = blockIdx.x, n_tile = blockIdx.y, split = blockIdx.z;
  const int c0 = m_tile * p.rows_per_tile;           // first input channel of the CTA's row tile
  const int rows_here = max(0, min(p.rows_per_tile, p.C - c0));   // tile rows that hold a channel
  const int o0 = n_tile * p.n_cols;                  // linear: first gradient column of the CTA
  const int u0 = n_tile * p.n_acc;                   // conv: first column unit of the CTA
  const int n_acc_here = (MODE == 0) ? p.n_acc : min(p.n_acc, p.n_units - u0);
  const int kt_begin = split * p.ktiles_per_split;
  const int kt_end = min(kt_begin + p.ktiles_per_split, p.total_ktiles);
  const int n_kt = kt_end - kt_begin;

  const uint32_t full_a = smem_u32(bars);
  const uint32_t empty_a = smem_u32(bars + kMaxAStages);
  const uint32_t full_b = smem_u32(bars + 2 * kMaxAStages);
  const uint32_t empty_b = smem_u32(bars + 2 * kMaxAStages + kMaxBStages);
  const uint32_t acc_bar = smem_u32(bars + 2 * kMaxAStages + 2 * kMaxBStages);
  if (tid == 0) {
    tma_prefetch_desc(&grad_map);
    for (int s = 0; s < p.a_stages; ++s) {
      mbar_init(full_a + 8 * s, (PAIR ? 2 : 1) * 8);   // the 8 warps (of each CTA) that rebuild a tile
      mbar_init(empty_a + 8 * s, 1);
    }
    for (int s = 0; s < p.b_stages; ++s) {
      mbar_init(full_b + 8 * s, 1);                    // the TMA thread (+ the bytes it expects)
      mbar_init(empty_b + 8 * s, 1);
    }
    mbar_init(acc_bar, 1);
    fail = 0;
    fence_barrier_init();
  }
  if (warp == 0) {
    if (PAIR) tmem_alloc_pair(smem_u32(&tmem_slot), p.tmem_cols);
    else tmem_alloc(smem_u32(&tmem_slot), p.tmem_cols);
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();          // both CTAs' barriers exist before either is arrived on
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  pdl_trigger();                         // the split reduction may be launched; it waits for this grid

  if (warp == 0) {
    // ================= MMA issuer (rank 0 of a pair) =================
    if (lane == 0 && cta_rank == 0) {
      const uint32_t idesc = make_idesc(PAIR ? 2 * kTileM : kTileM, p.acc_n) | (MODE == 0 ? ((1u << 15) | (1u << 16)) : 0u);
      const uint64_t a_base = (MODE == 0) ? make_desc_mn(smem_u32(smem)) : make_desc(smem_u32(smem));
      const uint64_t b_base = (MODE == 0) ? make_desc_mn(smem_u32(b_ring)) : make_desc(smem_u32(b_ring));
      const uint64_t a_inc = static_cast<uint64_t>(kATileBytes >> 4);
      const uint64_t b_inc = static_cast<uint64_t>(b_stage_bytes >> 4);
      const uint64_t acc_inc = static_cast<uint64_t>((acc_rows * 128) >> 4);
      constexpr int kStep = (MODE == 0) ? 128 : 2;
      uint64_t da = a_base, db = b_base;
      uint32_t pa = 0, pb = 0, accum = 0;
      int sa = 0, sb = 0;
      bool ok = true;
#ifdef SURGEON_DW_STATS
      // clock stamps of the issuing thread (a build with -DSURGEON_DW_STATS; read from the scratch
      // status area by paper_2503_20354_b200/diagnostics.py): where a K-tile's time goes
      long long st_g = 0, st_a = 0;
      const long long st_begin = clock64();
#endif
      for (int it = 0; it < n_kt; ++it) {
#ifdef SURGEON_DW_STATS
        const long long c0 = clock64();
        ok = mbar_wait_suspend(full_b + 8 * sb, pb);
        const long long c1 = clock64();
        ok = ok && (PAIR ? mbar_wait_suspend_cluster(full_a + 8 * sa, pa) : mbar_wait_suspend(full_a + 8 * sa, pa));
        st_g += c1 - c0; st_a += clock64() - c1;
#else
        ok = mbar_wait_suspend(full_b + 8 * sb, pb) &&
             (PAIR ? mbar_wait_suspend_cluster(full_a + 8 * sa, pa) : mbar_wait_suspend(full_a + 8 * sa, pa));
#endif
        if (!ok) break;
        tc_fence_after();
        if (n_acc_here == 1) umma_ktile<1, kStep, PAIR>(tmem_base, p.acc_n, da, db, acc_inc, idesc, accum);
        else if (n_acc_here == 2) umma_ktile<2, kStep, PAIR>(tmem_base, p.acc_n, da, db, acc_inc, idesc, accum);
        else if (n_acc_here == 3) umma_ktile<3, kStep, PAIR>(tmem_base, p.acc_n, da, db, acc_inc, idesc, accum);
        else umma_ktile<4, kStep, PAIR>(tmem_base, p.acc_n, da, db, acc_inc, idesc, accum);
        if (PAIR) { umma_commit_pair(empty_a + 8 * sa); umma_commit_pair(empty_b + 8 * sb); }
        else { umma_commit(empty_a + 8 * sa); umma_commit(empty_b + 8 * sb); }
        accum = 1;
        if (++sa == p.a_stages) { sa = 0; pa ^= 1; da = a_base; } else { da += a_inc; }
        if (++sb == p.b_stages) { sb = 0; pb ^= 1; db = b_base; } else { db += b_inc; }
      }
      if (!ok) { fail = 1; atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT)); }
#ifdef SURGEON_DW_STATS
      atomicAdd(reinterpret_cast<unsigned long long*>(status) + 4, static_cast<unsigned long long>(st_g));
      atomicAdd(reinterpret_cast<unsigned long long*>(status) + 5, static_cast<unsigned long long>(st_a));
      atomicAdd(reinterpret_cast<unsigned long long*>(status) + 6, static_cast<unsigned long long>(clock64() - st_begin));
      atomicAdd(reinterpret_cast<unsigned long long*>(status) + 7, static_cast<unsigned long long>(n_kt));
#endif
      if (PAIR) umma_commit_pair(acc_bar);
      else umma_commit(acc_bar);
    }
    __syncwarp();
  } else if (warp == 1) {
    // ================= gradient tiles by TMA =================
    if (lane == 0) {
      pdl_wait();                                      // the bf16 gradient copy is complete
      int sb = 0;
      uint32_t round = 0;
      int img = 0, kin = 0;                            // conv: image and K-tile within it
      if (MODE != 0) { img = kt_begin / p.tiles_per_img; kin = kt_begin - img * p.tiles_per_img; }
      for (int it = 0; it < n_kt; ++it) {
        if (round > 0 && !mbar_wait_suspend(empty_b + 8 * sb, (round - 1) & 1)) {
          fail = 1;
          atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
          break;
        }
        const uint32_t b_addr = smem_u32(b_ring + sb * b_stage_bytes);
        // rank 0 announces the bytes of both CTAs' loads of this tile
        if (cta_rank == 0)
          mbar_arrive_expect_tx(full_b + 8 * sb, static_cast<uint32_t>(n_acc_here * p.acc_n) * 128u);
        if (MODE == 0) {
          if (PAIR) {
            for (int a = 0; a < p.n_acc; ++a)
              for (int g = 0; g < acc_rows / 64; ++g)
                tma_load_2d_pair(b_addr + a * acc_rows * 128 + g * (kTileK * 128), &grad_map,
                                 o0 + a * p.acc_n + static_cast<int>(cta_rank) * acc_rows + g * 64,
                                 (kt_begin + it) * kTileK, full_b + 8 * sb);
          } else {
            for (int g = 0; g < p.n_cols / 64; ++g)
              tma_load_2d(b_addr + g * (kTileK * 128), &grad_map, o0 + g * 64, (kt_begin + it) * kTileK,
                          full_b + 8 * sb);
          }
        } else {
          const int p0 = kin * kTileK;
          for (int a = 0; a < n_acc_here; ++a) {
            // unit -> tap and channel range; the copy holding the tap's column shift, and the
            // tap's row shift as an offset along the flattened map
            const int u = u0 + a;
            const int tap = u / p.upt;
            const int o_lo = (u - tap * p.upt) * p.acc_n;
            int copy = tap, x = p0;
            if (p.row_shift) {
              const int r = tap / p.kw;
              copy = tap - r * p.kw;
              x = p0 + (p.pad - r) * p.in_w;
            }
            const int grow = copy * p.o_real + o_lo + static_cast<int>(cta_rank) * acc_rows;
            if (PAIR) tma_load_3d_pair(b_addr + a * acc_rows * 128, &grad_map, x, grow, img, full_b + 8 * sb);
            else tma_load_3d(b_addr + a * acc_rows * 128, &grad_map, x, grow, img, full_b + 8 * sb);
          }
          if (++kin == p.tiles_per_img) { kin = 0; ++img; }
        }
        if (++sb == p.b_stages) { sb = 0; ++round; }
      }
    }
    __syncwarp();
  } else {
    // ================= producers =================
    // Group g (warps 2 + 8g .. 9 + 8g) rebuilds the K-tiles g, g + kGroups, ... of this CTA's range.  A lane
    // owns one run of 32 consecutive elements per tile (linear: 32 channels of one row t; conv: 32
    // positions of one channel) = 64 bytes of the operand tile.
    const int pw = warp - 2;
    const int wg = pw >> 3, w8 = pw & 7;
    int row, part;                       // tile row and which run of the row
    if (MODE == 0) { row = 8 * w8 + static_cast<int>(lane >> 2); part = lane & 3; }   // k-row, 32-ch quarter
    else { row = 16 * w8 + static_cast<int>(lane >> 1); part = lane & 1; }            // channel, 32-pos half
    const uint32_t xr = row & 7;
    const uint32_t y = (MODE == 0) ? (part & 1) * 4 : part * 4;     // first 16-byte chunk of the run
    const uint32_t rowbase = (MODE == 0) ? (part >> 1) * (kTileK * 128) + row * 128 : row * 128;
    // per-warp staging of the packed values of a tile's rows (after the two rings)
    unsigned char* stg = b_ring + p.b_stages * b_stage_bytes + pw * kStageBytesPerWarp;
    const uint32_t n_keep = static_cast<uint32_t>(__ldg(p.n_keep_ptr));   // packed values in the store
    // ring position of this group's tile `it` (= it % a_stages) and how often it has wrapped
    int sa = wg % p.a_stages;
    uint32_t round = wg / p.a_stages;
    auto wait_stage = [&]() -> bool {
      if (round > 0 && lane == 0 && !mbar_wait_suspend(empty_a + 8 * sa, (round - 1) & 1)) {
        fail = 1;                                  // one lane polls; the warp follows
        atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
      }
      __syncwarp();
      return fail == 0;
    };
    auto next_stage = [&]() {
      sa += kGroups;
      while (sa >= p.a_stages) { sa -= p.a_stages; ++round; }
    };
    if (MODE != 0 && 16 * w8 >= rows_here) {
      // The warp's 16 rows hold no channel (the channels are spread evenly over the row tiles,
      // so every tile of a layer has idle warps when C is not a multiple of 128): they stay zero
      // in every stage, and the warp only keeps the barrier counts whole.
      for (int st = 0; st < p.a_stages; ++st) {
        unsigned char* dst_row = smem + st * kATileBytes + rowbase;
#pragma unroll
        for (int q = 0; q < 4; ++q)
          *reinterpret_cast<uint4*>(dst_row + (((y + q) ^ xr) << 4)) = make_uint4(0, 0, 0, 0);
      }
      for (int it = wg; it < n_kt; it += kGroups) {
        if (!wait_stage()) break;
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) { if (PAIR) mbar_arrive_rank0(full_a + 8 * sa); else mbar_arrive(full_a + 8 * sa); }
        next_stage();
      }
    } else if (MODE == 2) {
      // 1x1 stride-2 conv: the run's 32 output positions sample every other element of every
      // other input row.  Per output-row segment: 64 bitmap bits from the segment's first input
      // element, the even ones are the segment's bits; a kept element's place in the packed
      // vector counts the odd (skipped) bits before it as well.
      for (int it = wg; it < n_kt; it += kGroups) {
        const int kt = kt_begin + it;
        const int img = kt / p.tiles_per_img;
        const int q0 = (kt - img * p.tiles_per_img) * kTileK + 32 * part;     // first output position
        const int c = c0 + row;
        int left = (row < rows_here) ? min(32, p.T - q0) : 0;
        if (!wait_stage()) break;
        unsigned char* dst_row = smem + sa * kATileBytes + rowbase;
#pragma unroll
        for (int q = 0; q < 4; ++q)
          *reinterpret_cast<uint4*>(dst_row + (((y + q) ^ xr) << 4)) = make_uint4(0, 0, 0, 0);
        const long long plane = (static_cast<long long>(img) * p.C + c) * p.in_hw;
        int oy = q0 / p.ow, ox = q0 - oy * p.ow;
        int b0 = 0;                                    // position of the segment inside the run
        while (left > 0) {
          const int seg = min(left, p.ow - ox);
          const long long j = plane + static_cast<long long>(2 * oy) * p.in_w + 2 * ox;
          const long long blk = j >> kBlockShift;
          const long long wi = j >> 5;
          uint32_t rank = __ldg(offsets + blk);
          for (long long w = blk * kBlockWords; w < wi; ++w) rank += __popc(__ldg(bitmap + w));
          const uint32_t w0 = __ldg(bitmap + wi);
          const uint32_t w1 = (wi + 1 < p.n_words) ? __ldg(bitmap + wi + 1) : 0u;
          const uint32_t w2 = (wi + 2 < p.n_words) ? __ldg(bitmap + wi + 2) : 0u;
          const uint32_t sh = static_cast<uint32_t>(j & 31);
          rank += __popc(w0 & ((1u << sh) - 1u));
          unsigned long long win = (static_cast<unsigned long long>(__funnelshift_r(w1, w2, sh)) << 32) |
                                   __funnelshift_r(w0, w1, sh);
          // even bits of the window -> the segment's bits
          unsigned long long e = win & 0x5555555555555555ull;
          e = (e | (e >> 1)) & 0x3333333333333333ull;
          e = (e | (e >> 2)) & 0x0F0F0F0F0F0F0F0Full;
          e = (e | (e >> 4)) & 0x00FF00FF00FF00FFull;
          e = (e | (e >> 8)) & 0x0000FFFF0000FFFFull;
          e = (e | (e >> 16)) & 0x00000000FFFFFFFFull;
          uint32_t ev = static_cast<uint32_t>(e);
          ev = seg >= 32 ? ev : (ev & ((1u << seg) - 1u));
          // packed places of the kept samples are not contiguous (skipped odd elements lie
          // between them): eight loads in flight per round
          while (ev) {
            uint32_t vv[8];
            uint32_t e2 = ev;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const int i = e2 ? __ffs(e2) - 1 : 0;
              vv[u] = ld_packed<DT>(values, rank + __popcll(win & ((1ull << (2 * i)) - 1ull)), e2 != 0);
              e2 &= e2 - 1;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              if (ev) {
                const int b = b0 + __ffs(ev) - 1;
                ev &= ev - 1;
                const unsigned short h = (DT == 0) ? to_bf16_bits(__uint_as_float(vv[u]))
                                                   : static_cast<unsigned short>(vv[u]);
                *reinterpret_cast<unsigned short*>(dst_row + (((y + (b >> 3)) ^ xr) << 4) + ((b & 7) << 1)) = h;
              }
            }
          }
          b0 += seg; left -= seg; ox = 0; ++oy;
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) { if (PAIR) mbar_arrive_rank0(full_a + 8 * sa); else mbar_arrive(full_a + 8 * sa); }
        next_stage();
      }
    } else {
      // Flat index of the lane's run in the group's first tile, advanced by two tiles per round
      // without multiplications: linear j = t * C + c; conv j = (img * C + c) * T + position.
      const int kt_first = kt_begin + wg;
      long long j_run;                     // linear: flat index; conv: flat index of the row's image plane
      long long t_row = 0;                 // linear: row t of the run
      int kin = 0;                         // conv: K-tile within the image
      int n_run;                           // linear: channels of the run that exist (constant)
      if (MODE == 0) {
        const int c = c0 + 32 * part;
        n_run = max(0, min(32, p.C - c));
        t_row = static_cast<long long>(kt_first) * kTileK + row;
        j_run = t_row * p.C + c;
      } else {
        const int img = kt_first / p.tiles_per_img;
        kin = kt_first - img * p.tiles_per_img;
        n_run = (row < rows_here) ? 1 : 0;
        j_run = (static_cast<long long>(img) * p.C + (c0 + row)) * p.T;
      }
      const long long j_step = (MODE == 0) ? static_cast<long long>(kGroups) * kTileK * p.C : static_cast<long long>(p.C) * p.T;
      auto fetch = [&]() {                 // metadata of the run at the current position
        WordRaw r;
        r.base = 0; r.next = 0; r.words = make_uint4(0, 0, 0, 0); r.j = 0; r.nvalid = 0;
        long long j;
        int nvalid;
        if (MODE == 0) {
          nvalid = (t_row < p.T) ? n_run : 0;
          j = j_run;
        } else {
          const int pp = kin * kTileK + 32 * part;
          nvalid = n_run ? max(0, min(32, p.T - pp)) : 0;
          j = j_run + pp;
        }
        if (nvalid > 0) {
          r.nvalid = static_cast<uint32_t>(nvalid);
          r.j = static_cast<uint32_t>(j);
          const long long blk = j >> kBlockShift;
          const long long wi = j >> 5;
          r.base = __ldg(offsets + blk);
          if (static_cast<unsigned long long>(blk) != p.partial_blk) {
            r.words = __ldg(reinterpret_cast<const uint4*>(bitmap) + blk);
          } else {                                   // the last, partial block of the bitmap
            const long long w0 = blk * kBlockWords;
            r.words.x = __ldg(bitmap + w0);
            r.words.y = (w0 + 1 < p.n_words) ? __ldg(bitmap + w0 + 1) : 0u;
            r.words.z = (w0 + 2 < p.n_words) ? __ldg(bitmap + w0 + 2) : 0u;
            r.words.w = (w0 + 3 < p.n_words) ? __ldg(bitmap + w0 + 3) : 0u;
          }
          if ((r.j & 31u) && wi + 1 < p.n_words) r.next = __ldg(bitmap + wi + 1);
        }
        return r;
      };
      auto advance = [&]() {               // two K-tiles on
        if (MODE == 0) { t_row += kGroups * kTileK; j_run += j_step; }
        else {
          kin += kGroups;
          while (kin >= p.tiles_per_img) { kin -= p.tiles_per_img; j_run += j_step; }
        }
      };
      WordRaw cur = {};
      if (wg < n_kt) cur = fetch();
      for (int it = wg; it < n_kt; it += kGroups) {
        WordRaw nxt = {};
        advance();
        if (it + kGroups < n_kt) nxt = fetch();             // in flight while this tile is rebuilt
        // bits of the run and rank of its first kept element
        const uint32_t wq = (cur.j >> 5) & 3, sh = cur.j & 31;
        uint32_t rank = cur.base;
        rank += wq > 0 ? __popc(cur.words.x) : 0u;
        rank += wq > 1 ? __popc(cur.words.y) : 0u;
        rank += wq > 2 ? __popc(cur.words.z) : 0u;
        const uint32_t w0 = wq == 0 ? cur.words.x : (wq == 1 ? cur.words.y : (wq == 2 ? cur.words.z : cur.words.w));
        const uint32_t w1 = wq == 3 ? cur.next : (wq == 0 ? cur.words.y : (wq == 1 ? cur.words.z : cur.words.w));
        rank += __popc(w0 & ((1u << sh) - 1u));
        uint32_t bits = __funnelshift_r(w0, w1, sh);
        bits = cur.nvalid >= 32 ? bits : (bits & ((1u << cur.nvalid) - 1u));
        // ---- the packed values of the warp's rows -> shared memory, as bf16 ----
        // The lanes of a row (2 for conv, 4 for linear) hold consecutive runs, so a row's kept
        // values are one contiguous piece of the packed vector.  The warp copies every piece
        // with aligned 16-byte loads, lane by lane (coalesced; the lane-per-run loads they
        // replace touch a cache line per lane and saturate the L1 at low pruning ratios),
        // converting fp32 to bf16 on the way; each row has its own slot.
        constexpr int LPR = (MODE == 0) ? 4 : 2;              // lanes per row
        constexpr int RPW = 32 / LPR;                         // rows per warp
        constexpr int V = (DT == 0) ? 4 : 8;                  // packed values per 16-byte vector
        constexpr int VMAX = (32 * LPR + V - 1) / V + 1;      // vectors a row's piece can span
        constexpr int ITER = (RPW * VMAX + 31) / 32;
        constexpr int kSlot = 32 * LPR + 16;                  // bf16 values per row slot (piece + alignment slack)
        const uint32_t cnt = __popc(bits);
        uint4 chunk[4];
        // Dense tiles of fp32 activations (more than 55 % of the warp's 1024 elements kept) go
        // through the staging copy; for sparser ones the copy's fixed cost outweighs the
        // scattered loads it saves, and bf16 values (half as many cache lines per load) never
        // gain from it, so bf16 launches reserve no staging area.
        // Every run of the warp fully kept and its values 16-byte aligned: the layer that Eq. 7 gives
        // ratio 0 (there is one in every batch: the layer with the largest importance), or an
        // unpruned tensor.  The run is then 64 (128) consecutive bytes of the packed vector.
        const bool whole = __all_sync(0xFFFFFFFFu, bits == 0xFFFFFFFFu && (rank & static_cast<uint32_t>(V - 1)) == 0u);
        const bool dense = !whole && DT == 0 && __reduce_add_sync(0xFFFFFFFFu, cnt) > 560u;
        if (whole) {
          if (DT == 0) {
            const float4* src = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(values) + rank);
            float4 f[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) f[q] = __ldg(src + q);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              chunk[q].x = pack_bf16x2(f[2 * q].x, f[2 * q].y); chunk[q].y = pack_bf16x2(f[2 * q].z, f[2 * q].w);
              chunk[q].z = pack_bf16x2(f[2 * q + 1].x, f[2 * q + 1].y); chunk[q].w = pack_bf16x2(f[2 * q + 1].z, f[2 * q + 1].w);
            }
          } else {
            const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned short*>(values) + rank);
#pragma unroll
            for (int q = 0; q < 4; ++q) chunk[q] = __ldg(src + q);
          }
        } else if (dense) {
        uint32_t seg_len = cnt + __shfl_xor_sync(0xFFFFFFFFu, cnt, 1);
        if (MODE == 0) seg_len += __shfl_xor_sync(0xFFFFFFFFu, seg_len, 2);
        const uint32_t seg_start = __shfl_sync(0xFFFFFFFFu, rank, lane & ~(LPR - 1));
        const uint32_t a0 = seg_start & ~static_cast<uint32_t>(V - 1);
        const uint32_t nvec = seg_len ? (seg_start + seg_len - a0 + V - 1) / V : 0u;
        __syncwarp();                                         // the previous tile's slot reads are done
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
              else {                                          // the vector that ends past the last value
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
        // ---- the run as four 16-byte chunks of 8 elements, read from the row's slot ----
        const unsigned short* slot = reinterpret_cast<const unsigned short*>(
            stg + (lane / LPR) * (kSlot * 2)) + (rank - a0);
        uint32_t k = 0;                                       // kept elements of the run so far
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
          // sparse: one predicated global load per element, all of a lane's loads independent
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint32_t byte = (bits >> (8 * q)) & 0xFFu;
            uint32_t idx = rank + (q == 0 ? 0u : __popc(bits & ((1u << (8 * q)) - 1u)));
            uint32_t v[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const uint32_t on = (byte >> e) & 1u;
              v[e] = ld_packed<DT>(values, idx, on != 0);
              idx += on;
            }
            if (DT == 0) {
              chunk[q].x = pack_bf16x2(__uint_as_float(v[0]), __uint_as_float(v[1]));
              chunk[q].y = pack_bf16x2(__uint_as_float(v[2]), __uint_as_float(v[3]));
              chunk[q].z = pack_bf16x2(__uint_as_float(v[4]), __uint_as_float(v[5]));
              chunk[q].w = pack_bf16x2(__uint_as_float(v[6]), __uint_as_float(v[7]));
            } else {
              chunk[q].x = v[0] | (v[1] << 16); chunk[q].y = v[2] | (v[3] << 16);
              chunk[q].z = v[4] | (v[5] << 16); chunk[q].w = v[6] | (v[7] << 16);
            }
          }
        }
        if (!wait_stage()) break;
        unsigned char* dst_row = smem + sa * kATileBytes + rowbase;
#pragma unroll
        for (int q = 0; q < 4; ++q)
          *reinterpret_cast<uint4*>(dst_row + (((y + q) ^ xr) << 4)) = chunk[q];
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) { if (PAIR) mbar_arrive_rank0(full_a + 8 * sa); else mbar_arrive(full_a + 8 * sa); }
        next_stage();
        cur = nxt;
      }
    }
  }

  // ================= epilogue: TMEM -> scratch partial tile =================
  if (warp >= 2) {
    // a warp may read the 32 TMEM lanes of its quarter (warp % 4); the warps of a quarter take
    // the groups of 16 columns in turn
    const bool done = mbar_wait(acc_bar, 0, 64);
    tc_fence_after();
    if (done && !fail) {
      const int lane_grp = warp & 3;
      const int c = c0 + lane_grp * 32 + static_cast<int>(lane);
      float* out = partial + static_cast<long long>(split) * p.O * p.C;
      const int cols_here = n_acc_here * p.acc_n;
      for (int col = 16 * ((warp - 2) >> 2); col < cols_here; col += 16 * (kProdWarps / 4)) {
        uint32_t r[16];
        tmem_ld16(tmem_base + (static_cast<uint32_t>(lane_grp * 32) << 16) + col, r);
        int row0, n_ok;                   // first partial row of the 16 columns, how many exist
        if (MODE == 0) {
          row0 = o0 + col; n_ok = p.O - row0;
        } else {
          const int a = col / p.acc_n;
          const int u = u0 + a;
          const int tap = u / p.upt;
          const int o_lo = (u - tap * p.upt) * p.acc_n + (col - a * p.acc_n);
          row0 = tap * p.o_real + o_lo; n_ok = p.o_real - o_lo;
        }
        if (lane_grp * 32 + static_cast<int>(lane) < rows_here) {
#pragma unroll
          for (int e = 0; e < 16; ++e)
            if (e < n_ok && SURGEON_IN_BOUNDS(static_cast<long long>(split) * p.O * p.C +
                                                  static_cast<long long>(row0 + e) * p.C + c,
                                              static_cast<long long>(p.splits) * p.O * p.C, status))
              out[static_cast<long long>(row0 + e) * p.C + c] = __uint_as_float(r[e]);
        }
      }
    } else if (!done && lane == 0) {
      atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
    }
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();          // neither CTA leaves while the pair's MMAs or arrivals may touch it
  if (warp == 0) {
    if (PAIR) tmem_dealloc_pair(tmem_base, p.tmem_cols);
    else tmem_dealloc(tmem_base, p.tmem_cols);
  }
}

// Shifted bf16 copies of the output gradient of a k x k stride-1 convolution (Eq. 2 summed over
// input positions): out[img][tap * O + o][y' * W + x'] = g[img][o][y' + pad - r][x' + pad - s],
// zero where that lies outside the output map; tap = r * kw + s.  One thread writes 8 positions.
__global__ void __launch_bounds__(256)
grad_taps_bf16_kernel(const float* __restrict__ g, unsigned short* __restrict__ out,
                      long long chunks, DirectParams p) {
  pdl_trigger();
  const int per_row = p.pitch >> 3;
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < chunks;
       i += static_cast<long long>(gridDim.x) * blockDim.x) {
    const long long rowi = i / per_row;              // img * taps * O + tap * O + o
    const int chunk = static_cast<int>(i - rowi * per_row);
    const int v = static_cast<int>(rowi % p.O);
    const long long img = rowi / p.O;
    const int tap = v / p.o_real, o = v - tap * p.o_real;
    const int r = tap / p.kw, sft = tap - r * p.kw;
    const float* src = g + (img * p.o_real + o) * static_cast<long long>(p.oh) * p.ow;
    int pos = chunk * 8;
    int yy = pos / p.in_w, xx = pos - yy * p.in_w;   // input position
    float f[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int y = yy + p.pad - r, x = xx + p.pad - sft;
      f[e] = (pos < p.T && y >= 0 && y < p.oh && x >= 0 && x < p.ow) ? __ldg(src + y * p.ow + x) : 0.0f;
      ++pos; ++xx;
      if (xx == p.in_w) { xx = 0; ++yy; }
    }
    uint4 w;
    w.x = pack_bf16x2(f[0], f[1]); w.y = pack_bf16x2(f[2], f[3]);
    w.z = pack_bf16x2(f[4], f[5]); w.w = pack_bf16x2(f[6], f[7]);
    *reinterpret_cast<uint4*>(out + rowi * p.pitch + chunk * 8) = w;
  }
}

// The same for rows a multiple of 8 wide, where only the KW column shifts are materialised:
// out[img][s * O + o][y * W + x'] = g[img][o][y][x' + pad - s] for the OH gradient rows y (zero
// where the column lies outside the output map).  One thread reads a window of 8 + KW - 1
// gradient values and writes 8 positions of every shift.
// The same copies for a same-padded convolution (odd KW, padding (KW - 1) / 2, output map = input
// map): the source of input position pos under tap (r, s) is the flat index
// pos + (pad - r) * W + (pad - s) of the output gradient's plane, so one thread reads a window of
// 8 + KW - 1 consecutive values for a row shift r and writes the KW column shifts from it; a value
// is dropped where the shifted column leaves the row.
template <int KW>
__global__ void __launch_bounds__(256)
grad_taps_same_bf16_kernel(const float* __restrict__ g, unsigned short* __restrict__ out,
                           long long items, DirectParams p) {
  pdl_trigger();
  constexpr int H = (KW - 1) / 2;
  const int per_row = p.pitch >> 3;
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < items;
       i += static_cast<long long>(gridDim.x) * blockDim.x) {
    long long t = i / per_row;
    const int chunk = static_cast<int>(i - t * per_row);
    const int r = static_cast<int>(t % p.kh);
    t /= p.kh;
    const int o = static_cast<int>(t % p.o_real);
    const long long img = t / p.o_real;
    const float* src = g + (img * p.o_real + o) * static_cast<long long>(p.T);
    const int pos0 = chunk * 8;
    const int yy0 = pos0 / p.in_w;
    int xx = pos0 - yy0 * p.in_w;
    const int base = pos0 + (p.pad - r) * p.in_w - H;      // flat index of w[0]
    float w[8 + 2 * H];
#pragma unroll
    for (int j = 0; j < 8 + 2 * H; ++j) {
      const int q = base + j;
      w[j] = (q >= 0 && q < p.T) ? __ldg(src + q) : 0.0f;
    }
    int xe[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      xe[e] = (pos0 + e < p.T) ? xx : -64;                 // past the map: no column is valid
      if (++xx == p.in_w) xx = 0;
    }
#pragma unroll
    for (int sft = 0; sft < KW; ++sft) {
      float f[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int x = xe[e] + H - sft;
        f[e] = (x >= 0 && x < p.in_w) ? w[e + 2 * H - sft] : 0.0f;
      }
      uint4 v;
      v.x = pack_bf16x2(f[0], f[1]); v.y = pack_bf16x2(f[2], f[3]);
      v.z = pack_bf16x2(f[4], f[5]); v.w = pack_bf16x2(f[6], f[7]);
      const long long rowi = (img * p.taps + r * KW + sft) * p.o_real + o;
      *reinterpret_cast<uint4*>(out + rowi * p.pitch + chunk * 8) = v;
    }
  }
}

// SAME: padding (KW - 1) / 2 with KW odd, so the output map is as wide as the input (a multiple of
// 8): the 8 elements of a chunk are two aligned 16-byte loads, only the halo is fetched singly.
template <int KW, bool SAME>
__global__ void __launch_bounds__(256)
grad_cols_bf16_kernel(const float* __restrict__ g, unsigned short* __restrict__ out,
                      long long chunks, DirectParams p) {
  pdl_trigger();
  const int per_row = p.in_w >> 3;                     // chunks per map row
  const int per_plane = p.pitch >> 3;                  // pitch = OH * W
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < chunks;
       i += static_cast<long long>(gridDim.x) * blockDim.x) {
    const long long plane = i / per_plane;             // img * O + o
    const int chunk = static_cast<int>(i - plane * per_plane);
    const int y = chunk / per_row;
    const int x0 = (chunk - y * per_row) * 8;
    const long long img = plane / p.o_real;
    const int o = static_cast<int>(plane - img * p.o_real);
    const float* src = g + (plane * p.oh + y) * static_cast<long long>(p.ow);
    float f[8 + KW - 1];                               // f[j] = g[y][x0 + pad - (KW - 1) + j]
    if (SAME) {
      constexpr int H = (KW - 1) / 2;                  // f[j] = g[y][x0 - H + j]
      const float4 a = __ldg(reinterpret_cast<const float4*>(src + x0));
      const float4 b = __ldg(reinterpret_cast<const float4*>(src + x0 + 4));
      f[H] = a.x; f[H + 1] = a.y; f[H + 2] = a.z; f[H + 3] = a.w;
      f[H + 4] = b.x; f[H + 5] = b.y; f[H + 6] = b.z; f[H + 7] = b.w;
#pragma unroll
      for (int j = 0; j < H; ++j) {
        const int xl = x0 - H + j, xr = x0 + 8 + j;
        f[j] = xl >= 0 ? __ldg(src + xl) : 0.0f;
        f[H + 8 + j] = xr < p.ow ? __ldg(src + xr) : 0.0f;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 8 + KW - 1; ++j) {
        const int x = x0 + p.pad - (KW - 1) + j;
        f[j] = (x >= 0 && x < p.ow) ? __ldg(src + x) : 0.0f;
      }
    }
#pragma unroll
    for (int sft = 0; sft < KW; ++sft) {
      const int b = KW - 1 - sft;                      // element e of shift sft is f[e + b]
      uint4 w;
      w.x = pack_bf16x2(f[b], f[b + 1]); w.y = pack_bf16x2(f[b + 2], f[b + 3]);
      w.z = pack_bf16x2(f[b + 4], f[b + 5]); w.w = pack_bf16x2(f[b + 6], f[b + 7]);
      unsigned short* dst = out + ((img * KW + sft) * p.o_real + o) * static_cast<long long>(p.pitch) +
                            static_cast<long long>(chunk) * 8;
      *reinterpret_cast<uint4*>(dst) = w;
    }
  }
}

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                              CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                              CUtensorMapFloatOOBfill);

}  // namespace

// Shared memory: the staging area of the packed values (fp32 activations only), the gradient
// ring (as many tiles as fit beside four activation tiles, up to 4), then as many activation tiles
// as fit (up to 8).
static bool size_rings(DirectParams* p, int stage_bytes) {
  const int budget = 224 * 1024 - 1024 - stage_bytes;
  const int b_bytes = p->n_cols * (p->pair ? 64 : 128);
  int b_stages = (budget - 4 * kATileBytes) / b_bytes;
  if (b_stages > kMaxBStages) b_stages = kMaxBStages;
  if (b_stages < 2) b_stages = 2;
  if (b_stages * b_bytes + 2 * kATileBytes > budget) return false;
  int a_stages = (budget - b_stages * b_bytes) / kATileBytes;
  if (a_stages > kMaxAStages) a_stages = kMaxAStages;
  if (a_stages < 2) return false;
  p->a_stages = a_stages; p->b_stages = b_stages;
  p->smem_bytes = a_stages * kATileBytes + b_stages * b_bytes + stage_bytes + 1024;
  return true;
}

static bool compute_plan_direct(const surgeon_layer_desc& d, DirectParams* out) {
  DirectParams p{};
  if (d.kind == 0) {
    p.mode = 0;
    p.T = d.batch; p.imgs = 1;
    if (d.c_in % 8 != 0 || d.c_out % 8 != 0) return false;   // 16-byte units / TMA row pitch
  } else if (d.kind == 1 && d.kh == 1 && d.kw == 1 && d.stride == 1 && d.pad == 0) {
    p.mode = 1;
    p.T = d.h * d.w; p.imgs = d.batch;
  } else if (d.kind == 1 && d.kh == 1 && d.kw == 1 && d.stride == 2 && d.pad == 0) {
    p.mode = 2;                                    // output positions; the input is sampled
    p.ow = (d.w - 1) / 2 + 1;
    p.T = ((d.h - 1) / 2 + 1) * p.ow; p.imgs = d.batch;
    p.in_w = d.w; p.in_hw = d.h * d.w;
  } else if (d.kind == 1 && d.stride == 1 && d.kh * d.kw > 1 && d.kh <= 7 && d.kw <= 7 &&
             d.pad < d.kh && d.pad < d.kw) {
    // k x k, stride 1: the sum runs over INPUT positions, and tap (r, s) multiplies the
    // activation with the output gradient shifted by (pad - r, pad - s).  The shifted copies
    // (zero outside the map) are stacked as kh*kw*O gradient channels, which makes this the 1x1
    // problem with that many output channels; the activation operand is never expanded.
    // 8-16 channels fill an eighth of the tile's rows here; as im2col rows (channels x taps) they
    // fill a whole tile, and the gradient is read once instead of through shifted copies
    // (16 -> 160 channels, 3x3 on 32x32, batch 200: 145 against 181 us).  Fewer channels still
    // are quicker here (3 channels: 94 against 110 us).
    if (d.c_in >= 8 && d.c_in <= 16) return false;
    p.mode = 1;
    p.taps = d.kh * d.kw;
    p.kh = d.kh; p.kw = d.kw; p.pad = d.pad; p.in_h = d.h; p.in_w = d.w;
    p.oh = d.h + 2 * d.pad - d.kh + 1; p.ow = d.w + 2 * d.pad - d.kw + 1;
    if (p.oh < 1 || p.ow < 1) return false;
    p.T = d.h * d.w; p.imgs = d.batch;
    // Rows a multiple of 8 wide: only the kw column shifts need copies; a row shift is a
    // 16-byte-aligned offset of the TMA coordinate along the flattened map (zero fill outside).
    p.row_shift = (d.w % 8 == 0 && (d.kw == 2 || d.kw == 3 || d.kw == 5 || d.kw == 7)) ? 1 : 0;
  } else {
    return false;
  }
  if (p.taps == 0) p.taps = 1;
  p.o_real = d.c_out;
  if (static_cast<long long>(p.taps) * d.c_out > 2147483647LL / 256) return false;
  if (p.taps > 1 && d.c_out > 65535) return false;    // grid of the tap reduction
  p.C = d.c_in; p.O = p.taps * d.c_out;
  p.copies = p.row_shift ? p.kw : p.taps;
  p.g_len = p.row_shift ? p.oh * p.in_w : p.T;         // elements per row of the bf16 gradient copy
  p.pitch = (p.mode == 0) ? p.O : (p.g_len + 7) / 8 * 8;
  p.m_tiles = (p.C + kTileM - 1) / kTileM;
  // conv: the channels are spread evenly over the row tiles, in units of a warp's 16 rows
  p.rows_per_tile = (p.mode == 0) ? kTileM : ((p.C + p.m_tiles - 1) / p.m_tiles + 15) / 16 * 16;
  // Two or more row tiles: CTA pairs (each CTA 128 rows, the pair shares every gradient tile).
  p.pair = (p.m_tiles >= 2 && use_pairs()) ? 1 : 0;
  if (p.pair) p.m_tiles = (p.m_tiles + 1) / 2 * 2;
  if (p.mode == 0 && p.pair) {
    // accumulators of 128 columns (each CTA of the pair loads a 64-column slab of each), up to four
    const int units = (p.O + 127) / 128;
    p.acc_n = 128;
    int best_pad = -1;
    for (int na = 4; na >= 1; --na) {
      const int padded = (units + na - 1) / na * na;
      if (best_pad < 0 || padded < best_pad) { best_pad = padded; p.n_acc = na; }
    }
  } else if (p.mode == 0) {
    // columns come in slabs of 64; per CTA two accumulators of 192 or 128 columns, or one small one
    const int g = (p.O + 63) / 64;
    if (g <= 4) { p.n_acc = 1; p.acc_n = g * 64; }
    else {
      const int t6 = (g + 5) / 6 * 6, t4 = (g + 3) / 4 * 4;
      p.n_acc = 2;
      p.acc_n = (t6 <= t4) ? 192 : 128;
    }
  } else {
    // Columns come in units: one tap's output channels are cut into `upt` accumulators of acc_n
    // columns (a multiple of 16 with the fewest padded columns, then the widest); a CTA holds up
    // to three units (<= 512 TMEM columns).
    int best_waste = -1;
    for (int c = 256; c >= 16; c -= 16) {
      const int upt = (p.o_real + c - 1) / c;
      const int waste = upt * c - p.o_real;
      if (best_waste < 0 || waste < best_waste) { best_waste = waste; p.acc_n = c; p.upt = upt; }
    }
    p.n_units = p.taps * p.upt;
    const int col_cap = 512;
    p.n_acc = 1;
    while (p.n_acc < 3 && p.n_acc < p.n_units && (p.n_acc + 1) * p.acc_n <= col_cap) ++p.n_acc;
  }
  p.n_cols = p.acc_n * p.n_acc;
  p.n_tiles = (p.mode == 0) ? (p.O + p.n_cols - 1) / p.n_cols : (p.n_units + p.n_acc - 1) / p.n_acc;
  p.tiles_per_img = (p.T + kTileK - 1) / kTileK;
  const long long total = static_cast<long long>(p.imgs) * p.tiles_per_img;
  if (total > 2147483647LL / 4) return false;
  p.total_ktiles = static_cast<int>(total);
  const int sms = sm_count();
  const long long tiles_mn = static_cast<long long>(p.m_tiles) * p.n_tiles;
  const int max_splits = (p.total_ktiles + 7) / 8 < 1 ? 1 : (p.total_ktiles + 7) / 8;
  int best = 1;
  double best_cost = 1e30;
  for (int s = 1; s <= max_splits && s <= 128; ++s) {
    const long long ctas = tiles_mn * s;
    const long long waves = (ctas + sms - 1) / sms;
    const int kts = (p.total_ktiles + s - 1) / s;
    const double cost = static_cast<double>(waves) * (kts + 12) + 0.02 * s * tiles_mn / sms;
    if (cost < best_cost - 1e-9) { best_cost = cost; best = s; }
  }
  p.ktiles_per_split = (p.total_ktiles + best - 1) / best;
  p.splits = (p.total_ktiles + p.ktiles_per_split - 1) / p.ktiles_per_split;
  p.tmem_cols = 32;
  while (p.tmem_cols < p.n_cols) p.tmem_cols *= 2;
  if (!size_rings(&p, kStageBytes)) return false;   // the launcher sizes them again for the dtype
  *out = p;
  return true;
}

bool plan_direct(const surgeon_layer_desc& d, DirectParams* out) {
  struct Tag {};
  return memo_plan<Tag>(d, use_pairs() ? 1 : 0, out, [&](DirectParams* p) { return compute_plan_direct(d, p); });
}

size_t direct_grad_bf16_bytes(const DirectParams& p) {
  const size_t b = (p.mode == 0) ? static_cast<size_t>(p.T) * p.O * 2
                                 : static_cast<size_t>(p.imgs) * p.copies * p.o_real * p.pitch * 2;
  return (b + 255) & ~static_cast<size_t>(255);
}

// The bf16 copy (or shifted copies) of the output gradient that the tensor maps of the direct
// kernels read: one streaming pre-pass.
cudaError_t launch_direct_prepass(const DirectParams& p, const float* grad_out, void* grad_bf16,
                                  cudaStream_t stream) {
  cudaError_t e;
  if (p.row_shift) {
    const long long chunks = static_cast<long long>(p.imgs) * p.o_real * (p.pitch >> 3);
    const long long want = (chunks + 255) / 256;
    const long long cap = 32LL * sm_count();
    const int grid = static_cast<int>(want < 1 ? 1 : (want > cap ? cap : want));
    unsigned short* ob = static_cast<unsigned short*>(grad_bf16);
    const bool same = (p.kw & 1) && p.pad == (p.kw - 1) / 2 && p.ow == p.in_w &&
                      (reinterpret_cast<uintptr_t>(grad_out) & 15) == 0;
    switch (p.kw) {
      case 2: grad_cols_bf16_kernel<2, false><<<grid, 256, 0, stream>>>(grad_out, ob, chunks, p); break;
      case 3:
        if (same) grad_cols_bf16_kernel<3, true><<<grid, 256, 0, stream>>>(grad_out, ob, chunks, p);
        else grad_cols_bf16_kernel<3, false><<<grid, 256, 0, stream>>>(grad_out, ob, chunks, p);
        break;
      case 5:
        if (same) grad_cols_bf16_kernel<5, true><<<grid, 256, 0, stream>>>(grad_out, ob, chunks, p);
        else grad_cols_bf16_kernel<5, false><<<grid, 256, 0, stream>>>(grad_out, ob, chunks, p);
        break;
      default:
        if (same) grad_cols_bf16_kernel<7, true><<<grid, 256, 0, stream>>>(grad_out, ob, chunks, p);
        else grad_cols_bf16_kernel<7, false><<<grid, 256, 0, stream>>>(grad_out, ob, chunks, p);
        break;
    }
    note_launches(1);
    e = cudaGetLastError();
  } else if (p.taps > 1) {
    const long long chunks = static_cast<long long>(p.imgs) * p.O * (p.pitch >> 3);
    const long long want = (chunks + 255) / 256;
    const long long cap = 32LL * sm_count();
    const int grid = static_cast<int>(want < 1 ? 1 : (want > cap ? cap : want));
    unsigned short* ob = static_cast<unsigned short*>(grad_bf16);
    const bool same = (p.kw & 1) && p.kh == p.kw && p.pad == (p.kw - 1) / 2 && p.ow == p.in_w &&
                      p.oh == p.in_h && (p.kw == 3 || p.kw == 5 || p.kw == 7);
    if (same) {
      const long long items = chunks / p.kw;        // one thread per row shift writes the kw column shifts
      const long long want_s = (items + 255) / 256;
      const int grid_s = static_cast<int>(want_s < 1 ? 1 : (want_s > cap ? cap : want_s));
      if (p.kw == 3) grad_taps_same_bf16_kernel<3><<<grid_s, 256, 0, stream>>>(grad_out, ob, items, p);
      else if (p.kw == 5) grad_taps_same_bf16_kernel<5><<<grid_s, 256, 0, stream>>>(grad_out, ob, items, p);
      else grad_taps_same_bf16_kernel<7><<<grid_s, 256, 0, stream>>>(grad_out, ob, items, p);
    } else {
      grad_taps_bf16_kernel<<<grid, 256, 0, stream>>>(grad_out, ob, chunks, p);
    }
    note_launches(1);
    e = cudaGetLastError();
  } else if (p.mode != 0 && p.pitch != p.T)     // rows padded to a 16-byte pitch for the tensor map
    e = launch_grad_to_bf16_rows(grad_out, static_cast<long long>(p.imgs) * p.O, p.T, p.pitch,
                                 grad_bf16, stream);
  else
    e = launch_grad_to_bf16(grad_out, static_cast<long long>(p.imgs) * p.O * p.T, grad_bf16, stream);
  return e;
}

// Tensor map over the bf16 gradient copy.  Linear: [T rows][O columns], box 64 columns x 64 rows.
// Conv: [images][copies * O rows][g_len positions], box 64 positions x `box_rows` rows.
cudaError_t encode_direct_grad_map(const DirectParams& p, void* grad_bf16, int box_rows, CUtensorMap* out) {
  CUtensorMap& map = *out;
  const EncodeFn encode = reinterpret_cast<EncodeFn>(tensor_map_encode_fn());
  if (!encode) return cudaErrorNotSupported;
  CUresult r;
  if (p.mode == 0) {
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(p.O), static_cast<cuuint64_t>(p.T)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(p.O) * 2};
    const cuuint32_t box[2] = {64, static_cast<cuuint32_t>(kTileK)};
    const cuuint32_t estr[2] = {1, 1};
    r = encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, grad_bf16, dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {
    const cuuint64_t rows = static_cast<cuuint64_t>(p.copies) * p.o_real;
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(p.g_len), rows, static_cast<cuuint64_t>(p.imgs)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(p.pitch) * 2,
                                   static_cast<cuuint64_t>(p.pitch) * rows * 2};
    const cuuint32_t box[3] = {static_cast<cuuint32_t>(kTileK),
                               static_cast<cuuint32_t>(box_rows), 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    r = encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, grad_bf16, dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t launch_direct(const surgeon_compressed& act, const DirectParams& plan,
                          const float* grad_out, void* grad_bf16, float* partial,
                          uint32_t* status, cudaStream_t stream) {
  DirectParams p = plan;
  if (!size_rings(&p, act.dt == 0 ? kStageBytes : 0)) return cudaErrorInvalidValue;
  p.n_words = (act.n + 31) / 32;
  p.n_keep_ptr = reinterpret_cast<const long long*>(reinterpret_cast<const char*>(act.header) +
                                                    offsetof(surgeon_header, n_keep));
  p.partial_blk = (act.n % SURGEON_BLOCK) ? static_cast<unsigned>(act.n / SURGEON_BLOCK) : 0xFFFFFFFFu;
  cudaError_t e = launch_direct_prepass(p, grad_out, grad_bf16, stream);
  if (e != cudaSuccess) return e;
  CUtensorMap map;
  e = encode_direct_grad_map(p, grad_bf16, p.pair ? p.acc_n / 2 : p.acc_n, &map);
  if (e != cudaSuccess) return e;
  dim3 grid(p.m_tiles, p.n_tiles, p.splits);
  auto launch = [&](auto kernel) -> cudaError_t {
    cudaError_t err = allow_dynamic_smem(reinterpret_cast<const void*>(kernel), p.smem_bytes);
    if (err != cudaSuccess) return err;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = static_cast<size_t>(p.smem_bytes);
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = p.pair ? 2 : 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // starts while the gradient pre-pass drains: set-up and the first activation tiles overlap it
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, act.bitmap, act.values, act.block_offsets, map, partial,
                              status, p);
  };
  const int key = p.mode * 4 + (act.dt ? 2 : 0) + p.pair;
  switch (key) {
    case 0: e = launch(dw_direct_kernel<0, 0, 0>); break;
    case 1: e = launch(dw_direct_kernel<0, 0, 1>); break;
    case 2: e = launch(dw_direct_kernel<1, 0, 0>); break;
    case 3: e = launch(dw_direct_kernel<1, 0, 1>); break;
    case 4: e = launch(dw_direct_kernel<0, 1, 0>); break;
    case 5: e = launch(dw_direct_kernel<0, 1, 1>); break;
    case 6: e = launch(dw_direct_kernel<1, 1, 0>); break;
    case 7: e = launch(dw_direct_kernel<1, 1, 1>); break;
    case 8: e = launch(dw_direct_kernel<0, 2, 0>); break;
    case 9: e = launch(dw_direct_kernel<0, 2, 1>); break;
    case 10: e = launch(dw_direct_kernel<1, 2, 0>); break;
    default: e = launch(dw_direct_kernel<1, 2, 1>); break;
  }
  note_launches(1);
  return e;
}

}  // namespace surgeon

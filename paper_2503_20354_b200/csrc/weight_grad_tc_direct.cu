// Tensor-core weight gradient for layers whose im2col operand is the activation itself: linear
// layers ([T, C] activations) and 1x1 / stride 1 / pad 0 convolutions (NCHW).  Algorithm 1,
// Reshape and gradient steps with Eq. 2:  D[c, o] = sum_k A[k, c] * G[k, o].
//
//   c (input channel)  -> MMA M, 128 per CTA (TMEM lanes)
//   o (output channel) -> MMA N, one or two accumulators of up to 256 columns
//   k (row t, or image b and position p) -> MMA K, 64 per pipeline stage
//
// Operand layouts follow the memory order of the tensors, so that neither needs a transpose:
//   linear : A[t, c] and G[t, o] are contiguous along c / o -> both operands MN-major
//            (rows of 64 channels = 128 bytes, one row per k, 128-byte swizzle);
//   conv   : A[b, c, p] and G[b, o, p] are contiguous along p -> both operands K-major.
// The output gradient is converted to bf16 once by a streaming pre-pass and arrives by TMA.
// The activation operand is rebuilt from the compressed store by 16 producer warps: a thread
// owns units of 8 consecutive elements, finds their rank in the packed vector from the block
// offset and the 128 bitmap bits of their block, gathers the kept values and writes one 16-byte
// piece of the swizzled tile.  The loads of a unit are issued two units ahead of its store
// (metadata) and one unit ahead (values), so their latency overlaps the work on earlier units.
// One thread issues the MMAs, one the TMA loads; split-K partial tiles are reduced in a fixed
// order by the caller.  Every wait is bounded and ends in SURGEON_ERR_TIMEOUT.
#include <cuda.h>

#include "surgeon_internal.cuh"
#include "tc_common.cuh"
#include "weight_grad_tc_conv.cuh"

namespace surgeon {

namespace {

using namespace tc;

constexpr int kTileM = 128;
constexpr int kTileK = 64;
constexpr int kProdWarps = 16;
constexpr int kProdThreads = kProdWarps * 32;
constexpr int kThreads = 64 + kProdThreads;     // warp 0: MMA, warp 1: TMA, warps 2..17: producers
constexpr int kMaxStages = 4;
constexpr int kUnitsPerTile = kTileM * kTileK / 8;            // 1024
constexpr int kUnitsPerThread = kUnitsPerTile / kProdThreads; // 2
constexpr int kATileBytes = kTileM * kTileK * 2;              // 16 KB

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

// What a thread needs to decompress one unit: where it goes, and the raw metadata loads.
struct UnitMeta {
  uint32_t dst;        // byte offset inside the A tile; 0xFFFFFFFF = write zeros at `zdst`
  uint32_t zdst;
  uint32_t bitpos;     // position of the unit's first bit inside its 128-bit block
  uint32_t base;       // kept elements before the block
  uint4 words;         // the block's 128 bitmap bits
};

template <int DT>
__device__ __forceinline__ void gather_unit(const UnitMeta& m, const void* __restrict__ values,
                                            uint32_t (&v)[8]) {
  const uint32_t w[4] = {m.words.x, m.words.y, m.words.z, m.words.w};
  const uint32_t wi = m.bitpos >> 5, sh = m.bitpos & 31;
  uint32_t rank = m.base;
#pragma unroll
  for (int j = 0; j < 3; ++j) rank += (static_cast<uint32_t>(j) < wi) ? __popc(w[j]) : 0u;
  const uint32_t word = wi == 0 ? w[0] : (wi == 1 ? w[1] : (wi == 2 ? w[2] : w[3]));
  rank += __popc(word & ((1u << sh) - 1u));
  const uint32_t bits = (m.dst == 0xFFFFFFFFu) ? 0u : ((word >> sh) & 0xFFu);
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const bool on = (bits >> e) & 1u;
    const uint32_t idx = rank + __popc(bits & ((1u << e) - 1u));
    if (DT == 0) v[e] = on ? __ldg(reinterpret_cast<const uint32_t*>(values) + idx) : 0u;
    else v[e] = on ? static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(values) + idx)) : 0u;
  }
}

template <int DT>
__device__ __forceinline__ uint4 pack_unit(const uint32_t (&v)[8]) {
  uint4 o;
  if (DT == 0) {
    o.x = pack_bf16x2(__uint_as_float(v[0]), __uint_as_float(v[1]));
    o.y = pack_bf16x2(__uint_as_float(v[2]), __uint_as_float(v[3]));
    o.z = pack_bf16x2(__uint_as_float(v[4]), __uint_as_float(v[5]));
    o.w = pack_bf16x2(__uint_as_float(v[6]), __uint_as_float(v[7]));
  } else {
    o.x = v[0] | (v[1] << 16); o.y = v[2] | (v[3] << 16);
    o.z = v[4] | (v[5] << 16); o.w = v[6] | (v[7] << 16);
  }
  return o;
}

template <int DT, int MODE>
__global__ void __launch_bounds__(kThreads, 1)
dw_direct_kernel(const uint32_t* __restrict__ bitmap, const void* __restrict__ values,
                 const uint32_t* __restrict__ offsets, const __grid_constant__ CUtensorMap grad_map,
                 float* __restrict__ partial, uint32_t* __restrict__ status, DirectParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int stage_bytes = kATileBytes + p.n_cols * 128;
  __shared__ __align__(8) unsigned long long bars[2 * kMaxStages + 1];
  __shared__ uint32_t tmem_slot;
  __shared__ volatile uint32_t fail;

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const uint32_t lane = lane_id();
  const int m_tile = blockIdx.x, n_tile = blockIdx.y, split = blockIdx.z;
  const int c0 = m_tile * kTileM;
  const int o0 = n_tile * p.n_cols;
  const int kt_begin = split * p.ktiles_per_split;
  const int kt_end = min(kt_begin + p.ktiles_per_split, p.total_ktiles);
  const int n_kt = kt_end - kt_begin;

  const uint32_t full_bar = smem_u32(bars);
  const uint32_t empty_bar = smem_u32(bars + kMaxStages);
  const uint32_t acc_bar = smem_u32(bars + 2 * kMaxStages);
  if (tid == 0) {
    tma_prefetch_desc(&grad_map);
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(full_bar + 8 * s, kProdWarps + 1);   // 16 producer warps + the TMA thread
      mbar_init(empty_bar + 8 * s, 1);
    }
    mbar_init(acc_bar, 1);
    fail = 0;
    fence_barrier_init();
  }
  if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;

  if (warp == 0) {
    // ================= MMA issuer =================
    if (lane == 0) {
      const uint32_t idesc = make_idesc(kTileM, p.acc_n) | (MODE == 0 ? ((1u << 15) | (1u << 16)) : 0u);
      bool ok = true;
      for (int it = 0; it < n_kt; ++it) {
        const int s = it % p.stages;
        ok = mbar_wait(full_bar + 8 * s, (it / p.stages) & 1);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_addr = smem_u32(smem + s * stage_bytes);
        const uint32_t b_addr = a_addr + kATileBytes;
#pragma unroll
        for (int kk = 0; kk < kTileK / 16; ++kk) {
          if (MODE == 0) {
            const uint64_t da = make_desc_mn(a_addr + kk * 2048);
            for (int a = 0; a < p.n_acc; ++a)
              umma_bf16(tmem_base + a * p.acc_n, da,
                        make_desc_mn(b_addr + a * p.acc_n * 128 + kk * 2048), idesc,
                        (it > 0 || kk > 0) ? 1u : 0u);
          } else {
            const uint64_t da = make_desc(a_addr + kk * 32);
            for (int a = 0; a < p.n_acc; ++a)
              umma_bf16(tmem_base + a * p.acc_n, da,
                        make_desc(b_addr + a * p.acc_n * 128 + kk * 32), idesc,
                        (it > 0 || kk > 0) ? 1u : 0u);
          }
        }
        umma_commit(empty_bar + 8 * s);
      }
      if (!ok) { fail = 1; atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT)); }
      umma_commit(acc_bar);
    }
    __syncwarp();
  } else if (warp == 1) {
    // ================= gradient tiles by TMA =================
    if (lane == 0) {
      for (int it = 0; it < n_kt; ++it) {
        const int s = it % p.stages;
        if (it >= p.stages && !mbar_wait(empty_bar + 8 * s, ((it / p.stages) - 1) & 1)) {
          fail = 1;
          atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
          break;
        }
        const int kt = kt_begin + it;
        const uint32_t b_addr = smem_u32(smem + s * stage_bytes) + kATileBytes;
        mbar_arrive_expect_tx(full_bar + 8 * s, static_cast<uint32_t>(p.n_cols) * 128u);
        if (MODE == 0) {
          for (int g = 0; g < p.n_cols / 64; ++g)
            tma_load_2d(b_addr + g * (kTileK * 128), &grad_map, o0 + g * 64, kt * kTileK,
                        full_bar + 8 * s);
        } else {
          const int img = kt / p.tiles_per_img;
          const int p0 = (kt - img * p.tiles_per_img) * kTileK;
          for (int a = 0; a < p.n_acc; ++a)
            tma_load_3d(b_addr + a * p.acc_n * 128, &grad_map, p0, o0 + a * p.acc_n, img,
                        full_bar + 8 * s);
        }
      }
    }
    __syncwarp();
  } else {
    // ================= producers =================
    const int ptid = tid - 64;
    const int n_units = n_kt * kUnitsPerThread;
    // unit i of this thread: K-tile kt_begin + i/2, unit index (i&1)*512 + ptid inside the tile
    auto load_meta = [&](int i) {
      UnitMeta m;
      const int kt = kt_begin + (i >> 1);
      const int u = (i & 1) * kProdThreads + ptid;
      long long j;
      bool valid;
      if (MODE == 0) {
        const int k = u >> 4, h = u & 15;                   // k-row, 8-channel unit of the row
        const long long t = static_cast<long long>(kt) * kTileK + k;
        const int c = c0 + 8 * h;
        valid = t < p.T && c < p.C;
        j = t * p.C + c;
        m.zdst = static_cast<uint32_t>((h >> 3) * (kTileK * 128) + k * 128 + (((h & 7) ^ (k & 7)) << 4));
      } else {
        const int row = u >> 3, chunk = u & 7;              // channel row, 8-position unit
        const int img = kt / p.tiles_per_img;
        const int pp = (kt - img * p.tiles_per_img) * kTileK + 8 * chunk;
        const int c = c0 + row;
        valid = c < p.C && pp < p.T;
        j = (static_cast<long long>(img) * p.C + c) * p.T + pp;
        m.zdst = tile_off(row, chunk);
      }
      m.dst = valid ? m.zdst : 0xFFFFFFFFu;
      m.bitpos = 0; m.base = 0; m.words = make_uint4(0, 0, 0, 0);
      if (valid) {
        const long long blk = j >> kBlockShift;
        m.bitpos = static_cast<uint32_t>(j) & (SURGEON_BLOCK - 1);
        m.base = __ldg(offsets + blk);
        if (blk * kBlockWords + kBlockWords <= p.n_words) {
          m.words = __ldg(reinterpret_cast<const uint4*>(bitmap) + blk);
        } else {                                   // the last, partial block of the bitmap
          const long long w0 = blk * kBlockWords;
          m.words.x = __ldg(bitmap + w0);
          m.words.y = (w0 + 1 < p.n_words) ? __ldg(bitmap + w0 + 1) : 0u;
          m.words.z = (w0 + 2 < p.n_words) ? __ldg(bitmap + w0 + 2) : 0u;
          m.words.w = 0u;
        }
      }
      return m;
    };
    UnitMeta m_next = {};      // metadata of unit i+1
    uint32_t v_cur[8];         // values of unit i
    UnitMeta m_cur = {};
    if (n_units > 0) {
      m_cur = load_meta(0);
      m_next = (n_units > 1) ? load_meta(1) : m_cur;
      gather_unit<DT>(m_cur, values, v_cur);
    }
    bool ok = true;
    for (int i = 0; i < n_units; ++i) {
      UnitMeta m_after = {};
      if (i + 2 < n_units) m_after = load_meta(i + 2);
      uint32_t v_next[8];
      if (i + 1 < n_units) gather_unit<DT>(m_next, values, v_next);
      const int it = i >> 1;
      const int s = it % p.stages;
      if ((i & 1) == 0 && it >= p.stages) {
        if (!mbar_wait(empty_bar + 8 * s, ((it / p.stages) - 1) & 1)) {
          fail = 1;
          atomicMax(status, static_cast<uint32_t>(SURGEON_ERR_TIMEOUT));
        }
      }
      if (fail) { ok = false; break; }
      unsigned char* a_tile = smem + s * stage_bytes;
      *reinterpret_cast<uint4*>(a_tile + m_cur.zdst) = pack_unit<DT>(v_cur);
      if (i & 1) {
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(full_bar + 8 * s);
      }
      m_cur = m_next;
      m_next = m_after;
#pragma unroll
      for (int e = 0; e < 8; ++e) v_cur[e] = v_next[e];
    }
    (void)ok;
  }

  // ================= epilogue: TMEM -> scratch partial tile =================
  if (warp >= 2 && warp <= 5) {
    const bool done = mbar_wait(acc_bar, 0, 256);
    tc_fence_after();
    if (done && !fail) {
      const int lane_grp = warp & 3;              // TMEM lanes this warp may read
      const int c = c0 + lane_grp * 32 + static_cast<int>(lane);
      float* out = partial + static_cast<long long>(split) * p.O * p.C;
      for (int col = 0; col < p.n_cols; col += 16) {
        uint32_t r[16];
        tmem_ld16(tmem_base + (static_cast<uint32_t>(lane_grp * 32) << 16) + col, r);
        if (c < p.C) {
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const int o = o0 + col + e;
            if (o < p.O) out[static_cast<long long>(o) * p.C + c] = __uint_as_float(r[e]);
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

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                              CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                              CUtensorMapFloatOOBfill);

}  // namespace

bool plan_direct(const surgeon_layer_desc& d, DirectParams* out) {
  DirectParams p{};
  if (d.kind == 0) {
    p.mode = 0;
    p.T = d.batch; p.imgs = 1;
    if (d.c_in % 8 != 0 || d.c_out % 8 != 0) return false;   // 16-byte units / TMA row pitch
  } else if (d.kind == 1 && d.kh == 1 && d.kw == 1 && d.stride == 1 && d.pad == 0) {
    p.mode = 1;
    p.T = d.h * d.w; p.imgs = d.batch;
    if (p.T % 8 != 0) return false;                          // units never straddle a plane
  } else {
    return false;
  }
  p.C = d.c_in; p.O = d.c_out;
  if (p.mode == 0) {
    // columns come in slabs of 64; per CTA two accumulators of 192 or 128 columns, or one small one
    const int g = (p.O + 63) / 64;
    if (g <= 4) { p.n_acc = 1; p.acc_n = g * 64; }
    else {
      const int t6 = (g + 5) / 6 * 6, t4 = (g + 3) / 4 * 4;
      p.n_acc = 2;
      p.acc_n = (t6 <= t4) ? 192 : 128;
    }
  } else {
    int acc_n = 0;
    for (int c = 256; c >= 128; c -= 16)
      if (p.O % c == 0) { acc_n = c; break; }
    if (acc_n == 0) acc_n = (p.O <= 256) ? (p.O + 15) / 16 * 16 : 256;
    p.acc_n = acc_n;
    p.n_acc = (p.O + acc_n - 1) / acc_n >= 2 ? 2 : 1;
  }
  p.n_cols = p.acc_n * p.n_acc;
  p.n_tiles = (p.O + p.n_cols - 1) / p.n_cols;
  p.m_tiles = (p.C + kTileM - 1) / kTileM;
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
  const int stage_bytes = kATileBytes + p.n_cols * 128;
  int stages = (225 * 1024 - 1024) / stage_bytes;
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < 2) return false;
  p.stages = stages;
  p.smem_bytes = stages * stage_bytes + 1024;
  *out = p;
  return true;
}

size_t direct_grad_bf16_bytes(const DirectParams& p) {
  const size_t b = static_cast<size_t>(p.imgs) * p.O * p.T * 2;
  return (b + 255) & ~static_cast<size_t>(255);
}

cudaError_t launch_direct(const surgeon_compressed& act, const DirectParams& plan,
                          const float* grad_out, void* grad_bf16, float* partial,
                          uint32_t* status, cudaStream_t stream) {
  DirectParams p = plan;
  p.n_words = (act.n + 31) / 32;
  const long long gn = static_cast<long long>(p.imgs) * p.O * p.T;
  cudaError_t e = launch_grad_to_bf16(grad_out, gn, grad_bf16, stream);
  if (e != cudaSuccess) return e;
  const EncodeFn encode = reinterpret_cast<EncodeFn>(tensor_map_encode_fn());
  if (!encode) return cudaErrorNotSupported;
  CUtensorMap map;
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
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(p.T), static_cast<cuuint64_t>(p.O),
                                static_cast<cuuint64_t>(p.imgs)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(p.T) * 2,
                                   static_cast<cuuint64_t>(p.T) * p.O * 2};
    const cuuint32_t box[3] = {static_cast<cuuint32_t>(kTileK), static_cast<cuuint32_t>(p.acc_n), 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    r = encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, grad_bf16, dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
  dim3 grid(p.m_tiles, p.n_tiles, p.splits);
  auto launch = [&](auto kernel) -> cudaError_t {
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           p.smem_bytes);
    if (err != cudaSuccess) return err;
    kernel<<<grid, kThreads, p.smem_bytes, stream>>>(act.bitmap, act.values, act.block_offsets, map,
                                                     partial, status, p);
    return cudaGetLastError();
  };
  if (p.mode == 0) e = act.dt == 0 ? launch(dw_direct_kernel<0, 0>) : launch(dw_direct_kernel<1, 0>);
  else e = act.dt == 0 ? launch(dw_direct_kernel<0, 1>) : launch(dw_direct_kernel<1, 1>);
  note_launches(1);
  return e;
}

}  // namespace surgeon

// extern "C" entry points of libsurgeon: argument checks and host-side arithmetic; every step
// that touches tensor data is a kernel launched from the other translation units.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>

#include <atomic>

#include "surgeon_internal.cuh"

namespace surgeon {

static std::atomic<unsigned long long> g_launches{0};
void note_launches(int n) { g_launches.fetch_add(static_cast<unsigned long long>(n), std::memory_order_relaxed); }
unsigned long long launches_so_far() { return g_launches.load(std::memory_order_relaxed); }

void* tensor_map_encode_fn() {
  static void* fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return p;
  }();
  return fn;
}

cudaError_t allow_dynamic_smem(const void* kernel, int bytes) {
  struct Seen { const void* fn; int dev; std::atomic<int> bytes; };
  static Seen seen[256];
  static std::atomic<int> n_seen{0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) dev = 0;
  const int n = n_seen.load(std::memory_order_acquire);
  Seen* hit = nullptr;
  for (int i = 0; i < n; ++i)
    if (seen[i].fn == kernel && seen[i].dev == dev) { hit = &seen[i]; break; }
  if (hit && hit->bytes.load(std::memory_order_relaxed) >= bytes) return cudaSuccess;
  const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return e;
  // two threads may both set the attribute (harmless: the larger value is set again by whoever
  // needs it); the table only grows
  if (hit) {
    hit->bytes.store(bytes, std::memory_order_relaxed);
  } else {
    const int slot = n_seen.load(std::memory_order_relaxed);
    if (slot < 256) {
      seen[slot].fn = kernel; seen[slot].dev = dev; seen[slot].bytes.store(bytes, std::memory_order_relaxed);
      n_seen.store(slot + 1, std::memory_order_release);
    }
  }
  return cudaSuccess;
}

int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
      n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Algorithm 1: prune step: kept count for `ratio`; one double multiply, one floor.
inline int64_t kept_count(int64_t n, double ratio) {
  double pruned = floor(ratio * static_cast<double>(n));
  if (pruned < 0.0) pruned = 0.0;
  int64_t np = static_cast<int64_t>(pruned);
  if (np > n) np = n;
  return n - np;
}

bool desc_ok(const surgeon_layer_desc* d, surgeon_status* why) {
  *why = SURGEON_ERR_INVALID_ARG;
  if (!d) return false;
  if (d->kind != 0 && d->kind != 1) return false;
  if (d->path != 0 && d->path != 1) return false;
  if (d->batch <= 0 || d->c_in <= 0 || d->c_out <= 0 || d->h <= 0 || d->w <= 0) return false;
  if (d->kh <= 0 || d->kw <= 0 || d->stride <= 0 || d->pad < 0) return false;
  if (d->kind == 0 && (d->h != 1 || d->w != 1 || d->kh != 1 || d->kw != 1 || d->stride != 1 ||
                       d->pad != 0))
    return false;
  if (d->h + 2 * d->pad < d->kh || d->w + 2 * d->pad < d->kw) return false;
  if (d->groups < 0) return false;
  if (d->groups > 1 && (d->kind != 1 || d->c_in % d->groups != 0 || d->c_out % d->groups != 0)) return false;
  *why = SURGEON_ERR_UNSUPPORTED;
  const long long oh = (d->h + 2 * d->pad - d->kh) / d->stride + 1;
  const long long ow = (d->w + 2 * d->pad - d->kw) / d->stride + 1;
  const long long lim = 2147483647LL;
  if (static_cast<long long>(d->batch) * d->c_in * d->h * d->w > lim) return false;
  if (static_cast<long long>(d->batch) * d->c_out * oh * ow > lim) return false;
  if (static_cast<long long>(d->c_out) * d->c_in * d->kh * d->kw > lim) return false;
  if (d->pad >= d->kh || d->pad >= d->kw) return false;  // windows entirely in the padding
  *why = SURGEON_OK;
  return true;
}

}  // namespace
}  // namespace surgeon

using namespace surgeon;

extern "C" {

surgeon_status surgeon_layer_ratios(const double* gi, const double* lam, int32_t n_layers,
                                    double* ratios_out) {
  if (!gi || !lam || !ratios_out || n_layers <= 0) return SURGEON_ERR_INVALID_ARG;
  double total = 0.0, g_max = 0.0;
  for (int i = 0; i < n_layers; ++i) {
    if (!isfinite(gi[i]) || gi[i] < 0.0 || !isfinite(lam[i]) || !(lam[i] > 0.0))
      return SURGEON_ERR_INVALID_ARG;
    total += lam[i];
    if (gi[i] > g_max) g_max = gi[i];
  }
  // Eq. 5: M_i = -log(m_i / sum m); kept in ratios_out until Eq. 6 overwrites it.
  double m_max = 0.0;
  for (int i = 0; i < n_layers; ++i) {
    const double mi = -log(lam[i] / total);
    ratios_out[i] = mi;
    if (mi > m_max) m_max = mi;
  }
  // Eq. 6: I_i = (M_i / max M) * (G_i / max G).
  double i_max = 0.0;
  for (int i = 0; i < n_layers; ++i) {
    const double imp = (m_max > 0.0 && g_max > 0.0) ? (ratios_out[i] / m_max) * (gi[i] / g_max) : 0.0;
    ratios_out[i] = imp;
    if (imp > i_max) i_max = imp;
  }
  if (!(i_max > 0.0)) {
    for (int i = 0; i < n_layers; ++i) ratios_out[i] = 0.0;
    return SURGEON_ERR_DEGENERATE;
  }
  // Eq. 7: p_i = 1 - I_i / max I.
  for (int i = 0; i < n_layers; ++i) ratios_out[i] = 1.0 - ratios_out[i] / i_max;
  return SURGEON_OK;
}

surgeon_status surgeon_layer_ratios_rule(const double* gi, const double* lam, int32_t n_layers,
                                         surgeon_ratio_rule rule, double static_ratio,
                                         double* ratios_out) {
  if (!ratios_out || n_layers <= 0) return SURGEON_ERR_INVALID_ARG;
  if (rule == SURGEON_RULE_BOTH) return surgeon_layer_ratios(gi, lam, n_layers, ratios_out);
  if (rule == SURGEON_RULE_STATIC) {
    if (!(static_ratio >= 0.0 && static_ratio <= 1.0)) return SURGEON_ERR_INVALID_ARG;
    for (int i = 0; i < n_layers; ++i) ratios_out[i] = static_ratio;
    return SURGEON_OK;
  }
  double i_max = 0.0;
  if (rule == SURGEON_RULE_NO_GRADIENT) {
    // Eq. 5, then Eq. 6 with the gradient factor taken as 1: I_i = M_i / max M
    if (!lam) return SURGEON_ERR_INVALID_ARG;
    double total = 0.0;
    for (int i = 0; i < n_layers; ++i) {
      if (!isfinite(lam[i]) || !(lam[i] > 0.0)) return SURGEON_ERR_INVALID_ARG;
      total += lam[i];
    }
    for (int i = 0; i < n_layers; ++i) {
      ratios_out[i] = -log(lam[i] / total);
      if (ratios_out[i] > i_max) i_max = ratios_out[i];
    }
  } else if (rule == SURGEON_RULE_NO_MEMORY) {
    // Eq. 6 with the memory factor taken as 1: I_i = G_i / max G
    if (!gi) return SURGEON_ERR_INVALID_ARG;
    for (int i = 0; i < n_layers; ++i) {
      if (!isfinite(gi[i]) || gi[i] < 0.0) return SURGEON_ERR_INVALID_ARG;
      ratios_out[i] = gi[i];
      if (gi[i] > i_max) i_max = gi[i];
    }
  } else {
    return SURGEON_ERR_INVALID_ARG;
  }
  if (!(i_max > 0.0)) {
    for (int i = 0; i < n_layers; ++i) ratios_out[i] = 0.0;
    return SURGEON_ERR_DEGENERATE;
  }
  // Eq. 7 (the inner normalisation cancels against the outer one)
  for (int i = 0; i < n_layers; ++i) ratios_out[i] = 1.0 - ratios_out[i] / i_max;
  return SURGEON_OK;
}

surgeon_status surgeon_compact_sizes(int64_t n, surgeon_dtype dt, double ratio, int64_t* n_keep,
                                     size_t* bitmap_bytes, size_t* values_bytes,
                                     size_t* offsets_bytes, size_t* workspace_bytes) {
  if (n < 0 || !(ratio >= 0.0 && ratio <= 1.0) || (dt != SURGEON_F32 && dt != SURGEON_BF16))
    return SURGEON_ERR_INVALID_ARG;
  if (n > SURGEON_MAX_N) return SURGEON_ERR_UNSUPPORTED;
  const int64_t k = kept_count(n, ratio);
  if (n_keep) *n_keep = k;
  if (bitmap_bytes) *bitmap_bytes = static_cast<size_t>((n + 31) / 32) * 4;
  if (values_bytes) *values_bytes = static_cast<size_t>(k) * (dt == SURGEON_F32 ? 4 : 2);
  if (offsets_bytes)
    *offsets_bytes = static_cast<size_t>((n + SURGEON_BLOCK - 1) / SURGEON_BLOCK + 1) * 4;
  if (workspace_bytes) *workspace_bytes = prune_workspace_bytes(n, static_cast<int>(dt));
  return SURGEON_OK;
}

surgeon_status surgeon_prune_compact(const void* x, int64_t n, surgeon_dtype dt, double ratio,
                                     surgeon_compressed* out, void* workspace,
                                     size_t workspace_bytes, void* cuda_stream) {
  return surgeon_prune_compact_flags(x, n, dt, ratio, 0u, out, workspace, workspace_bytes, cuda_stream);
}

surgeon_status surgeon_prune_compact_flags(const void* x, int64_t n, surgeon_dtype dt, double ratio,
                                           uint32_t flags, surgeon_compressed* out, void* workspace,
                                           size_t workspace_bytes, void* cuda_stream) {
  if (flags & ~static_cast<uint32_t>(SURGEON_STORE_DROP_ZEROS | SURGEON_DEBUG_STALL_BARRIER))
    return SURGEON_ERR_INVALID_ARG;
  if (!out || n < 0 || !(ratio >= 0.0 && ratio <= 1.0) ||
      (dt != SURGEON_F32 && dt != SURGEON_BF16))
    return SURGEON_ERR_INVALID_ARG;
  if (n > SURGEON_MAX_N) return SURGEON_ERR_UNSUPPORTED;
  const int64_t k = kept_count(n, ratio);
  if (!out->header || !out->block_offsets || !workspace) return SURGEON_ERR_INVALID_ARG;
  if (n > 0 && (!x || !out->bitmap)) return SURGEON_ERR_INVALID_ARG;
  if (k > 0 && !out->values) return SURGEON_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(out->bitmap) || !aligned16(out->values) ||
      !aligned16(out->block_offsets) || !aligned16(out->header) || !aligned16(workspace))
    return SURGEON_ERR_INVALID_ARG;
  if (workspace_bytes < prune_workspace_bytes(n, static_cast<int>(dt))) return SURGEON_ERR_BUFFER_TOO_SMALL;
  out->n = n;
  out->dt = static_cast<int32_t>(dt);
  out->reserved = 0;
  const cudaError_t e = launch_prune_compact(x, n, static_cast<int>(dt), k, *out, workspace,
                                             static_cast<cudaStream_t>(cuda_stream),
                                             (flags & SURGEON_STORE_DROP_ZEROS) ? 1 : 0,
                                             (flags & SURGEON_DEBUG_STALL_BARRIER) ? 1 : 0);
  return e == cudaSuccess ? SURGEON_OK : SURGEON_ERR_CUDA;
}

size_t surgeon_weight_grad_workspace(const surgeon_layer_desc* d) {
  surgeon_status why;
  if (!desc_ok(d, &why)) return 0;
  const size_t b = d->groups > 1 ? weight_grad_grouped_workspace(*d)
                   : (d->path == 1 ? weight_grad_fp32_workspace(*d) : weight_grad_tc_workspace(*d));
  return (b + 255) & ~static_cast<size_t>(255);
}

surgeon_status surgeon_weight_grad(const surgeon_compressed* act, const surgeon_layer_desc* d,
                                   const float* grad_out, float* dw, int32_t accumulate,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
  surgeon_status why;
  if (!desc_ok(d, &why)) return why;
  if (!act || !grad_out || !dw || !act->bitmap || !act->block_offsets) return SURGEON_ERR_INVALID_ARG;
  if (act->dt != SURGEON_F32 && act->dt != SURGEON_BF16) return SURGEON_ERR_INVALID_ARG;
  if (act->n != static_cast<int64_t>(d->batch) * d->c_in * d->h * d->w) return SURGEON_ERR_INVALID_ARG;
  if (!aligned16(act->bitmap) || !aligned16(act->values) || !aligned16(act->block_offsets) ||
      !aligned16(grad_out) || !aligned16(dw) || !aligned16(workspace))
    return SURGEON_ERR_INVALID_ARG;
  const size_t need = surgeon_weight_grad_workspace(d);
  if (need > 0 && (!workspace || workspace_bytes < need)) return SURGEON_ERR_BUFFER_TOO_SMALL;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (d->groups > 1 && need == 0) return SURGEON_ERR_UNSUPPORTED;
  const cudaError_t e =
      d->groups > 1 ? launch_weight_grad_grouped(*act, *d, grad_out, dw, accumulate ? 1 : 0, workspace, s)
      : d->path == 1 ? launch_weight_grad_fp32(*act, *d, grad_out, dw, accumulate ? 1 : 0, workspace, s)
                     : launch_weight_grad_tc(*act, *d, grad_out, dw, accumulate ? 1 : 0, workspace, s);
  if (e == cudaErrorNotSupported) return SURGEON_ERR_UNSUPPORTED;
  if (e != cudaSuccess && getenv("SURGEON_VERBOSE"))
    fprintf(stderr, "surgeon_weight_grad: %s\n", cudaGetErrorString(e));
  return e == cudaSuccess ? SURGEON_OK : SURGEON_ERR_CUDA;
}

surgeon_status surgeon_decompress(const surgeon_compressed* act, void* x_out, void* cuda_stream) {
  if (!act || act->n < 0 || (act->dt != SURGEON_F32 && act->dt != SURGEON_BF16))
    return SURGEON_ERR_INVALID_ARG;
  if (act->n > 0 && (!x_out || !act->bitmap || !act->block_offsets)) return SURGEON_ERR_INVALID_ARG;
  if (!aligned16(x_out) || !aligned16(act->bitmap) || !aligned16(act->values) ||
      !aligned16(act->block_offsets))
    return SURGEON_ERR_INVALID_ARG;
  const cudaError_t e = launch_decompress(*act, x_out, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? SURGEON_OK : SURGEON_ERR_CUDA;
}

surgeon_status surgeon_gradient_importance(const float* dw, int64_t n_weights, double* gi_out,
                                           void* workspace, size_t workspace_bytes,
                                           void* cuda_stream) {
  if (!gi_out || !workspace || n_weights < 0 || (n_weights > 0 && !dw)) return SURGEON_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 7u) || (reinterpret_cast<uintptr_t>(gi_out) & 7u) ||
      (reinterpret_cast<uintptr_t>(dw) & 3u))
    return SURGEON_ERR_INVALID_ARG;
  if (workspace_bytes < SURGEON_GI_WORKSPACE_BYTES) return SURGEON_ERR_BUFFER_TOO_SMALL;
  const cudaError_t e = launch_gradient_importance(dw, n_weights, gi_out, workspace,
                                                   static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? SURGEON_OK : SURGEON_ERR_CUDA;
}

uint64_t surgeon_launch_count(void) { return launches_so_far(); }

const char* surgeon_status_string(surgeon_status s) {
  switch (s) {
    case SURGEON_OK: return "ok";
    case SURGEON_ERR_INVALID_ARG: return "invalid argument";
    case SURGEON_ERR_BUFFER_TOO_SMALL: return "buffer too small";
    case SURGEON_ERR_DEGENERATE: return "degenerate input (ratio rule is 0/0)";
    case SURGEON_ERR_UNSUPPORTED: return "unsupported geometry, dtype or size";
    case SURGEON_ERR_CUDA: return "CUDA runtime error";
    case SURGEON_ERR_TIMEOUT: return "device-side bounded wait expired";
    case SURGEON_ERR_INTERNAL: return "device-side self-check failed";
  }
  return "unknown status";
}

}  // extern "C"

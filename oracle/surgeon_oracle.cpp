// CPU oracle for the dynamic-activation-sparsity path of arXiv 2503.20354.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the CUDA library is
// checked against.  It shares no code, header, table or helper with the CUDA path, and nothing
// in the product may call it.  Every function takes the steps in the order the paper states
// them; there is no blocking, fusion or reordering.  Arithmetic is IEEE double.
//
// What the paper fixes and what is a reading of it is listed next to each function.  Every
// function here is pinned by CPU tests against hand-worked values, closed forms, brute force
// on tiny inputs or an independent library routine; none is "parity unpinned".
//
// Build: g++ -O2 -std=c++17 -fopenmp -shared -fPIC surgeon_oracle.cpp -o libsurgeon_oracle.so

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// Magnitude key: the element's bit pattern with the sign bit cleared, read as an unsigned
// integer.  For finite values this orders exactly like |x|; -0 equals +0; Inf sits above every
// finite value and NaN above Inf.  (The paper gives no pruning criterion beyond "prune with
// ratio p", Algorithm 1: prune step; magnitude is the criterion of the activation-pruning works it
// builds on, Section 2.)
inline uint32_t key_of(const void* x, int64_t j, int dt) {
  if (dt == 0) {
    uint32_t b;
    std::memcpy(&b, static_cast<const char*>(x) + 4 * j, 4);
    return b & 0x7FFFFFFFu;
  }
  uint16_t h;
  std::memcpy(&h, static_cast<const char*>(x) + 2 * j, 2);
  return static_cast<uint32_t>(h & 0x7FFFu);
}

// Element j widened to double (fp32 exactly; bf16 = the upper 16 bits of an fp32).
inline double value_of(const void* x, int64_t j, int dt) {
  uint32_t b;
  if (dt == 0) {
    std::memcpy(&b, static_cast<const char*>(x) + 4 * j, 4);
  } else {
    uint16_t h;
    std::memcpy(&h, static_cast<const char*>(x) + 2 * j, 2);
    b = static_cast<uint32_t>(h) << 16;
  }
  float f;
  std::memcpy(&f, &b, 4);
  return static_cast<double>(f);
}

struct KeyIdx {
  uint32_t key;
  int64_t idx;
};

// Total order of the selection: larger key first; equal keys by ascending flat index.
inline bool before(const KeyIdx& a, const KeyIdx& b) {
  if (a.key != b.key) return a.key > b.key;
  return a.idx < b.idx;
}

}  // namespace

extern "C" {

// Eq. 5, Eq. 6, Eq. 7, evaluated in the order the paper writes them.
//   m_i = size(A_i);  M_i = -log(m_i / sum_j m_j)                   (Eq. 5, natural log)
//   I_i = Norm(M_i) * Norm(G_i),  Norm(v)_i = v_i / max_j v_j       (Eq. 6, "Max Normalization")
//   p_i = 1 - I_i / max_j I_j                                       (Eq. 7)
// Returns 0, or 3 when max_j I_j is zero (Eq. 7 would be 0/0): p is then all zeros.
int oracle_layer_ratios(const double* G, const double* m, int l, double* p) {
  double total = 0.0;
  for (int i = 0; i < l; ++i) total += m[i];
  std::vector<double> M(l), I(l);
  for (int i = 0; i < l; ++i) M[i] = -std::log(m[i] / total);
  double maxM = 0.0, maxG = 0.0;
  for (int i = 0; i < l; ++i) {
    maxM = std::max(maxM, M[i]);
    maxG = std::max(maxG, G[i]);
  }
  double maxI = 0.0;
  for (int i = 0; i < l; ++i) {
    double normM = (maxM > 0.0) ? M[i] / maxM : 0.0;
    double normG = (maxG > 0.0) ? G[i] / maxG : 0.0;
    I[i] = normM * normG;
    maxI = std::max(maxI, I[i]);
  }
  if (!(maxI > 0.0)) {
    for (int i = 0; i < l; ++i) p[i] = 0.0;
    return 3;
  }
  for (int i = 0; i < l; ++i) p[i] = 1.0 - I[i] / maxI;
  return 0;
}

// Eq. 4: Gradient Importance of one layer, G = sqrt( sum_j (dw_j)^2 / N ), the root mean square
// of the layer's N weight-gradient entries.  One pass in index order, squares and sum in double.
// N = 0 has no mean: returns 0.
double oracle_gradient_importance(const float* dw, int64_t n) {
  if (n <= 0) return 0.0;
  double sum = 0.0;
  for (int64_t j = 0; j < n; ++j) {
    const double v = static_cast<double>(dw[j]);
    sum += v * v;
  }
  return std::sqrt(sum / static_cast<double>(n));
}

// The ratio rule with one factor of Eq. 6 left out, as in the paper's ablation (Section 5.3,
// the table of strategies), and the global static ratio it is compared with (Section 5.3,
// "global static sparsity").  The paper names the variants without formulas; the reading is:
//   rule 0  "Ours"    I_i = Norm(M_i) * Norm(G_i)        (Eq. 6 as printed)
//   rule 1  "w/o G"   I_i = Norm(M_i)                    (the gradient factor replaced by 1)
//   rule 2  "w/o M"   I_i = Norm(G_i)                    (the memory factor replaced by 1)
//   rule 3  static    p_i = p_static for every layer     (no importance at all)
// followed by Eq. 7 unchanged for rules 0-2.  Returns 0, or 3 when max_j I_j is zero.
int oracle_layer_ratios_rule(const double* G, const double* m, int l, int rule, double p_static,
                             double* p) {
  if (rule == 3) {
    for (int i = 0; i < l; ++i) p[i] = p_static;
    return 0;
  }
  double total = 0.0;
  for (int i = 0; i < l; ++i) total += m[i];
  std::vector<double> M(l), I(l);
  for (int i = 0; i < l; ++i) M[i] = -std::log(m[i] / total);
  double maxM = 0.0, maxG = 0.0;
  for (int i = 0; i < l; ++i) {
    maxM = std::max(maxM, M[i]);
    maxG = std::max(maxG, G[i]);
  }
  double maxI = 0.0;
  for (int i = 0; i < l; ++i) {
    const double normM = (rule == 2) ? 1.0 : ((maxM > 0.0) ? M[i] / maxM : 0.0);
    const double normG = (rule == 1) ? 1.0 : ((maxG > 0.0) ? G[i] / maxG : 0.0);
    I[i] = normM * normG;
    maxI = std::max(maxI, I[i]);
  }
  if (!(maxI > 0.0)) {
    for (int i = 0; i < l; ++i) p[i] = 0.0;
    return 3;
  }
  for (int i = 0; i < l; ++i) p[i] = 1.0 - I[i] / maxI;
  return 0;
}

// Algorithm 1: prune step: how many elements "ratio p" removes.  The paper does not state the
// rounding; the reading is n_prune = floor(p*n) with the product taken once in double, and
// the kept count is what remains.
int64_t oracle_n_keep(int64_t n, double p) {
  int64_t n_prune = static_cast<int64_t>(std::floor(p * static_cast<double>(n)));
  if (n_prune < 0) n_prune = 0;
  if (n_prune > n) n_prune = n;
  return n - n_prune;
}

// Algorithm 1: prune step: the kept set = the k elements that come first when all elements are
// ordered by magnitude key descending, equal keys by ascending flat index.
//   method 0: stable sort of all indices by key (the definition written out);
//   method 1: std::nth_element on (key, index) pairs under the same total order (same result,
//             linear time; for large n).
// keep[j] (n bytes) is set to 1 for kept elements, else 0.  tau = key of the k-th element in
// that order (all ones for k == 0: 0xFFFFFFFF for fp32, 0xFFFF for bf16), c_gt = number of
// keys strictly above tau, q = k - c_gt.
void oracle_select(const void* x, int64_t n, int dt, int64_t k, int method, uint8_t* keep,
                   uint32_t* tau, int64_t* c_gt, int64_t* q) {
  std::memset(keep, 0, static_cast<size_t>(n));
  if (k <= 0) {
    *tau = (dt == 0) ? 0xFFFFFFFFu : 0xFFFFu;
    *c_gt = 0;
    *q = 0;
    return;
  }
  std::vector<KeyIdx> v(static_cast<size_t>(n));
  for (int64_t j = 0; j < n; ++j) v[j] = KeyIdx{key_of(x, j, dt), j};
  if (method == 0) {
    std::stable_sort(v.begin(), v.end(),
                     [](const KeyIdx& a, const KeyIdx& b) { return a.key > b.key; });
  } else {
    std::nth_element(v.begin(), v.begin() + (k - 1), v.end(), before);
  }
  uint32_t t = v[k - 1].key;
  int64_t greater = 0;
  for (int64_t r = 0; r < k; ++r) {
    keep[v[r].idx] = 1;
    if (v[r].key > t) ++greater;
  }
  *tau = t;
  *c_gt = greater;
  *q = k - greater;
}

// Algorithm 1: decompose step / Section 4.2: decompose the pruned activation into the vector of kept
// elements (ascending flat index, bit copies) and an index of 1 bit per element.  Bit (j & 31)
// of 32-bit word (j >> 5) belongs to flat index j.  offsets[b] = kept elements below b*block;
// offsets[ceil(n/block)] = total kept.  Returns the kept count.
int64_t oracle_compact(const void* x, int64_t n, int dt, const uint8_t* keep, int64_t block,
                       uint32_t* bitmap, void* values, uint64_t* offsets) {
  const int64_t n_words = (n + 31) / 32;
  for (int64_t w = 0; w < n_words; ++w) bitmap[w] = 0u;
  const size_t es = (dt == 0) ? 4 : 2;
  int64_t r = 0;
  for (int64_t j = 0; j < n; ++j) {
    if (j % block == 0) offsets[j / block] = static_cast<uint64_t>(r);
    if (keep[j]) {
      bitmap[j >> 5] |= (1u << (j & 31));
      std::memcpy(static_cast<char*>(values) + es * r, static_cast<const char*>(x) + es * j, es);
      ++r;
    }
  }
  offsets[(n + block - 1) / block] = static_cast<uint64_t>(r);
  return r;
}

// Algorithm 1: Reshape step: Reshape(values, index) -> dense tensor with +0 where nothing is kept.
void oracle_decompress(const uint32_t* bitmap, const void* values, int64_t n, int dt,
                       void* x_out) {
  const size_t es = (dt == 0) ? 4 : 2;
  std::memset(x_out, 0, es * static_cast<size_t>(n));
  int64_t r = 0;
  for (int64_t j = 0; j < n; ++j) {
    if ((bitmap[j >> 5] >> (j & 31)) & 1u) {
      std::memcpy(static_cast<char*>(x_out) + es * j, static_cast<const char*>(values) + es * r,
                  es);
      ++r;
    }
  }
}

// Eq. 2 for a bias-free linear layer, in the weight's own layout (the transpose of the
// paper's A^T * dL/dA_{i+1}):  dw[o, c] = sum_t g[t, o] * a[t, c].
// a: [T, C] of dt (dense, already pruned); g: [T, O] fp32; dw: [O, C] double.
void oracle_dw_linear(const void* a, int dt, const float* g, int64_t T, int64_t C, int64_t O,
                      double* dw) {
#pragma omp parallel for schedule(static)
  for (int64_t o = 0; o < O; ++o) {
    for (int64_t c = 0; c < C; ++c) {
      double acc = 0.0;
      for (int64_t t = 0; t < T; ++t)
        acc += static_cast<double>(g[t * O + o]) * value_of(a, t * C + c, dt);
      dw[o * C + c] = acc;
    }
  }
}

// Weight gradient of a 2-D cross-correlation layer (the layer type the paper defers to its
// appendix; standard definition, dilation 1, groups 1, no bias):
//   dw[o, c, r, s] = sum_{b, y, x} g[b, o, y, x] * a[b, c, y*stride + r - pad, x*stride + s - pad]
// with out-of-range input positions contributing zero;  OH = (H + 2*pad - KH)/stride + 1.
// a: NCHW [B, C, H, W] of dt; g: [B, O, OH, OW] fp32; dw: [O, C, KH, KW] double.
void oracle_dw_conv2d(const void* a, int dt, const float* g, int64_t B, int64_t C, int64_t H,
                      int64_t W, int64_t O, int64_t KH, int64_t KW, int64_t stride, int64_t pad,
                      double* dw) {
  const int64_t OH = (H + 2 * pad - KH) / stride + 1;
  const int64_t OW = (W + 2 * pad - KW) / stride + 1;
#pragma omp parallel for schedule(static)
  for (int64_t o = 0; o < O; ++o) {
    for (int64_t c = 0; c < C; ++c) {
      for (int64_t r = 0; r < KH; ++r) {
        for (int64_t s = 0; s < KW; ++s) {
          double acc = 0.0;
          for (int64_t b = 0; b < B; ++b) {
            for (int64_t y = 0; y < OH; ++y) {
              const int64_t iy = y * stride + r - pad;
              if (iy < 0 || iy >= H) continue;
              for (int64_t xo = 0; xo < OW; ++xo) {
                const int64_t ix = xo * stride + s - pad;
                if (ix < 0 || ix >= W) continue;
                acc += static_cast<double>(g[((b * O + o) * OH + y) * OW + xo]) *
                       value_of(a, ((b * C + c) * H + iy) * W + ix, dt);
              }
            }
          }
          dw[((o * C + c) * KH + r) * KW + s] = acc;
        }
      }
    }
  }
}

// One entry of the conv2d weight gradient (for spot checks at sizes where the full tensor
// would take minutes).
double oracle_dw_conv2d_entry(const void* a, int dt, const float* g, int64_t B, int64_t C,
                              int64_t H, int64_t W, int64_t O, int64_t KH, int64_t KW,
                              int64_t stride, int64_t pad, int64_t o, int64_t c, int64_t r,
                              int64_t s) {
  const int64_t OH = (H + 2 * pad - KH) / stride + 1;
  const int64_t OW = (W + 2 * pad - KW) / stride + 1;
  double acc = 0.0;
  for (int64_t b = 0; b < B; ++b) {
    for (int64_t y = 0; y < OH; ++y) {
      const int64_t iy = y * stride + r - pad;
      if (iy < 0 || iy >= H) continue;
      for (int64_t xo = 0; xo < OW; ++xo) {
        const int64_t ix = xo * stride + s - pad;
        if (ix < 0 || ix >= W) continue;
        acc += static_cast<double>(g[((b * O + o) * OH + y) * OW + xo]) *
               value_of(a, ((b * C + c) * H + iy) * W + ix, dt);
      }
    }
  }
  return acc;
}

// Weight gradient of a GROUPED 2-D cross-correlation (the layer type of ResNeXt's 3x3 convolutions
// and of a depthwise convolution; the paper adapts ResNeXt-29 on CIFAR100-C, Section 5.1).  The
// standard definition: input and output channels are cut into `groups` equal consecutive ranges,
// output channel o belongs to group g = o / (O / groups) and sees only the C / groups input
// channels of that group:
//   dw[o, c', r, s] = sum_{b, y, x} g[b, o, y, x] * a[b, g*(C/groups) + c', y*stride + r - pad,
//                                                      x*stride + s - pad]
// a: NCHW [B, C, H, W] of dt; g: [B, O, OH, OW] fp32; dw: [O, C/groups, KH, KW] double.
void oracle_dw_conv2d_grouped(const void* a, int dt, const float* g, int64_t B, int64_t C,
                              int64_t H, int64_t W, int64_t O, int64_t KH, int64_t KW,
                              int64_t stride, int64_t pad, int64_t groups, double* dw) {
  const int64_t OH = (H + 2 * pad - KH) / stride + 1;
  const int64_t OW = (W + 2 * pad - KW) / stride + 1;
  const int64_t Cg = C / groups, Og = O / groups;
#pragma omp parallel for schedule(static)
  for (int64_t o = 0; o < O; ++o) {
    const int64_t grp = o / Og;
    for (int64_t cl = 0; cl < Cg; ++cl) {
      const int64_t c = grp * Cg + cl;
      for (int64_t r = 0; r < KH; ++r) {
        for (int64_t s = 0; s < KW; ++s) {
          double acc = 0.0;
          for (int64_t b = 0; b < B; ++b) {
            for (int64_t y = 0; y < OH; ++y) {
              const int64_t iy = y * stride + r - pad;
              if (iy < 0 || iy >= H) continue;
              for (int64_t xo = 0; xo < OW; ++xo) {
                const int64_t ix = xo * stride + s - pad;
                if (ix < 0 || ix >= W) continue;
                acc += static_cast<double>(g[((b * O + o) * OH + y) * OW + xo]) *
                       value_of(a, ((b * C + c) * H + iy) * W + ix, dt);
              }
            }
          }
          dw[((o * Cg + cl) * KH + r) * KW + s] = acc;
        }
      }
    }
  }
}

// One entry of the linear weight gradient.
double oracle_dw_linear_entry(const void* a, int dt, const float* g, int64_t T, int64_t C,
                              int64_t O, int64_t o, int64_t c) {
  double acc = 0.0;
  for (int64_t t = 0; t < T; ++t)
    acc += static_cast<double>(g[t * O + o]) * value_of(a, t * C + c, dt);
  return acc;
}

int oracle_num_threads() {
#ifdef _OPENMP
  int n = 1;
#pragma omp parallel
  {
#pragma omp single
    n = omp_get_num_threads();
  }
  return n;
#else
  return 1;
#endif
}

}  // extern "C"

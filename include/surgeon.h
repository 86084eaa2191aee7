/*
 * surgeon.h — C ABI of the B200-native dynamic-activation-sparsity hot path.
 *
 * The library implements one path of "SURGEON: Memory-Adaptive Fully Test-Time
 * Adaptation via Dynamic Activation Sparsity" (arXiv 2503.20354):
 *
 *   per-layer pruning ratio (Eq. 5-7)  ->  prune the saved activation A_i at
 *   that ratio (Algorithm 1: prune step)   ->  store it as packed kept values plus a
 *   1-bit-per-element index (Algorithm 1: decompose step; Section 4.2, "Algorithm"
 *   paragraph)  ->  rebuild the sparse activation and form the weight gradient
 *   from it (Algorithm 1: Reshape and gradient steps; Eq. 2).
 *
 * Conventions shared by every entry point
 *   - Every function returns a surgeon_status; argument errors are found on the
 *     host before anything is launched.
 *   - "device pointer" = global memory of the current CUDA device, owned by the
 *     caller, at least 16-byte aligned (else SURGEON_ERR_INVALID_ARG).
 *     "host pointer" = ordinary host memory.
 *   - The library never allocates or frees device memory, never synchronises the
 *     device and keeps no pointer after a call returns.  All device work of a call is
 *     enqueued on the caller's stream (`cuda_stream` is a cudaStream_t passed as
 *     void*; NULL = the legacy default stream).
 *   - Conditions that only the device can see (a bounded wait that ran out, an
 *     internal count that does not add up) are reported in
 *     surgeon_header::status, never by a trap.  Once one is seen, the kernels of
 *     that call that have not run yet store nothing to the outputs.
 *   - Flat index j of an activation element = its row-major index in the tensor
 *     as given: NCHW for conv2d inputs, [T, C] for linear inputs.
 */
#ifndef SURGEON_H_
#define SURGEON_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SURGEON_OK = 0,
  SURGEON_ERR_INVALID_ARG = 1,      /* null / misaligned pointer, negative size, ratio outside [0,1] */
  SURGEON_ERR_BUFFER_TOO_SMALL = 2, /* workspace smaller than the size query says                    */
  SURGEON_ERR_DEGENERATE = 3,       /* Eq. 7 is 0/0 for this input; output filled with zeros          */
  SURGEON_ERR_UNSUPPORTED = 4,      /* layer geometry / dtype / size the library does not implement   */
  SURGEON_ERR_CUDA = 5,             /* a CUDA runtime call failed                                     */
  SURGEON_ERR_TIMEOUT = 6,          /* device-side bounded wait expired (only in surgeon_header)      */
  SURGEON_ERR_INTERNAL = 7          /* device-side self-check failed, e.g. the kept count does not
                                       add up (only in surgeon_header)                                */
} surgeon_status;

typedef enum { SURGEON_F32 = 0, SURGEON_BF16 = 1 } surgeon_dtype;

/* Elements covered by one entry of surgeon_compressed::block_offsets. */
#define SURGEON_BLOCK 128
/* Largest supported element count of one activation tensor (counts are packed in 31 bits). */
#define SURGEON_MAX_N 2147483647LL

/* ------------------------------------------------------------------------------------------
 * Eq. 5-7: per-layer pruning ratios from Gradient Importance G_i and activation size m_i.
 *   M_i = -log(m_i / sum_j m_j)                              (Eq. 5)
 *   I_i = (M_i / max_j M_j) * (G_i / max_j G_j)              (Eq. 6, max-normalisation)
 *   p_i = 1 - I_i / max_j I_j                                (Eq. 7)
 * gi, lam, ratios_out: HOST pointers to n_layers doubles.  lam[i] is size(A_i) in any one unit
 * (bytes or elements).  ratios_out[i] is in [0,1]; at least one layer gets exactly 0.
 * Errors: INVALID_ARG for null pointers, n_layers <= 0, a non-finite or negative gi, a
 * non-finite or non-positive lam.  DEGENERATE when max_j I_j == 0 (one layer only, or every
 * gi zero): ratios_out is filled with 0 (no pruning) and the code is returned.
 * ---------------------------------------------------------------------------------------- */
surgeon_status surgeon_layer_ratios(const double* gi, const double* lam, int32_t n_layers,
                                    double* ratios_out);

/* ------------------------------------------------------------------------------------------
 * Section 5.3 (the ablation's strategies) and the global static ratio it is compared with: the
 * rule of Eq. 5-7 with one factor of Eq. 6 left out.  The paper names the variants without
 * formulas; here the missing factor is 1 and Eq. 7 is unchanged:
 *   SURGEON_RULE_BOTH         I_i = Norm(M_i) * Norm(G_i)   (= surgeon_layer_ratios)
 *   SURGEON_RULE_NO_GRADIENT  I_i = Norm(M_i)               ("w/o G"; gi may be NULL)
 *   SURGEON_RULE_NO_MEMORY    I_i = Norm(G_i)               ("w/o M"; lam may be NULL)
 *   SURGEON_RULE_STATIC       p_i = static_ratio            (gi and lam may be NULL)
 * Arguments, units and errors as for surgeon_layer_ratios; static_ratio outside [0,1] or an
 * unknown rule is INVALID_ARG.
 * ---------------------------------------------------------------------------------------- */
typedef enum {
  SURGEON_RULE_BOTH = 0,
  SURGEON_RULE_NO_GRADIENT = 1,
  SURGEON_RULE_NO_MEMORY = 2,
  SURGEON_RULE_STATIC = 3
} surgeon_ratio_rule;
surgeon_status surgeon_layer_ratios_rule(const double* gi, const double* lam, int32_t n_layers,
                                         surgeon_ratio_rule rule, double static_ratio,
                                         double* ratios_out);

/* ------------------------------------------------------------------------------------------
 * Eq. 4: Gradient Importance of one layer, G = sqrt( sum_j (dw_j)^2 / N ): the root mean square
 * of the N entries of the layer's weight gradient, the G_i that surgeon_layer_ratios takes.
 * dw: DEVICE pointer to n_weights fp32 values (as written by surgeon_weight_grad).  gi_out:
 * DEVICE pointer to one double.  workspace: DEVICE scratch of at least
 * SURGEON_GI_WORKSPACE_BYTES bytes, 8-byte aligned, owned by the caller, not shared with a call
 * in flight.  Squares and sums are taken in double, in a fixed order, so the result is bitwise
 * reproducible.  n_weights = 0 gives 0.  Asynchronous on cuda_stream.
 * Errors: INVALID_ARG (null pointer, n_weights < 0), BUFFER_TOO_SMALL, CUDA.
 * ---------------------------------------------------------------------------------------- */
#define SURGEON_GI_WORKSPACE_BYTES 8192
surgeon_status surgeon_gradient_importance(const float* dw, int64_t n_weights, double* gi_out,
                                           void* workspace, size_t workspace_bytes,
                                           void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Algorithm 1: prune step ("prune A_i with ratio p"): the kept count and the buffer sizes.
 * Pure host arithmetic.  n_prune = floor(ratio * n) evaluated in IEEE double, n_keep = n -
 * n_prune.  Any out pointer may be NULL.  bitmap_bytes = 4*ceil(n/32); values_bytes =
 * n_keep*sizeof(dt); offsets_bytes = 4*(ceil(n/SURGEON_BLOCK)+1); workspace_bytes = scratch
 * surgeon_prune_compact needs for this n and dt (independent of ratio).
 * Errors: INVALID_ARG (n < 0, ratio not in [0,1], bad dt), UNSUPPORTED (n > SURGEON_MAX_N).
 * ---------------------------------------------------------------------------------------- */
surgeon_status surgeon_compact_sizes(int64_t n, surgeon_dtype dt, double ratio, int64_t* n_keep,
                                     size_t* bitmap_bytes, size_t* values_bytes,
                                     size_t* offsets_bytes, size_t* workspace_bytes);

/* Result header written by the device (32 bytes, device memory). */
typedef struct surgeon_header {
  uint32_t threshold_key; /* magnitude key (bit pattern with the sign cleared) of the n_keep-th
                             largest element; all ones (0xFFFFFFFF / 0xFFFF) when n_keep == 0   */
  uint32_t status;        /* surgeon_status seen by the device, SURGEON_OK if none              */
  int64_t n_keep;         /* kept count                                                         */
  int64_t n_greater;      /* elements whose key is strictly above threshold_key                 */
  int64_t tie_quota;      /* n_keep - n_greater: elements with key == threshold_key that are
                             kept; they are the ones with the lowest flat indices               */
} surgeon_header;

/* The compressed activation store: Section 4.2 caches the pruned activation as the vector of
 * kept elements plus an index of 1 bit per element.  All pointers are DEVICE pointers owned by
 * the caller.  block_offsets is this library's own addition so that a reader can start in the
 * middle of the tensor without a scan. */
typedef struct surgeon_compressed {
  int64_t n;               /* element count of the dense tensor                                 */
  int32_t dt;              /* surgeon_dtype of x and of values                                  */
  int32_t reserved;
  uint32_t* bitmap;        /* ceil(n/32) words; bit (j & 31) of word (j >> 5) is 1 iff flat
                              index j is kept; pad bits of the last word are 0                  */
  void* values;            /* n_keep elements of dt in ascending flat index, bit copies of x    */
  uint32_t* block_offsets; /* ceil(n/SURGEON_BLOCK)+1 entries; entry b = number of kept elements
                              with flat index < b*SURGEON_BLOCK; the last entry = n_keep        */
  surgeon_header* header;  /* 32 bytes                                                          */
} surgeon_compressed;

/* ------------------------------------------------------------------------------------------
 * Algorithm 1: prune and decompose steps: prune the activation x (n elements of dt, device pointer, not
 * modified) by magnitude at `ratio` and write the compressed store.
 * Kept set: the n_keep elements with the largest magnitude key (bit pattern with the sign bit
 * cleared, compared as an unsigned integer: equals |x| order on finite data, -0 ties with +0,
 * Inf above finite, NaN above Inf); among elements whose key equals the threshold the ones
 * with the lowest flat index are kept.  Kept zeros are stored like any other kept element.
 * out->n and out->dt are set by the call; the four pointers in *out must be device buffers of
 * at least the sizes surgeon_compact_sizes reports for (n, dt, ratio).  workspace: device
 * scratch of workspace_bytes >= the reported size; contents are undefined afterwards.
 * Asynchronous on cuda_stream.  n == 0 is legal (header only).
 * Errors: INVALID_ARG, BUFFER_TOO_SMALL, UNSUPPORTED, CUDA.
 * ---------------------------------------------------------------------------------------- */
surgeon_status surgeon_prune_compact(const void* x, int64_t n, surgeon_dtype dt, double ratio,
                                     surgeon_compressed* out, void* workspace,
                                     size_t workspace_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Algorithm 1, decompose step ("the non-zero values ... and a 1-bit index"): the same call with
 * store options.  SURGEON_STORE_DROP_ZEROS: the selection is unchanged, but a kept element that
 * is exactly zero (+0 or -0; post-ReLU data at a low ratio has many) gets no bit and no value.
 * The dense tensor the store stands for, and every weight gradient computed from it, are the
 * same; header->n_keep and the last block offset then give the number of STORED values, which is
 * at most the count surgeon_compact_sizes reports (size the buffers from that).  flags = 0 is
 * surgeon_prune_compact.  Unknown flag bits: INVALID_ARG.
 * ---------------------------------------------------------------------------------------- */
#define SURGEON_STORE_DROP_ZEROS 1u
/* Diagnostic without a counterpart in the paper, for testing the error path of the bounded
 * device-side waits: the select's grid-wide barrier is given an arrival target it cannot reach
 * and a cap of 1024 polls, so it gives up after some tens of microseconds.  Every kernel of the
 * call then returns without storing to bitmap, values or block_offsets, and
 * surgeon_header::status reads SURGEON_ERR_TIMEOUT; the other header fields are undefined.
 * Nothing faults and nothing spins past the cap. */
#define SURGEON_DEBUG_STALL_BARRIER 0x80000000u
surgeon_status surgeon_prune_compact_flags(const void* x, int64_t n, surgeon_dtype dt, double ratio,
                                           uint32_t flags, surgeon_compressed* out, void* workspace,
                                           size_t workspace_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * No counterpart in the paper: surgeon_prune_compact for callers that cannot allocate device
 * memory.  A hook that runs while the framework's allocator is locked or its pool is frozen, a
 * plug-in behind an interface that forbids cudaMalloc, or a process that gave away its whole
 * memory budget at start-up still owns x and the four output buffers of *out, but has no scratch
 * to pass as `workspace`.  This variant takes none: the scratch is a fixed array inside the
 * library (about 1.3 MB of global data on every GPU that loads the library, held until the
 * process exits), so neither the caller nor the library allocates or frees anything.
 * Same arguments, results, ordering on cuda_stream and error codes as surgeon_prune_compact,
 * except:
 *   - n may not exceed SURGEON_STATIC_MAX_N elements; a larger n returns
 *     SURGEON_ERR_UNSUPPORTED before anything is launched (use surgeon_prune_compact with your
 *     own workspace for such tensors);
 *   - the first call on each device looks up the array's device address (one host-side
 *     runtime query, with that device current) and keeps it for the life of the process: the
 *     one exception to "keeps no pointer after a call returns".  Make that first call outside
 *     any stream capture; later calls on the device do no set-up.  The kept address does not
 *     survive cudaDeviceReset (or any other teardown of the device's primary context): do not
 *     call this entry point on a device after resetting it;
 *   - all calls on one device share the one array.  Each call clears what it needs before use,
 *     so calls that follow each other on a stream, or are otherwise ordered, are independent;
 *     two calls whose kernels can run at the same time on one GPU (different streams without an
 *     event between them) race on the array and give undefined results.
 * ---------------------------------------------------------------------------------------- */
#define SURGEON_STATIC_MAX_N (1LL << 22)
surgeon_status surgeon_prune_compact_static(const void* x, int64_t n, surgeon_dtype dt,
                                            double ratio, surgeon_compressed* out,
                                            void* cuda_stream);

/* Layer geometry for the weight gradient.  Dilation 1. */
typedef struct surgeon_layer_desc {
  int32_t kind;  /* 0 = linear: activation [batch, c_in] (batch = rows T; h = w = kh = kw = 1,
                    stride = 1, pad = 0);  1 = conv2d: activation NCHW [batch, c_in, h, w]       */
  int32_t batch, c_in, h, w;
  int32_t c_out, kh, kw, stride, pad;
  int32_t path;  /* 0 = tensor-core path (bf16 x bf16 -> fp32, tcgen05/TMEM);
                    1 = fp32 CUDA-core path                                                      */
  int32_t groups; /* conv2d: channel groups (0 or 1 = an ordinary convolution).  groups > 1 (the
                    3x3 layers of ResNeXt, the network the paper adapts on CIFAR100-C in Section
                    5.1; groups = c_in = c_out is a depthwise convolution): c_in and c_out must
                    be multiples of it, output channel o reads only the c_in / groups input
                    channels of group o / (c_out / groups), and dw is [c_out, c_in / groups, kh,
                    kw].  A group's problem is far smaller than a tensor-core tile, so both
                    values of `path` run the same fp32 CUDA-core kernel for such a layer.       */
} surgeon_layer_desc;

/* Device scratch (bytes) surgeon_weight_grad needs for this layer and path; 0 on a bad desc. */
size_t surgeon_weight_grad_workspace(const surgeon_layer_desc* d);

/* ------------------------------------------------------------------------------------------
 * Algorithm 1: Reshape and gradient steps with Eq. 2 (weight gradient only): rebuild the sparse activation
 * from the store on chip and contract it with the output gradient.
 *   linear:  dw[o, c]       = sum_t        grad_out[t, o]       * A[t, c]
 *   conv2d:  dw[o, c, r, s] = sum_{b,y,x}  grad_out[b, o, y, x] * A[b, c, y*stride + r - pad,
 *                                                                   x*stride + s - pad]
 *            (terms outside the input are zero; oh = (h + 2*pad - kh)/stride + 1, same for ow;
 *            with groups > 1, c counts inside the group of o: input channel
 *            (o / (c_out/groups)) * (c_in/groups) + c)
 * where A is the pruned activation (zero where the bitmap bit is 0).  dw has the layout of a
 * PyTorch weight, [c_out, c_in, kh, kw], i.e. the transpose of Eq. 2's A^T * dL/dA_{i+1}.
 * act: HOST pointer to a struct of DEVICE pointers written by surgeon_prune_compact on the
 * same stream (or earlier); act->n must equal batch*c_in*h*w.  grad_out: device, fp32,
 * [batch, c_out, oh, ow] (conv2d) or [batch, c_out] (linear).  dw: device, fp32.
 * accumulate = 0 overwrites dw, 1 adds to it.  The summation order is fixed, so results are
 * bitwise reproducible from call to call.  Asynchronous on cuda_stream.
 * Errors: INVALID_ARG, BUFFER_TOO_SMALL, UNSUPPORTED (dilation is not expressible; sizes beyond
 * 2^31-1 elements; a grouped layer whose group has more than 1024 blocks of
 * (8 output channels) x (c_in/groups * kh * kw) weights), CUDA.
 * ---------------------------------------------------------------------------------------- */
surgeon_status surgeon_weight_grad(const surgeon_compressed* act, const surgeon_layer_desc* d,
                                   const float* grad_out, float* dw, int32_t accumulate,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Algorithm 1: Reshape step ("Reshape") as a stand-alone utility: x_out[j] = kept ? value : +0 for
 * all j < act->n, in act->dt.  x_out: device pointer to n elements.  surgeon_weight_grad does
 * not call this (it rebuilds tiles in shared memory); tests use it.  Asynchronous.
 * ---------------------------------------------------------------------------------------- */
surgeon_status surgeon_decompress(const surgeon_compressed* act, void* x_out, void* cuda_stream);

/* Static text for a status code. */
const char* surgeon_status_string(surgeon_status s);

/* Diagnostic without a counterpart in the paper: how many kernels this library has launched in
 * this process so far (all streams, all devices).  Benchmarks report the difference around a
 * timed region. */
uint64_t surgeon_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SURGEON_H_ */

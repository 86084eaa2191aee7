"""CPU oracle of the dynamic-activation-sparsity path (arXiv 2503.20354) — TEST INFRASTRUCTURE.

A thin numpy/ctypes front for ``surgeon_oracle.cpp`` (plain C++17, fp64).  Only the test-suite,
the repository's smoke check and the benchmark's CPU-baseline leg may import this package; the
CUDA library and its Python binding never do, and the oracle imports nothing of theirs.

Arrays cross as numpy: fp32 activations as ``float32``, bf16 activations as ``uint16`` bit
patterns (``dt=1``).  Section / equation numbers in the docstrings are the paper's.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "surgeon_oracle.cpp")
_LIB = os.path.join(_HERE, "libsurgeon_oracle.so")

BLOCK = 128  # elements per block-offset entry of the store that is compared with the library's
F32, BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2 -fopenmp) next to its source; returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-fopenmp", "-shared", "-fPIC", _SRC, "-o", tmp]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c = ctypes
        lib.oracle_layer_ratios.restype = c.c_int
        lib.oracle_layer_ratios.argtypes = [c.c_void_p, c.c_void_p, c.c_int, c.c_void_p]
        lib.oracle_gradient_importance.restype = c.c_double
        lib.oracle_gradient_importance.argtypes = [c.c_void_p, c.c_int64]
        lib.oracle_layer_ratios_rule.restype = c.c_int
        lib.oracle_layer_ratios_rule.argtypes = [c.c_void_p, c.c_void_p, c.c_int, c.c_int, c.c_double,
                                                 c.c_void_p]
        lib.oracle_n_keep.restype = c.c_int64
        lib.oracle_n_keep.argtypes = [c.c_int64, c.c_double]
        lib.oracle_select.restype = None
        lib.oracle_select.argtypes = [c.c_void_p, c.c_int64, c.c_int, c.c_int64, c.c_int,
                                      c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
        lib.oracle_compact.restype = c.c_int64
        lib.oracle_compact.argtypes = [c.c_void_p, c.c_int64, c.c_int, c.c_void_p, c.c_int64,
                                       c.c_void_p, c.c_void_p, c.c_void_p]
        lib.oracle_decompress.restype = None
        lib.oracle_decompress.argtypes = [c.c_void_p, c.c_void_p, c.c_int64, c.c_int, c.c_void_p]
        lib.oracle_dw_linear.restype = None
        lib.oracle_dw_linear.argtypes = [c.c_void_p, c.c_int, c.c_void_p] + [c.c_int64] * 3 + [
            c.c_void_p]
        lib.oracle_dw_conv2d.restype = None
        lib.oracle_dw_conv2d.argtypes = [c.c_void_p, c.c_int, c.c_void_p] + [c.c_int64] * 9 + [
            c.c_void_p]
        lib.oracle_dw_conv2d_grouped.restype = None
        lib.oracle_dw_conv2d_grouped.argtypes = [c.c_void_p, c.c_int, c.c_void_p] + [c.c_int64] * 10 + [
            c.c_void_p]
        lib.oracle_dw_conv2d_entry.restype = c.c_double
        lib.oracle_dw_conv2d_entry.argtypes = [c.c_void_p, c.c_int, c.c_void_p] + [c.c_int64] * 13
        lib.oracle_dw_linear_entry.restype = c.c_double
        lib.oracle_dw_linear_entry.argtypes = [c.c_void_p, c.c_int, c.c_void_p] + [c.c_int64] * 5
        lib.oracle_num_threads.restype = c.c_int
        lib.oracle_num_threads.argtypes = []
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _dt_of(x: np.ndarray) -> int:
    if x.dtype == np.float32:
        return F32
    if x.dtype == np.uint16:
        return BF16
    raise TypeError("activation must be float32 or uint16 (bf16 bit patterns), got %s" % x.dtype)


def num_threads() -> int:
    """Threads the OpenMP loops of the weight-gradient oracle use."""
    return int(_load().oracle_num_threads())


def layer_ratios(gi, lam):
    """Eq. 5-7: (status, p) with p the per-layer pruning ratios; status 3 = degenerate (0/0)."""
    g = np.ascontiguousarray(gi, dtype=np.float64)
    m = np.ascontiguousarray(lam, dtype=np.float64)
    assert g.ndim == 1 and g.shape == m.shape
    p = np.empty_like(g)
    st = _load().oracle_layer_ratios(_ptr(g), _ptr(m), int(g.size), _ptr(p))
    return int(st), p


RULE_BOTH, RULE_NO_GRADIENT, RULE_NO_MEMORY, RULE_STATIC = 0, 1, 2, 3


def layer_ratios_rule(gi, lam, rule: int, p_static: float = 0.0):
    """Eq. 5-7 with one factor of Eq. 6 left out ("w/o G", "w/o M") or a global static ratio."""
    g = np.ascontiguousarray(gi, dtype=np.float64)
    m = np.ascontiguousarray(lam, dtype=np.float64)
    assert g.ndim == 1 and g.shape == m.shape
    p = np.empty_like(g)
    st = _load().oracle_layer_ratios_rule(_ptr(g), _ptr(m), int(g.size), int(rule), float(p_static),
                                          _ptr(p))
    return int(st), p


def gradient_importance(dw) -> float:
    """Eq. 4: root mean square of a layer's weight-gradient entries (fp32 in, double out)."""
    w = np.ascontiguousarray(dw, dtype=np.float32).reshape(-1)
    return float(_load().oracle_gradient_importance(_ptr(w), int(w.size)))


def n_keep(n: int, ratio: float) -> int:
    """Algorithm 1: prune step: kept count for ``ratio`` = n - floor(ratio*n)."""
    return int(_load().oracle_n_keep(int(n), float(ratio)))


def select(x: np.ndarray, k: int, method: int = 1):
    """Algorithm 1: prune step: the k largest-magnitude elements, ties by lowest flat index.

    Returns (keep uint8[n], tau, c_gt, q).  method 0 = full stable sort, 1 = nth_element."""
    x = np.ascontiguousarray(x).reshape(-1)
    dt = _dt_of(x)
    keep = np.zeros(x.size, dtype=np.uint8)
    tau = ctypes.c_uint32(0)
    cgt = ctypes.c_int64(0)
    q = ctypes.c_int64(0)
    _load().oracle_select(_ptr(x), x.size, dt, int(k), int(method), _ptr(keep),
                          ctypes.byref(tau), ctypes.byref(cgt), ctypes.byref(q))
    return keep, int(tau.value), int(cgt.value), int(q.value)


def compact(x: np.ndarray, keep: np.ndarray, block: int = BLOCK):
    """Algorithm 1: decompose step: (bitmap uint32[ceil(n/32)], values[k], offsets uint64[ceil(n/block)+1])."""
    x = np.ascontiguousarray(x).reshape(-1)
    dt = _dt_of(x)
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    assert keep.size == x.size
    n = x.size
    bitmap = np.zeros((n + 31) // 32, dtype=np.uint32)
    values = np.zeros(int(keep.sum(dtype=np.int64)), dtype=x.dtype)
    offsets = np.zeros((n + block - 1) // block + 1, dtype=np.uint64)
    r = _load().oracle_compact(_ptr(x), n, dt, _ptr(keep), block, _ptr(bitmap), _ptr(values),
                               _ptr(offsets))
    assert r == values.size
    return bitmap, values, offsets


def decompress(bitmap: np.ndarray, values: np.ndarray, n: int) -> np.ndarray:
    """Algorithm 1: Reshape step: dense tensor (flat) from the store, +0 where the bit is clear."""
    bitmap = np.ascontiguousarray(bitmap, dtype=np.uint32)
    values = np.ascontiguousarray(values)
    dt = _dt_of(values)
    out = np.zeros(n, dtype=values.dtype)
    _load().oracle_decompress(_ptr(bitmap), _ptr(values), int(n), dt, _ptr(out))
    return out


def magnitude_keys(x: np.ndarray) -> np.ndarray:
    """The bit pattern of every element with the sign bit cleared (0 for +0 and -0)."""
    x = np.ascontiguousarray(x).reshape(-1)
    return (x.view(np.uint32) & np.uint32(0x7FFFFFFF)) if _dt_of(x) == 0 else \
        (x.view(np.uint16) & np.uint16(0x7FFF)).astype(np.uint32)


def prune_compact(x: np.ndarray, ratio: float, method: int = 1, block: int = BLOCK,
                  drop_zeros: bool = False):
    """Algorithm 1: prune and decompose steps in one call: dict with tau, k, c_gt, q, keep, bitmap, values, offsets.

    drop_zeros: the store variant that does not spend a value on a kept element that is exactly
    zero (Algorithm 1's decompose step caches "non-zero values"): the selection is the same, then
    the zeros among the kept elements are taken out again.  The dense tensor it stands for is
    unchanged, so is every weight gradient; k becomes the number of stored values."""
    x = np.ascontiguousarray(x).reshape(-1)
    k = n_keep(x.size, ratio)
    keep, tau, cgt, q = select(x, k, method)
    if drop_zeros:
        keep = keep.copy()
        keep[magnitude_keys(x) == 0] = 0
        k = int(keep.sum(dtype=np.int64))
        if tau == 0:
            q = 0
    bitmap, values, offsets = compact(x, keep, block)
    return dict(k=k, tau=tau, c_gt=cgt, q=q, keep=keep, bitmap=bitmap, values=values,
                offsets=offsets)


def dw_linear(a: np.ndarray, g: np.ndarray) -> np.ndarray:
    """Eq. 2 (weight layout): dw[o,c] = sum_t g[t,o] a[t,c]; a [T,C] (f32/bf16 bits), g [T,O] f32."""
    a = np.ascontiguousarray(a)
    g = np.ascontiguousarray(g, dtype=np.float32)
    T, C = a.shape
    O = g.shape[1]
    assert g.shape[0] == T
    dw = np.zeros((O, C), dtype=np.float64)
    _load().oracle_dw_linear(_ptr(a), _dt_of(a), _ptr(g), T, C, O, _ptr(dw))
    return dw


def conv_out_hw(h, w, kh, kw, stride, pad):
    return (h + 2 * pad - kh) // stride + 1, (w + 2 * pad - kw) // stride + 1


def dw_conv2d(a: np.ndarray, g: np.ndarray, kh: int, kw: int, stride: int, pad: int) -> np.ndarray:
    """Conv2d weight gradient, a NCHW [B,C,H,W], g [B,O,OH,OW] f32 -> dw [O,C,KH,KW] float64."""
    a = np.ascontiguousarray(a)
    g = np.ascontiguousarray(g, dtype=np.float32)
    B, C, H, W = a.shape
    O = g.shape[1]
    oh, ow = conv_out_hw(H, W, kh, kw, stride, pad)
    assert g.shape == (B, O, oh, ow), (g.shape, (B, O, oh, ow))
    dw = np.zeros((O, C, kh, kw), dtype=np.float64)
    _load().oracle_dw_conv2d(_ptr(a), _dt_of(a), _ptr(g), B, C, H, W, O, kh, kw, stride, pad,
                             _ptr(dw))
    return dw


def dw_conv2d_grouped(a: np.ndarray, g: np.ndarray, kh: int, kw: int, stride: int, pad: int,
                      groups: int) -> np.ndarray:
    """Weight gradient of a grouped conv2d (ResNeXt's 3x3 layers, depthwise convolutions):
    a NCHW [B,C,H,W], g [B,O,OH,OW] f32 -> dw [O,C/groups,KH,KW] float64."""
    a = np.ascontiguousarray(a)
    g = np.ascontiguousarray(g, dtype=np.float32)
    B, C, H, W = a.shape
    O = g.shape[1]
    assert groups >= 1 and C % groups == 0 and O % groups == 0, (C, O, groups)
    oh, ow = conv_out_hw(H, W, kh, kw, stride, pad)
    assert g.shape == (B, O, oh, ow), (g.shape, (B, O, oh, ow))
    dw = np.zeros((O, C // groups, kh, kw), dtype=np.float64)
    _load().oracle_dw_conv2d_grouped(_ptr(a), _dt_of(a), _ptr(g), B, C, H, W, O, kh, kw, stride,
                                     pad, groups, _ptr(dw))
    return dw


def dw_conv2d_entry(a, g, kh, kw, stride, pad, o, c, r, s) -> float:
    """One entry dw[o,c,r,s] of the conv2d weight gradient."""
    a = np.ascontiguousarray(a)
    g = np.ascontiguousarray(g, dtype=np.float32)
    B, C, H, W = a.shape
    O = g.shape[1]
    return float(_load().oracle_dw_conv2d_entry(_ptr(a), _dt_of(a), _ptr(g), B, C, H, W, O, kh,
                                                kw, stride, pad, o, c, r, s))


def dw_linear_entry(a, g, o, c) -> float:
    """One entry dw[o,c] of the linear weight gradient."""
    a = np.ascontiguousarray(a)
    g = np.ascontiguousarray(g, dtype=np.float32)
    T, C = a.shape
    O = g.shape[1]
    return float(_load().oracle_dw_linear_entry(_ptr(a), _dt_of(a), _ptr(g), T, C, O, o, c))

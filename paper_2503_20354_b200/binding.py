"""ctypes binding of libsurgeon.so: the same names as ``include/surgeon.h``.

Argument marshalling only — every step of the path runs in the library's CUDA kernels.  PyTorch
supplies device memory and the current stream.  There is no fallback: if the shared library is
missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# SURGEON_LIB names another build of the same library (the checked build libsurgeon_bounds.so)
LIB_PATH = os.environ.get("SURGEON_LIB") or os.path.join(_HERE, "libsurgeon.so")

SURGEON_OK = 0
SURGEON_ERR_INVALID_ARG = 1
SURGEON_ERR_BUFFER_TOO_SMALL = 2
SURGEON_ERR_DEGENERATE = 3
SURGEON_ERR_UNSUPPORTED = 4
SURGEON_ERR_CUDA = 5
SURGEON_ERR_TIMEOUT = 6
SURGEON_ERR_INTERNAL = 7
SURGEON_F32, SURGEON_BF16 = 0, 1
SURGEON_BLOCK = 128
PATH_TENSOR_CORE, PATH_FP32 = 0, 1


class SurgeonError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__("%s: %s (status %d)" % (where, status_string(status), status))


class Header(C.Structure):
    _fields_ = [("threshold_key", C.c_uint32), ("status", C.c_uint32), ("n_keep", C.c_int64),
                ("n_greater", C.c_int64), ("tie_quota", C.c_int64)]


class Compressed(C.Structure):
    _fields_ = [("n", C.c_int64), ("dt", C.c_int32), ("reserved", C.c_int32),
                ("bitmap", C.c_void_p), ("values", C.c_void_p), ("block_offsets", C.c_void_p),
                ("header", C.c_void_p)]


class LayerDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("kind", "batch", "c_in", "h", "w", "c_out", "kh", "kw",
                                         "stride", "pad", "path", "groups")]


_lib = None


def lib():
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libsurgeon.so is missing at %s: build it with "
                "`python -m paper_2503_20354_b200.build` (there is no CPU fallback)" % LIB_PATH)
        l = C.CDLL(LIB_PATH)
        l.surgeon_layer_ratios.restype = C.c_int
        l.surgeon_layer_ratios.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
        l.surgeon_layer_ratios_rule.restype = C.c_int
        l.surgeon_layer_ratios_rule.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int, C.c_double,
                                                C.c_void_p]
        l.surgeon_gradient_importance.restype = C.c_int
        l.surgeon_gradient_importance.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p,
                                                  C.c_size_t, C.c_void_p]
        l.surgeon_compact_sizes.restype = C.c_int
        l.surgeon_compact_sizes.argtypes = [C.c_int64, C.c_int, C.c_double, C.c_void_p, C.c_void_p,
                                            C.c_void_p, C.c_void_p, C.c_void_p]
        l.surgeon_prune_compact.restype = C.c_int
        l.surgeon_prune_compact.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_double,
                                            C.POINTER(Compressed), C.c_void_p, C.c_size_t, C.c_void_p]
        l.surgeon_prune_compact_flags.restype = C.c_int
        l.surgeon_prune_compact_flags.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_double, C.c_uint32,
                                                  C.POINTER(Compressed), C.c_void_p, C.c_size_t, C.c_void_p]
        l.surgeon_prune_compact_static.restype = C.c_int
        l.surgeon_prune_compact_static.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_double,
                                                   C.POINTER(Compressed), C.c_void_p]
        l.surgeon_weight_grad_workspace.restype = C.c_size_t
        l.surgeon_weight_grad_workspace.argtypes = [C.POINTER(LayerDesc)]
        l.surgeon_weight_grad.restype = C.c_int
        l.surgeon_weight_grad.argtypes = [C.POINTER(Compressed), C.POINTER(LayerDesc), C.c_void_p,
                                          C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t, C.c_void_p]
        l.surgeon_decompress.restype = C.c_int
        l.surgeon_decompress.argtypes = [C.POINTER(Compressed), C.c_void_p, C.c_void_p]
        l.surgeon_launch_count.restype = C.c_uint64
        l.surgeon_launch_count.argtypes = []
        l.surgeon_status_string.restype = C.c_char_p
        l.surgeon_status_string.argtypes = [C.c_int]
        _lib = l
    return _lib


def status_string(status: int) -> str:
    return lib().surgeon_status_string(int(status)).decode()


def surgeon_launch_count() -> int:
    """Kernels launched by the library in this process so far."""
    return int(lib().surgeon_launch_count())


def _check(status: int, where: str, allow=()):
    if status != SURGEON_OK and status not in allow:
        raise SurgeonError(status, where)
    return status


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _scratch(nbytes: int, device, stream: Optional[torch.cuda.Stream]) -> torch.Tensor:
    """A scratch tensor made here (the caller passed none).  It is dropped when the call returns,
    while the kernels that use it are still queued on ``stream``: the allocator is told, so that
    the block is not handed out again before they are done."""
    t = torch.empty(max(int(nbytes), 16), dtype=torch.uint8, device=device)
    if stream is not None:
        t.record_stream(stream)
    return t


def dtype_code(t: torch.dtype) -> int:
    if t == torch.float32:
        return SURGEON_F32
    if t == torch.bfloat16:
        return SURGEON_BF16
    raise TypeError("activation dtype must be float32 or bfloat16, got %s" % t)


# ---------------------------------------------------------------------------------------------
# surgeon_layer_ratios (Eq. 5-7) and surgeon_compact_sizes (Algorithm 1: prune step): host arithmetic
# ---------------------------------------------------------------------------------------------

def surgeon_layer_ratios(gi, lam, allow_degenerate: bool = False) -> np.ndarray:
    """Per-layer pruning ratios from Gradient Importance ``gi`` and activation sizes ``lam``."""
    g = np.ascontiguousarray(gi, dtype=np.float64)
    m = np.ascontiguousarray(lam, dtype=np.float64)
    if g.ndim != 1 or g.shape != m.shape:
        raise ValueError("gi and lam must be 1-D and of equal length")
    out = np.empty_like(g)
    st = lib().surgeon_layer_ratios(g.ctypes.data, m.ctypes.data, int(g.size), out.ctypes.data)
    _check(st, "surgeon_layer_ratios", allow=(SURGEON_ERR_DEGENERATE,) if allow_degenerate else ())
    return out


SURGEON_RULE_BOTH, SURGEON_RULE_NO_GRADIENT, SURGEON_RULE_NO_MEMORY, SURGEON_RULE_STATIC = 0, 1, 2, 3
SURGEON_GI_WORKSPACE_BYTES = 8192


def surgeon_layer_ratios_rule(gi, lam, rule: int, static_ratio: float = 0.0,
                              allow_degenerate: bool = False) -> np.ndarray:
    """The ratio rule with one factor left out ("w/o G", "w/o M") or a global static ratio."""
    g = None if gi is None else np.ascontiguousarray(gi, dtype=np.float64)
    m = None if lam is None else np.ascontiguousarray(lam, dtype=np.float64)
    ref = g if g is not None else m
    if ref is None or ref.ndim != 1 or (g is not None and m is not None and g.shape != m.shape):
        raise ValueError("gi and lam must be 1-D and of equal length (one of them may be None)")
    out = np.empty(ref.shape, dtype=np.float64)
    st = lib().surgeon_layer_ratios_rule(None if g is None else g.ctypes.data,
                                         None if m is None else m.ctypes.data, int(ref.size),
                                         int(rule), float(static_ratio), out.ctypes.data)
    _check(st, "surgeon_layer_ratios_rule",
           allow=(SURGEON_ERR_DEGENERATE,) if allow_degenerate else ())
    return out


def surgeon_gradient_importance(dw: torch.Tensor, out: Optional[torch.Tensor] = None,
                                workspace: Optional[torch.Tensor] = None,
                                stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Eq. 4 on the device: a one-element float64 tensor holding sqrt(mean(dw^2))."""
    if not dw.is_cuda or not dw.is_contiguous() or dw.dtype != torch.float32:
        raise ValueError("dw must be a contiguous fp32 CUDA tensor")
    if out is None:
        out = torch.empty(1, dtype=torch.float64, device=dw.device)
    if workspace is None:
        workspace = _scratch(SURGEON_GI_WORKSPACE_BYTES, dw.device, stream)
    st = lib().surgeon_gradient_importance(dw.data_ptr() if dw.numel() else None, dw.numel(),
                                           out.data_ptr(), workspace.data_ptr(),
                                           workspace.numel() * workspace.element_size(),
                                           _stream_ptr(stream))
    _check(st, "surgeon_gradient_importance")
    return out


@dataclass
class CompactSizes:
    n_keep: int
    bitmap_bytes: int
    values_bytes: int
    offsets_bytes: int
    workspace_bytes: int


def surgeon_compact_sizes(n: int, dt: int, ratio: float) -> CompactSizes:
    k = C.c_int64(0)
    b, v, o, w = C.c_size_t(0), C.c_size_t(0), C.c_size_t(0), C.c_size_t(0)
    st = lib().surgeon_compact_sizes(int(n), int(dt), float(ratio), C.byref(k), C.byref(b),
                                     C.byref(v), C.byref(o), C.byref(w))
    _check(st, "surgeon_compact_sizes")
    return CompactSizes(k.value, b.value, v.value, o.value, w.value)


# ---------------------------------------------------------------------------------------------
# The compressed store and surgeon_prune_compact (Algorithm 1: prune and decompose steps)
# ---------------------------------------------------------------------------------------------

class CompressedActivation:
    """Device buffers of one compressed activation plus the C struct that points at them."""

    def __init__(self, n: int, dt: int, ratio: float, device, sizes: Optional[CompactSizes] = None):
        s = sizes or surgeon_compact_sizes(n, dt, ratio)
        self.n, self.dt, self.ratio, self.sizes = int(n), int(dt), float(ratio), s
        self.bitmap = torch.empty(max(s.bitmap_bytes // 4, 1), dtype=torch.int32, device=device)
        vt = torch.float32 if dt == SURGEON_F32 else torch.bfloat16
        self.values = torch.empty(max(s.n_keep, 1), dtype=vt, device=device)
        self.block_offsets = torch.empty(s.offsets_bytes // 4, dtype=torch.int32, device=device)
        self.header = torch.zeros(4, dtype=torch.int64, device=device)
        self.c = Compressed(self.n, self.dt, 0, self.bitmap.data_ptr(), self.values.data_ptr(),
                            self.block_offsets.data_ptr(), self.header.data_ptr())

    @property
    def n_keep(self) -> int:
        return self.sizes.n_keep

    @property
    def stored_bytes(self) -> int:
        """Bytes of the cached form: packed values + 1 bit per element + block offsets."""
        return self.sizes.values_bytes + self.sizes.bitmap_bytes + self.sizes.offsets_bytes

    def read_header(self) -> Header:
        """Synchronising device->host read of the 32-byte result header."""
        raw = self.header.cpu().numpy().tobytes()
        return Header.from_buffer_copy(raw)

    def to_numpy(self):
        """Host copies for comparison: (bitmap uint32, values, offsets uint32, Header)."""
        nw = (self.n + 31) // 32
        bitmap = self.bitmap[:nw].cpu().numpy().view(np.uint32)
        hdr = self.read_header()
        vals = self.values[: int(hdr.n_keep)].cpu()    # the stored count (= n_keep unless zeros are dropped)
        vals = vals.view(torch.int16).numpy().view(np.uint16) if self.dt == SURGEON_BF16 else vals.numpy()
        offs = self.block_offsets[: self.sizes.offsets_bytes // 4].cpu().numpy().view(np.uint32)
        return bitmap, vals, offs, hdr


SURGEON_STORE_DROP_ZEROS = 1
SURGEON_DEBUG_STALL_BARRIER = 0x80000000


def surgeon_prune_compact(x: torch.Tensor, ratio: float, out: Optional[CompressedActivation] = None,
                          workspace: Optional[torch.Tensor] = None,
                          stream: Optional[torch.cuda.Stream] = None,
                          flags: int = 0) -> CompressedActivation:
    """Prune ``x`` (CUDA tensor, fp32 or bf16, contiguous) at ``ratio`` into a compressed store.
    ``flags=SURGEON_STORE_DROP_ZEROS``: kept zeros get no bit and no value (the header's n_keep
    is then the stored count; ``out.sizes.n_keep`` stays the upper bound the buffers are sized for)."""
    if not x.is_cuda or not x.is_contiguous():
        raise ValueError("x must be a contiguous CUDA tensor")
    dt = dtype_code(x.dtype)
    n = x.numel()
    sizes = surgeon_compact_sizes(n, dt, ratio)
    if out is None:
        out = CompressedActivation(n, dt, ratio, x.device, sizes)
    else:
        if out.n != n or out.dt != dt or out.values.numel() < sizes.n_keep:
            raise ValueError("output store does not fit this tensor / ratio")
        out.ratio, out.sizes = float(ratio), sizes
    if workspace is None:
        workspace = _scratch(sizes.workspace_bytes, x.device, stream)
    st = lib().surgeon_prune_compact_flags(x.data_ptr(), n, dt, float(ratio), int(flags), C.byref(out.c),
                                           workspace.data_ptr(),
                                           workspace.numel() * workspace.element_size(),
                                           _stream_ptr(stream))
    _check(st, "surgeon_prune_compact")
    return out


SURGEON_STATIC_MAX_N = 1 << 22


def surgeon_prune_compact_static(x: torch.Tensor, ratio: float, out: CompressedActivation,
                                 stream: Optional[torch.cuda.Stream] = None) -> CompressedActivation:
    """``surgeon_prune_compact`` without a workspace, for callers that must not allocate device
    memory (a hook running while the allocator is locked, a frozen memory pool): the scratch is
    a fixed array inside the library.  ``out`` must already exist and be large enough for this
    ratio (build it once with ``CompressedActivation(n, dt, 0.0, device)``); this function
    creates no tensor.  Tensors of more than ``SURGEON_STATIC_MAX_N`` elements are refused.
    Calls on one GPU share the scratch, so they must not overlap in time."""
    if not x.is_cuda or not x.is_contiguous():
        raise ValueError("x must be a contiguous CUDA tensor")
    dt = dtype_code(x.dtype)
    n = x.numel()
    if n > SURGEON_STATIC_MAX_N:
        raise SurgeonError(SURGEON_ERR_UNSUPPORTED, "surgeon_prune_compact_static: %d elements "
                           "exceed the built-in scratch (limit %d)" % (n, SURGEON_STATIC_MAX_N))
    sizes = surgeon_compact_sizes(n, dt, ratio)
    if out.n != n or out.dt != dt or out.values.numel() < sizes.n_keep:
        raise ValueError("output store does not fit this tensor / ratio")
    out.ratio, out.sizes = float(ratio), sizes
    st = lib().surgeon_prune_compact_static(x.data_ptr(), n, dt, float(ratio), C.byref(out.c),
                                            _stream_ptr(stream))
    _check(st, "surgeon_prune_compact_static")
    return out


def surgeon_decompress(act: CompressedActivation, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Dense flat tensor rebuilt from the store (test utility; Algorithm 1: Reshape step)."""
    vt = torch.float32 if act.dt == SURGEON_F32 else torch.bfloat16
    out = torch.empty(max(act.n, 1), dtype=vt, device=act.bitmap.device)
    if stream is not None:
        out.record_stream(stream)
    st = lib().surgeon_decompress(C.byref(act.c), out.data_ptr(), _stream_ptr(stream))
    _check(st, "surgeon_decompress")
    return out[: act.n]


# ---------------------------------------------------------------------------------------------
# surgeon_weight_grad (Algorithm 1: Reshape and gradient steps, Eq. 2)
# ---------------------------------------------------------------------------------------------

def layer_desc(layer, path: int) -> LayerDesc:
    """LayerDesc from any object with kind/batch/c_in/h/w/c_out/kh/kw/stride/pad attributes."""
    return LayerDesc(layer.kind, layer.batch, layer.c_in, layer.h, layer.w, layer.c_out, layer.kh,
                     layer.kw, layer.stride, layer.pad, int(path), int(getattr(layer, "groups", 1)))


def surgeon_weight_grad_workspace(desc: LayerDesc) -> int:
    return int(lib().surgeon_weight_grad_workspace(C.byref(desc)))


def surgeon_weight_grad(act: CompressedActivation, desc: LayerDesc, grad_out: torch.Tensor,
                        dw: Optional[torch.Tensor] = None, accumulate: bool = False,
                        workspace: Optional[torch.Tensor] = None,
                        stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """dW of the layer from the compressed activation and fp32 ``grad_out``; returns ``dw``."""
    if grad_out.dtype != torch.float32 or not grad_out.is_cuda or not grad_out.is_contiguous():
        raise ValueError("grad_out must be a contiguous fp32 CUDA tensor")
    shape = (desc.c_out, desc.c_in // max(desc.groups, 1), desc.kh, desc.kw) if desc.kind == 1 else (desc.c_out, desc.c_in)
    if dw is None:
        if accumulate:
            raise ValueError("accumulate needs an existing dw")
        dw = torch.empty(shape, dtype=torch.float32, device=grad_out.device)
    need = surgeon_weight_grad_workspace(desc)
    if workspace is None:
        workspace = _scratch(need, grad_out.device, stream)
    st = lib().surgeon_weight_grad(C.byref(act.c), C.byref(desc), grad_out.data_ptr(), dw.data_ptr(),
                                   1 if accumulate else 0, workspace.data_ptr(),
                                   workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    _check(st, "surgeon_weight_grad")
    return dw

"""Helpers shared by the GPU parity tests (not a test module)."""
import numpy as np
import torch

import oracle
from paper_2503_20354_b200 import binding as B
from paper_2503_20354_b200 import workloads as W


def assert_store_equals_oracle(x_cpu: torch.Tensor, ratio: float, comp=None, method: int = 1,
                               drop_zeros: bool = False):
    """Run surgeon_prune_compact on the GPU copy of x_cpu and compare every output bit-exactly
    with the oracle: threshold key, kept count, tie quota, bitmap, packed values, block offsets."""
    xb = W.as_numpy_bits(x_cpu).reshape(-1)
    ref = oracle.prune_compact(xb, ratio, method=method, drop_zeros=drop_zeros)
    if comp is None:
        comp = B.surgeon_prune_compact(x_cpu.cuda().contiguous(), ratio,
                                       flags=B.SURGEON_STORE_DROP_ZEROS if drop_zeros else 0)
    torch.cuda.synchronize()
    bitmap, vals, offs, hdr = comp.to_numpy()
    assert hdr.status == B.SURGEON_OK, B.status_string(hdr.status)
    assert hdr.n_keep == ref["k"] and (drop_zeros or hdr.n_keep == comp.n_keep)
    assert hdr.threshold_key == ref["tau"], (hex(hdr.threshold_key), hex(ref["tau"]))
    assert hdr.n_greater == ref["c_gt"] and hdr.tie_quota == ref["q"]
    assert np.array_equal(bitmap, ref["bitmap"])
    assert np.array_equal(vals.view(np.uint8), ref["values"].view(np.uint8))
    assert np.array_equal(offs, ref["offsets"])
    return comp, ref


def rel_frobenius(got: np.ndarray, ref: np.ndarray) -> float:
    got = np.asarray(got, dtype=np.float64)
    den = float(np.linalg.norm(ref))
    num = float(np.linalg.norm(got - ref))
    if den == 0.0:
        return 0.0 if num == 0.0 else float("inf")
    return num / den


def oracle_dw(layer, a_bits: np.ndarray, g: np.ndarray) -> np.ndarray:
    if layer.kind == 1:
        return oracle.dw_conv2d(a_bits.reshape(layer.act_shape), g, layer.kh, layer.kw,
                                layer.stride, layer.pad)
    return oracle.dw_linear(a_bits.reshape(layer.act_shape), g)

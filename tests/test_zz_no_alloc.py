"""GPU check of surgeon_prune_compact_static, the variant of surgeon_prune_compact for callers
that cannot allocate device memory (their scratch is an array built into the library).

The file name sorts last on purpose: a run that stops at the first failure has then already gone
through every other test.  Each test calls the no-workspace entry point twice in a row through the
C ABI, on different inputs, and requires every output of each call (header, bitmap, packed values,
block offsets) to equal, bit for bit, what the ordinary entry point with a caller-owned workspace
produces for the same input.  The second call reuses the scratch the first one dirtied, which is
what the comparison is there to catch."""
import ctypes as C

import numpy as np
import oracle
import pytest
import torch

from paper_2503_20354_b200 import binding as B
from paper_2503_20354_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _same_store(a, b):
    for u, v in zip(a.to_numpy()[:3], b.to_numpy()[:3]):
        assert np.array_equal(u.view(np.uint8), v.view(np.uint8))
    ha, hb = a.read_header(), b.read_header()
    assert ha.status == hb.status == B.SURGEON_OK
    assert (ha.threshold_key, ha.n_keep, ha.n_greater, ha.tie_quota) == \
           (hb.threshold_key, hb.n_keep, hb.n_greater, hb.tie_quota)


@pytest.mark.parametrize("bf16", [False, True])
def test_two_calls_in_a_row_match_the_workspace_entry_point(bf16):
    cases = [("relu_normal", (1 << 20) + 777, 0.6), ("ties16", 300_001, 0.35)]
    # outputs exist before the calls under test; those calls create nothing on the device
    outs = []
    for dist, n, ratio in cases:
        x = W.draw(dist, n, seed=11, tag=n)
        x = (x.to(torch.bfloat16) if bf16 else x).cuda()
        outs.append((x, ratio, B.CompressedActivation(n, B.dtype_code(x.dtype), 0.0, x.device)))
    torch.cuda.synchronize()
    allocations = lambda: torch.cuda.memory_stats()["allocation.all.allocated"]  # event count
    before = allocations()
    for x, ratio, out in outs:                       # two calls in a row, same scratch
        B.surgeon_prune_compact_static(x, ratio, out)
    assert allocations() == before                   # the binding allocated nothing either
    torch.cuda.synchronize()
    for x, ratio, out in outs:
        _same_store(out, B.surgeon_prune_compact(x, ratio))


@pytest.mark.parametrize("bf16", [False, True])
def test_largest_size_against_the_oracle_too(bf16):
    """n = SURGEON_STATIC_MAX_N exactly (the scratch is laid out for this size; both dtypes take
    the streamed select here), twice in a row, against the ordinary entry point and the oracle."""
    n = B.SURGEON_STATIC_MAX_N
    x = W.draw("relu_normal", n, seed=12)
    x = x.to(torch.bfloat16) if bf16 else x
    xd = x.cuda()
    out = B.CompressedActivation(n, B.dtype_code(xd.dtype), 0.0, xd.device)
    for ratio in (0.8, 0.25):
        B.surgeon_prune_compact_static(xd, ratio, out)
        _same_store(out, B.surgeon_prune_compact(xd, ratio))
        ref = oracle.prune_compact(W.as_numpy_bits(x).reshape(-1), ratio)
        bitmap, vals, offs, hdr = out.to_numpy()
        assert hdr.threshold_key == ref["tau"] and hdr.n_keep == ref["k"]
        assert np.array_equal(bitmap, ref["bitmap"]) and np.array_equal(offs, ref["offsets"])
        assert np.array_equal(vals.view(np.uint8), ref["values"].view(np.uint8))


def test_same_input_twice_and_size_limit():
    n = 123_457
    x = W.draw("normal", n, seed=5).cuda()
    out = B.CompressedActivation(n, B.SURGEON_F32, 0.0, x.device)
    ref = B.surgeon_prune_compact(x, 0.9)
    for _ in range(2):
        B.surgeon_prune_compact_static(x, 0.9, out)
        _same_store(out, ref)
    # beyond the built-in scratch: refused on the host, nothing launched
    st = B.lib().surgeon_prune_compact_static(x.data_ptr(), B.SURGEON_STATIC_MAX_N + 1,
                                              B.SURGEON_F32, 0.5, C.byref(out.c), None)
    assert st == B.SURGEON_ERR_UNSUPPORTED
    with pytest.raises(B.SurgeonError):
        big = torch.empty(B.SURGEON_STATIC_MAX_N + 1, dtype=torch.bfloat16, device="cuda")
        B.surgeon_prune_compact_static(big, 0.5, out)

"""GPU parity: surgeon_gradient_importance (Eq. 4) through the C ABI vs the fp64 oracle.

Both sides square and add in double; only the order of the additions differs, so the tolerance
is a relative 1e-12.  The summation order on the device is fixed: repeated calls agree bitwise."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_20354_b200 import binding as B
from paper_2503_20354_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n", [1, 2, 255, 256, 257, 4095, 4096, 4097, 1000003, 4096 * 1024 + 5,
                               640 * 640 * 9])
def test_matches_oracle(n):
    g = torch.Generator().manual_seed(n)
    dw = torch.randn(n, generator=g, dtype=torch.float32) * 1e-3
    got = B.surgeon_gradient_importance(dw.cuda())
    again = B.surgeon_gradient_importance(dw.cuda())
    torch.cuda.synchronize()
    ref = oracle.gradient_importance(dw.numpy())
    assert abs(got.item() - ref) <= 1e-12 * ref
    assert got.item() == again.item()                  # fixed summation order


def test_empty_constant_and_scratch_reuse():
    ws = torch.empty(B.SURGEON_GI_WORKSPACE_BYTES, dtype=torch.uint8, device="cuda")
    out = torch.full((1,), -1.0, dtype=torch.float64, device="cuda")
    B.surgeon_gradient_importance(torch.empty(0, dtype=torch.float32, device="cuda"), out=out, workspace=ws)
    assert out.item() == 0.0
    B.surgeon_gradient_importance(torch.full((70001,), -2.5, device="cuda"), out=out, workspace=ws)
    assert out.item() == 2.5                           # a constant vector gives its magnitude
    B.surgeon_gradient_importance(torch.ones(3, device="cuda"), out=out, workspace=ws)
    assert out.item() == 1.0                           # stale partials of the larger call are not read


def test_of_a_weight_gradient_feeds_the_ratio_rule():
    """dW of two layers -> G_i on the device -> Eq. 5-7: the loop of Algorithm 1 without a dense pass."""
    layers = [W.conv("gi_a", 2, 16, 16, 32, 3), W.conv("gi_b", 2, 32, 8, 32, 3)]
    gis, refs = [], []
    for i, l in enumerate(layers):
        a = W.activation(l, 11 + i).cuda()
        g = W.grad_out(l, 11 + i).cuda()
        comp = B.surgeon_prune_compact(a, 0.9)            # the importance pass runs at a high static ratio
        dw = B.surgeon_weight_grad(comp, B.layer_desc(l, B.PATH_FP32), g)
        gis.append(B.surgeon_gradient_importance(dw).item())
        refs.append(oracle.gradient_importance(dw.cpu().numpy()))
    np.testing.assert_allclose(gis, refs, rtol=1e-12, atol=0)
    lam = [l.act_bytes for l in layers]
    _, p_ref = oracle.layer_ratios(refs, lam)
    np.testing.assert_allclose(B.surgeon_layer_ratios(gis, lam), p_ref, rtol=0, atol=1e-12)


def test_argument_errors():
    dw = torch.ones(8, device="cuda")
    with pytest.raises(B.SurgeonError) as e:
        B.surgeon_gradient_importance(dw, workspace=torch.empty(64, dtype=torch.uint8, device="cuda"))
    assert e.value.status == B.SURGEON_ERR_BUFFER_TOO_SMALL
    with pytest.raises(ValueError):
        B.surgeon_gradient_importance(dw.double())

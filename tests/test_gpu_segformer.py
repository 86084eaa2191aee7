"""GPU parity on Segformer-B5-shaped linear layers (Section 5.1: the segmentation model, batch 1):
widths 64 / 128 / 320 / 512, MLP ratio 4, keys and values on a reduced token grid.  One block per
stage on a 256x256 image (4096 / 1024 / 256 / 64 tokens), ratios from Eq. 5-7 over the stack:
stores bit for bit, weight gradients within the path's tolerance of the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_20354_b200 import binding as B
from paper_2503_20354_b200 import workloads as W
from gpu_util import assert_store_equals_oracle, oracle_dw, rel_frobenius

pytestmark = pytest.mark.gpu

TOL = {B.PATH_FP32: 1e-5, B.PATH_TENSOR_CORE: 5e-3}
LAYERS = W.segformer_b5(image=256, depths=(1, 1, 1, 1))


def _ratios():
    gi = W.gradient_importance(len(LAYERS), seed=3)
    lam = np.array([l.act_bytes for l in LAYERS], dtype=np.float64)
    return B.surgeon_layer_ratios(gi, lam)


def test_stack_shape():
    full = W.segformer_b5()
    assert len(full) == 5 * (3 + 6 + 40 + 3)
    assert [l.batch for l in full[:5]] == [65536, 1024, 65536, 65536, 65536]
    assert (full[-1].c_in, full[-1].c_out, full[-1].batch) == (2048, 512, 1024)
    assert len(LAYERS) == 20 and LAYERS[1].batch == 64      # a 64 x 64 token grid reduced 8 times per side


@pytest.mark.parametrize("path", [B.PATH_TENSOR_CORE, B.PATH_FP32])
@pytest.mark.parametrize("li", range(len(LAYERS)))
def test_layer_store_and_weight_gradient(li, path):
    layer = LAYERS[li]
    ratio = float(_ratios()[li])
    a = W.activation(layer, 5, li)
    g = W.grad_out(layer, 5, li)
    comp, ref = assert_store_equals_oracle(a, ratio)
    dw = B.surgeon_weight_grad(comp, B.layer_desc(layer, path), g.cuda())
    torch.cuda.synchronize()
    pruned = oracle.decompress(ref["bitmap"], ref["values"], layer.n_act)
    want = oracle_dw(layer, pruned, g.numpy())
    assert dw.shape == (layer.c_out, layer.c_in)
    if not want.any():
        assert not dw.cpu().numpy().any()
    else:
        assert rel_frobenius(dw.cpu().numpy(), want) <= TOL[path]

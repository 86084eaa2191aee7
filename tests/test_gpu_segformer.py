"""GPU parity on the layers of Segformer-B5-shaped blocks (Section 5.1: the segmentation model, batch
1): widths 64 / 128 / 320 / 512, MLP ratio 4, keys and values on a token grid reduced by a strided
convolution, a depthwise 3x3 convolution inside the MLP.  One block per stage on a 256x256 image
(4096 / 1024 / 256 / 64 tokens), ratios from Eq. 5-7 over the stack: stores bit for bit, weight
gradients within the path's tolerance of the fp64 oracle (the depthwise layers run the fp32
grouped kernel on both paths)."""
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
    lin = W.segformer_b5(convs=False)
    assert len(lin) == 5 * (3 + 6 + 40 + 3)
    assert [l.batch for l in lin[:5]] == [65536, 1024, 65536, 65536, 65536]
    assert (lin[-1].c_in, lin[-1].c_out, lin[-1].batch) == (2048, 512, 1024)
    full = W.segformer_b5()
    assert len(full) == len(lin) + (3 + 6 + 40) + (3 + 6 + 40 + 3)      # reductions in stages 1-3, a depthwise conv per block
    sr, dwc = full[1], full[5]
    assert (sr.name, sr.kh, sr.stride, sr.pad, sr.h, sr.c_in, sr.c_out) == ("s0b0.sr", 8, 8, 0, 256, 64, 64)
    assert (dwc.name, dwc.groups, dwc.c_in, dwc.kh, dwc.h) == ("s0b0.dwconv", 256, 256, 3, 256)
    assert len(LAYERS) == 20 + 3 + 4 and LAYERS[2].batch == 64      # a 64 x 64 token grid reduced 8 times per side


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
    if layer.groups > 1:
        want = oracle.dw_conv2d_grouped(pruned.reshape(layer.act_shape), g.numpy(), layer.kh, layer.kw,
                                        layer.stride, layer.pad, layer.groups)
    else:
        want = oracle_dw(layer, pruned, g.numpy())
    assert tuple(dw.shape) == tuple(layer.dw_shape)
    tol = 1e-5 if layer.groups > 1 else TOL[path]
    if not want.any():
        assert not dw.cpu().numpy().any()
    else:
        assert rel_frobenius(dw.cpu().numpy(), want) <= tol

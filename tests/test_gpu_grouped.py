"""GPU parity: the weight gradient of grouped convolutions (ResNeXt's 3x3 layers, depthwise
convolutions) through the C ABI vs the fp64 oracle.  A group's problem is too small for a
tensor-core tile, so both values of `path` run the fp32 CUDA-core kernel: tolerance 1e-5 for both."""
from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
from paper_2503_20354_b200 import binding as B
from paper_2503_20354_b200 import workloads as W
from gpu_util import rel_frobenius

pytestmark = pytest.mark.gpu

SHAPES = [
    W.conv("x3x3_g8", 3, 32, 16, 32, 3, groups=8),                  # ResNeXt-like: 4 -> 4 channels per group
    W.conv("x3x3_g8_s2", 2, 64, 16, 64, 3, 2, groups=8),            # stride 2, 8 channels per group
    W.conv("x3x3_g4_c16", 2, 64, 8, 64, 3, groups=4),               # 16 channels per group: 144 columns, 2 blocks
    W.conv("depthwise3x3", 2, 24, 14, 24, 3, groups=24),            # one channel per group
    W.conv("depthwise3x3_s2_odd", 3, 10, 15, 10, 3, 2, groups=10),
    W.conv("g2_og20", 2, 12, 9, 40, 3, groups=2),                   # 20 output channels per group: a ragged block of 8
    W.conv("g3_1x1", 4, 18, 7, 12, 1, 1, 0, groups=3),
    W.conv("depthwise5x5_w40", 1, 6, 40, 6, 5, 1, 2, groups=6),
    W.conv("tall_map_bands", 1, 4, 200, 4, 3, groups=2),            # a map too tall for one band of shared memory
    # the register-tiled 3x3 kernel (output rows a multiple of 8 wide): every tile shape, both strides,
    # batches that do not divide into rounds, rows of 8, 16, 32, 40 and 64
    W.conv("t22_w32", 5, 16, 32, 16, 3, groups=4),                  # 4 -> 4 per group: 2 x 2 tiles
    W.conv("t41_w16", 3, 6, 16, 24, 3, groups=6),                   # 1 -> 4 per group
    W.conv("t14_w8", 7, 16, 8, 4, 3, groups=4),                     # 4 -> 1 per group
    W.conv("t21_t12_w40", 2, 6, 40, 6, 3, groups=3),                # 2 -> 2: 2 x 2; rows wider than a warp
    W.conv("t12_w24", 2, 4, 24, 6, 3, groups=2),                    # 2 -> 3 per group: 1 x 2 tiles
    W.conv("t21_w8_s2", 3, 9, 16, 6, 3, 2, groups=3),               # 3 -> 2 per group, stride 2: 2 x 1 tiles
    W.conv("depthwise_w64_s2", 2, 5, 128, 5, 3, 2, groups=5),       # 1 x 1 tiles, two column chunks per row
    W.conv("depthwise_w16", 9, 12, 16, 12, 3, groups=12),
    W.conv("t22_s2_w16", 3, 32, 32, 32, 3, 2, groups=4),            # 8 -> 8 per group, stride 2
    replace(W.conv("t22_tall_bands", 1, 8, 64, 8, 3, groups=2), h=240),   # several bands of output rows
]


@pytest.mark.parametrize("path", [B.PATH_FP32, B.PATH_TENSOR_CORE])
@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("layer", SHAPES, ids=lambda l: l.name)
def test_grouped_layer_shapes(layer, bf16, path):
    layer = replace(layer, dt=W.BF16 if bf16 else W.F32)
    a = W.activation(layer, seed=6)
    g = W.grad_out(layer, seed=6)
    a_bits = W.as_numpy_bits(a).reshape(-1)
    for ratio in (0.0, 0.7, 1.0):
        comp = B.surgeon_prune_compact(a.cuda(), ratio)
        dw = B.surgeon_weight_grad(comp, B.layer_desc(layer, path), g.cuda()).cpu().numpy()
        assert dw.shape == layer.dw_shape
        r = oracle.prune_compact(a_bits, ratio)
        pruned = oracle.decompress(r["bitmap"], r["values"], a_bits.size).reshape(layer.act_shape)
        ref = oracle.dw_conv2d_grouped(pruned, g.numpy(), layer.kh, layer.kw, layer.stride, layer.pad, layer.groups)
        if ratio == 1.0:
            assert not dw.any()
        else:
            assert rel_frobenius(dw, ref) <= 1e-5, (layer.name, ratio)


def test_grouped_accumulate_and_reproducible():
    layer = SHAPES[0]
    a, g = W.activation(layer, seed=7).cuda(), W.grad_out(layer, seed=7).cuda()
    comp = B.surgeon_prune_compact(a, 0.5)
    desc = B.layer_desc(layer, B.PATH_FP32)
    d1 = B.surgeon_weight_grad(comp, desc, g)
    d2 = B.surgeon_weight_grad(comp, desc, g)
    assert torch.equal(d1, d2)
    acc = d1.clone()
    B.surgeon_weight_grad(comp, desc, g, dw=acc, accumulate=True)
    assert torch.allclose(acc, 2 * d1, rtol=1e-6, atol=0)


def test_grouped_argument_errors():
    bad = W.conv("bad", 2, 10, 8, 12, 3, groups=4)        # 10 input channels do not split into 4 groups
    a = torch.zeros(bad.act_shape, device="cuda")
    comp = B.surgeon_prune_compact(a, 0.5)
    with pytest.raises(B.SurgeonError) as e:
        B.surgeon_weight_grad(comp, B.layer_desc(bad, B.PATH_FP32), torch.zeros(bad.grad_shape, device="cuda"),
                              dw=torch.zeros(12, 2, 3, 3, device="cuda"))
    assert e.value.status == B.SURGEON_ERR_INVALID_ARG


def test_resnext29_grouped_layer_at_bench_size_on_sampled_entries():
    """The 3x3 grouped convolution of ResNeXt-29's first stage at batch 200 (26 M activation
    elements): store bit for bit, weight gradient on every entry of a sample of output channels."""
    from gpu_util import assert_store_equals_oracle
    layer = next(l for l in W.resnext29() if l.name == "s1b1.conv2")
    a = W.activation(layer, seed=0)
    g = W.grad_out(layer, seed=0)
    comp, ref = assert_store_equals_oracle(a.reshape(-1), 0.7)
    dw = B.surgeon_weight_grad(comp, B.layer_desc(layer, B.PATH_TENSOR_CORE), g.cuda()).cpu().numpy()
    pruned = oracle.decompress(ref["bitmap"], ref["values"], layer.n_act).reshape(layer.act_shape)
    # the oracle on the channels of three groups (first, a middle one, last): every entry of those
    og, cg = layer.c_out // layer.groups, layer.c_in // layer.groups
    for grp in (0, 13, layer.groups - 1):
        sub = oracle.dw_conv2d(pruned[:, grp * cg:(grp + 1) * cg], g.numpy()[:, grp * og:(grp + 1) * og], 3, 3, 1, 1)
        assert rel_frobenius(dw[grp * og:(grp + 1) * og], sub) <= 1e-5

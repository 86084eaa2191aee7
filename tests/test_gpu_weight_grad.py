"""GPU parity: surgeon_weight_grad through the C ABI vs the fp64 oracle.

Tolerance (relative Frobenius error against the fp64 oracle): 1e-5 for the fp32 CUDA-core path,
5e-3 for the tensor-core path (bf16 operands, fp32 accumulation)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_20354_b200 import binding as B
from paper_2503_20354_b200 import workloads as W
from gpu_util import oracle_dw, rel_frobenius

pytestmark = pytest.mark.gpu

TOL = {B.PATH_FP32: 1e-5, B.PATH_TENSOR_CORE: 5e-3}
PATHS = [B.PATH_FP32, B.PATH_TENSOR_CORE]


def run_layer(layer, ratio, path, seed=0, sigma=0.01):
    a = W.activation(layer, seed)
    g = W.grad_out(layer, seed, sigma=sigma)
    comp = B.surgeon_prune_compact(a.cuda(), ratio)
    dw = B.surgeon_weight_grad(comp, B.layer_desc(layer, path), g.cuda())
    torch.cuda.synchronize()
    a_bits = W.as_numpy_bits(a).reshape(-1)
    r = oracle.prune_compact(a_bits, ratio)
    pruned = oracle.decompress(r["bitmap"], r["values"], a_bits.size)
    ref = oracle_dw(layer, pruned, g.numpy())
    return dw.cpu().numpy(), ref, a_bits, g.numpy()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("ratio", [0.0, 0.3, 0.6, 0.9, 1.0])
def test_config1_tiny_conv(ratio, path):
    layer = W.tiny_conv()[0]
    dw, ref, a_bits, g = run_layer(layer, ratio, path)
    assert dw.shape == (64, 64, 3, 3)
    if ratio == 1.0:
        assert not dw.any()                     # empty store: exactly zero
    else:
        assert rel_frobenius(dw, ref) <= TOL[path]
    if ratio == 0.0:                            # dense gradient computed from x itself
        dense = oracle_dw(layer, a_bits, g)
        assert rel_frobenius(dw, dense) <= TOL[path]


SHAPES = [
    # ragged tiles, strides, 1x1, 7x7 stem, FC-like and token-major linears
    W.conv("c3x3_s2", 3, 20, 18, 24, 3, 2),
    W.conv("c3x3_odd", 2, 17, 13, 70, 3, 1),
    W.conv("c1x1", 4, 40, 14, 96, 1, 1, 0),
    W.conv("c1x1_s2", 4, 64, 14, 130, 1, 2, 0),
    W.conv("stem7x7", 2, 3, 64, 64, 7, 2, 3, dist="normal"),
    W.conv("c3x3_7x7map", 5, 32, 7, 48, 3, 1),
    W.conv("c3x3_nopad", 2, 8, 10, 8, 3, 1, 0),
    # stride-1 3x3 / 1x1 convs with rows a multiple of 8 wide (the two-group fast kernel)
    W.conv("f3x3_w16_partial_ch", 3, 20, 16, 24, 3),
    W.conv("f3x3_w8_two_acc", 4, 32, 8, 320, 3),
    W.conv("f3x3_w56", 2, 8, 56, 16, 3),
    W.conv("f3x3_w32_cout640", 2, 16, 32, 640, 3),
    W.conv("f3x3_w32_cout272_padded", 2, 16, 32, 272, 3),
    W.Layer("f3x3_h12w8_tail_ktile", 1, 3, 8, 12, 8, 32, 3, 3, 1, 1),
    W.Layer("f3x3_h5w16_tail_ktile", 1, 2, 8, 5, 16, 16, 3, 3, 1, 1),
    W.conv("f1x1_w8", 5, 200, 8, 48, 1, 1, 0),
    W.conv("f1x1_w56", 2, 64, 56, 256, 1, 1, 0),
    W.Layer("f1x1_h12w8_tail_ktile", 1, 3, 40, 12, 8, 32, 1, 1, 1, 0),
    W.conv("f3x3_s2_w32", 3, 20, 32, 40, 3, 2),
    W.conv("f3x3_s2_w16_two_acc", 4, 16, 16, 320, 3, 2),
    W.conv("f1x1_s2_w32", 3, 150, 32, 48, 1, 2, 0),
    W.conv("f1x1_s2_w16", 5, 24, 16, 320, 1, 2, 0),
    W.linear("fc", 64, 2048, 1000, dist="abs_normal", dt=W.F32),
    W.linear("tokens", 2 * 197, 768, 256, dist="normal", dt=W.F32),
    W.linear("tiny", 5, 7, 3, dist="normal", dt=W.F32),
    # layers whose im2col operand is the activation itself (the direct kernel): linear layers
    # with two 192-column accumulators, ragged channel / row counts; 1x1 convs on 14x14 and 7x7
    # maps (the bf16 gradient copy gets a padded row pitch)
    W.linear("lin_two_acc192", 3 * 64 + 17, 256, 768, dist="normal", dt=W.F32),
    W.linear("lin_c40_o520", 200, 40, 520, dist="gelu_normal", dt=W.F32),
    W.conv("d1x1_hw14", 3, 136, 14, 264, 1, 1, 0),
    W.conv("d1x1_hw7", 5, 72, 7, 48, 1, 1, 0),
    # 1x1 stride 2 (the residual downsample shortcut): even and odd map sizes, output rows
    # shorter and longer than one 32-position run, channels past one tile
    W.conv("d1x1s2_hw56", 2, 72, 56, 136, 1, 2, 0),
    W.conv("d1x1s2_hw28", 3, 264, 28, 520, 1, 2, 0),
    W.conv("d1x1s2_hw15", 3, 40, 15, 48, 1, 2, 0),
    W.conv("d1x1s2_hw70", 1, 16, 70, 32, 1, 2, 0),
    # k x k stride 1 through shifted gradient copies: 5x5, a 2x3 kernel with less padding than
    # "same", channels past one tile on a 14x14 map
    W.conv("t5x5_hw12", 2, 24, 12, 40, 5, 1, 2),
    W.Layer("t2x3_pad1", 1, 3, 16, 9, 11, 24, 2, 3, 1, 1),
    W.conv("t3x3_hw14_c136", 2, 136, 14, 72, 3),
    # the two-group im2col kernel: 3x3 stride 2 on 28- and 14-wide maps with channels past one
    # patch group, 5x5 stride 2, 7x7 stride 3, an output row shorter than a chunk of 8
    W.conv("g3x3s2_hw28_c40", 2, 40, 28, 136, 3, 2),
    W.conv("g3x3s2_hw14_c136", 3, 136, 14, 24, 3, 2),
    W.conv("g5x5s2_hw19", 2, 6, 19, 16, 5, 2, 2),
    W.conv("g7x7s3_hw30", 1, 5, 30, 8, 7, 3, 3, dist="normal"),
    W.conv("g3x3s2_hw10", 4, 8, 10, 8, 3, 2),
]


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("layer", SHAPES, ids=lambda l: l.name)
def test_layer_shapes(layer, bf16, path):
    from dataclasses import replace
    layer = replace(layer, dt=W.BF16 if bf16 else W.F32)
    for ratio in (0.0, 0.7):
        dw, ref, _, _ = run_layer(layer, ratio, path, seed=3)
        assert rel_frobenius(dw, ref) <= TOL[path], (layer.name, ratio)


@pytest.mark.parametrize("path", PATHS)
def test_accumulate_and_reproducible(path):
    layer = W.conv("acc", 2, 16, 16, 32, 3)
    a = W.activation(layer, 9).cuda()
    g = W.grad_out(layer, 9).cuda()
    comp = B.surgeon_prune_compact(a, 0.5)
    d = B.layer_desc(layer, path)
    dw1 = B.surgeon_weight_grad(comp, d, g)
    dw2 = B.surgeon_weight_grad(comp, d, g)
    assert torch.equal(dw1, dw2)                       # fixed summation order
    acc = dw1.clone()
    B.surgeon_weight_grad(comp, d, g, dw=acc, accumulate=True)
    torch.testing.assert_close(acc, 2 * dw1, rtol=1e-6, atol=0)


@pytest.mark.parametrize("path", PATHS)
def test_one_hot_gradient_gives_shifted_copy(path):
    layer = W.conv("onehot", 2, 3, 6, 2, 3, 2, 1, dist="normal")
    a = torch.arange(layer.n_act, dtype=torch.float32).reshape(layer.act_shape) + 1.0
    g = torch.zeros(layer.grad_shape)
    g[1, 1, 0, 2] = 1.0
    comp = B.surgeon_prune_compact(a.cuda(), 0.0)
    dw = B.surgeon_weight_grad(comp, B.layer_desc(layer, path), g.cuda()).cpu().numpy()
    ref = oracle.dw_conv2d(a.numpy(), g.numpy(), 3, 3, 2, 1)
    assert rel_frobenius(dw, ref) <= TOL[path] and not dw[0].any()


def test_cta_pairs():
    """The cta_group::2 variant of the direct kernel (off by default) in a child process."""
    import os
    import subprocess
    import sys
    worker = os.path.join(os.path.dirname(os.path.abspath(__file__)), "pairs_worker.py")
    out = subprocess.run([sys.executable, worker], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "PAIRS_OK" in out.stdout, out.stdout[-2000:] + out.stderr[-2000:]


def test_exchanged_roles_on_cta_pairs():
    """The kernel with the operand roles exchanged on CTA pairs (off by default) in a child process."""
    import os
    import subprocess
    import sys
    worker = os.path.join(os.path.dirname(os.path.abspath(__file__)), "swap_worker.py")
    out = subprocess.run([sys.executable, worker], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "SWAP_OK" in out.stdout, out.stdout[-2000:] + out.stderr[-2000:]


def test_weight_grad_argument_errors():
    layer = W.conv("err", 2, 4, 8, 4, 3)
    a = W.activation(layer, 1).cuda()
    g = W.grad_out(layer, 1).cuda()
    comp = B.surgeon_prune_compact(a, 0.5)
    d = B.layer_desc(layer, B.PATH_FP32)
    with pytest.raises(B.SurgeonError) as e:
        B.surgeon_weight_grad(comp, d, g, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == B.SURGEON_ERR_BUFFER_TOO_SMALL
    wrong = B.layer_desc(W.conv("err2", 3, 4, 8, 4, 3), B.PATH_FP32)   # activation size mismatch
    with pytest.raises(B.SurgeonError) as e:
        B.surgeon_weight_grad(comp, wrong, g)
    assert e.value.status == B.SURGEON_ERR_INVALID_ARG


@pytest.mark.parametrize("path", PATHS)
def test_one_store_feeds_the_two_layers_that_read_the_same_input(path):
    """A residual block's first convolution and its 1x1 shortcut take the same tensor: it is pruned
    once and both weight gradients are formed from the one store."""
    conv1 = W.conv("b0.conv1", 3, 48, 16, 72, 3, 2)
    short = W.conv("b0.shortcut", 3, 48, 16, 72, 1, 2, 0)
    assert W.shared_inputs([conv1, short]) == {1: 0}
    a = W.activation(conv1, seed=4)
    comp = B.surgeon_prune_compact(a.cuda(), 0.6)
    ref = oracle.prune_compact(W.as_numpy_bits(a).reshape(-1), 0.6)
    pruned = oracle.decompress(ref["bitmap"], ref["values"], conv1.n_act)
    for layer in (conv1, short):
        g = W.grad_out(layer, seed=4, index=1 + layer.kh)
        dw = B.surgeon_weight_grad(comp, B.layer_desc(layer, path), g.cuda()).cpu().numpy()
        want = oracle_dw(layer, pruned, g.numpy())
        assert rel_frobenius(dw, want) <= TOL[path], layer.name
    assert comp.read_header().status == 0


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("layer", [SHAPES[1], SHAPES[2], SHAPES[4], SHAPES[10], SHAPES[19], SHAPES[22], SHAPES[36]],
                         ids=lambda l: l.name)
def test_output_and_scratch_stay_inside_their_buffers(layer, path):
    """dw and the scratch sit at the front of larger buffers filled with a pattern: the words after
    `dw` and after the size surgeon_weight_grad_workspace reports must come back untouched."""
    a, g = W.activation(layer, seed=5).cuda(), W.grad_out(layer, seed=5).cuda()
    comp = B.surgeon_prune_compact(a, 0.6)
    desc = B.layer_desc(layer, path)
    need = B.surgeon_weight_grad_workspace(desc)
    n_dw = int(np.prod(layer.dw_shape))
    big_dw = torch.full((n_dw + 256,), 777.0, device="cuda")
    big_ws = torch.full((need + 1024,), 0x5A, dtype=torch.uint8, device="cuda")
    dw = big_dw[:n_dw].view(layer.dw_shape)
    B.surgeon_weight_grad(comp, desc, g, dw=dw, workspace=big_ws[:need])
    torch.cuda.synchronize()
    assert bool((big_dw[n_dw:] == 777.0).all()) and bool((big_ws[need:] == 0x5A).all())
    ref = B.surgeon_weight_grad(comp, desc, g)
    assert torch.equal(dw, ref)

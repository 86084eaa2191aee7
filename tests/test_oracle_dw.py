"""Pins for the oracle's weight gradient (Eq. 2; Algorithm 1: Reshape and gradient steps).

Independent references: PyTorch's fp64 autograd through conv2d / matmul (a library routine, not
the oracle's loops), finite differences of a scalar loss, the 1x1-conv == linear identity,
linearity in the activation, one-hot inputs with a hand-derivable answer, and the two ends of
the ratio range (0 -> dense gradient, 1 -> exactly zero).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_20354_b200 import workloads as W


def _torch_dw_conv(a64, g64, kh, kw, stride, pad):
    a = torch.from_numpy(a64)
    g = torch.from_numpy(g64)
    w = torch.zeros(g.shape[1], a.shape[1], kh, kw, dtype=torch.float64, requires_grad=True)
    y = torch.nn.functional.conv2d(a, w, None, stride=stride, padding=pad)
    assert y.shape == g.shape
    (y * g).sum().backward()
    return w.grad.numpy()


CONV_CASES = [
    # B, C, H, W, O, k, stride, pad
    (2, 3, 8, 8, 4, 3, 1, 1),
    (2, 4, 9, 7, 3, 3, 2, 1),
    (1, 2, 12, 12, 5, 7, 2, 3),
    (3, 5, 6, 6, 2, 1, 1, 0),
    (2, 4, 8, 8, 6, 1, 2, 0),
    (2, 2, 5, 5, 2, 3, 1, 0),
    (1, 3, 4, 6, 2, 2, 2, 1),
]


@pytest.mark.parametrize("case", CONV_CASES)
def test_conv_matches_torch_autograd_fp64(case):
    B, C, H, Wd, O, k, s, p = case
    rng = np.random.default_rng(7)
    a = rng.standard_normal((B, C, H, Wd)).astype(np.float32)
    oh, ow = oracle.conv_out_hw(H, Wd, k, k, s, p)
    g = rng.standard_normal((B, O, oh, ow)).astype(np.float32)
    dw = oracle.dw_conv2d(a, g, k, k, s, p)
    ref = _torch_dw_conv(a.astype(np.float64), g.astype(np.float64), k, k, s, p)
    np.testing.assert_allclose(dw, ref, rtol=1e-12, atol=1e-12)
    # single-entry routine agrees with the full one
    assert oracle.dw_conv2d_entry(a, g, k, k, s, p, O - 1, C - 1, k - 1, 0) == pytest.approx(
        dw[O - 1, C - 1, k - 1, 0], rel=1e-14, abs=1e-14)


def test_conv_bf16_input_matches_torch():
    B, C, H, Wd, O, k, s, p = 2, 3, 8, 8, 4, 3, 1, 1
    a_bf = torch.randn(B, C, H, Wd, generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    g = np.random.default_rng(3).standard_normal((B, O, 8, 8)).astype(np.float32)
    dw = oracle.dw_conv2d(W.as_numpy_bits(a_bf), g, k, k, s, p)
    ref = _torch_dw_conv(a_bf.to(torch.float64).numpy(), g.astype(np.float64), k, k, s, p)
    np.testing.assert_allclose(dw, ref, rtol=1e-12, atol=1e-12)


def test_linear_matches_matmul_and_paper_orientation():
    rng = np.random.default_rng(11)
    T, C, O = 37, 19, 23
    a = rng.standard_normal((T, C)).astype(np.float32)
    g = rng.standard_normal((T, O)).astype(np.float32)
    dw = oracle.dw_linear(a, g)
    # Eq. 2 writes A^T * dL/dA_{i+1} ([in, out]); the weight layout is its transpose.
    eq2 = a.astype(np.float64).T @ g.astype(np.float64)
    np.testing.assert_allclose(dw, eq2.T, rtol=1e-12, atol=1e-12)
    assert oracle.dw_linear_entry(a, g, 5, 7) == pytest.approx(eq2[7, 5], rel=1e-13)
    # autograd through y = a @ w^T
    w = torch.zeros(O, C, dtype=torch.float64, requires_grad=True)
    (torch.from_numpy(a.astype(np.float64)) @ w.T * torch.from_numpy(g.astype(np.float64))).sum().backward()
    np.testing.assert_allclose(dw, w.grad.numpy(), rtol=1e-12, atol=1e-12)


def test_conv1x1_equals_linear_on_nhwc_view():
    rng = np.random.default_rng(13)
    B, C, H, Wd, O = 3, 6, 5, 4, 7
    a = rng.standard_normal((B, C, H, Wd)).astype(np.float32)
    g = rng.standard_normal((B, O, H, Wd)).astype(np.float32)
    dw_conv = oracle.dw_conv2d(a, g, 1, 1, 1, 0)[:, :, 0, 0]
    a_rows = np.ascontiguousarray(a.transpose(0, 2, 3, 1).reshape(-1, C))
    g_rows = np.ascontiguousarray(g.transpose(0, 2, 3, 1).reshape(-1, O))
    np.testing.assert_allclose(dw_conv, oracle.dw_linear(a_rows, g_rows), rtol=1e-13, atol=1e-13)


def test_finite_difference_of_scalar_loss():
    # L(w) = sum(conv(a, w) * g) is linear in w, so a central difference is exact up to rounding.
    rng = np.random.default_rng(17)
    B, C, H, Wd, O, k, s, p = 2, 2, 4, 4, 2, 3, 1, 1
    a = rng.standard_normal((B, C, H, Wd)).astype(np.float32)
    g = rng.standard_normal((B, O, H, Wd)).astype(np.float32)
    dw = oracle.dw_conv2d(a, g, k, k, s, p)
    a_t, g_t = torch.from_numpy(a).double(), torch.from_numpy(g).double()

    def loss(w):
        return float((torch.nn.functional.conv2d(a_t, w, None, stride=s, padding=p) * g_t).sum())

    w0 = torch.from_numpy(rng.standard_normal((O, C, k, k)))
    for (o, c, r, q) in [(0, 0, 0, 0), (1, 1, 2, 2), (0, 1, 1, 0), (1, 0, 0, 2)]:
        e = torch.zeros_like(w0)
        e[o, c, r, q] = 0.5
        fd = loss(w0 + e) - loss(w0 - e)
        assert fd == pytest.approx(dw[o, c, r, q], rel=1e-10, abs=1e-10)


def test_one_hot_gives_shifted_copy():
    # One non-zero gradient entry g[b0,o0,y0,x0] = 1: dw[o0,c,r,s] = a[b0,c,y0*st+r-p,x0*st+s-p].
    B, C, H, Wd, O, k, s, p = 2, 3, 6, 6, 2, 3, 2, 1
    a = np.arange(B * C * H * Wd, dtype=np.float32).reshape(B, C, H, Wd) + 1.0
    oh, ow = oracle.conv_out_hw(H, Wd, k, k, s, p)
    g = np.zeros((B, O, oh, ow), dtype=np.float32)
    b0, o0, y0, x0 = 1, 1, 0, 2
    g[b0, o0, y0, x0] = 1.0
    dw = oracle.dw_conv2d(a, g, k, k, s, p)
    assert not dw[0].any()
    for c in range(C):
        for r in range(k):
            for q in range(k):
                iy, ix = y0 * s + r - p, x0 * s + q - p
                exp = a[b0, c, iy, ix] if 0 <= iy < H and 0 <= ix < Wd else 0.0
                assert dw[o0, c, r, q] == exp


@pytest.mark.parametrize("bf16", [False, True])
def test_ratio_ends_and_linearity_through_the_store(bf16):
    layer = W.conv("t", 2, 4, 8, 5, 3, dt=W.BF16 if bf16 else W.F32)
    a_t = W.activation(layer, seed=21)
    a = W.as_numpy_bits(a_t)
    g = W.grad_out(layer, seed=21).numpy()
    n = a.size
    dense = oracle.dw_conv2d(a, g, 3, 3, 1, 1)      # computed from x itself, never from a store
    # ratio 0: the store round-trips, so dW from the store equals the dense dW exactly
    r0 = oracle.prune_compact(a, 0.0)
    a0 = oracle.decompress(r0["bitmap"], r0["values"], n).reshape(a.shape)
    assert np.array_equal(oracle.dw_conv2d(a0, g, 3, 3, 1, 1), dense)
    # ratio 1: empty store, dW exactly zero
    r1 = oracle.prune_compact(a, 1.0)
    a1 = oracle.decompress(r1["bitmap"], r1["values"], n).reshape(a.shape)
    assert not oracle.dw_conv2d(a1, g, 3, 3, 1, 1).any()
    # linearity: dW(pruned) + dW(removed part) = dW(dense)
    r = oracle.prune_compact(a, 0.6)
    kept = oracle.decompress(r["bitmap"], r["values"], n).reshape(a.shape)
    removed = a.copy().reshape(-1)
    removed[r["keep"] == 1] = 0
    removed = removed.reshape(a.shape)
    s = oracle.dw_conv2d(kept, g, 3, 3, 1, 1) + oracle.dw_conv2d(removed, g, 3, 3, 1, 1)
    np.testing.assert_allclose(s, dense, rtol=1e-12, atol=1e-14)


# ---- grouped convolutions (ResNeXt's 3x3 layers, depthwise convolutions) --------------------------

GROUPED_CASES = [
    # B, C, H, W, O, k, stride, pad, groups
    (2, 8, 7, 7, 12, 3, 1, 1, 4),
    (2, 6, 8, 6, 6, 3, 2, 1, 6),      # depthwise, stride 2
    (1, 4, 9, 9, 8, 3, 1, 0, 2),
    (3, 6, 5, 5, 9, 1, 1, 0, 3),
    (1, 4, 10, 10, 4, 5, 2, 2, 4),    # depthwise 5x5
]


@pytest.mark.parametrize("case", GROUPED_CASES)
def test_grouped_conv_matches_torch_autograd_fp64(case):
    B, C, H, Wd, O, k, s, p, groups = case
    rng = np.random.default_rng(11)
    a32 = rng.standard_normal((B, C, H, Wd)).astype(np.float32)
    oh, ow = oracle.conv_out_hw(H, Wd, k, k, s, p)
    g32 = rng.standard_normal((B, O, oh, ow)).astype(np.float32)
    a = torch.from_numpy(a32.astype(np.float64))
    g = torch.from_numpy(g32.astype(np.float64))
    w = torch.zeros(O, C // groups, k, k, dtype=torch.float64, requires_grad=True)
    y = torch.nn.functional.conv2d(a, w, None, stride=s, padding=p, groups=groups)
    (y * g).sum().backward()
    got = oracle.dw_conv2d_grouped(a32, g32, k, k, s, p, groups)
    assert got.shape == (O, C // groups, k, k)
    np.testing.assert_allclose(got, w.grad.numpy(), rtol=1e-12, atol=1e-12)


def test_one_group_is_the_ungrouped_gradient():
    rng = np.random.default_rng(12)
    a = rng.standard_normal((2, 5, 6, 7)).astype(np.float32)
    g = rng.standard_normal((2, 4, 6, 7)).astype(np.float32)
    assert np.array_equal(oracle.dw_conv2d_grouped(a, g, 3, 3, 1, 1, 1), oracle.dw_conv2d(a, g, 3, 3, 1, 1))


def test_groups_are_independent_ungrouped_problems():
    """Group g of a grouped layer is the ungrouped layer on its own slices of the channels."""
    rng = np.random.default_rng(13)
    a = rng.standard_normal((2, 6, 6, 6)).astype(np.float32)
    g = rng.standard_normal((2, 9, 3, 3)).astype(np.float32)
    full = oracle.dw_conv2d_grouped(a, g, 3, 3, 2, 1, 3)
    for grp in range(3):
        part = oracle.dw_conv2d(a[:, 2 * grp:2 * grp + 2], g[:, 3 * grp:3 * grp + 3], 3, 3, 2, 1)
        assert np.array_equal(full[3 * grp:3 * grp + 3], part)


def test_depthwise_2x2_worked_by_hand():
    """One image, two channels, 2x2 maps, 1x1 kernel, groups = channels: each weight is the plain
    correlation of its own channel's gradient and activation."""
    a = np.array([[[[1, 2], [3, 4]], [[-1, 0], [2, 5]]]], dtype=np.float32)
    g = np.array([[[[1, 0], [0, 2]], [[3, 1], [1, 1]]]], dtype=np.float32)
    dw = oracle.dw_conv2d_grouped(a, g, 1, 1, 1, 0, 2)
    # channel 0: 1*1 + 0*2 + 0*3 + 2*4 = 9;  channel 1: 3*(-1) + 1*0 + 1*2 + 1*5 = 4
    assert dw.reshape(-1).tolist() == [9.0, 4.0]
    # a 2x2 kernel without padding has one output position: dw = g * a window
    g1 = np.array([[[[2.0]], [[-1.0]]]], dtype=np.float32)
    dw2 = oracle.dw_conv2d_grouped(a, g1, 2, 2, 1, 0, 2)
    assert np.array_equal(dw2[0, 0], 2.0 * a[0, 0]) and np.array_equal(dw2[1, 0], -1.0 * a[0, 1])

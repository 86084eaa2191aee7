"""GPU parity at the sizes and in the configuration `bench.py` times.

Stores of whole bench layers are compared with the oracle bit for bit (its nth_element select
takes seconds at 10-40 M elements); a 2^28-element tensor is checked through the properties that
define the store (every one of them is decided on the device with plain torch ops, none uses the
library); weight gradients of whole bench layers are compared with the oracle on sampled
entries, which it computes one by one."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_20354_b200 import binding as B
from paper_2503_20354_b200 import workloads as W
from gpu_util import assert_store_equals_oracle

pytestmark = pytest.mark.gpu


def _layer(stack, name):
    return next(l for l in stack if l.name == name)


@pytest.mark.parametrize("which,name,ratio", [
    ("wrn", "g1b1.conv1", 0.2), ("wrn", "g1b1.conv1", 0.7), ("wrn", "g3b1.conv1", 0.0),
    ("vit", "blk0.fc2", 0.7), ("vit", "blk0.qkv", 0.3), ("r50", "layer1.0.conv1", 0.6),
])
def test_store_of_a_whole_bench_layer(which, name, ratio):
    stack = {"wrn": W.wrn28_10, "vit": W.vit_b16, "r50": W.resnet50}[which]()
    layer = _layer(stack, name)
    x = W.activation(layer, seed=0)
    assert_store_equals_oracle(x.reshape(-1), ratio)


def _keys(x):
    if x.dtype == torch.float32:
        return x.view(torch.int32) & 0x7FFFFFFF
    return (x.view(torch.int16) & 0x7FFF).to(torch.int32)


@pytest.mark.parametrize("lg,bf16,ratio", [(28, False, 0.5), (28, False, 0.1), (28, True, 0.9),
                                            (30, False, 0.9), (30, True, 0.5)])
def test_store_properties_at_sweep_size(lg, bf16, ratio):
    """2^28 and 2^30 elements (the largest tensor of the bandwidth sweep: 4 GiB of fp32, where
    byte offsets need 64 bits)."""
    n = 1 << lg
    x = W.draw("relu_normal", n, seed=3, device="cuda")
    if bf16:
        x = x.to(torch.bfloat16)
    comp = B.surgeon_prune_compact(x, ratio)
    torch.cuda.synchronize()
    h = comp.read_header()
    assert h.status == 0 and h.n_keep == oracle.n_keep(n, ratio)
    # bitmap -> kept mask, 2^24 elements at a time
    keys = _keys(x)
    tau = int(h.threshold_key)
    shifts = torch.arange(32, device="cuda", dtype=torch.int32)
    kept_total = kept_ties = 0
    last_kept_tie, first_dropped_tie = -1, n
    vals = comp.values.view(torch.int32 if not bf16 else torch.int16)
    xbits = x.view(torch.int32 if not bf16 else torch.int16)
    offs = comp.block_offsets[: n // 128 + 1].to(torch.int64)
    step = 1 << 24
    for lo in range(0, n, step):
        words = comp.bitmap[lo // 32:(lo + step) // 32]
        mask = ((words.unsqueeze(1) >> shifts) & 1).reshape(-1).bool()
        k = keys[lo:lo + step]
        assert bool((k[mask] >= tau).all()) and bool((k[~mask] <= tau).all())
        ties = k == tau
        kt = mask & ties
        dt_ = (~mask) & ties
        if bool(kt.any()):
            last_kept_tie = max(last_kept_tie, lo + int(kt.nonzero()[-1]))
        if bool(dt_.any()):
            first_dropped_tie = min(first_dropped_tie, lo + int(dt_.nonzero()[0]))
        cnt = int(mask.sum())
        # packed values = the kept elements in index order; block offsets = running kept count
        assert torch.equal(vals[kept_total:kept_total + cnt], xbits[lo:lo + step][mask])
        per_block = mask.view(-1, 128).sum(dim=1)
        run = torch.cumsum(per_block, 0) - per_block + kept_total
        assert torch.equal(offs[lo // 128:(lo + step) // 128], run)
        kept_total += cnt
        kept_ties += int(kt.sum())
    assert kept_total == h.n_keep == int(offs[-1])
    assert kept_ties == h.tie_quota and h.n_greater + h.tie_quota == h.n_keep
    assert last_kept_tie < first_dropped_tie          # ties are kept by lowest flat index


def _stratified_entries(shape, rng, k_len):
    """Entries of a weight-gradient tensor that reach every part of the launch grid: one random
    entry in every cell of (16 output channels) x (16 input channels) x (kernel tap) - no tile of
    rows, column unit, tap or accumulator of any kernel is wider than such a cell - plus random
    entries over the whole tensor, fewer for long reductions (an entry costs k_len terms)."""
    O, C = shape[0], shape[1]
    taps = [(r, s) for r in range(shape[2]) for s in range(shape[3])] if len(shape) == 4 else [()]
    cells = []
    for tap in taps:
        for o0 in range(0, O, 16):
            for c0 in range(0, C, 16):
                cells.append((int(rng.integers(o0, min(o0 + 16, O))),
                              int(rng.integers(c0, min(c0 + 16, C)))) + tap)
    budget = int(2.5e8 // max(k_len, 1))                 # terms the CPU adds up per case
    if len(cells) > budget:                              # thin the cells evenly, keep the strata
        cells = [cells[i] for i in np.linspace(0, len(cells) - 1, budget).astype(int)]
    n_rand = int(min(2000, max(64, budget - len(cells))))
    rand = [tuple(int(rng.integers(0, d)) for d in shape) for _ in range(n_rand)]
    return cells + rand


_SIGMA = {"wrn": 0.01, "vit": 1e-3, "r50": 1e-3}


@pytest.mark.parametrize("ratio", [0.0, 0.3, 0.95])
@pytest.mark.parametrize("which,name", [
    ("wrn", "g1b1.conv1"),            # 160 channels, 32x32: tap stacking, two row tiles of 80 rows
    ("wrn", "g2b1.conv1"),            # 320 channels, 16x16
    ("wrn", "g3b1.conv1"),            # 640 channels, 8x8: five row tiles, twelve column tiles
    ("wrn", "g2b0.conv1"),            # 3x3 stride 2 (shared-memory patch kernel)
    ("wrn", "g2b0.shortcut"),         # 1x1 stride 2
    ("vit", "blk0.qkv"), ("vit", "blk0.fc1"), ("vit", "blk0.fc2"),
    ("r50", "layer1.0.conv3"),        # 1x1 64 -> 256 on 56x56: bound by the gradient read
    ("r50", "layer3.0.conv2"),        # 3x3 stride 2 on 28x28 (im2col kernel)
    ("r50", "stem"),                  # 7x7 stride 2
    ("r50", "layer2.0.downsample"),   # 1x1 stride 2 on 56x56
    ("r50", "layer4.1.conv2"),        # 3x3 on 7x7 maps (rows not a multiple of 8 wide)
    ("r50", "fc"),
])
def test_weight_gradient_of_a_whole_bench_layer_on_sampled_entries(which, name, ratio):
    """A whole bench layer at a ratio the rule produces (0: the layer Eq. 7 leaves dense; 0.3: the
    dense-tile path of the producers; 0.95).  The oracle prunes the activation itself; the GPU
    store must equal the oracle's bit for bit, and the weight gradient is compared with the
    oracle's on a stratified sample of entries computed from the ORACLE's pruned activation."""
    stack = {"wrn": W.wrn28_10, "vit": W.vit_b16, "r50": W.resnet50}[which]()
    layer = _layer(stack, name)
    a = W.activation(layer, seed=0)
    g = W.grad_out(layer, seed=0, sigma=_SIGMA[which])
    comp, ref = assert_store_equals_oracle(a.reshape(-1), ratio)
    pruned = oracle.decompress(ref["bitmap"], ref["values"], layer.n_act).reshape(layer.act_shape)
    dw = B.surgeon_weight_grad(comp, B.layer_desc(layer, B.PATH_TENSOR_CORE), g.cuda())
    dwh = dw.cpu().numpy()
    gh = g.numpy()
    rng = np.random.default_rng(5)
    got, want = [], []
    for idx in _stratified_entries(dwh.shape, rng, layer.gemm_k):
        if layer.kind == 1:
            r = oracle.dw_conv2d_entry(pruned, gh, layer.kh, layer.kw, layer.stride, layer.pad, *idx)
        else:
            r = oracle.dw_linear_entry(pruned, gh, *idx)
        got.append(float(dwh[idx])); want.append(r)
    got, want = np.array(got), np.array(want)
    # the tolerance of the tensor-core path, taken over the sample
    assert np.linalg.norm(got - want) <= 5e-3 * np.linalg.norm(want)
    assert np.isfinite(dwh).all()
    assert comp.read_header().status == 0


@pytest.mark.parametrize("ratio", [0.0, 0.3, 0.95])
@pytest.mark.parametrize("name", ["s1b1.conv2",      # 32 groups of 4 channels, 32x32
                                  "s2b0.conv2",      # 8 channels per group, stride 2, 32x32 -> 16x16
                                  "s3b1.conv2"])     # 16 channels per group, 8x8
def test_grouped_weight_gradient_of_a_whole_resnext_layer_on_sampled_entries(name, ratio):
    """The grouped 3x3 layers of the ResNeXt-29-shaped stack at batch 200, from the oracle's own store
    (asserted equal to the GPU's bit for bit), at a ratio that takes the mostly-kept rebuild path
    (0, 0.3) and one that takes the sparse path (0.95).  An entry (o, c', r, s) of a grouped layer
    is the ungrouped entry (o, group(o) * C/G + c', r, s), so the entry-wise oracle serves; the
    sample has one entry in every 16 x 16 x tap cell plus random ones.  fp32 kernel: 1e-5."""
    layer = _layer(W.resnext29(), name)
    assert layer.groups == 32
    a = W.activation(layer, seed=0)
    g = W.grad_out(layer, seed=0, sigma=0.01)
    comp, ref = assert_store_equals_oracle(a.reshape(-1), ratio)
    pruned = oracle.decompress(ref["bitmap"], ref["values"], layer.n_act).reshape(layer.act_shape)
    dwh = B.surgeon_weight_grad(comp, B.layer_desc(layer, B.PATH_TENSOR_CORE), g.cuda()).cpu().numpy()
    assert dwh.shape == layer.dw_shape
    gh = g.numpy()
    cg, og = layer.c_in // layer.groups, layer.c_out // layer.groups
    rng = np.random.default_rng(6)
    got, want = [], []
    for (o, cl, r, s_) in _stratified_entries(dwh.shape, rng, layer.gemm_k):
        c = (o // og) * cg + cl
        want.append(oracle.dw_conv2d_entry(pruned, gh, layer.kh, layer.kw, layer.stride, layer.pad, o, c, r, s_))
        got.append(float(dwh[o, cl, r, s_]))
    got, want = np.array(got), np.array(want)
    assert np.linalg.norm(got - want) <= 1e-5 * np.linalg.norm(want)
    assert np.isfinite(dwh).all()


@pytest.mark.parametrize("which,name,ratio", [
    ("wrn", "g1b1.conv1", 0.2), ("r50", "layer1.0.conv1", 0.3), ("vit", "blk0.fc2", 0.4),
])
def test_store_without_kept_zeros_at_bench_size(which, name, ratio):
    """The store variant that spends no bit on a kept zero, on whole bench layers whose data hold
    exact zeros in the kept set (post-ReLU at a ratio below one half) or none at all (GELU)."""
    stack = {"wrn": W.wrn28_10, "vit": W.vit_b16, "r50": W.resnet50}[which]()
    layer = _layer(stack, name)
    x = W.activation(layer, seed=0)
    assert_store_equals_oracle(x.reshape(-1), ratio, drop_zeros=True)

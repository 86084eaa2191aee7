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


@pytest.mark.parametrize("bf16,ratio", [(False, 0.5), (False, 0.1), (True, 0.9)])
def test_store_properties_at_sweep_size(bf16, ratio):
    n = 1 << 28
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


@pytest.mark.parametrize("which,name", [
    ("wrn", "g3b1.conv1"), ("wrn", "g1b1.conv1"), ("wrn", "g2b0.conv1"), ("vit", "blk0.qkv"),
    ("r50", "layer3.0.conv2"), ("r50", "stem"), ("r50", "layer2.0.downsample"),
])
def test_weight_gradient_of_a_whole_bench_layer_on_sampled_entries(which, name):
    stack = {"wrn": W.wrn28_10, "vit": W.vit_b16, "r50": W.resnet50}[which]()
    layer = _layer(stack, name)
    a = W.activation(layer, seed=0, device="cuda")
    g = W.grad_out(layer, seed=0, sigma=1e-3, device="cuda")
    comp = B.surgeon_prune_compact(a, 0.7)
    dw = B.surgeon_weight_grad(comp, B.layer_desc(layer, B.PATH_TENSOR_CORE), g)
    pruned = W.as_numpy_bits(B.surgeon_decompress(comp)).reshape(layer.act_shape)
    gh = g.cpu().numpy()
    dwh = dw.cpu().numpy()
    rng = np.random.default_rng(5)
    got, ref = [], []
    for _ in range(24):
        idx = tuple(int(rng.integers(0, d)) for d in dwh.shape)
        if layer.kind == 1:
            r = oracle.dw_conv2d_entry(pruned, gh, layer.kh, layer.kw, layer.stride, layer.pad, *idx)
        else:
            r = oracle.dw_linear_entry(pruned, gh, *idx)
        got.append(float(dwh[idx])); ref.append(r)
    got, ref = np.array(got), np.array(ref)
    # the tolerance of the tensor-core path, taken over the sample
    assert np.linalg.norm(got - ref) <= 5e-3 * np.linalg.norm(ref)
    assert comp.read_header().status == 0

"""GPU parity: surgeon_prune_compact / surgeon_decompress through the C ABI vs the CPU oracle,
bit for bit (threshold key, kept count, tie quota, bitmap, packed values, block offsets)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_20354_b200 import binding as B
from paper_2503_20354_b200 import workloads as W
from gpu_util import assert_store_equals_oracle

pytestmark = pytest.mark.gpu

RATIOS_CFG1 = (0.0, 0.3, 0.6, 0.9, 1.0)


def _as(x32: torch.Tensor, bf16: bool) -> torch.Tensor:
    return x32.to(torch.bfloat16) if bf16 else x32


@pytest.mark.parametrize("ratio", RATIOS_CFG1)
def test_config1_tiny_conv_activation(ratio):
    layer = W.tiny_conv()[0]
    x = W.activation(layer, seed=0)
    comp, ref = assert_store_equals_oracle(x, ratio)
    # decompress on the device gives the oracle's dense pruned tensor bitwise
    dense = B.surgeon_decompress(comp).cpu().numpy()
    exp = oracle.decompress(ref["bitmap"], ref["values"], x.numel())
    assert np.array_equal(dense.view(np.uint8), exp.view(np.uint8))


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("n", [1, 2, 31, 32, 33, 1023, 1024, 1025, 8191, 8192, 8193, 65536 + 7,
                               3 * 8192 + 1000])
def test_edge_sizes(n, bf16):
    x = _as(W.draw("relu_normal", n, seed=1, tag=n), bf16)
    for ratio in (0.0, 0.5, 0.77, 1.0):
        assert_store_equals_oracle(x, ratio, method=0 if n < 5000 else 1)


@pytest.mark.parametrize("bf16", [False, True])
def test_empty_tensor(bf16):
    x = torch.empty(0, dtype=torch.bfloat16 if bf16 else torch.float32, device="cuda")
    comp = B.surgeon_prune_compact(x, 0.5)
    torch.cuda.synchronize()
    _, _, offs, hdr = comp.to_numpy()
    assert hdr.n_keep == 0 and hdr.status == 0 and offs.tolist() == [0]
    assert hdr.threshold_key == (0xFFFF if bf16 else 0xFFFFFFFF)


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("dist", ["relu_normal", "normal", "student_t2", "ties16", "gelu_normal"])
@pytest.mark.parametrize("log2n", [20, 23])       # below / above the size where the sampled path starts
def test_distributions_and_ratios(dist, log2n, bf16):
    n = (1 << log2n) + 4321   # many tiles and a ragged tail
    x = _as(W.draw(dist, n, seed=2), bf16)
    for ratio in (0.1, 0.5, 0.9, 0.99):
        assert_store_equals_oracle(x, ratio)


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("n", [1000, 65536 + 7, 300000, (1 << 23) + 77])
def test_store_without_kept_zeros(n, bf16):
    """SURGEON_STORE_DROP_ZEROS: bit-exact with the oracle's variant; at ratios that keep more than
    the non-zero half of post-ReLU data the threshold key is 0 and the zeros are left out."""
    x = _as(W.draw("relu_normal", n, seed=6, tag=n), bf16)
    for ratio in (0.0, 0.3, 0.45, 0.6, 1.0):
        comp, ref = assert_store_equals_oracle(x, ratio, drop_zeros=True, method=0 if n < 5000 else 1)
        if ratio <= 0.45:
            assert ref["tau"] == 0 and ref["k"] < oracle.n_keep(n, ratio)
    # the dense tensor is the one of the plain store
    a = B.surgeon_decompress(B.surgeon_prune_compact(x.cuda(), 0.3)).cpu()
    b = B.surgeon_decompress(B.surgeon_prune_compact(x.cuda(), 0.3, flags=B.SURGEON_STORE_DROP_ZEROS)).cpu()
    assert torch.equal(a.float(), b.float())
    # all zeros: nothing is stored
    z = torch.zeros(n, dtype=x.dtype)
    assert_store_equals_oracle(z, 0.25, drop_zeros=True, method=0 if n < 5000 else 1)


def test_store_without_kept_zeros_gives_the_same_weight_gradient():
    layer = W.conv("nz", 4, 72, 16, 96, 3)
    a = W.activation(layer, 13).cuda()
    g = W.grad_out(layer, 13).cuda()
    for path in (B.PATH_FP32, B.PATH_TENSOR_CORE):
        d = B.layer_desc(layer, path)
        dw_a = B.surgeon_weight_grad(B.surgeon_prune_compact(a, 0.2), d, g)
        dw_b = B.surgeon_weight_grad(B.surgeon_prune_compact(a, 0.2, flags=B.SURGEON_STORE_DROP_ZEROS), d, g)
        assert torch.equal(dw_a, dw_b)
    with pytest.raises(B.SurgeonError) as e:
        B.surgeon_prune_compact(a, 0.2, flags=6)
    assert e.value.status == B.SURGEON_ERR_INVALID_ARG


@pytest.mark.parametrize("bf16", [False, True])
def test_special_values(bf16):
    x = W.draw("normal", 5000, seed=3)
    x[7] = float("nan"); x[100] = float("inf"); x[101] = -float("inf"); x[9] = -0.0; x[10] = 0.0
    x[4000:4100] = 0.0
    x = _as(x, bf16)
    for ratio in (0.0, 0.2, 0.999, 0.9998, 1.0):
        assert_store_equals_oracle(x, ratio, method=0)


@pytest.mark.parametrize("bf16", [False, True])
def test_all_equal_and_two_level(bf16):
    # every key equal: the kept set is the first n_keep indices
    x = _as(torch.full((20000,), 1.5), bf16)
    for ratio in (0.25, 0.5, 0.9999):
        comp, ref = assert_store_equals_oracle(x, ratio)
        assert ref["c_gt"] == 0 and ref["q"] == ref["k"]
    x = torch.zeros(30000)
    x[::3] = -2.0
    for ratio in (0.1, 0.6667, 0.9):
        assert_store_equals_oracle(_as(x, bf16), ratio)


@pytest.mark.parametrize("bf16", [False, True])
def test_massive_ties_on_the_sampled_path(bf16):
    """Tensors large enough for the sampled select in which one magnitude holds far more elements
    than a chunk's candidate slot: every key inside the bracket is then one key, which the select
    takes as the threshold without a fall-back pass.  The tie quota ends in the middle of the
    tensor, at its very start and at its very end; a second magnitude close by (the next key up)
    makes the bracket hold two keys, which must take the fall-back and still agree."""
    n = (1 << 22) + 77
    g = torch.Generator().manual_seed(11)
    u = torch.rand(n, generator=g)
    sign = torch.where(torch.rand(n, generator=g) < 0.5, -1.0, 1.0)
    x = torch.where(u < 0.6, 1.0, 2.0) * sign                 # 60 % at |1|, 40 % at |2|
    for ratio in (0.3, 0.6, 0.7, 0.95, 1.0 - 1.0 / n, 1.0 / n):
        assert_store_equals_oracle(_as(x, bf16), ratio)
    x = torch.full((n,), -0.75)                                # every key equal
    for ratio in (0.5, 0.001):
        comp, ref = assert_store_equals_oracle(_as(x, bf16), ratio)
        assert ref["c_gt"] == 0 and ref["q"] == ref["k"]
    up = torch.tensor(1.0).view(torch.int32) + 1 if not bf16 else None
    y = torch.where(u < 0.5, 1.0, 1.0078125 if bf16 else float(up.view(torch.float32)))   # two adjacent keys
    for ratio in (0.25, 0.5, 0.75):
        assert_store_equals_oracle(_as(y, bf16), ratio)


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("odd", [1, 3, 5, 7])
def test_fully_kept_chunks_behind_a_misaligned_kept_count(odd, bf16):
    # A head of small magnitudes of which an odd number is kept, then large magnitudes that are all
    # kept: every later 4 KB piece is written out whole, starting at a packed position that is not
    # a multiple of a 16-byte vector.
    n_head, n = 3 * 4096 + 40, 1 << 23
    g = torch.Generator().manual_seed(17 + odd)
    x = torch.empty(n)
    x[:n_head] = torch.rand(n_head, generator=g) * 0.5 + 0.01
    x[n_head:] = (torch.rand(n - n_head, generator=g) * 8.0 + 2.0) * torch.where(
        torch.rand(n - n_head, generator=g) < 0.5, -1.0, 1.0)
    keep_head = 1000 + odd
    ratio = (n_head - keep_head + 0.5) / n            # n - floor(ratio * n) = n - n_head + keep_head
    comp, ref = assert_store_equals_oracle(_as(x, bf16), ratio)
    assert ref["k"] == n - n_head + keep_head


def test_repeat_calls_are_bitwise_identical_and_reuse_buffers():
    x = W.draw("ties16", 300000, seed=5).cuda()
    comp = B.surgeon_prune_compact(x, 0.7)
    a = [t.copy() if isinstance(t, np.ndarray) else t for t in comp.to_numpy()[:3]]
    ws = torch.empty(comp.sizes.workspace_bytes, dtype=torch.uint8, device="cuda")
    for _ in range(3):
        B.surgeon_prune_compact(x, 0.7, out=comp, workspace=ws)
        b = comp.to_numpy()[:3]
        assert all(np.array_equal(u, v) for u, v in zip(a, b))


def test_non_default_stream_and_canaries():
    # outputs sit inside larger buffers; the words after each output must stay untouched
    n = 50000 + 13
    x = W.draw("normal", n, seed=6).cuda()
    sizes = B.surgeon_compact_sizes(n, B.SURGEON_F32, 0.4)
    comp = B.CompressedActivation(n, B.SURGEON_F32, 0.4, x.device, sizes)
    pad = 64
    big_bitmap = torch.full((sizes.bitmap_bytes // 4 + pad,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    big_vals = torch.full((sizes.n_keep + pad,), 12345.0, dtype=torch.float32, device="cuda")
    big_offs = torch.full((sizes.offsets_bytes // 4 + pad,), 0x1234567, dtype=torch.int32, device="cuda")
    comp.bitmap, comp.values, comp.block_offsets = big_bitmap, big_vals, big_offs
    comp.c.bitmap, comp.c.values, comp.c.block_offsets = (big_bitmap.data_ptr(), big_vals.data_ptr(),
                                                          big_offs.data_ptr())
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        B.surgeon_prune_compact(x, 0.4, out=comp, stream=s)
    s.synchronize()
    assert_store_equals_oracle(x.cpu(), 0.4, comp=comp)
    assert torch.all(big_bitmap[sizes.bitmap_bytes // 4:] == 0x5A5A5A5A)
    assert torch.all(big_vals[sizes.n_keep:] == 12345.0)
    assert torch.all(big_offs[sizes.offsets_bytes // 4:] == 0x1234567)


def test_argument_errors_on_device():
    x = torch.zeros(1024, device="cuda")
    comp = B.CompressedActivation(1024, 0, 0.5, x.device)
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SurgeonError) as e:
        B.surgeon_prune_compact(x, 0.5, out=comp, workspace=small)
    assert e.value.status == B.SURGEON_ERR_BUFFER_TOO_SMALL
    with pytest.raises(B.SurgeonError) as e:
        B.surgeon_prune_compact(x[1:], 0.5)      # 4-byte aligned only
    assert e.value.status == B.SURGEON_ERR_INVALID_ARG


@pytest.mark.parametrize("bf16", [False, True])
def test_bounded_wait_that_runs_out_reports_timeout_and_stores_nothing(bf16):
    """The select's grid barrier is given a target it cannot reach and a cap of 1024 polls
    (SURGEON_DEBUG_STALL_BARRIER): the wait gives up, the header says so, and no kernel of the call
    has touched bitmap, values or block offsets.  The next ordinary call is unaffected."""
    n = 5000
    x = _as(W.draw("normal", n, seed=8), bf16).cuda()
    comp = B.CompressedActivation(n, B.dtype_code(x.dtype), 0.0, x.device)
    comp.bitmap.fill_(0x5A5A5A5A); comp.block_offsets.fill_(0x1234567)
    comp.values.view(torch.int16 if bf16 else torch.int32).fill_(0x4D4D)
    ws = torch.empty(comp.sizes.workspace_bytes, dtype=torch.uint8, device="cuda")
    B.surgeon_prune_compact(x, 0.5, out=comp, workspace=ws, flags=B.SURGEON_DEBUG_STALL_BARRIER)
    torch.cuda.synchronize()
    assert comp.read_header().status == B.SURGEON_ERR_TIMEOUT
    assert bool((comp.bitmap == 0x5A5A5A5A).all()) and bool((comp.block_offsets == 0x1234567).all())
    assert bool((comp.values.view(torch.int16 if bf16 else torch.int32) == 0x4D4D).all())
    assert_store_equals_oracle(x.cpu(), 0.5, comp=B.surgeon_prune_compact(x, 0.5, out=comp, workspace=ws))

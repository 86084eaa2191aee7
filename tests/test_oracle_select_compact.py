"""Pins for the oracle's magnitude top-k selection and compressed store (Algorithm 1: prune, decompose and Reshape steps).

Brute force in pure Python on tiny tensors, invariants that fix the result uniquely, the
round trip at ratio 0, and special values.  Both selection routes (full stable sort and
nth_element) are held to the same pins.
"""
import struct

import numpy as np
import pytest

import oracle
from paper_2503_20354_b200 import workloads as W


def _bf16_bits(x32: np.ndarray) -> np.ndarray:
    import torch
    return W.as_numpy_bits(torch.from_numpy(np.asarray(x32, dtype=np.float32)).to(torch.bfloat16))


def _brute_force_keep(x: np.ndarray, k: int):
    """Kept set by sorting Python tuples (-|x| by bit pattern, index): independent of the oracle."""
    if x.dtype == np.float32:
        keys = [struct.unpack("<I", struct.pack("<f", float(v)))[0] & 0x7FFFFFFF for v in x]
    else:
        keys = [int(v) & 0x7FFF for v in x]
    order = sorted(range(len(keys)), key=lambda j: (-keys[j], j))
    keep = np.zeros(len(keys), dtype=np.uint8)
    keep[order[:k]] = 1
    tau = keys[order[k - 1]] if k > 0 else None
    return keep, tau, keys


@pytest.mark.parametrize("method", [0, 1])
@pytest.mark.parametrize("dist", ["relu_normal", "normal", "ties16", "student_t2"])
@pytest.mark.parametrize("bf16", [False, True])
def test_brute_force_all_ratios_tiny(method, dist, bf16):
    for n in (1, 2, 7, 33, 97):
        x = W.draw(dist, n, seed=3, tag=n).numpy()
        if bf16:
            x = _bf16_bits(x)
        for k in range(0, n + 1):
            keep, tau, cgt, q = oracle.select(x, k, method)
            ref_keep, ref_tau, keys = _brute_force_keep(x, k)
            assert np.array_equal(keep, ref_keep), (n, k)
            if k > 0:
                assert tau == ref_tau
                assert cgt == sum(1 for key in keys if key > tau)
                assert q == k - cgt
            else:
                assert tau == (0xFFFF if bf16 else 0xFFFFFFFF) and cgt == 0 and q == 0


def test_magnitude_criterion_against_abs_values():
    # On finite data the key order is the |x| order: every kept |x| >= every dropped |x|.
    x = W.draw("normal", 4096, seed=5).numpy()
    for ratio in (0.1, 0.5, 0.9):
        r = oracle.prune_compact(x, ratio, method=0)
        kept = np.abs(x[r["keep"] == 1])
        dropped = np.abs(x[r["keep"] == 0])
        assert kept.size == r["k"] == oracle.n_keep(4096, ratio)
        assert kept.min() >= dropped.max()
        # no ties in continuous data: the threshold is the k-th largest |x| of a numpy sort
        assert np.float32(np.sort(np.abs(x))[::-1][r["k"] - 1]).view(np.uint32) == r["tau"]


@pytest.mark.parametrize("method", [0, 1])
def test_ties_keep_lowest_indices(method):
    # 16-level data: many equal magnitudes.  Among keys == tau exactly q are kept and they are the
    # first q in index order; +x and -x tie.
    x = W.draw("ties16", 5000, seed=9).numpy()
    keys = np.abs(x).view(np.uint32)
    for k in (1, 17, 1234, 2500, 4999, 5000):
        keep, tau, cgt, q = oracle.select(x, k, method)
        assert keep.sum() == k
        assert np.all(keep[keys > tau] == 1) and np.all(keep[keys < tau] == 0)
        tie_idx = np.nonzero(keys == tau)[0]
        assert keep[tie_idx].sum() == q == k - cgt and q >= 1
        assert np.all(keep[tie_idx[:q]] == 1) and np.all(keep[tie_idx[q:]] == 0)
    # explicit tiny case: |values| = 2 2 1 2 1, k = 2 -> indices 0 and 1
    x = np.array([2.0, -2.0, 1.0, 2.0, -1.0], dtype=np.float32)
    keep, tau, cgt, q = oracle.select(x, 2, method)
    assert keep.tolist() == [1, 1, 0, 0, 0] and cgt == 0 and q == 2
    keep, tau, cgt, q = oracle.select(x, 4, method)
    assert keep.tolist() == [1, 1, 1, 1, 0] and cgt == 3 and q == 1


def test_relu_zeros_inside_kept_set():
    # Post-ReLU data at a low ratio: more elements are kept than are non-zero, so the threshold
    # key is 0 and the kept zeros are the lowest-index ones.
    x = W.draw("relu_normal", 1 << 12, seed=0).numpy()
    nnz = int((x != 0).sum())
    r = oracle.prune_compact(x, 0.3)
    assert r["k"] > nnz and r["tau"] == 0 and r["c_gt"] == nnz and r["q"] == r["k"] - nnz
    zero_idx = np.nonzero(x == 0)[0]
    assert np.all(r["keep"][zero_idx[: r["q"]]] == 1) and np.all(r["keep"][zero_idx[r["q"]:]] == 0)
    assert np.all(r["keep"][x != 0] == 1)


@pytest.mark.parametrize("method", [0, 1])
def test_special_values_order(method):
    # -0 ties with +0; Inf above finite; NaN above Inf.
    x = np.array([0.0, -0.0, 1.0, -np.inf, np.nan, -3.0, np.inf, 1e-45], dtype=np.float32)
    expected_order = [4, 3, 6, 5, 2, 7, 0, 1]   # NaN, Inf(idx3), Inf(idx6), 3, 1, denormal, 0, -0
    for k in range(0, 9):
        keep, tau, cgt, q = oracle.select(x, k, method)
        assert sorted(np.nonzero(keep)[0].tolist()) == sorted(expected_order[:k])
    xb = _bf16_bits(x)
    for k in range(0, 9):
        keep, _, _, _ = oracle.select(xb, k, method)
        # 1e-45 rounds to 0 in bf16: order becomes NaN, Inf, Inf, 3, 1, then zeros by index (0,1,7)
        exp = [4, 3, 6, 5, 2, 0, 1, 7]
        assert sorted(np.nonzero(keep)[0].tolist()) == sorted(exp[:k])


@pytest.mark.parametrize("bf16", [False, True])
def test_sort_and_nth_element_agree(bf16):
    for dist in W.DISTS:
        x = W.draw(dist, 20000, seed=11).numpy()
        if bf16:
            x = _bf16_bits(x)
        for ratio in (0.0, 0.1, 0.5, 0.9, 0.99, 1.0):
            k = oracle.n_keep(x.size, ratio)
            a = oracle.select(x, k, 0)
            b = oracle.select(x, k, 1)
            assert np.array_equal(a[0], b[0]) and a[1:] == b[1:]


@pytest.mark.parametrize("bf16", [False, True])
def test_store_format_and_round_trip(bf16):
    n = 3 * 1024 + 77    # three full offset blocks and a ragged tail
    x = W.draw("normal", n, seed=13).numpy()
    x[5] = -0.0
    x[6] = np.float32(np.nan)
    if bf16:
        x = _bf16_bits(x)
    # ratio 0: everything kept, values == x bitwise, decompress is the identity bitwise
    r = oracle.prune_compact(x, 0.0)
    assert r["k"] == n and np.array_equal(r["values"].view(np.uint8), x.view(np.uint8))
    back = oracle.decompress(r["bitmap"], r["values"], n)
    assert np.array_equal(back.view(np.uint8), x.view(np.uint8))
    # ratio 1: nothing kept
    r = oracle.prune_compact(x, 1.0)
    assert r["k"] == 0 and r["values"].size == 0 and not r["bitmap"].any()
    assert not oracle.decompress(r["bitmap"], r["values"], n).view(np.uint8).any()
    # general ratio: format invariants written out with numpy bit operations
    r = oracle.prune_compact(x, 0.6)
    bits = np.unpackbits(r["bitmap"].view(np.uint8), bitorder="little")
    assert bits.size == 32 * ((n + 31) // 32)
    assert np.array_equal(bits[:n], r["keep"]) and not bits[n:].any()        # bit j <-> index j; pad 0
    assert bits.sum() == r["k"] == oracle.n_keep(n, 0.6)                      # 1 bit per kept element
    assert np.array_equal(r["values"].view(np.uint8).reshape(r["k"], -1),
                          x[np.nonzero(r["keep"])[0]].view(np.uint8).reshape(r["k"], -1))
    csum = np.concatenate([[0], np.cumsum(r["keep"], dtype=np.int64)])
    nb = (n + oracle.BLOCK - 1) // oracle.BLOCK
    assert r["offsets"].size == nb + 1
    assert [int(v) for v in r["offsets"][:nb]] == [int(csum[b * oracle.BLOCK]) for b in range(nb)]
    assert int(r["offsets"][nb]) == r["k"]
    # stored bytes = kept values + 1 bit per element (Section 4.2)
    es = 2 if bf16 else 4
    assert r["values"].nbytes + r["bitmap"].nbytes == r["k"] * es + 4 * ((n + 31) // 32)
    # decompress puts every value back at its own index and +0 elsewhere
    back = oracle.decompress(r["bitmap"], r["values"], n)
    keep = r["keep"].astype(bool)
    assert np.array_equal(back[keep].view(np.uint8), x[keep].view(np.uint8))
    assert not back[~keep].view(np.uint8).any()


def test_empty_and_single():
    x = np.zeros(0, dtype=np.float32)
    r = oracle.prune_compact(x, 0.5)
    assert r["k"] == 0 and r["bitmap"].size == 0 and r["offsets"].tolist() == [0]
    x = np.array([-2.5], dtype=np.float32)
    r = oracle.prune_compact(x, 0.5)
    assert r["k"] == 1 and r["bitmap"].tolist() == [1] and r["values"].tolist() == [-2.5]
    r = oracle.prune_compact(x, 1.0)
    assert r["k"] == 0 and r["bitmap"].tolist() == [0] and r["tau"] == 0xFFFFFFFF


def test_config1_kept_counts_and_zero_threshold():
    # The tiny-conv configuration: [16,64,32,32] post-ReLU fp32, seed 0.
    layer = W.tiny_conv()[0]
    x = W.as_numpy_bits(W.activation(layer, seed=0)).reshape(-1)
    assert x.size == 1 << 20
    for ratio, k in ((0.0, 1048576), (0.3, 734004), (0.6, 419431), (0.9, 104858), (1.0, 0)):
        r = oracle.prune_compact(x, ratio)
        assert r["k"] == k == int(r["keep"].sum())
        if ratio == 0.3:   # k exceeds the ~50 % non-zeros: threshold key 0, kept zeros by index
            assert r["tau"] == 0 and r["q"] > 0


def test_drop_zeros_variant():
    """The store that spends no value on kept zeros: a hand-worked case, the unchanged dense tensor,
    and equality with the plain store when nothing kept is zero."""
    x = np.array([0.0, 3.0, -0.0, -1.0, 2.0, 0.0], dtype=np.float32)
    # ratio 1/6 removes one element: the kept five are 3, 2, -1 and the zeros at 0 and 2 (lowest indices)
    a = oracle.prune_compact(x, 1.0 / 6.0)
    assert a["k"] == 5 and a["bitmap"].tolist() == [0b011111]
    b = oracle.prune_compact(x, 1.0 / 6.0, drop_zeros=True)
    assert b["k"] == 3 and b["bitmap"].tolist() == [0b011010]
    assert b["values"].tolist() == [3.0, -1.0, 2.0] and b["offsets"].tolist() == [0, 3]
    rng = np.random.default_rng(8)
    for dt in (np.float32, "bf16"):
        r = np.maximum(rng.standard_normal(5000), 0).astype(np.float32)           # half zeros
        xx = r if dt is np.float32 else (r.view(np.uint32) >> 16).astype(np.uint16)
        for ratio in (0.0, 0.3, 0.6):
            a = oracle.prune_compact(xx, ratio)
            b = oracle.prune_compact(xx, ratio, drop_zeros=True)
            da = oracle.decompress(a["bitmap"], a["values"], xx.size)
            db = oracle.decompress(b["bitmap"], b["values"], xx.size)
            assert np.array_equal(da, db)                                          # same dense tensor
            keys = oracle.magnitude_keys(xx)
            assert b["k"] == int(((a["keep"] == 1) & (keys != 0)).sum()) == b["values"].size
            assert not (oracle.magnitude_keys(b["values"]) == 0).any()
            assert b["offsets"][-1] == b["k"]
        pos = xx[keys != 0]
        a = oracle.prune_compact(pos, 0.4)
        b = oracle.prune_compact(pos, 0.4, drop_zeros=True)
        assert np.array_equal(a["bitmap"], b["bitmap"]) and np.array_equal(a["values"], b["values"])

"""Pins for the oracle's per-layer ratio rule (Eq. 5-7) and kept count (Algorithm 1: prune step).

The expected values come from hand-worked fixtures, from a closed form that follows from the
equations (the two inner normalisations cancel: p_i = 1 - M_i G_i / max_j M_j G_j), and from
invariances the equations imply.  None of them re-types the oracle's own steps.
"""
import math
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield line


def test_hand_worked_ratio_examples():
    n = 0
    for line in _rows("ratios_hand_worked.txt"):
        m, g, p, tol = [part.split() for part in line.split("|")]
        st, got = oracle.layer_ratios([float(v) for v in g], [float(v) for v in m])
        assert st == 0
        np.testing.assert_allclose(got, [float(v) for v in p], rtol=0, atol=float(tol[0]))
        n += 1
    assert n >= 4


def test_kept_count_fixture():
    n_rows = 0
    for line in _rows("kept_count_hand_worked.txt"):
        n, p, k = line.split()
        assert oracle.n_keep(int(n), float(p)) == int(k), line
        n_rows += 1
    assert n_rows >= 10


def test_kept_count_properties():
    for n in (1, 2, 31, 1000, 12345, 1 << 20, (1 << 31) - 1):
        assert oracle.n_keep(n, 0.0) == n
        assert oracle.n_keep(n, 1.0) == 0
        prev = n
        for i in range(0, 101):
            k = oracle.n_keep(n, i / 100.0)
            assert 0 <= k <= prev  # monotone non-increasing in p
            prev = k
            # exact rational check: floor(i*n/100) differs from the double product only when
            # i*n/100 sits within rounding of an integer
            exact = n - (i * n) // 100
            assert abs(k - exact) <= 1


def _closed_form(g, m):
    g = np.asarray(g, dtype=np.float64)
    m = np.asarray(m, dtype=np.float64)
    M = np.array([math.log2(m.sum() / v) for v in m])  # base 2 on purpose: the base cancels
    prod = M * g
    return 1.0 - prod / prod.max()


def test_closed_form_and_log_base():
    rng = np.random.default_rng(1)
    for l in (2, 3, 7, 28, 54):
        g = np.exp(rng.standard_normal(l))
        m = rng.integers(1, 1 << 24, size=l).astype(np.float64)
        st, p = oracle.layer_ratios(g, m)
        assert st == 0
        np.testing.assert_allclose(p, _closed_form(g, m), rtol=0, atol=1e-13)
        assert p.min() == 0.0 and p.max() <= 1.0  # the arg-max layer is never pruned
        assert np.all(p >= 0.0)


def test_invariances():
    rng = np.random.default_rng(2)
    l = 11
    g = np.exp(rng.standard_normal(l))
    m = rng.integers(1000, 1 << 22, size=l).astype(np.float64)
    _, p = oracle.layer_ratios(g, m)
    _, p_gs = oracle.layer_ratios(g * 37.5, m)          # scale of G cancels (Eq. 6 normalisation)
    _, p_ms = oracle.layer_ratios(g, m * 4.0)           # unit of size cancels (Eq. 5 is a fraction)
    perm = rng.permutation(l)
    _, p_perm = oracle.layer_ratios(g[perm], m[perm])   # layers are exchangeable
    np.testing.assert_allclose(p_gs, p, rtol=0, atol=1e-13)
    np.testing.assert_allclose(p_ms, p, rtol=0, atol=1e-13)
    np.testing.assert_allclose(p_perm, p[perm], rtol=0, atol=1e-13)


def test_monotone_in_gradient_and_size():
    # Section 4.2: large gradients -> low ratio; large activations -> high ratio.
    g = np.array([1.0, 2.0, 3.0, 5.0])
    m = np.array([4096.0, 1024.0, 2048.0, 512.0])
    _, p0 = oracle.layer_ratios(g, m)
    top = int(np.argmin(p0))
    for i in range(4):
        if i == top:
            continue
        g2 = g.copy()
        g2[i] *= 1.2   # small enough that the arg-max layer stays the same
        _, p1 = oracle.layer_ratios(g2, m)
        if int(np.argmin(p1)) == top:
            assert p1[i] < p0[i]
    # a layer that grows (others fixed) gets a larger ratio relative to an equal-G twin
    g = np.array([1.0, 1.0, 1.0])
    _, pa = oracle.layer_ratios(g, [100.0, 100.0, 50.0])
    _, pb = oracle.layer_ratios(g, [400.0, 100.0, 50.0])
    assert pb[0] > pa[0]
    assert pb[0] > pb[1] > pb[2] == 0.0


def test_deeper_smaller_layers_have_higher_memory_importance():
    # Section 5.4 (visualisation): M rises as the activation shrinks with depth.
    from paper_2503_20354_b200 import workloads as W
    layers = [l for l in W.wrn28_10(200) if l.name.endswith("conv2")]
    m = np.array([l.act_bytes for l in layers], dtype=np.float64)
    _, p = oracle.layer_ratios(np.ones(len(m)), m)
    # with equal G the ratio falls (importance rises) as the size falls
    order = np.argsort(-m, kind="stable")
    assert np.all(np.diff(p[order]) <= 1e-15)


def test_degenerate_inputs():
    st, p = oracle.layer_ratios([3.0], [10.0])         # one layer: M = 0 -> 0/0
    assert st == 3 and p.tolist() == [0.0]
    st, p = oracle.layer_ratios([0.0, 0.0], [1.0, 3.0])  # all G zero
    assert st == 3 and p.tolist() == [0.0, 0.0]
    st, p = oracle.layer_ratios([0.0, 2.0, 1.0], [1.0, 3.0, 3.0])  # one G zero: fully pruned
    assert st == 0 and p[0] == 1.0 and p.min() == 0.0

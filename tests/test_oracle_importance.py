"""Pins for the oracle's Gradient Importance (Eq. 4) and the ablation's ratio-rule variants.

Expected values: a hand-worked fixture, closed forms and identities that follow from the
equations, and numpy's norm as an independent library routine.  None re-types the oracle's loop.
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


def test_hand_worked_importance_examples():
    n = 0
    for line in _rows("gradient_importance_hand_worked.txt"):
        w, g, tol = [part.split() for part in line.split("|")]
        got = oracle.gradient_importance([float(v) for v in w])
        assert abs(got - float(g[0])) <= float(tol[0])
        n += 1
    assert n >= 5


def test_importance_against_library_norm_and_identities():
    rng = np.random.default_rng(4)
    w = rng.standard_normal(10007).astype(np.float32)
    g = oracle.gradient_importance(w)
    ref = np.linalg.norm(w.astype(np.float64)) / math.sqrt(w.size)     # ||w||_2 / sqrt(N)
    assert abs(g - ref) <= 1e-12 * ref
    # scaling by a power of two is exact in fp32: G(a w) = |a| G(w)
    assert oracle.gradient_importance(-4.0 * w) == pytest.approx(4.0 * g, rel=1e-15)
    # a one-hot vector: 1 / sqrt(N); order of the entries does not matter
    e = np.zeros(64, dtype=np.float32); e[17] = 1.0
    assert oracle.gradient_importance(e) == pytest.approx(0.125, abs=0)
    assert oracle.gradient_importance(w[::-1].copy()) == pytest.approx(g, rel=1e-13)
    # two layers joined: N G^2 adds up
    a, b = w[:3000], w[3000:]
    lhs = w.size * g * g
    rhs = a.size * oracle.gradient_importance(a) ** 2 + b.size * oracle.gradient_importance(b) ** 2
    assert lhs == pytest.approx(rhs, rel=1e-12)
    assert oracle.gradient_importance(np.zeros(0, dtype=np.float32)) == 0.0


def test_ratio_rule_variants():
    m = np.array([8.0, 4.0, 2.0, 2.0])
    g = np.array([3.0, 3.0, 1.0, 2.0])
    # rule 0 is Eq. 5-7 as printed
    st0, p0 = oracle.layer_ratios_rule(g, m, oracle.RULE_BOTH)
    st, p = oracle.layer_ratios(g, m)
    assert st0 == st == 0 and np.array_equal(p0, p)
    # "w/o M": p_i = 1 - G_i / max G, whatever the sizes
    st, p = oracle.layer_ratios_rule(g, m, oracle.RULE_NO_MEMORY)
    np.testing.assert_allclose(p, [0.0, 0.0, 2.0 / 3.0, 1.0 / 3.0], rtol=0, atol=1e-15)
    st, p2 = oracle.layer_ratios_rule(g, m[::-1].copy(), oracle.RULE_NO_MEMORY)
    assert np.array_equal(p, p2)
    # "w/o G": fractions (1/2,1/4,1/8,1/8) -> M = (1,2,3,3) ln 2 -> p = (2/3, 1/3, 0, 0), whatever G
    st, p = oracle.layer_ratios_rule(g, m, oracle.RULE_NO_GRADIENT)
    np.testing.assert_allclose(p, [2.0 / 3.0, 1.0 / 3.0, 0.0, 0.0], rtol=0, atol=1e-12)
    st, p2 = oracle.layer_ratios_rule(g[::-1].copy(), m, oracle.RULE_NO_GRADIENT)
    assert np.array_equal(p, p2)
    # equal sizes: "w/o G" prunes nothing
    st, p = oracle.layer_ratios_rule(g, np.full(4, 5.0), oracle.RULE_NO_GRADIENT)
    assert st == 0 and not p.any()
    # static: the same ratio everywhere
    st, p = oracle.layer_ratios_rule(g, m, oracle.RULE_STATIC, 0.8)
    assert st == 0 and np.array_equal(p, np.full(4, 0.8))
    # the product rule is the product of the one-factor importances: 1 - p0 = (1 - pG)(1 - pM) / max
    _, pm = oracle.layer_ratios_rule(g, m, oracle.RULE_NO_GRADIENT)
    _, pg = oracle.layer_ratios_rule(g, m, oracle.RULE_NO_MEMORY)
    prod = (1 - pm) * (1 - pg)
    np.testing.assert_allclose(1 - p0, prod / prod.max(), rtol=1e-12, atol=1e-15)
    # every gradient zero: Eq. 7 is 0/0 for the rules that use G
    st, p = oracle.layer_ratios_rule(np.zeros(4), m, oracle.RULE_NO_MEMORY)
    assert st == 3 and not p.any()

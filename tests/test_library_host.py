"""CPU-side checks of libsurgeon.so: it builds for sm_100a, loads, exports every symbol that
include/surgeon.h declares, and its host-only entry points (ratio rule, size arithmetic, argument
checks) agree with the oracle.  No kernel is launched here."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2503_20354_b200 import binding as B
from paper_2503_20354_b200 import build as lib_build
from paper_2503_20354_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    lib_build.build()


def test_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "surgeon.h")).read()
    names = set(re.findall(r"\b(surgeon_[a-z_0-9]+)\s*\(", text))
    assert {"surgeon_layer_ratios", "surgeon_compact_sizes", "surgeon_prune_compact",
            "surgeon_weight_grad", "surgeon_weight_grad_workspace", "surgeon_decompress",
            "surgeon_status_string", "surgeon_layer_ratios_rule",
            "surgeon_gradient_importance"} <= names
    l = ctypes.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(l, n), n


def test_struct_layouts_match_header():
    assert ctypes.sizeof(B.Header) == 32
    assert ctypes.sizeof(B.Compressed) == 48
    assert ctypes.sizeof(B.LayerDesc) == 48


def test_ratios_match_oracle_and_fixture():
    st, p = oracle.layer_ratios([2, 1, 4], [4, 2, 2])
    got = B.surgeon_layer_ratios([2, 1, 4], [4, 2, 2])
    assert got.tolist() == [0.75, 0.75, 0.0] == p.tolist()
    rng = np.random.default_rng(4)
    for layers in (W.wrn28_10(), W.resnet50(), W.vit_b16()):
        gi = W.gradient_importance(len(layers), seed=0)
        lam = np.array([l.act_bytes for l in layers], dtype=np.float64)
        _, ref = oracle.layer_ratios(gi, lam)
        np.testing.assert_allclose(B.surgeon_layer_ratios(gi, lam), ref, rtol=0, atol=1e-14)


def test_ratios_errors():
    with pytest.raises(B.SurgeonError) as e:
        B.surgeon_layer_ratios([1.0], [5.0])
    assert e.value.status == B.SURGEON_ERR_DEGENERATE
    assert B.surgeon_layer_ratios([1.0], [5.0], allow_degenerate=True).tolist() == [0.0]
    for gi, lam in (([1.0, -1.0], [1.0, 1.0]), ([1.0, np.nan], [1.0, 1.0]), ([1.0, 1.0], [0.0, 1.0]),
                    ([1.0, 1.0], [np.inf, 1.0])):
        with pytest.raises(B.SurgeonError) as e:
            B.surgeon_layer_ratios(gi, lam)
        assert e.value.status == B.SURGEON_ERR_INVALID_ARG


def test_ratio_rule_variants_match_oracle():
    for layers in (W.wrn28_10(), W.resnet50(), W.vit_b16()):
        gi = W.gradient_importance(len(layers), seed=1)
        lam = np.array([l.act_bytes for l in layers], dtype=np.float64)
        for rule in (oracle.RULE_BOTH, oracle.RULE_NO_GRADIENT, oracle.RULE_NO_MEMORY):
            _, ref = oracle.layer_ratios_rule(gi, lam, rule)
            np.testing.assert_allclose(B.surgeon_layer_ratios_rule(gi, lam, rule), ref, rtol=0, atol=1e-14)
        _, ref = oracle.layer_ratios_rule(gi, lam, oracle.RULE_STATIC, 0.9)
        assert np.array_equal(B.surgeon_layer_ratios_rule(gi, lam, B.SURGEON_RULE_STATIC, 0.9), ref)
    # the factor that is left out need not be passed
    np.testing.assert_allclose(B.surgeon_layer_ratios_rule(None, [8, 4, 2, 2], B.SURGEON_RULE_NO_GRADIENT),
                               [2 / 3, 1 / 3, 0, 0], rtol=0, atol=1e-12)
    np.testing.assert_allclose(B.surgeon_layer_ratios_rule([3, 3, 1, 2], None, B.SURGEON_RULE_NO_MEMORY),
                               [0, 0, 2 / 3, 1 / 3], rtol=0, atol=1e-15)
    for args in (([1.0, 2.0], [1.0, 1.0], 7, 0.0), ([1.0, 2.0], [1.0, 1.0], B.SURGEON_RULE_STATIC, 1.5),
                 (None, [1.0, 1.0], B.SURGEON_RULE_NO_MEMORY, 0.0), ([1.0, -2.0], None, B.SURGEON_RULE_NO_MEMORY, 0.0)):
        with pytest.raises(B.SurgeonError) as e:
            B.surgeon_layer_ratios_rule(*args)
        assert e.value.status == B.SURGEON_ERR_INVALID_ARG
    with pytest.raises(B.SurgeonError) as e:
        B.surgeon_layer_ratios_rule([0.0, 0.0], None, B.SURGEON_RULE_NO_MEMORY)
    assert e.value.status == B.SURGEON_ERR_DEGENERATE


def test_compact_sizes_match_oracle_kept_count():
    for n in (0, 1, 31, 32, 33, 1023, 1024, 1025, 1 << 20, 12345677, (1 << 31) - 1):
        for ratio in (0.0, 0.1, 0.3, 0.5, 0.6, 0.9, 0.99, 1.0):
            for dt, es in ((B.SURGEON_F32, 4), (B.SURGEON_BF16, 2)):
                s = B.surgeon_compact_sizes(n, dt, ratio)
                assert s.n_keep == oracle.n_keep(n, ratio)
                assert s.bitmap_bytes == 4 * ((n + 31) // 32)
                assert s.values_bytes == s.n_keep * es
                assert s.offsets_bytes == 4 * ((n + 127) // 128 + 1)
                assert s.workspace_bytes > 0 and s.workspace_bytes % 256 == 0
    for bad in ((-1, 0, 0.5), (10, 0, 1.5), (10, 0, -0.1), (10, 2, 0.5), (10, 0, float("nan"))):
        with pytest.raises(B.SurgeonError) as e:
            B.surgeon_compact_sizes(*bad)
        assert e.value.status == B.SURGEON_ERR_INVALID_ARG
    with pytest.raises(B.SurgeonError) as e:
        B.surgeon_compact_sizes(1 << 31, 0, 0.5)
    assert e.value.status == B.SURGEON_ERR_UNSUPPORTED


def test_argument_checks_need_no_device():
    l = B.lib()
    comp = B.Compressed(16, 0, 0, 0, 0, 0, 0)
    assert l.surgeon_prune_compact(0, 16, 0, 0.5, ctypes.byref(comp), 0, 0, 0) == B.SURGEON_ERR_INVALID_ARG
    assert l.surgeon_prune_compact(0, 16, 0, 2.0, ctypes.byref(comp), 0, 0, 0) == B.SURGEON_ERR_INVALID_ARG
    d = B.LayerDesc(1, 2, 3, 8, 8, 4, 3, 3, 1, 1, 1)
    assert B.surgeon_weight_grad_workspace(d) > 0
    bad = B.LayerDesc(0, 2, 3, 8, 8, 4, 3, 3, 1, 1, 1)     # linear with a spatial extent
    assert B.surgeon_weight_grad_workspace(bad) == 0
    assert l.surgeon_weight_grad(ctypes.byref(comp), ctypes.byref(bad), 16, 16, 0, 0, 0, 0) == B.SURGEON_ERR_INVALID_ARG
    assert B.status_string(B.SURGEON_ERR_TIMEOUT).startswith("device-side")

"""Child process of test_cta_pairs: the tensor-core weight gradient with CTA pairs switched on
(the switch is read once per process), checked against the fp64 oracle."""
import os
import sys

os.environ["SURGEON_DW_PAIRS"] = "1"
sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from dataclasses import replace  # noqa: E402

from paper_2503_20354_b200 import binding as B  # noqa: E402
from paper_2503_20354_b200 import workloads as W  # noqa: E402
from gpu_util import rel_frobenius  # noqa: E402
from test_gpu_weight_grad import run_layer  # noqa: E402

SHAPES = [
    W.linear("pair_lin", 3 * 64 + 17, 256, 768, dist="normal", dt=W.F32),       # two row tiles
    W.linear("pair_lin_odd_tiles", 200, 264, 520, dist="gelu_normal", dt=W.F32),  # three, padded to four
    W.conv("pair_1x1", 3, 136, 14, 264, 1, 1, 0),
    W.conv("pair_1x1_s2", 2, 264, 28, 72, 1, 2, 0),
    W.conv("pair_3x3_w8", 4, 160, 8, 160, 3),                                    # row-shifted taps
    W.conv("pair_3x3_hw14", 2, 136, 14, 72, 3),                                  # nine tap copies
]

for layer in SHAPES:
    for bf16 in (False, True):
        lay = replace(layer, dt=W.BF16 if bf16 else W.F32)
        for ratio in (0.0, 0.7):
            dw, ref, _, _ = run_layer(lay, ratio, B.PATH_TENSOR_CORE, seed=5)
            err = rel_frobenius(dw, ref)
            assert err <= 5e-3, (lay.name, bf16, ratio, err)
print("PAIRS_OK")

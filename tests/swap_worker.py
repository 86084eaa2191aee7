"""Child process of test_exchanged_roles_on_cta_pairs: the tensor-core weight gradient on CTA pairs
with the operand roles exchanged (gradient rows as MMA M, input channels as the N operand both CTAs
rebuild a half of), switched on for this process, checked against the fp64 oracle."""
import os
import sys

os.environ["SURGEON_DW_SWAP"] = "1"
sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from dataclasses import replace  # noqa: E402

from paper_2503_20354_b200 import binding as B  # noqa: E402
from paper_2503_20354_b200 import workloads as W  # noqa: E402
from gpu_util import rel_frobenius  # noqa: E402
from test_gpu_weight_grad import run_layer  # noqa: E402

SHAPES = [
    W.linear("swap_lin_c256", 3 * 64 + 17, 256, 768, dist="normal", dt=W.F32),   # 128 channels per CTA, K tail
    W.linear("swap_lin_c128_o520", 200, 128, 520, dist="gelu_normal", dt=W.F32),  # gradient columns past the last unit
    W.conv("swap_1x1", 3, 136, 14, 264, 1, 1, 0),                                  # 264 = 2 * 128 + 8: remainder boxes
    W.conv("swap_1x1_o96", 4, 40, 14, 96, 1, 1, 0),
    W.conv("swap_3x3_w8_o160", 4, 160, 8, 160, 3),                                 # row-shifted taps, 128 + 32 rows per tap
    W.conv("swap_3x3_w16_o320", 2, 64, 16, 320, 3),                                # 2 * 128 + 64 rows per tap
    W.conv("swap_3x3_hw14", 2, 136, 14, 72, 3),                                    # nine tap copies, 72 -> boxes of 128 rows, partly filled
    W.conv("swap_3x3_w32_o64", 2, 64, 32, 64, 3),                                  # two taps to an accumulator
]

for layer in SHAPES:
    for bf16 in (False, True):
        lay = replace(layer, dt=W.BF16 if bf16 else W.F32)
        for ratio in (0.0, 0.7):
            dw, ref, _, _ = run_layer(lay, ratio, B.PATH_TENSOR_CORE, seed=5)
            err = rel_frobenius(dw, ref)
            assert err <= 5e-3, (lay.name, bf16, ratio, err)
print("SWAP_OK")

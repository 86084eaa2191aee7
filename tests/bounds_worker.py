"""Worker of test_gpu_bounds_build.py: runs in a process whose SURGEON_LIB names the checked build
(-DSURGEON_BOUNDS: every guarded global store tests its index against the buffer size the host
computed).  A small list of shapes goes through prune+compact and both weight-gradient paths; the
results must match the oracle and no status word may report an index out of bounds."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import numpy as np
import torch

import oracle
from paper_2503_20354_b200 import binding as B
from paper_2503_20354_b200 import workloads as W
from gpu_util import assert_store_equals_oracle, oracle_dw, rel_frobenius


def main():
    assert B.LIB_PATH.endswith("libsurgeon_bounds.so"), B.LIB_PATH
    shapes = [W.conv("c3x3", 3, 40, 16, 72, 3), W.conv("c3x3_s2", 3, 24, 16, 40, 3, 2),
              W.conv("c1x1", 4, 40, 14, 96, 1, 1, 0), W.conv("c1x1_s2", 2, 72, 28, 136, 1, 2, 0),
              W.conv("stem", 2, 3, 32, 16, 7, 2, 3, dist="normal"), W.conv("c3x3_hw7", 5, 32, 7, 48, 3),
              W.linear("tokens", 2 * 197, 256, 200, dist="normal", dt=W.F32),
              W.linear("odd", 37, 24, 40, dist="normal", dt=W.F32)]
    for bf16 in (False, True):
        for layer in shapes:
            from dataclasses import replace
            layer = replace(layer, dt=W.BF16 if bf16 else W.F32)
            a, g = W.activation(layer, seed=9), W.grad_out(layer, seed=9)
            for ratio in (0.0, 0.8):
                comp, ref = assert_store_equals_oracle(a.reshape(-1), ratio)
                pruned = oracle.decompress(ref["bitmap"], ref["values"], layer.n_act)
                want = oracle_dw(layer, pruned, g.numpy())
                for path, tol in ((B.PATH_FP32, 1e-5), (B.PATH_TENSOR_CORE, 5e-3)):
                    desc = B.layer_desc(layer, path)
                    ws = torch.zeros(max(B.surgeon_weight_grad_workspace(desc), 256), dtype=torch.uint8, device="cuda")
                    dw = B.surgeon_weight_grad(comp, desc, g.cuda(), workspace=ws).cpu().numpy()
                    assert rel_frobenius(dw, want) <= tol, (layer.name, ratio, path)
                    if path == B.PATH_TENSOR_CORE:       # its scratch starts with the status word
                        assert int(ws[:4].view(torch.int32)[0]) == 0, "scratch status word"
                assert comp.read_header().status == 0
    # streamed select / compaction at a size with a ragged tail
    for bf16 in (False, True):
        x = W.draw("relu_normal", (1 << 23) + 4321, seed=9)
        assert_store_equals_oracle(x.to(torch.bfloat16) if bf16 else x, 0.6)
    print("BOUNDS_OK")


if __name__ == "__main__":
    main()

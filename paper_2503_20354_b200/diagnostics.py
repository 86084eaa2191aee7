"""Clock stamps of the tensor-core weight-gradient kernels: where a K-tile's time goes.

Builds an instrumented copy of the library (-DSURGEON_DW_STATS: the thread that issues the MMAs
stamps the clock around its two waits - for the gradient tile, which TMA delivers, and for the
activation tile, which the producer warps rebuild - and, in the kernel on CTA pairs, a producer
warp stamps its phases) next to the ordinary one, runs one layer of a bench workload through it and
prints the averages per K-tile.  The instrumented copy does the same work as the ordinary build;
its timings are a few per cent slower.

  python -m paper_2503_20354_b200.diagnostics [--workload wrn28|vit|resnet50] [--layer NAME]
                                              [--ratio P] [--swap]
"""
from __future__ import annotations

import argparse
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)


def build_instrumented() -> str:
    from paper_2503_20354_b200 import build as lib_build
    lib = os.path.join(HERE, "libsurgeon_stats.so")
    deps = lib_build.sources()
    if os.path.exists(lib) and all(os.path.getmtime(p) <= os.path.getmtime(lib) for p in deps):
        return lib
    flags = [f for f in lib_build.NVCC_FLAGS if not f.startswith("--use_fast_math")] + ["-DSURGEON_DW_STATS"]
    cmd = [os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")] + flags + [
        "-I", os.path.join(ROOT, "include"), "-I", lib_build.CSRC] + deps + ["-o", lib]
    subprocess.check_call(cmd)
    return lib


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="vit", choices=["wrn28", "vit", "resnet50"])
    ap.add_argument("--layer", default=None)
    ap.add_argument("--ratio", type=float, default=0.7)
    ap.add_argument("--swap", action="store_true", help="the kernel on CTA pairs with exchanged operand roles")
    args = ap.parse_args()
    os.environ["SURGEON_LIB"] = build_instrumented()
    if args.swap:
        os.environ["SURGEON_DW_SWAP"] = "1"
    if ROOT not in sys.path:
        sys.path.insert(0, ROOT)
    import torch
    from paper_2503_20354_b200 import binding as B
    from paper_2503_20354_b200 import workloads as W
    stack = {"wrn28": W.wrn28_10, "vit": W.vit_b16, "resnet50": W.resnet50}[args.workload]()
    name = args.layer or {"wrn28": "g3b1.conv1", "vit": "blk0.qkv", "resnet50": "layer3.1.conv2"}[args.workload]
    layer = next(l for l in stack if l.name == name)
    a = W.activation(layer, 0, device="cuda")
    g = W.grad_out(layer, 0, device="cuda")
    comp = B.surgeon_prune_compact(a, args.ratio)
    desc = B.layer_desc(layer, B.PATH_TENSOR_CORE)
    ws = torch.zeros(B.surgeon_weight_grad_workspace(desc), dtype=torch.uint8, device="cuda")
    dw = torch.empty(layer.dw_shape, device="cuda")
    for _ in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        B.surgeon_weight_grad(comp, desc, g, dw=dw, workspace=ws)
        e1.record()
        e1.synchronize()
    st = ws[:256].view(torch.int64).cpu().tolist()
    wait_g, wait_a, total, n_kt = st[4:8]
    print("%s %s, ratio %.2f: whole call %.1f us" % (args.workload, name, args.ratio, e0.elapsed_time(e1) * 1e3))
    if n_kt == 0:
        print("  no stamps: this layer runs a kernel without them")
        return
    print("  issuing thread, clocks per K-tile: total %.0f = wait for the gradient tile %.0f + wait for the "
          "activation tile %.0f + issue (MMA back-pressure) %.0f" % (total / n_kt, wait_g / n_kt, wait_a / n_kt,
                                                                      (total - wait_g - wait_a) / n_kt))
    if args.swap and st[10]:
        ph = [x / n_kt for x in st[17:23]]
        print("  producer warp, clocks per K-tile (times the number of groups = per tile): metadata fetch %.0f | "
              "pack %.0f | wait for a free stage %.0f | stores %.0f | loads of the next tile %.0f | proxy fence + arrive %.0f"
              % tuple(ph))


if __name__ == "__main__":
    main()

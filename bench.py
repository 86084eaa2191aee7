#!/usr/bin/env python
"""Benchmark of the dynamic-activation-sparsity hot path on B200.

One step = one pass of the whole path over one batch of a layer stack: per-layer ratios (Eq. 5-7),
prune+compact of every saved activation (Algorithm 1: prune and decompose steps), and the weight
gradient of every layer from its compressed store (its Reshape and gradient steps).  Prints ONE
JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload all|vit|wrn28|resnet50|resnet50_uniform|resnext29|tiny|segformer|sweep]
                  [--batch B] [--path tc|fp32]

The default workload `all` runs, in one process, the ViT-B/16-shaped stack (the headline: `value`,
`ms_per_step`, `roofline`, `e2e` and `cpu_baseline` are its figures), the WideResNet-28-10-shaped
and ResNet-50-shaped stacks (the latter with ratios from Eq. 5-7 and with ratios drawn uniformly
in [0.5, 0.95]) and the largest tensors of the prune+compact bandwidth sweep; every one of them
reports under `workloads` with a roofline entry for prune+compact (HBM) and one for the weight
gradient (tensor cores).

N > 1 (launched with torch.distributed.run): every rank runs an independent replica of the
step on its own GPU (the path has no exchange step); time is the max over ranks.
`--impl reference` times the CPU oracle on a bounded sample of the headline workload (rank 0 only).
"""
from __future__ import annotations

import argparse
import glob
import hashlib
import json
import os
import re
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

METRIC = "prune+compact GB/s and sparse-act dW TFLOP/s, as % of B200 HBM/tensor peak"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL = {"hbm_gbs": 7700.0, "bf16_tflops": 2250.0}
# fp32 CUDA-core peak for the fp32 path: 148 SMs x 128 FMA lanes x 2 flop x 1.965 GHz
FP32_ALU_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12
HEADLINE = "vit"


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


def kernel_sources_hash() -> str:
    """Hash of the CUDA sources: DRAM counters taken under ncu hold for the kernels as they were."""
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2503_20354_b200", "csrc")
    for p in sorted(glob.glob(os.path.join(csrc, "*.cu")) + glob.glob(os.path.join(csrc, "*.cuh"))):
        with open(p, "rb") as f:
            h.update(os.path.basename(p).encode() + b"\0" + f.read())
    return h.hexdigest()[:16]


def recorded_traffic(workload: str, part: str):
    """DRAM bytes per step (dram__bytes_read.sum + dram__bytes_write.sum over the launches of one
    step, from an ncu capture) that `profiles/dram_traffic_per_step.md` records for this workload
    and part ("prune_compact" / "weight_grad"); None when there is no record or the kernels'
    sources have changed since the counters were taken."""
    p = os.path.join(ROOT, "profiles", "dram_traffic_per_step.md")
    if not os.path.exists(p):
        return None
    text = open(p).read()
    m = re.search(r"sources hash:\s*`?([0-9a-f]{16})`?", text)
    if not m or m.group(1) != kernel_sources_hash():
        return None
    m = re.search(r"^\|\s*%s\s*\|\s*%s\s*\|\s*([0-9]+)\s*\|" % (re.escape(workload), re.escape(part)), text, re.M)
    return int(m.group(1)) if m else None


def get_layers(workload: str, batch):
    from paper_2503_20354_b200 import workloads as W
    if workload == "wrn28":
        return W.wrn28_10(batch or 200), "WideResNet-28-10-shaped stack, 32x32, batch %d, fp32 activations" % (batch or 200)
    if workload == "tiny":
        return W.tiny_conv(batch or 16), "tiny conv 3x3 64->64 on [%d,64,32,32] fp32" % (batch or 16)
    if workload in ("resnet50", "resnet50_uniform"):
        return W.resnet50(batch or 64), "ResNet-50-shaped stack, 224x224, batch %d, bf16 activations" % (batch or 64)
    if workload == "vit":
        return W.vit_b16(batch or 64), "ViT-B/16-shaped stack, batch %d, bf16 activations" % (batch or 64)
    if workload == "resnext29":
        return W.resnext29(batch or 200), "ResNeXt-29 (32x4d)-shaped stack, 32x32, batch %d, fp32 activations, grouped 3x3 convolutions" % (batch or 200)
    if workload == "segformer":
        return W.segformer_b5(1024, batch or 1), "blocks of a Segformer-B5-shaped encoder (linear layers, reduction and depthwise convolutions), 1024x1024, batch %d, bf16 activations" % (batch or 1)
    raise SystemExit("unknown workload %r" % workload)


# output-gradient scale per workload (the tiny and WideResNet configs: 0.01; ResNet-50 / ViT: 1e-3)
SIGMA = {"wrn28": 0.01, "tiny": 0.01, "segformer": 0.01, "resnext29": 0.01, "resnet50": 1e-3, "resnet50_uniform": 1e-3, "vit": 1e-3}


def prune_alg_bytes(layer, n_keep: int) -> int:
    """Algorithmic bytes of prune+compact: two reads of the tensor (one to find the threshold,
    one to emit), the bitmap, the packed values and the block offsets."""
    es = 4 if layer.dt == 0 else 2
    n = layer.n_act
    return 2 * n * es + (n + 7) // 8 + n_keep * es + 4 * ((n + 127) // 128 + 1)


def dw_min_bytes(layer, n_keep: int) -> int:
    """Least bytes the weight gradient of a layer moves: the fp32 output gradient once, the
    compressed store once, the fp32 weight gradient once."""
    es = 4 if layer.dt == 0 else 2
    n = layer.n_act
    store = n_keep * es + (n + 7) // 8 + 4 * ((n + 127) // 128 + 1)
    return 4 * int(np.prod(layer.grad_shape)) + store + 4 * layer.n_weight


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.lines, self.proc, self.idx = [], None, device_index
        self.nvml, self.samples, self.stop_flag, self.t = None, [], False, None

    def _nvml_loop(self):
        n = self.nvml
        h = self.handle
        while not self.stop_flag:
            try:
                sm = n.nvmlDeviceGetClockInfo(h, n.NVML_CLOCK_SM)
                mx = n.nvmlDeviceGetMaxClockInfo(h, n.NVML_CLOCK_SM)
                try:
                    r = n.nvmlDeviceGetCurrentClocksEventReasons(h)
                except Exception:
                    r = n.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                self.samples.append((sm, mx, int(r)))
            except Exception:
                pass
            time.sleep(0.01)

    def start(self):
        # NVML in a thread (a sample every 10 ms, reading only); nvidia-smi as the fall-back
        try:
            import pynvml
            pynvml.nvmlInit()
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            if vis and not vis.split(",")[self.idx].isdigit():
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(vis.split(",")[self.idx])
            else:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(int(vis.split(",")[self.idx]) if vis else self.idx)
            self.nvml = pynvml
            self.t = threading.Thread(target=self._nvml_loop, daemon=True)
            self.t.start()
            return
        except Exception:
            self.nvml = None
        try:
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            idx = vis.split(",")[self.idx] if vis else str(self.idx)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", idx, "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        if self.nvml is not None:
            self.stop_flag = True
            self.t.join(timeout=2)
            bits = {"sw_power_cap": 0x4, "hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20,
                    "hw_thermal_slowdown": 0x40}
            reasons = sorted(k for k, b in bits.items() if any(r & b for _, _, r in self.samples))
            sm = [x[0] for x in self.samples]
            mx = [x[1] for x in self.samples]
            return {"sm_mhz": float(np.median(sm)) if sm else None,
                    "sm_max_mhz": float(max(mx)) if mx else None,
                    "samples": len(sm), "reasons": reasons, "source": "nvml, 10 ms"}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for l in self.lines:
            f = [v.strip() for v in l.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(mx)) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons), "source": "nvidia-smi, 100 ms"}


def dist_setup(n_gpus: int):
    """(rank, world, device).  One process per GPU; rendezvous from the torchrun environment."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        if torch.cuda.is_available():
            torch.cuda.set_device(local)
        dist.init_process_group(backend=backend)
    elif torch.cuda.is_available():
        torch.cuda.set_device(0)
    return rank, world, local


def max_over_ranks(value: float, world: int, device) -> float:
    """Max of a per-rank scalar (the job's time is its slowest rank's)."""
    if world == 1:
        return float(value)
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


# ------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------

class Stack:
    """Device-resident inputs, stores, outputs and scratch of one replica of the workload."""

    def __init__(self, layers, path: int, seed: int, device, n_streams=1, sigma=0.01, ratios="rule", share=True):
        from paper_2503_20354_b200 import binding as B
        from paper_2503_20354_b200 import workloads as W
        self.B, self.layers, self.path, self.device = B, layers, path, device
        self.gi = W.gradient_importance(len(layers), seed)
        self.lam = np.array([l.act_bytes for l in layers], dtype=np.float64)
        if isinstance(ratios, str):
            self.fixed_ratios = W.uniform_ratios(len(layers), seed) if ratios == "uniform" else None
        else:                       # given per layer (a profiling subset keeps the whole stack's ratios)
            self.fixed_ratios = np.asarray(ratios, dtype=np.float64)
        # A residual block's shortcut convolution reads the same tensor as the block's first
        # convolution: that tensor is pruned once, at the smaller of the two layers' ratios (the
        # one that keeps more), and both weight gradients read the one store.
        self.shared = W.shared_inputs(layers) if share else {}
        self.x = [None if i in self.shared else W.activation(l, seed, i, device=device) for i, l in enumerate(layers)]
        for j, i in self.shared.items():
            self.x[j] = self.x[i]
        self.g = [W.grad_out(l, seed, i, sigma=sigma, device=device) for i, l in enumerate(layers)]
        self.desc = [B.layer_desc(l, path) for l in layers]
        self.dw = [torch.empty(l.dw_shape, dtype=torch.float32, device=device) for l in layers]
        # stores sized for ratio 0: ratios change every batch, the buffers do not
        self.store = [None if i in self.shared else B.CompressedActivation(l.n_act, l.dt, 0.0, device)
                      for i, l in enumerate(layers)]
        for j, i in self.shared.items():
            self.store[j] = self.store[i]
        ws1 = max(s.sizes.workspace_bytes for s in self.store)
        self.own = [i for i in range(len(layers)) if i not in self.shared]    # layers that prune their input
        ws2 = max(B.surgeon_weight_grad_workspace(d) for d in self.desc)
        # Layers are independent of one another (a layer's store is written once in the forward
        # pass and read once in the backward pass), so they are issued round-robin on n_streams
        # streams, each with its own scratch: the short dependent kernels of one layer overlap
        # with those of its neighbours.  Both loops fork from and join the caller's stream.
        self.n_streams = max(1, int(n_streams))
        self.streams = [torch.cuda.Stream(device=device) for _ in range(self.n_streams)] if self.n_streams > 1 else []
        self.ws = [torch.empty(max(ws1, ws2, 256), dtype=torch.uint8, device=device)
                   for _ in range(self.n_streams)]
        self.ratios = None

    def _fork(self):
        main = torch.cuda.current_stream(self.device)
        for st in self.streams:
            st.wait_stream(main)

    def _join(self):
        main = torch.cuda.current_stream(self.device)
        for st in self.streams:
            main.wait_stream(st)

    def stream_of(self, k):
        return self.streams[k] if self.streams else None

    def compute_ratios(self):
        if self.fixed_ratios is not None:
            self.ratios = self.fixed_ratios
        else:
            self.ratios = self.B.surgeon_layer_ratios(self.gi, self.lam, allow_degenerate=True)   # Eq. 5-7
        if self.shared:
            self.ratios = np.array(self.ratios, dtype=np.float64)
            for j, i in self.shared.items():
                self.ratios[i] = self.ratios[j] = min(self.ratios[i], self.ratios[j])
        return self.ratios

    def step(self, ev=None, x_ready=None, g_ready=None, dw_done=None):
        """One pass.  `ev`: three events (start, after the forward loop, end).  The host-buffer leg
        passes per-layer events: a layer's prune waits for x_ready[i], its weight gradient for
        g_ready[i], and dw_done[i] is recorded after it."""
        B = self.B
        if ev: ev[0].record()
        self.compute_ratios()
        self._fork()
        for n, i in enumerate(self.own):                                                 # forward
            k = n % self.n_streams
            st = self.stream_of(k)
            if x_ready is not None:
                (st or torch.cuda.current_stream(self.device)).wait_event(x_ready[i])
            B.surgeon_prune_compact(self.x[i], float(self.ratios[i]), out=self.store[i], workspace=self.ws[k],
                                    stream=st)
        self._join()
        if ev: ev[1].record()
        self._fork()
        for j, i in enumerate(reversed(range(len(self.layers)))):                        # backward
            k = j % self.n_streams
            st = self.stream_of(k)
            if g_ready is not None:
                (st or torch.cuda.current_stream(self.device)).wait_event(g_ready[i])
            B.surgeon_weight_grad(self.store[i], self.desc[i], self.g[i], dw=self.dw[i], workspace=self.ws[k],
                                  stream=st)
            if dw_done is not None:
                dw_done[i].record(st or torch.cuda.current_stream(self.device))
        self._join()
        if ev: ev[2].record()

    def per_layer_dw_us(self, reps=3):
        """Each layer's weight gradient alone on the GPU (one stream, L2 not flushed: a layer's
        gradient alone exceeds L2 on the large layers), median of `reps`."""
        B = self.B
        out = []
        for i in range(len(self.layers)):
            ts = []
            for _ in range(reps + 1):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                B.surgeon_weight_grad(self.store[i], self.desc[i], self.g[i], dw=self.dw[i], workspace=self.ws[0])
                e1.record()
                e1.synchronize()
                ts.append(e0.elapsed_time(e1) * 1e3)
            out.append(float(np.median(ts[1:])))
        return out


def frac_entry(kind, achieved, peaks, path_tc=True, traffic=None, extra=None):
    """A roofline entry.  HBM: against the measured copy bandwidth.  Tensor: against the measured
    burst cuBLAS bf16 rate (a timed region of a fraction of a second runs at full clock, before
    the power cap settles), with the sustained and the nominal fractions beside it."""
    if kind == "hbm":
        peak = float(peaks["hbm_gbs"])
        d = {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
             "frac": round(achieved / peak, 4), "traffic": traffic,
             "peak_source": peaks["_source"] + " copy bandwidth",
             "frac_nominal": round(achieved / NOMINAL["hbm_gbs"], 4)}
    elif path_tc:
        peak = float(peaks["bf16_tflops"])
        sus = float(peaks.get("bf16_tflops_sustained", peak))
        d = {"bound": "tensor", "achieved": round(achieved, 3), "peak": round(peak, 1), "unit": "TFLOP/s",
             "frac": round(achieved / peak, 4), "traffic": traffic,
             "peak_source": peaks["_source"] + " bf16 cuBLAS, burst",
             "frac_sustained": round(achieved / sus, 4), "peak_sustained": round(sus, 1),
             "frac_nominal": round(achieved / NOMINAL["bf16_tflops"], 4)}
    else:
        d = {"bound": "alu", "achieved": round(achieved, 3), "peak": round(FP32_ALU_TFLOPS, 1), "unit": "TFLOP/s",
             "frac": round(achieved / FP32_ALU_TFLOPS, 4), "traffic": traffic,
             "peak_source": "derived: 148 SMs x 128 fp32 FMA lanes x 2 x 1.965 GHz"}
    if extra:
        d.update(extra)
    return d


def run_stack(key, args, rank, world, device, peaks, path, keep_stack=False, sampler=None):
    """Times one layer stack; returns (result dict, stack or None).  `sampler` records the clocks
    during the timed region."""
    from paper_2503_20354_b200 import binding as B
    layers, desc_text = get_layers(key, args.batch)
    uniform = key == "resnet50_uniform"
    recipe = "uniform" if uniform else "rule"
    if args.layers:      # profiling aid: keep only the named layers of the stack, at the ratios they have in the whole stack
        from paper_2503_20354_b200 import binding as B
        from paper_2503_20354_b200 import workloads as W
        keep = set(args.layers.split(","))
        idx = [i for i, l in enumerate(layers) if l.name in keep]
        if not idx:
            raise SystemExit("--layers names no layer of the stack")
        if uniform:
            full = np.asarray(W.uniform_ratios(len(layers), args.seed + rank), dtype=np.float64)
        else:
            full = np.asarray(B.surgeon_layer_ratios(W.gradient_importance(len(layers), args.seed + rank),
                                                     np.array([l.act_bytes for l in layers], dtype=np.float64),
                                                     allow_degenerate=True), dtype=np.float64)
        for j, i in W.shared_inputs(layers).items():
            full[i] = full[j] = min(full[i], full[j])
        recipe = full[idx]
        layers = [layers[i] for i in idx]
        desc_text += " (layers %s only)" % args.layers
    stack = Stack(layers, path, args.seed + rank, device, n_streams=args.streams, sigma=SIGMA[key],
                  ratios=recipe)
    torch.cuda.synchronize()
    for _ in range(args.warmup):
        stack.step()
    torch.cuda.synchronize()
    barrier(world)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    launches0 = B.surgeon_launch_count()
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    if sampler is not None:
        sampler.start()
    t_begin.record()
    for s in range(args.steps):
        stack.step(evs[s])
    t_end.record()
    torch.cuda.synchronize()
    barrier(world)
    launches = B.surgeon_launch_count() - launches0
    if sampler is not None:
        res_clocks = sampler.stop()
    total_ms = max_over_ranks(t_begin.elapsed_time(t_end), world, device)
    prune_ms = sum(e[0].elapsed_time(e[1]) for e in evs) / args.steps
    dw_ms = sum(e[1].elapsed_time(e[2]) for e in evs) / args.steps
    ms_per_step = total_ms / args.steps
    # device-side status of every store (one small read per layer, outside the timed region)
    for s in stack.store:
        h = s.read_header()
        if h.status != 0:
            raise SystemExit("device status %d in a compressed store" % h.status)
    flops = sum(l.flops for l in layers)
    own = stack.own                      # a tensor two layers read is pruned and stored once
    pbytes = sum(prune_alg_bytes(layers[i], stack.store[i].sizes.n_keep) for i in own)
    stored = sum(stack.store[i].stored_bytes for i in own)
    dense = sum(layers[i].act_bytes for i in own)
    prune_gbs = pbytes / (prune_ms * 1e-3) / 1e9
    dw_tflops = flops / (dw_ms * 1e-3) / 1e12
    full = args.batch is None and args.layers is None
    tc = path == B.PATH_TENSOR_CORE
    # per-layer roofline time of the weight gradient: the slower of the tensor cores on the
    # dense-equivalent flops and HBM on the least bytes (fp32 gradient + store + dW)
    tpeak = float(peaks["bf16_tflops"]) * 1e12 if tc else FP32_ALU_TFLOPS * 1e12
    hpeak = float(peaks["hbm_gbs"]) * 1e9
    roof_us = [max(l.flops / tpeak, dw_min_bytes(l, s.sizes.n_keep) / hpeak) * 1e6
               for l, s in zip(layers, stack.store)]
    dw_entry = frac_entry("tensor", dw_tflops, peaks, tc,
                          recorded_traffic(key, "weight_grad") if (full and tc) else None,
                          {"kernel": "weight gradient (all layers of one step)", "ms": round(dw_ms, 4), "flops": flops,
                           "roofline_ms": round(sum(roof_us) / 1e3, 4),
                           "frac_of_layer_rooflines": round(sum(roof_us) / 1e3 / dw_ms, 4)})
    pc_entry = frac_entry("hbm", prune_gbs, peaks, True,
                          recorded_traffic(key, "prune_compact") if full else None,
                          {"kernel": "surgeon_prune_compact (all kernels of all layers of one step)",
                           "ms": round(prune_ms, 4), "algorithmic_bytes": pbytes})
    res = {
        "workload": desc_text, "layers": len(layers),
        "ratios": "uniform in [0.5, 0.95]" if uniform else "Eq. 5-7, G_i ~ LogNormal(0,1)",
        "mean_ratio": round(float(np.mean(stack.ratios)), 4),
        "ms_per_step": round(ms_per_step, 4), "step_TFLOP/s": round(world * flops / (ms_per_step * 1e-3) / 1e12, 3),
        "prune_compact": pc_entry, "weight_grad": dw_entry,
        "store_bytes": stored, "dense_bytes": dense, "gpu_launches": int(launches),
        "read_GB_per_step": round((dense + sum(g.numel() * 4 for g in stack.g)) / 1e9, 2),
        "shared_inputs": len(stack.shared),
    }
    if args.per_layer or key.startswith("resnet50"):
        us = stack.per_layer_dw_us()
        res["weight_grad"]["per_layer"] = {
            "note": "each layer's call alone on one stream; roofline_us = max(flops / tensor peak, least bytes / HBM peak)",
            "name": [l.name for l in layers], "ratio": [round(float(r), 3) for r in stack.ratios],
            "us": [round(u, 1) for u in us], "roofline_us": [round(r, 1) for r in roof_us],
            "sum_us": round(sum(us), 1), "sum_roofline_us": round(sum(roof_us), 1),
            "frac": round(sum(roof_us) / sum(us), 4)}
    if sampler is not None:
        res["clocks"] = res_clocks
    if keep_stack:
        return res, stack
    del stack
    torch.cuda.empty_cache()
    return res, None


SWEEP_DISTS = ("relu_normal", "normal", "student_t2", "ties16")
SWEEP_RATIOS = (0.1, 0.5, 0.9, 0.99)


def run_sweep_cases(args, device, peaks, sizes, dists, ratios, steps, warmup):
    """Prune+compact on single tensors of 2^lg elements, fp32 and bf16; L2 flushed (256 MB written)
    before every timed call.  Returns the list of cases."""
    from paper_2503_20354_b200 import binding as B
    from paper_2503_20354_b200 import workloads as W
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    cases = []
    for bf16 in (False, True):
        for lg in sizes:
            n = 1 << lg
            es = 2 if bf16 else 4
            for dist in dists:
                x = W.draw(dist, n, args.seed, device=device)
                if bf16:
                    x = x.to(torch.bfloat16)
                out = B.CompressedActivation(n, B.dtype_code(x.dtype), 0.0, device)
                ws = torch.empty(out.sizes.workspace_bytes, dtype=torch.uint8, device=device)
                for ratio in ratios:
                    ts = []
                    for it in range(warmup + steps):
                        flush.zero_()
                        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        e0.record()
                        B.surgeon_prune_compact(x, ratio, out=out, workspace=ws)
                        e1.record()
                        e1.synchronize()
                        if it >= warmup:
                            ts.append(e0.elapsed_time(e1))
                    ms = float(np.median(ts))
                    k = out.sizes.n_keep
                    balg = 2 * n * es + n // 8 + k * es + 4 * (n // 128 + 1)
                    if out.read_header().status != 0:
                        raise SystemExit("device status in sweep case")
                    gbs = balg / ms / 1e6
                    cases.append({"dtype": "bf16" if bf16 else "f32", "log2_n": lg, "dist": dist, "ratio": ratio,
                                  "us": round(ms * 1e3, 1), "GB/s": round(gbs, 1),
                                  "frac": round(gbs / float(peaks["hbm_gbs"]), 4)})
                del x, out, ws
    del flush
    torch.cuda.empty_cache()
    return cases


def sweep_summary(cases, peaks, sizes):
    """Median GB/s per dtype at the largest size, as roofline entries (ties16 apart: it takes the
    exact fall-back select)."""
    out = {"l2": "flushed before every call", "cases": cases}
    top = sizes[-1]
    for dt in ("f32", "bf16"):
        main = [c["GB/s"] for c in cases if c["dtype"] == dt and c["log2_n"] == top and c["dist"] != "ties16"]
        ties = [c["GB/s"] for c in cases if c["dtype"] == dt and c["log2_n"] == top and c["dist"] == "ties16"]
        if main:
            out["%s_2^%d" % (dt, top)] = frac_entry("hbm", float(np.median(main)), peaks, True, None,
                                                    {"kernel": "surgeon_prune_compact (all kernels of a call)",
                                                     "min_GB/s": round(min(main), 1), "max_GB/s": round(max(main), 1)})
        if ties:
            out["%s_2^%d_ties16" % (dt, top)] = {"min_GB/s": round(min(ties), 1), "max_GB/s": round(max(ties), 1)}
    return out


def run_sweep_line(args, device, peaks):
    from paper_2503_20354_b200 import binding as B
    sizes = [20, 22, 24, 26, 28, 30][: args.sweep_sizes]
    launches0 = B.surgeon_launch_count()
    cases = run_sweep_cases(args, device, peaks, sizes, SWEEP_DISTS, SWEEP_RATIOS, args.steps, args.warmup)
    summ = sweep_summary(cases, peaks, sizes)
    big = [c["GB/s"] for c in cases if c["log2_n"] == sizes[-1]]
    val = float(np.median(big))
    print(json.dumps({
        "metric": METRIC, "value": round(val, 1), "unit": "GB/s (algorithmic bytes / call time, median at the largest size)",
        "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u32", "data": "synthetic",
        "config": {"workload": "prune+compact sweep, 2^20..2^%d elements, fp32 and bf16" % sizes[-1],
                   "l2": "flushed before every call"},
        "roofline": frac_entry("hbm", val, peaks, True, None, {"kernel": "surgeon_prune_compact (all kernels of a call)"}),
        "gpu_launches": int(B.surgeon_launch_count() - launches0), "sweep": summ}))


def run_ours(args, rank, world, local):
    from paper_2503_20354_b200 import binding as B
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    B.lib()
    device = torch.device("cuda", local if world > 1 else 0)
    peaks = load_peaks()
    if args.workload == "sweep":
        if rank == 0:
            run_sweep_line(args, device, peaks)
        return
    path = B.PATH_FP32 if args.path == "fp32" else B.PATH_TENSOR_CORE
    head_key = HEADLINE if args.workload == "all" else args.workload
    others = ["wrn28", "resnet50", "resnet50_uniform"] if args.workload == "all" else []

    sampler = ClockSampler(local if world > 1 else 0)
    head, stack = run_stack(head_key, args, rank, world, device, peaks, path, keep_stack=True, sampler=sampler)
    clocks = head.pop("clocks")
    layers = stack.layers
    flops = sum(l.flops for l in layers)
    # ---- end to end through the C ABI with host buffers --------------------------------------
    e2e = run_e2e(stack, layers, args, world, device, flops) if args.e2e else None
    del stack
    torch.cuda.empty_cache()

    results = {head_key: head}
    for key in others:
        results[key], _ = run_stack(key, args, rank, world, device, peaks, path)
    if args.workload == "all" and rank == 0:
        # the top of the bandwidth sweep: 2^28 and 2^30 elements, three distributions, two ratios
        # (+ the many-ties case at one ratio), 5 timed calls each
        sizes = [28, 30]
        cases = run_sweep_cases(args, device, peaks, sizes, ("relu_normal", "normal", "student_t2"), (0.5, 0.9), 5, 3)
        cases += run_sweep_cases(args, device, peaks, sizes, ("ties16",), (0.9,), 5, 3)
        results["sweep"] = sweep_summary(cases, peaks, sizes)
        for lg in sizes[:-1]:
            for dt in ("f32", "bf16"):
                sub = [c["GB/s"] for c in cases if c["dtype"] == dt and c["log2_n"] == lg and c["dist"] != "ties16"]
                results["sweep"]["%s_2^%d" % (dt, lg)] = frac_entry("hbm", float(np.median(sub)), peaks, True, None,
                                                                   {"min_GB/s": round(min(sub), 1), "max_GB/s": round(max(sub), 1)})
    barrier(world)

    roofline = dict(head["weight_grad"])
    roofline.pop("per_layer", None)
    out = {
        "metric": METRIC, "value": head["step_TFLOP/s"], "unit": "TFLOP/s (dense-equivalent dW flops / whole-step time)",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": head["ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if path == B.PATH_TENSOR_CORE else "f32", "data": "synthetic",
        "config": {"workload": head["workload"], "layers": head["layers"], "ratios": head["ratios"],
                   "path": args.path, "l2": "inputs larger than L2 (%.2f GB read per step)" % head["read_GB_per_step"],
                   "replicas": world, "streams": args.streams,
                   "also_timed": [k for k in results if k != head_key]},
        "roofline": roofline,
        "roofline_prune_compact": head["prune_compact"],
        "workloads": results,
        "e2e": e2e, "gpu_launches": int(sum(r.get("gpu_launches", 0) for r in results.values() if isinstance(r, dict))),
        "clocks": clocks,
    }
    if rank == 0:
        if args.cpu_baseline:
            args_head = argparse.Namespace(**vars(args))
            args_head.workload = head_key
            out["cpu_baseline"] = cpu_baseline(args_head, budget_s=20.0)
        print(json.dumps(out))


def run_e2e(stack, layers, args, world, device, flops):
    """The same step with HOST inputs: per step every activation and output gradient is copied in
    from pinned host memory and every dW is copied back to pinned host memory.  The copies run on
    their own streams in layer order; a layer's kernels wait only for that layer's tensors, so
    the transfers of later layers overlap the work on earlier ones."""
    steps = max(1, min(args.steps, args.e2e_steps))
    n = len(layers)
    hx = [torch.empty(x.shape, dtype=x.dtype).pin_memory() for x in stack.x]
    hg = [torch.empty(g.shape, dtype=g.dtype).pin_memory() for g in stack.g]
    hdw = [torch.empty(d.shape, dtype=d.dtype).pin_memory() for d in stack.dw]
    for h, d in zip(hx + hg, stack.x + stack.g):
        h.copy_(d)
    torch.cuda.synchronize()
    h2d = sum(hx[i].numel() * hx[i].element_size() for i in stack.own) + sum(t.numel() * t.element_size() for t in hg)
    d2h = sum(t.numel() * t.element_size() for t in hdw)
    s_in, s_out = torch.cuda.Stream(device=device), torch.cuda.Stream(device=device)
    main = torch.cuda.current_stream(device)

    def one():
        x_ready = [torch.cuda.Event() for _ in range(n)]
        g_ready = [torch.cuda.Event() for _ in range(n)]
        dw_done = [torch.cuda.Event() for _ in range(n)]
        s_in.wait_stream(main)
        with torch.cuda.stream(s_in):
            for i in stack.own:                      # forward order; a shared tensor crosses once
                stack.x[i].copy_(hx[i], non_blocking=True)
                x_ready[i].record(s_in)
            for i in reversed(range(n)):             # backward order
                stack.g[i].copy_(hg[i], non_blocking=True)
                g_ready[i].record(s_in)
        stack.step(x_ready=x_ready, g_ready=g_ready, dw_done=dw_done)
        with torch.cuda.stream(s_out):
            for i in reversed(range(n)):
                s_out.wait_event(dw_done[i])
                hdw[i].copy_(stack.dw[i], non_blocking=True)
        main.wait_stream(s_out)
        main.wait_stream(s_in)

    one()
    torch.cuda.synchronize()
    barrier(world)
    b, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    b.record()
    for _ in range(steps):
        one()
    e.record()
    torch.cuda.synchronize()
    barrier(world)
    ms = max_over_ranks(b.elapsed_time(e), world, device) / steps
    return {"value": round(world * flops / (ms * 1e-3) / 1e12, 4), "unit": "TFLOP/s", "ms_per_step": round(ms, 3),
            "steps": steps, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "note": "PCIe-bound: copies of later layers overlap the kernels of earlier ones"}


# ------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------

def oracle_step(layers, inputs, ratios):
    """The oracle's pass over `layers`: ratios, prune+compact, decompress, dW (fp64)."""
    import oracle
    for l, (a, g), p in zip(layers, inputs, ratios):
        r = oracle.prune_compact(a.reshape(-1), float(p))
        pruned = oracle.decompress(r["bitmap"], r["values"], a.size).reshape(l.act_shape)
        if l.kind == 1 and l.groups > 1:
            oracle.dw_conv2d_grouped(pruned, g, l.kh, l.kw, l.stride, l.pad, l.groups)
        elif l.kind == 1:
            oracle.dw_conv2d(pruned, g, l.kh, l.kw, l.stride, l.pad)
        else:
            oracle.dw_linear(pruned, g)


def oracle_sample(args, budget_s: float, grow: bool = False):
    """A bounded sample of the workload for the CPU: the same stack at batch 1, thinned to every
    `stride`-th layer until one pass fits the budget; with `grow`, the batch is then raised (up to
    16) so that one pass takes a sizeable part of the budget."""
    import oracle
    from paper_2503_20354_b200 import workloads as W
    full, _ = get_layers(args.workload, args.batch)
    batch = 1
    small = W.shrink(full, batch)
    gi = W.gradient_importance(len(small), args.seed)
    lam = np.array([l.act_bytes for l in full], dtype=np.float64)
    _, ratios = oracle.layer_ratios(gi, lam)
    stride = 1
    while True:
        idx = list(range(0, len(small), stride))
        layers = [small[i] for i in idx]
        inputs = [(W.as_numpy_bits(W.activation(small[i], args.seed, i)), W.grad_out(small[i], args.seed, i, sigma=SIGMA.get(args.workload, 0.01)).numpy())
                  for i in idx]
        t0 = time.perf_counter()
        oracle_step(layers, inputs, ratios[idx])
        dt = time.perf_counter() - t0
        if grow and batch == 1 and dt < budget_s / 4:
            batch = max(2, min(16, int(0.6 * budget_s / dt)))
            small = W.shrink(full, batch)
            continue
        if dt <= budget_s or len(layers) == 1 or batch > 1:
            break
        stride *= 2
    text = "%s at batch %d, %d of %d layers (every %d-th)" % (args.workload, batch, len(layers), len(small), stride)
    return layers, inputs, ratios[idx], dt, text


def cpu_baseline(args, budget_s: float):
    import oracle
    layers, inputs, ratios, dt, text = oracle_sample(args, budget_s, grow=True)
    flops = sum(l.flops for l in layers)
    return {"value": round(flops / dt / 1e12, 6), "unit": "TFLOP/s", "cores": oracle.num_threads(),
            "kind": "oracle", "sample": text, "seconds": round(dt, 3)}


def run_reference(args, rank, world):
    """The CPU oracle as the reference arm (rank 0 only)."""
    if rank != 0:
        return
    import oracle
    total = max(1, args.steps + args.warmup)
    layers, inputs, ratios, dt, text = oracle_sample(args, budget_s=max(0.5, 120.0 / total))
    for _ in range(args.warmup):
        oracle_step(layers, inputs, ratios)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(layers, inputs, ratios)
    ms = (time.perf_counter() - t0) * 1e3 / max(1, args.steps)
    flops = sum(l.flops for l in layers)
    v = round(flops / (ms * 1e-3) / 1e12, 6)
    _, desc_text = get_layers(args.workload, args.batch)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": "TFLOP/s (dense-equivalent dW flops / whole-step time)",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": desc_text, "sample": text},
        "cpu_baseline": {"value": v, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle", "sample": text},
        "e2e": {"value": v, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="all",
                    choices=["all", "vit", "wrn28", "resnet50", "resnet50_uniform", "resnext29", "tiny", "segformer", "sweep"])
    ap.add_argument("--sweep-sizes", type=int, default=6, help="how many of 2^20,22,24,26,28,30 the sweep covers")
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--layers", default=None, help="comma-separated layer names: run only these (profiling)")
    ap.add_argument("--path", default="tc", choices=["tc", "fp32"])
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--streams", type=int, default=8,
                    help="streams the independent layers are issued on (1 = the caller's stream only)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--per-layer", action="store_true", help="time every layer's weight gradient alone as well")
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--no-e2e", dest="e2e", action="store_false", help="skip the host-buffer leg (profiling runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        if args.workload in ("all", "sweep"):
            args.workload = HEADLINE
        rank = int(os.environ.get("RANK", "0"))
        run_reference(args, rank, int(os.environ.get("WORLD_SIZE", "1")))
        return
    rank, world, local = dist_setup(args.gpus)
    try:
        run_ours(args, rank, world, local)
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


if __name__ == "__main__":
    main()

"""Seeded synthetic workloads: layer shape tables and input generators.

This module holds no arithmetic of the method (no ratios, thresholds, pruning or gradients):
only the shapes of the networks the paper adapts (Section 5.1: WideResNet-28-10 at batch 200,
ResNet-50 at batch 64, the linear layers of Segformer-B5 at batch 1) plus a ViT-B/16-shaped
stack, and random tensors with the value
distributions of their saved activations.  The tensors stand in for CIFAR10-C / ImageNet-C
batches flowing through pre-trained backbones, which are not available offline.  The same bytes
are handed to the CUDA library and to the CPU oracle by the tests and the benchmark.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import List

import numpy as np
import torch

F32, BF16 = 0, 1


@dataclass(frozen=True)
class Layer:
    """One weight layer whose input activation is saved for the backward pass."""
    name: str
    kind: int          # 0 linear, 1 conv2d
    batch: int         # images (conv2d) or rows T (linear)
    c_in: int
    h: int
    w: int
    c_out: int
    kh: int = 1
    kw: int = 1
    stride: int = 1
    pad: int = 0
    dist: str = "relu_normal"   # distribution of the saved input activation
    dt: int = F32               # dtype of the saved activation
    rows_per_sample: int = 0    # linear layers: rows T per sample (0: see shrink)
    groups: int = 1             # conv2d: channel groups (c_in = c_out = groups: depthwise)

    @property
    def oh(self) -> int:
        return (self.h + 2 * self.pad - self.kh) // self.stride + 1

    @property
    def ow(self) -> int:
        return (self.w + 2 * self.pad - self.kw) // self.stride + 1

    @property
    def n_act(self) -> int:
        return self.batch * self.c_in * self.h * self.w

    @property
    def act_shape(self):
        return (self.batch, self.c_in, self.h, self.w) if self.kind == 1 else (self.batch, self.c_in)

    @property
    def grad_shape(self):
        return (self.batch, self.c_out, self.oh, self.ow) if self.kind == 1 else (self.batch, self.c_out)

    @property
    def dw_shape(self):
        return (self.c_out, self.c_in // self.groups, self.kh, self.kw) if self.kind == 1 else (self.c_out, self.c_in)

    @property
    def n_weight(self) -> int:
        return self.c_out * (self.c_in // self.groups) * self.kh * self.kw

    @property
    def gemm_k(self) -> int:
        return self.batch * self.oh * self.ow

    @property
    def flops(self) -> int:
        """Dense-equivalent flops of the weight gradient: 2 * Cout * (Cin*kh*kw) * (B*OH*OW)."""
        return 2 * self.n_weight * self.gemm_k

    @property
    def macs_per_sample(self) -> int:
        return self.n_weight * self.oh * self.ow if self.kind == 1 else self.n_weight

    @property
    def act_bytes(self) -> int:
        return self.n_act * (4 if self.dt == F32 else 2)


def conv(name, batch, c_in, hw, c_out, k, stride=1, pad=None, dist="relu_normal", dt=F32, groups=1) -> Layer:
    if pad is None:
        pad = k // 2
    return Layer(name, 1, batch, c_in, hw, hw, c_out, k, k, stride, pad, dist, dt, 0, groups)


def linear(name, rows, c_in, c_out, dist="normal", dt=BF16, rows_per_sample=0) -> Layer:
    return Layer(name, 0, rows, c_in, 1, 1, c_out, 1, 1, 1, 0, dist, dt, rows_per_sample)


def tiny_conv(batch: int = 16) -> List[Layer]:
    """One 3x3 conv 64->64, stride 1, pad 1, on [batch,64,32,32] fp32 post-ReLU input."""
    return [conv("conv3x3_64", batch, 64, 32, 64, 3)]


def wrn28_10(batch: int = 200, dt: int = F32) -> List[Layer]:
    """The 28 conv layers of WideResNet-28-10 on 32x32 inputs (4 blocks per group, widths
    160/320/640, a 1x1 shortcut conv in the first block of each group)."""
    L = [conv("conv1", batch, 3, 32, 16, 3, dist="normal", dt=dt)]
    c_prev, hw = 16, 32
    for g, (width, stride) in enumerate([(160, 1), (320, 2), (640, 2)], start=1):
        for b in range(4):
            s = stride if b == 0 else 1
            L.append(conv(f"g{g}b{b}.conv1", batch, c_prev, hw, width, 3, s, dt=dt))
            hw_out = hw // s
            L.append(conv(f"g{g}b{b}.conv2", batch, width, hw_out, width, 3, 1, dt=dt))
            if b == 0:
                L.append(conv(f"g{g}b{b}.shortcut", batch, c_prev, hw, width, 1, s, 0, dt=dt))
            c_prev, hw = width, hw_out
    return L


def resnet50(batch: int = 64, dt: int = BF16) -> List[Layer]:
    """The 53 conv layers and the FC layer of ResNet-50 at 224x224 (bottlenecks with the stride
    on the 3x3 conv)."""
    L = [conv("stem", batch, 3, 224, 64, 7, 2, 3, dist="normal", dt=dt)]
    c_prev, hw = 64, 56
    for li, (width, blocks, stride) in enumerate([(64, 3, 1), (128, 4, 2), (256, 6, 2), (512, 3, 2)],
                                                 start=1):
        for b in range(blocks):
            s = stride if b == 0 else 1
            p = f"layer{li}.{b}"
            L.append(conv(p + ".conv1", batch, c_prev, hw, width, 1, 1, 0, dt=dt))
            L.append(conv(p + ".conv2", batch, width, hw, width, 3, s, 1, dt=dt))
            hw_out = hw // s
            L.append(conv(p + ".conv3", batch, width, hw_out, width * 4, 1, 1, 0, dt=dt))
            if b == 0:
                L.append(conv(p + ".downsample", batch, c_prev, hw, width * 4, 1, s, 0, dt=dt))
            c_prev, hw = width * 4, hw_out
    L.append(linear("fc", batch, 2048, 1000, dist="abs_normal", dt=dt))
    return L


def resnext29(batch: int = 200, dt: int = F32, cardinality: int = 32, base_width: int = 4) -> List[Layer]:
    """The conv layers and the FC layer of ResNeXt-29 (32x4d) on 32x32 inputs, the network the paper
    adapts on CIFAR100-C (Section 5.1) and times on the embedded board (Section 5.5): a 3x3 stem,
    three stages of three bottleneck blocks (1x1 reduce, GROUPED 3x3 with `cardinality` groups,
    1x1 expand; a 1x1 shortcut convolution in the first block of a stage), stage outputs
    256 / 512 / 1024 channels on 32 / 16 / 8 wide maps."""
    L = [conv("conv1", batch, 3, 32, 64, 3, dist="normal", dt=dt)]
    c_prev, hw = 64, 32
    for st in range(3):
        d = cardinality * base_width * (2 ** st)          # width of the grouped convolution
        c_out = 256 * (2 ** st)
        for b in range(3):
            s = 2 if (st > 0 and b == 0) else 1
            n = f"s{st + 1}b{b}"
            L.append(conv(n + ".conv1", batch, c_prev, hw, d, 1, 1, 0, dt=dt))
            L.append(conv(n + ".conv2", batch, d, hw, d, 3, s, 1, dt=dt, groups=cardinality))
            hw_out = hw // s
            L.append(conv(n + ".conv3", batch, d, hw_out, c_out, 1, 1, 0, dt=dt))
            if b == 0:
                L.append(conv(n + ".shortcut", batch, c_prev, hw, c_out, 1, s, 0, dt=dt))
            c_prev, hw = c_out, hw_out
    L.append(linear("fc", batch, 1024, 100, dist="abs_normal", dt=dt))
    return L


def vit_b16(batch: int = 64, dt: int = BF16, blocks: int = 12) -> List[Layer]:
    """qkv / proj / fc1 / fc2 linears of ViT-B/16 at 224x224: 197 tokens, width 768, MLP 3072."""
    T = batch * 197
    L = []
    for b in range(blocks):
        L.append(linear(f"blk{b}.qkv", T, 768, 2304, "normal", dt))
        L.append(linear(f"blk{b}.proj", T, 768, 768, "normal", dt))
        L.append(linear(f"blk{b}.fc1", T, 768, 3072, "normal", dt))
        L.append(linear(f"blk{b}.fc2", T, 3072, 768, "gelu_normal", dt))
    return L


def segformer_b5(image: int = 1024, batch: int = 1, dt: int = BF16, depths=(3, 6, 40, 3),
                 convs: bool = True) -> List[Layer]:
    """The layers of a Segformer-B5-shaped encoder's blocks (Section 5.1: semantic segmentation at
    batch 1) on an image x image input: four stages of widths 64 / 128 / 320 / 512 on token grids
    of 1/4, 1/8, 1/16 and 1/32 of the image side, attention with keys and values on a grid reduced
    8 / 4 / 2 / 1 times per side, MLP ratio 4.  Per block the linear layers q, kv, proj, fc1, fc2
    and, with `convs`, the two convolutions: the spatial reduction before kv (kernel = stride =
    the reduction, stages 1-3) and the depthwise 3x3 between fc1 and fc2 (groups = channels).  The
    overlapping patch embeddings between the stages are not part of this stack."""
    widths, reductions = (64, 128, 320, 512), (8, 4, 2, 1)
    L = []
    for s in range(4):
        side = image // (4 << s)
        t_q = side * side
        t_kv = (side // reductions[s]) ** 2
        c = widths[s]
        for b in range(depths[s]):
            n = f"s{s}b{b}"
            L.append(linear(n + ".q", batch * t_q, c, c, "normal", dt, t_q))
            if convs and reductions[s] > 1:
                L.append(conv(n + ".sr", batch, c, side, c, reductions[s], reductions[s], 0, "normal", dt))
            L.append(linear(n + ".kv", batch * t_kv, c, 2 * c, "normal", dt, t_kv))
            L.append(linear(n + ".proj", batch * t_q, c, c, "normal", dt, t_q))
            L.append(linear(n + ".fc1", batch * t_q, c, 4 * c, "normal", dt, t_q))
            if convs:
                L.append(conv(n + ".dwconv", batch, 4 * c, side, 4 * c, 3, 1, 1, "normal", dt, groups=4 * c))
            L.append(linear(n + ".fc2", batch * t_q, 4 * c, c, "gelu_normal", dt, t_q))
    return L


def shared_inputs(layers: List[Layer]) -> dict:
    """Layers that read the same saved tensor as an earlier layer of the stack: the 1x1 shortcut /
    downsample convolution of a residual block takes the block's input, like the block's first
    convolution.  Returns {index of the later layer: index of the layer whose input it shares}."""
    by_name = {l.name: i for i, l in enumerate(layers)}
    out = {}
    for j, l in enumerate(layers):
        for suffix in (".shortcut", ".downsample"):
            if l.name.endswith(suffix):
                i = by_name.get(l.name[: -len(suffix)] + ".conv1")
                if i is not None and layers[i].act_shape == l.act_shape and layers[i].dt == l.dt:
                    out[j] = i
    return out


def shrink(layers: List[Layer], batch: int) -> List[Layer]:
    """Same stack at a smaller batch (rows scale with the batch for linear layers)."""
    out = []
    for l in layers:
        if l.kind == 1:
            out.append(replace(l, batch=batch))
        else:
            full = l.batch
            per = l.rows_per_sample or (197 if full % 197 == 0 else 1)
            out.append(replace(l, batch=batch * per))
    return out


# ------------------------------------------------------------------------------------------
# Random tensors.  A torch generator seeded with (seed, tag) drives everything, on the CPU or
# on the GPU; tests that compare with the oracle draw on the CPU and upload the bytes.
# ------------------------------------------------------------------------------------------

DISTS = ("relu_normal", "normal", "abs_normal", "student_t2", "ties16", "gelu_normal")


def _gen(seed: int, tag: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1000003 + int(tag)) & 0x7FFFFFFFFFFFFFFF)
    return g


def draw(dist: str, n: int, seed: int, tag: int = 0, device="cpu") -> torch.Tensor:
    """n fp32 samples of the named distribution.

    relu_normal: max(z,0), z~N(0,1) (about half exact +0, post-BN+ReLU activations);
    normal: N(0,1) (LayerNorm outputs, image inputs); abs_normal: |z|;
    student_t2: z / sqrt(e), e~Exp(1) (Student-t with 2 degrees of freedom, heavy tails);
    ties16: N(0,1) rounded to the 16 levels {-4, -3.5, ..., 3.5} (many equal magnitudes);
    gelu_normal: z * Phi(z) (exact erf GELU of a N(0,1) pre-activation)."""
    g = _gen(seed, tag, device)
    z = torch.randn(n, generator=g, device=device, dtype=torch.float32)
    if dist == "normal":
        return z
    if dist == "relu_normal":
        return torch.relu_(z)
    if dist == "abs_normal":
        return torch.abs_(z)
    if dist == "student_t2":
        u = torch.rand(n, generator=g, device=device, dtype=torch.float32)
        e = -torch.log(torch.clamp_(u, min=1e-30))
        return z / torch.sqrt(e)
    if dist == "ties16":
        return torch.clamp_(torch.round(z * 2.0), -8.0, 7.0) * 0.5
    if dist == "gelu_normal":
        return torch.nn.functional.gelu(z)
    raise ValueError("unknown distribution %r" % dist)


def activation(layer: Layer, seed: int, index: int = 0, device="cpu") -> torch.Tensor:
    """Saved input activation of `layer` (fp32, or bf16 rounded to nearest-even from fp32)."""
    x = draw(layer.dist, layer.n_act, seed, 2 * index, device).reshape(layer.act_shape)
    return x if layer.dt == F32 else x.to(torch.bfloat16)


def grad_out(layer: Layer, seed: int, index: int = 0, sigma: float = 0.01, device="cpu") -> torch.Tensor:
    """Output gradient of `layer`: fp32 ~ N(0, sigma^2)."""
    n = int(np.prod(layer.grad_shape))
    g = draw("normal", n, seed, 2 * index + 1, device)
    return g.mul_(sigma).reshape(layer.grad_shape)


def gradient_importance(n_layers: int, seed: int) -> np.ndarray:
    """Synthetic per-layer Gradient Importance (Eq. 4 is an input here): LogNormal(0,1)."""
    rng = np.random.Generator(np.random.Philox(int(seed) + 7919))
    return np.exp(rng.standard_normal(n_layers))


def uniform_ratios(n_layers: int, seed: int, lo: float = 0.5, hi: float = 0.95) -> np.ndarray:
    rng = np.random.Generator(np.random.Philox(int(seed) + 104729))
    return lo + (hi - lo) * rng.random(n_layers)


def as_numpy_bits(t: torch.Tensor) -> np.ndarray:
    """CPU numpy view for the oracle: float32 stays float32, bf16 becomes its uint16 bits."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()

"""Seeded synthetic inputs and layer shapes for tests and benchmarks.

Holds no DyBit arithmetic: only shapes (ResNet-18 / ResNet-50 topologies as
lists of convolution geometries) and random tensors with the distributions
the workloads call for (Kaiming-normal weights, half-normal post-ReLU
activations, N(0,1) / Laplace(0,1) for the quantize sweep).  The same buffers
are handed to the CUDA library and to the CPU oracle.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class ConvLayer:
    name: str
    n: int
    h: int
    w: int
    c: int
    k: int
    r: int
    s: int
    stride: int
    pad: int

    @property
    def oh(self) -> int:
        return (self.h + 2 * self.pad - (self.r - 1) - 1) // self.stride + 1

    @property
    def ow(self) -> int:
        return (self.w + 2 * self.pad - (self.s - 1) - 1) // self.stride + 1

    @property
    def gemm_m(self) -> int:
        return self.n * self.oh * self.ow

    @property
    def gemm_n(self) -> int:
        return self.k

    @property
    def gemm_k(self) -> int:
        return self.r * self.s * self.c

    @property
    def macs(self) -> int:
        return self.gemm_m * self.gemm_n * self.gemm_k

    def with_batch(self, n: int) -> "ConvLayer":
        return ConvLayer(self.name, n, self.h, self.w, self.c, self.k, self.r, self.s, self.stride, self.pad)


def _conv(name, n, hw, c, k, ksz, stride):
    return ConvLayer(name, n, hw, hw, c, k, ksz, ksz, stride, ksz // 2)


def resnet18_layers(batch: int = 32):
    """The 20 convolutions and the FC of a ResNet-18 at 224x224 (FC as a 1x1 conv on a 1x1 map)."""
    L = [_conv("conv1", batch, 224, 3, 64, 7, 2)]
    hw, cin = 56, 64
    for stage, cout in enumerate((64, 128, 256, 512)):
        for block in range(2):
            stride = 2 if (stage > 0 and block == 0) else 1
            L.append(_conv(f"layer{stage + 1}.{block}.conv1", batch, hw, cin, cout, 3, stride))
            hw_out = hw // stride
            L.append(_conv(f"layer{stage + 1}.{block}.conv2", batch, hw_out, cout, cout, 3, 1))
            if stride != 1 or cin != cout:
                L.append(_conv(f"layer{stage + 1}.{block}.downsample", batch, hw, cin, cout, 1, stride))
            hw, cin = hw_out, cout
    L.append(ConvLayer("fc", batch, 1, 1, 512, 1000, 1, 1, 1, 0))
    return L


def resnet50_layers(batch: int = 64):
    """The 53 convolutions and the FC of a ResNet-50 (stride on the 3x3 of each bottleneck)."""
    L = [_conv("conv1", batch, 224, 3, 64, 7, 2)]
    hw, cin = 56, 64
    for stage, (width, blocks) in enumerate(((64, 3), (128, 4), (256, 6), (512, 3))):
        cout = width * 4
        for block in range(blocks):
            stride = 2 if (stage > 0 and block == 0) else 1
            L.append(_conv(f"layer{stage + 1}.{block}.conv1", batch, hw, cin, width, 1, 1))
            L.append(_conv(f"layer{stage + 1}.{block}.conv2", batch, hw, width, width, 3, stride))
            hw_out = hw // stride
            L.append(_conv(f"layer{stage + 1}.{block}.conv3", batch, hw_out, width, cout, 1, 1))
            if block == 0:
                L.append(_conv(f"layer{stage + 1}.{block}.downsample", batch, hw, cin, cout, 1, stride))
            hw, cin = hw_out, cout
    L.append(ConvLayer("fc", batch, 1, 1, 2048, 1000, 1, 1, 1, 0))
    return L


def mobilenetv2_depthwise_layers(batch: int = 32):
    """The 17 depth-wise 3x3 convolutions of a MobileNetV2 (width 1.0, 224x224 input): the middle layer of every
    inverted-residual block, on t * c_in channels, with the block's stride; k == c marks them as depth-wise."""
    L = []
    hw, cin = 112, 32
    for t, c, n, s in ((1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2), (6, 96, 3, 1), (6, 160, 3, 2),
                       (6, 320, 1, 1)):
        for i in range(n):
            stride = s if i == 0 else 1
            hidden = cin * t
            L.append(ConvLayer(f"block{len(L)}.dw", batch, hw, hw, hidden, hidden, 3, 3, stride, 1))
            hw //= stride
            cin = c
    return L


MIXED_BITS = (2, 3, 4, 5, 6, 8)


def mixed_bitwidths(num_layers: int, seed: int = 0):
    """Per-layer (weight bits, activation bits) drawn independently from MIXED_BITS."""
    g = torch.Generator().manual_seed(seed)
    w = torch.randint(0, len(MIXED_BITS), (num_layers,), generator=g).tolist()
    a = torch.randint(0, len(MIXED_BITS), (num_layers,), generator=g).tolist()
    return [(MIXED_BITS[i], MIXED_BITS[j]) for i, j in zip(w, a)]


def _gen(seed: int, device):
    return torch.Generator(device=device).manual_seed(int(seed))


def normal(shape, seed: int, std: float = 1.0, device="cpu") -> torch.Tensor:
    return torch.randn(shape, generator=_gen(seed, device), device=device, dtype=torch.float32) * std


def half_normal(shape, seed: int, device="cpu") -> torch.Tensor:
    """|N(0,1)|: the distribution of a post-ReLU activation."""
    return torch.randn(shape, generator=_gen(seed, device), device=device, dtype=torch.float32).abs_()


def laplace(shape, seed: int, device="cpu") -> torch.Tensor:
    """Laplace(0,1) by inverse CDF of a uniform draw."""
    u = torch.rand(shape, generator=_gen(seed, device), device=device, dtype=torch.float32) - 0.5
    mag = u.abs().clamp_(max=0.5 - 2.0 ** -25)          # rand() may return exactly 0: keep the log finite
    return -torch.sign(u) * torch.log1p(-2.0 * mag)


def kaiming_normal(k: int, r: int, s: int, c: int, seed: int, device="cpu") -> torch.Tensor:
    """Weights [k][r][s][c] ~ N(0, 2 / fan_in), fan_in = c*r*s."""
    return normal((k, r, s, c), seed, std=math.sqrt(2.0 / (c * r * s)), device=device)


DISTRIBUTIONS = {"normal": normal, "laplace": laplace, "half_normal": half_normal}

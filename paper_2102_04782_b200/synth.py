"""Seeded synthetic inputs shaped like the paper's CNN workloads.

This module holds input generators and layer-shape tables only: none of the method's arithmetic
(no statistics, clipping, quantization or convolution) lives here, so the CPU oracle and the CUDA
path can both be fed from it without sharing any computation.

Recipes (all numpy, Philox counter-based bit generator, deterministic in the seed):
  * activations  X  = ReLU(N(0, 1))
  * weights      W  ~ N(0, sqrt(2 / (Cin*R*S)))                       (He initialisation)
  * gradients    dY : every output channel c is independently "bell-shaped" N(0, sigma_c) or
                      "sharp, long-tailed" Laplace(0, sigma_c / sqrt(2)) (both have standard
                      deviation sigma_c), each with probability 1/2, sigma_c log-uniform in
                      [1e-6, 1e-3]  -- the two channel-wise shapes of Fig. 1.
  * bf16 variants round each value to bfloat16 (round to nearest even) and return both the 16-bit
    patterns and the exactly representable fp32 values.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Tuple

import numpy as np


def _rng(seed: int, salt: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed) & 0xFFFFFFFFFFFFFFFF, int(salt)]))


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bfloat16 bit patterns (uint16), round to nearest even.  Finite inputs only."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """fp32 values rounded to the nearest bfloat16, returned as fp32."""
    return bf16_bits_to_f32(to_bf16_bits(x))


def activations(N: int, C: int, H: int, W: int, seed: int) -> np.ndarray:
    """X = ReLU(N(0,1)), NCHW fp32."""
    x = _rng(seed, 1).standard_normal((N, C, H, W), dtype=np.float32)
    np.maximum(x, 0.0, out=x)
    return x


def weights(Cout: int, Cin: int, R: int, S: int, seed: int) -> np.ndarray:
    """W ~ N(0, sqrt(2/(Cin*R*S))), (Cout,Cin,R,S) fp32."""
    w = _rng(seed, 2).standard_normal((Cout, Cin, R, S), dtype=np.float32)
    w *= np.float32(np.sqrt(2.0 / (Cin * R * S)))
    return w


def channel_mixed_grad(N: int, C: int, H: int, W: int, seed: int):
    """dY with per-channel bell-shaped / long-tailed mix.  Returns (dY NCHW fp32,
    is_bell[C] bool, sigma[C] float64)."""
    meta = _rng(seed, 3)
    is_bell = meta.random(C) < 0.5
    sigma = 10.0 ** meta.uniform(-6.0, -3.0, size=C)
    g = np.empty((N, C, H, W), np.float32)
    for c in range(C):
        r = _rng(seed, 1000 + c)
        if is_bell[c]:
            v = r.standard_normal((N, H, W), dtype=np.float32) * np.float32(sigma[c])
        else:
            v = r.laplace(0.0, sigma[c] / np.sqrt(2.0), size=(N, H, W)).astype(np.float32)
        g[:, c] = v
    return g, is_bell, sigma


# ------------------------------------------------------------------------------------------------
# Layer-shape tables.  A layer is (name, Cin, Cout, H, W, R, S, stride, pad); H, W are input extents.
# ------------------------------------------------------------------------------------------------
@dataclass(frozen=True)
class ConvLayer:
    name: str
    Cin: int
    Cout: int
    H: int
    W: int
    R: int
    S: int
    stride: int
    pad: int

    @property
    def P(self) -> int:
        return (self.H + 2 * self.pad - self.R) // self.stride + 1

    @property
    def Q(self) -> int:
        return (self.W + 2 * self.pad - self.S) // self.stride + 1

    def macs(self, N: int) -> int:
        return N * self.P * self.Q * self.Cout * self.Cin * self.R * self.S


def config1_layer() -> ConvLayer:
    return ConvLayer("conv3x3_64_14", 64, 64, 14, 14, 3, 3, 1, 1)


def resnet50_conv2x_block() -> List[ConvLayer]:
    """One bottleneck of stage conv2_x (input 256 channels, 56x56)."""
    return [ConvLayer("conv2_x.1x1a", 256, 64, 56, 56, 1, 1, 1, 0),
            ConvLayer("conv2_x.3x3", 64, 64, 56, 56, 3, 3, 1, 1),
            ConvLayer("conv2_x.1x1b", 64, 256, 56, 56, 1, 1, 1, 0)]


def resnet50_convs() -> List[ConvLayer]:
    """All 53 convolutions of ResNet-50 at 224x224 input (stride on the 3x3 of the first block of
    stages 3-5, projection shortcut in the first block of every stage)."""
    layers = [ConvLayer("stem", 3, 64, 224, 224, 7, 7, 2, 3)]
    in_ch, hw = 64, 56
    for stage, (mid, blocks) in enumerate([(64, 3), (128, 4), (256, 6), (512, 3)], start=2):
        out_ch = 4 * mid
        for b in range(blocks):
            stride = 2 if (b == 0 and stage > 2) else 1
            pre = f"conv{stage}_{b + 1}"
            layers.append(ConvLayer(pre + ".1x1a", in_ch, mid, hw, hw, 1, 1, 1, 0))
            layers.append(ConvLayer(pre + ".3x3", mid, mid, hw, hw, 3, 3, stride, 1))
            if b == 0:
                layers.append(ConvLayer(pre + ".proj", in_ch, out_ch, hw, hw, 1, 1, stride, 0))
            hw //= stride
            layers.append(ConvLayer(pre + ".1x1b", mid, out_ch, hw, hw, 1, 1, 1, 0))
            in_ch = out_ch
    assert len(layers) == 53
    return layers


def mobilenetv2_pointwise() -> List[ConvLayer]:
    """The 34 pointwise (1x1) convolutions of MobileNetV2 width 1.0 at 224x224 input."""
    layers: List[ConvLayer] = []
    cfg = [(1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2), (6, 96, 3, 1),
           (6, 160, 3, 2), (6, 320, 1, 1)]
    in_ch, hw = 32, 112
    for bi, (t, c, n, s) in enumerate(cfg):
        for i in range(n):
            stride = s if i == 0 else 1
            hidden = in_ch * t
            if t != 1:
                layers.append(ConvLayer(f"b{bi}_{i}.expand", in_ch, hidden, hw, hw, 1, 1, 1, 0))
            hw //= stride  # the depthwise 3x3 (excluded) carries the stride
            layers.append(ConvLayer(f"b{bi}_{i}.project", hidden, c, hw, hw, 1, 1, 1, 0))
            in_ch = c
    layers.append(ConvLayer("head", 320, 1280, 7, 7, 1, 1, 1, 0))
    assert len(layers) == 34
    return layers


def vgg16_convs() -> List[ConvLayer]:
    """The thirteen 3x3 pad-1 convolutions of VGG-16 at 224x224 input."""
    plan = [(3, 64, 224), (64, 64, 224), (64, 128, 112), (128, 128, 112), (128, 256, 56),
            (256, 256, 56), (256, 256, 56), (256, 512, 28), (512, 512, 28), (512, 512, 28),
            (512, 512, 14), (512, 512, 14), (512, 512, 14)]
    return [ConvLayer(f"conv{i + 1}", ci, co, hw, hw, 3, 3, 1, 1)
            for i, (ci, co, hw) in enumerate(plan)]


def layer_inputs(layer: ConvLayer, N: int, seed: int, bf16: bool) -> Tuple[np.ndarray, ...]:
    """(X, W, dY, is_bell, sigma) for one layer; all fp32 arrays (bf16-representable if bf16)."""
    x = activations(N, layer.Cin, layer.H, layer.W, seed)
    w = weights(layer.Cout, layer.Cin, layer.R, layer.S, seed)
    g, is_bell, sigma = channel_mixed_grad(N, layer.Cout, layer.P, layer.Q, seed)
    if bf16:
        x, w, g = round_to_bf16(x), round_to_bf16(w), round_to_bf16(g)
    return x, w, g, is_bell, sigma


def device_layer_inputs(layer: ConvLayer, N: int, seed: int, device):
    """The same recipes drawn by torch on `device` (for workloads too large to generate on the host
    in reasonable time): (X NHWC bf16, W (Cout,Cin,R,S) bf16, dY NHWC bf16).  The per-channel shape
    and sigma_c of dY come from the same seeded draw as channel_mixed_grad; the samples themselves
    are torch's, so these tensors feed timing runs, not comparisons with host-generated ones."""
    import torch
    gen = torch.Generator(device=device).manual_seed(int(seed) & 0x7FFFFFFF)
    bf = torch.bfloat16
    x = torch.randn((N, layer.H, layer.W, layer.Cin), device=device, generator=gen, dtype=torch.float32)
    x = torch.relu_(x).to(bf)
    w = torch.randn((layer.Cout, layer.Cin, layer.R, layer.S), device=device, generator=gen, dtype=torch.float32)
    w = (w * float(np.sqrt(2.0 / (layer.Cin * layer.R * layer.S)))).to(bf)
    meta = _rng(seed, 3)
    is_bell = torch.from_numpy(meta.random(layer.Cout) < 0.5).to(device)
    sigma = torch.from_numpy((10.0 ** meta.uniform(-6.0, -3.0, size=layer.Cout)).astype(np.float32)).to(device)
    g = torch.empty((N, layer.P, layer.Q, layer.Cout), device=device, dtype=bf)
    for n0 in range(0, N, 8):      # in slabs of 8 images to bound the fp32 temporaries
        n1 = min(N, n0 + 8)
        shape = (n1 - n0, layer.P, layer.Q, layer.Cout)
        normal = torch.randn(shape, device=device, generator=gen, dtype=torch.float32)
        # Laplace(0, b) by inversion: -b sign(u) ln(1 - 2|u|), u uniform in (-1/2, 1/2); b = sigma / sqrt(2)
        u = torch.rand(shape, device=device, generator=gen, dtype=torch.float32) - 0.5
        lap = -torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp_(max=0.49999997)) * (1.0 / np.sqrt(2.0))
        g[n0:n1] = (torch.where(is_bell, normal, lap) * sigma).to(bf)
    return x, w, g

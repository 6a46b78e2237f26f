"""Seeded synthetic inputs for the five benchmark configurations.

Serves both the CPU oracle's tests and the CUDA path's tests/bench.  It holds no
arithmetic of the method: it only draws bitwidths, integer codes, scales and fp32
tensors with numpy's counter-based ``default_rng``.  The synthetic tensors stand in
for the paper's CIFAR-10 (32x32) and ImageNet (224x224 crops) workloads: same tensor
shapes and code ranges, no dataset and no trained weights.

Codes are returned in the paper's order: activations ``[N, C, H, W]`` (unsigned,
``[0, 2^Ab - 1]``), weights ``[C_out, C_in, kh, kw]`` (signed two's complement,
``[-2^(Wb-1), 2^(Wb-1) - 1]``), dtype int32.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

from .nets import ConvLayer, gemm_as_conv, resnet18_imagenet, resnet50_imagenet, resnet_cifar


@dataclass(frozen=True)
class LayerSpec:
    """A layer plus everything drawn for it."""
    index: int
    layer: ConvLayer
    w_bits: int
    a_bits: int
    w_scale: float
    a_scale: float
    batch: int
    dist: str                 # "uniform" | "gaussian"
    seed: int


def _rng(seed: int, layer_index: int, stream: int) -> np.random.Generator:
    return np.random.default_rng([int(seed), int(layer_index), int(stream)])


def weight_codes(spec: LayerSpec) -> np.ndarray:
    L = spec.layer
    rng = _rng(spec.seed, spec.index, 0)
    lo, hi = -(1 << (spec.w_bits - 1)), (1 << (spec.w_bits - 1)) - 1
    shape = (L.c_out, L.c_in, L.k, L.k)
    if spec.dist == "uniform":
        return rng.integers(lo, hi + 1, size=shape, dtype=np.int32)
    z = rng.standard_normal(size=shape)
    return np.clip(np.floor(z * (1 << (spec.w_bits - 1)) / 3.0 + 0.5), lo, hi).astype(np.int32)


def act_codes(spec: LayerSpec, batch: Optional[int] = None, h_in: Optional[int] = None) -> np.ndarray:
    L = spec.layer
    rng = _rng(spec.seed, spec.index, 1)
    n = spec.batch if batch is None else batch
    h = L.h_in if h_in is None else h_in
    w = L.w_in if h_in is None else h_in
    hi = (1 << spec.a_bits) - 1
    shape = (n, L.c_in, h, w)
    if spec.dist == "uniform":
        return rng.integers(0, hi + 1, size=shape, dtype=np.int32)
    z = np.abs(rng.standard_normal(size=shape, dtype=np.float32))
    return np.clip(np.floor(z * (hi / 3.0) + 0.5), 0, hi).astype(np.int32)


def fp32_from_codes(codes: np.ndarray, scale: float, seed: int, jitter: float = 0.3) -> np.ndarray:
    """fp32 values that quantize back to ``codes`` at step ``scale`` (|jitter| < 0.5 steps)."""
    rng = np.random.default_rng([int(seed), 977])
    noise = rng.uniform(-jitter, jitter, size=codes.shape)
    return ((codes.astype(np.float64) + noise) * float(scale)).astype(np.float32)


def _draw(seed: int, layers: Sequence[ConvLayer], bit_choices: Sequence[int], batch: int, dist: str,
          a_bit_choices: Optional[Sequence[int]] = None) -> List[LayerSpec]:
    """Per-layer (Wb, Ab) in layer order, Wb then Ab; non-quantized layers stay at 8/8."""
    rng = np.random.default_rng(int(seed))
    wch = np.asarray(bit_choices)
    ach = np.asarray(bit_choices if a_bit_choices is None else a_bit_choices)
    specs = []
    for i, L in enumerate(layers):
        if L.quantized:
            wb = int(wch[rng.integers(0, len(wch))])
            ab = int(ach[rng.integers(0, len(ach))])
        else:
            wb, ab = 8, 8
        s_w, s_a = (float(v) for v in rng.uniform(0.01, 0.1, size=2))
        specs.append(LayerSpec(i, L, wb, ab, s_w, s_a, batch, dist, int(seed)))
    return specs


def config1(seed: int = 0) -> List[LayerSpec]:
    """One 3x3 convolution, N=1, 64->64 channels, 32x32, W2A2, uniform codes."""
    L = ConvLayer("c1_3x3_64", 64, 64, 3, 1, 1, 32, 32)
    rng = np.random.default_rng(int(seed))
    s_w, s_a = (float(v) for v in rng.uniform(0.01, 0.1, size=2))
    return [LayerSpec(0, L, 2, 2, s_w, s_a, 1, "uniform", int(seed))]


def config2(seed: int = 0, batch: int = 128) -> List[LayerSpec]:
    """CIFAR ResNet-20 stack, (Wb, Ab) in {1..4}^2, first conv and classifier at 8 bits."""
    return _draw(seed, resnet_cifar(3), [1, 2, 3, 4], batch, "uniform")


def config3(seed: int = 0, batch: int = 64) -> List[LayerSpec]:
    """ImageNet ResNet-18 quantized conv layers, (Wb, Ab) in {2..6}^2, Gaussian / half-normal codes."""
    layers = [L for L in resnet18_imagenet() if L.quantized]
    return _draw(seed, layers, [2, 3, 4, 5, 6], batch, "gaussian")


def config4(w_bits: int, a_bits: int, seed: int = 0, mg: int = 4096, ng: int = 4096,
            kg: int = 4096) -> LayerSpec:
    """One (Wb, Ab) point of the bit-plane GEMM sweep, as a 1x1 convolution over mg pixels."""
    L = gemm_as_conv(mg, ng, kg)
    return LayerSpec(w_bits * 8 + a_bits, L, w_bits, a_bits, 0.05, 0.05, 1, "uniform", int(seed))


def config5(seed: int = 0, batch: int = 256) -> List[LayerSpec]:
    """ImageNet ResNet-50 bottleneck stack, (Wb, Ab) in {2..8}^2, Gaussian weight codes.

    A shortcut convolution reads the same tensor as its block's first convolution,
    so it takes that layer's activation bitwidth.
    """
    layers = [L for L in resnet50_imagenet() if L.quantized]
    specs = _draw(seed, layers, [2, 3, 4, 5, 6, 7, 8], batch, "gaussian")
    by_name = {s.layer.name: s for s in specs}
    out = []
    for s in specs:
        if s.layer.role == "shortcut":
            first = by_name[s.layer.name[:-2] + "c1"]
            s = LayerSpec(s.index, s.layer, s.w_bits, first.a_bits, s.w_scale, first.a_scale, s.batch,
                          s.dist, s.seed)
        out.append(s)
    return out


def binary_ops(spec: LayerSpec, batch: Optional[int] = None) -> int:
    """2 * MACs * Wb * Ab: one AND and one bitcount-accumulate per bit pair (Sec. 4.3, complexity)."""
    n = spec.batch if batch is None else batch
    return 2 * n * spec.layer.macs * spec.w_bits * spec.a_bits


def resnet_cifar_network(blocks_per_stage: int, seed: int = 0, batch: int = 128) -> List[LayerSpec]:
    """A CIFAR ResNet (3/5/9 blocks per stage = ResNet-20/32/56) with config2's bitwidth recipe, wired as a
    network: a projection shortcut takes the activation bitwidth of its block's first convolution."""
    specs = _draw(seed, resnet_cifar(blocks_per_stage), [1, 2, 3, 4], batch, "uniform")
    return _share_shortcut_inputs(specs)


def resnet20_network(seed: int = 0, batch: int = 128) -> List[LayerSpec]:
    """The ResNet-20 stack of config2 wired as a network: a projection shortcut reads the same
    tensor as its block's first convolution, so it takes that layer's activation bitwidth."""
    return _share_shortcut_inputs(config2(seed, batch))


def resnet18_network(seed: int = 0, batch: int = 32) -> List[LayerSpec]:
    """The ImageNet ResNet-18 of config3 wired as a network (first convolution and classifier at 8 bits, a projection
    shortcut reads the same tensor as its block's first convolution); 224x224 images, a 3x3 stride-2 max pooling follows
    the first convolution."""
    return _share_shortcut_inputs(_draw(seed, resnet18_imagenet(), [2, 3, 4, 5, 6], batch, "gaussian"))


def _share_shortcut_inputs(specs: List[LayerSpec]) -> List[LayerSpec]:
    by_name = {s.layer.name: s for s in specs}
    out = []
    for s in specs:
        if s.layer.role == "shortcut":
            first = by_name[s.layer.name[:-2] + "c1"]
            s = LayerSpec(s.index, s.layer, s.w_bits, first.a_bits, s.w_scale, first.a_scale, s.batch, s.dist, s.seed)
        out.append(s)
    return out


def images_u8(seed: int, batch: int, h: int = 32, w: int = 32, c: int = 3) -> np.ndarray:
    """Synthetic 8-bit images [N, C, H, W]: smooth per-image gradients plus noise, so that pixel
    statistics differ between images and channels the way natural images' do."""
    rng = np.random.default_rng([int(seed), 4242])
    yy, xx = np.meshgrid(np.linspace(0, 1, h), np.linspace(0, 1, w), indexing="ij")
    gx = rng.uniform(-1, 1, size=(batch, c, 1, 1))
    gy = rng.uniform(-1, 1, size=(batch, c, 1, 1))
    base = rng.uniform(0.2, 0.8, size=(batch, c, 1, 1))
    img = base + 0.3 * gx * xx + 0.3 * gy * yy + 0.08 * rng.standard_normal(size=(batch, c, h, w))
    return np.clip(np.floor(img * 255.0 + 0.5), 0, 255).astype(np.int32)

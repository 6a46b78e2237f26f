"""Layer lists (shapes only) of the networks the paper evaluates, used to build synthetic workloads.

No arithmetic of the method lives here: a layer is a plain record of sizes.  The
CIFAR ResNets use 1x1 stride-2 convolution shortcuts, the only variant that
reproduces the multiply-accumulate totals the paper prints in Table 1 (40.81 M for
ResNet-20, 69.12 M for ResNet-32, 125.7 M for ResNet-56); ResNet-18 reproduces
Table 2's 1.82 G.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import List


@dataclass(frozen=True)
class ConvLayer:
    name: str
    c_in: int
    c_out: int
    k: int
    stride: int
    pad: int
    h_in: int
    w_in: int
    quantized: bool = True      # False: first conv / classifier, kept at 8 bits (Appendix B)
    role: str = "conv"          # "conv" | "shortcut" | "first" | "fc"

    @property
    def h_out(self) -> int:
        return (self.h_in + 2 * self.pad - self.k) // self.stride + 1

    @property
    def w_out(self) -> int:
        return (self.w_in + 2 * self.pad - self.k) // self.stride + 1

    @property
    def macs(self) -> int:
        """Multiply-accumulates per image."""
        return self.c_in * self.c_out * self.k * self.k * self.h_out * self.w_out


def _conv(name, c_in, c_out, k, stride, h, pad=None, **kw) -> ConvLayer:
    return ConvLayer(name, c_in, c_out, k, stride, k // 2 if pad is None else pad, h, h, **kw)


def resnet_cifar(blocks_per_stage: int, num_classes: int = 10) -> List[ConvLayer]:
    """ResNet-20/32/56 for 32x32 inputs (blocks_per_stage = 3/5/9)."""
    layers = [_conv("conv1", 3, 16, 3, 1, 32, quantized=False, role="first")]
    c_in, h = 16, 32
    for stage, c in enumerate([16, 32, 64]):
        for b in range(blocks_per_stage):
            stride = 2 if (stage > 0 and b == 0) else 1
            first = _conv(f"s{stage + 1}b{b + 1}c1", c_in, c, 3, stride, h)
            layers.append(first)
            layers.append(_conv(f"s{stage + 1}b{b + 1}c2", c, c, 3, 1, first.h_out))
            if stride == 2:
                layers.append(_conv(f"s{stage + 1}b{b + 1}ds", c_in, c, 1, 2, h, pad=0, role="shortcut"))
            c_in, h = c, first.h_out
    layers.append(ConvLayer("fc", 64, num_classes, 1, 1, 0, 1, 1, quantized=False, role="fc"))
    return layers


def resnet18_imagenet(num_classes: int = 1000) -> List[ConvLayer]:
    layers = [_conv("conv1", 3, 64, 7, 2, 224, pad=3, quantized=False, role="first")]
    c_in, h = 64, 56            # after the 3x3 stride-2 max pool
    for stage, c in enumerate([64, 128, 256, 512]):
        for b in range(2):
            stride = 2 if (stage > 0 and b == 0) else 1
            first = _conv(f"l{stage + 1}b{b + 1}c1", c_in, c, 3, stride, h)
            layers.append(first)
            layers.append(_conv(f"l{stage + 1}b{b + 1}c2", c, c, 3, 1, first.h_out))
            if stride == 2:
                layers.append(_conv(f"l{stage + 1}b{b + 1}ds", c_in, c, 1, 2, h, pad=0, role="shortcut"))
            c_in, h = c, first.h_out
    layers.append(ConvLayer("fc", 512, num_classes, 1, 1, 0, 1, 1, quantized=False, role="fc"))
    return layers


def resnet50_imagenet(num_classes: int = 1000) -> List[ConvLayer]:
    """Bottleneck ResNet-50 with the stride on the 3x3 convolution of a stage's first block."""
    layers = [_conv("conv1", 3, 64, 7, 2, 224, pad=3, quantized=False, role="first")]
    c_in, h = 64, 56
    for stage, (width, blocks) in enumerate(zip([64, 128, 256, 512], [3, 4, 6, 3])):
        for b in range(blocks):
            stride = 2 if (stage > 0 and b == 0) else 1
            tag = f"l{stage + 1}b{b + 1}"
            layers.append(_conv(tag + "c1", c_in, width, 1, 1, h, pad=0))
            mid = _conv(tag + "c2", width, width, 3, stride, h)
            layers.append(mid)
            layers.append(_conv(tag + "c3", width, 4 * width, 1, 1, mid.h_out, pad=0))
            if b == 0:
                layers.append(_conv(tag + "ds", c_in, 4 * width, 1, stride, h, pad=0, role="shortcut"))
            c_in, h = 4 * width, mid.h_out
    layers.append(ConvLayer("fc", 2048, num_classes, 1, 1, 0, 1, 1, quantized=False, role="fc"))
    return layers


def gemm_as_conv(mg: int, ng: int, kg: int) -> ConvLayer:
    """A bit-plane GEMM (mg x kg) by (kg x ng) expressed as a 1x1 convolution over mg pixels."""
    side = int(round(mg ** 0.5))
    assert side * side == mg, "mg must be a perfect square to lay the rows out as an image"
    return ConvLayer("gemm", kg, ng, 1, 1, 0, side, side)


def total_macs(layers: List[ConvLayer]) -> int:
    return sum(layer.macs for layer in layers)


def scaled(layer: ConvLayer, h_in: int) -> ConvLayer:
    """The same layer on a smaller image (for oracle-sized parity cases)."""
    return replace(layer, h_in=h_in, w_in=h_in)

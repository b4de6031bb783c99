"""Layer shapes of the five workloads and the paper's memory-transfer model.

Pure data and integer arithmetic; no device code is touched here.

The byte model is Sec. 6 of the paper: Eq. 4 (static quantization: weights + input +
8-bit output) and Eq. 5 (dynamic quantization: weights + input + 32-bit output written,
32-bit output read back, 8-bit output written), with b_w = b_a = 8 and b_acc = 32.
"""
from __future__ import annotations

from dataclasses import dataclass, replace


@dataclass(frozen=True)
class ConvShape:
    name: str
    N: int
    H: int
    W: int
    C: int          # input channels
    K: int          # output channels
    R: int = 1
    S: int = 1
    stride: int = 1
    pad: int = 0
    groups: int = 1

    @property
    def Ho(self) -> int:
        return (self.H + 2 * self.pad - self.R) // self.stride + 1

    @property
    def Wo(self) -> int:
        return (self.W + 2 * self.pad - self.S) // self.stride + 1

    @property
    def depthwise(self) -> bool:
        return self.groups != 1

    def with_batch(self, n: int) -> "ConvShape":
        return replace(self, N=n)

    # ---- algorithmic work -------------------------------------------------------
    @property
    def weight_elems(self) -> int:
        return self.K * self.R * self.S * (1 if self.depthwise else self.C)

    @property
    def in_elems(self) -> int:
        return self.N * self.H * self.W * self.C

    @property
    def out_elems(self) -> int:
        return self.N * self.Ho * self.Wo * self.K

    @property
    def ops(self) -> int:
        """2 x multiply-accumulates of the dense definition (padding taps counted)."""
        k = self.R * self.S * (1 if self.depthwise else self.C)
        return 2 * self.out_elems * k


@dataclass(frozen=True)
class LinearShape:
    name: str
    M: int
    N: int
    K: int

    @property
    def weight_elems(self) -> int:
        return self.N * self.K

    @property
    def in_elems(self) -> int:
        return self.M * self.K

    @property
    def out_elems(self) -> int:
        return self.M * self.N

    @property
    def ops(self) -> int:
        return 2 * self.M * self.N * self.K


def static_bytes(weight_elems: int, in_elems: int, out_elems: int, b_w: int = 8, b_a: int = 8) -> float:
    """Eq. 4: bits moved with a range known in advance, returned in bytes."""
    return (weight_elems * b_w + in_elems * b_a + out_elems * b_a) / 8.0


def dynamic_bytes(weight_elems: int, in_elems: int, out_elems: int, b_w: int = 8, b_a: int = 8, b_acc: int = 32) -> float:
    """Eq. 5: the accumulator output is saved, loaded again, then saved quantized."""
    return (weight_elems * b_w + in_elems * b_a + 2 * out_elems * b_acc + out_elems * b_a) / 8.0


def layer_static_bytes(s, bwd: bool = False) -> float:
    """Eq. 4 for a layer; backward data swaps the roles of input and output (Sec. 6)."""
    i, o = (s.out_elems, s.in_elems) if bwd else (s.in_elems, s.out_elems)
    return static_bytes(s.weight_elems, i, o)


def layer_dynamic_bytes(s, bwd: bool = False) -> float:
    i, o = (s.out_elems, s.in_elems) if bwd else (s.in_elems, s.out_elems)
    return dynamic_bytes(s.weight_elems, i, o)


# ---- the five workloads -------------------------------------------------------------
CFG1_LINEAR = LinearShape("linear256", M=256, N=128, K=256)
CFG2_CONV = ConvShape("resnet_conv3x3_64", N=64, H=56, W=56, C=64, K=64, R=3, S=3, stride=1, pad=1)
# backward data of a 256->256 3x3 conv at 14x14: the forward layer's shape is given, dY has its output shape
CFG3_BWD = ConvShape("resnet_conv3x3_256_bwd", N=256, H=14, W=14, C=256, K=256, R=3, S=3, stride=1, pad=1)
CFG4_EXPAND = ConvShape("mbv2_expand", N=256, H=56, W=56, C=24, K=144)
CFG4_DW = ConvShape("mbv2_dw3x3", N=256, H=56, W=56, C=144, K=144, R=3, S=3, stride=1, pad=1, groups=144)
CFG4_PROJECT = ConvShape("mbv2_project", N=256, H=56, W=56, C=144, K=24)


def resnet18_layers(batch: int = 128):
    """All convolutions of ResNet-18 at 224x224 plus the final linear layer.

    Returns (convs, fc): convs is a list of ConvShape in network order (stem, then
    per stage the 3x3 convolutions and the 1x1 stride-2 shortcut), fc a LinearShape.
    """
    L = [ConvShape("stem7x7", batch, 224, 224, 3, 64, 7, 7, 2, 3)]
    L += [ConvShape(f"layer1.{i}", batch, 56, 56, 64, 64, 3, 3, 1, 1) for i in range(4)]
    c, h = 64, 56
    for stage in (2, 3, 4):
        k = 2 * c
        L.append(ConvShape(f"layer{stage}.0a", batch, h, h, c, k, 3, 3, 2, 1))
        L.append(ConvShape(f"layer{stage}.ds", batch, h, h, c, k, 1, 1, 2, 0))
        h //= 2
        L += [ConvShape(f"layer{stage}.{i}", batch, h, h, k, k, 3, 3, 1, 1) for i in range(1, 4)]
        c = k
    return L, LinearShape("fc", batch, 1000, 512)

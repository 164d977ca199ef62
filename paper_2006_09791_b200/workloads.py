"""Layer tables of the synthetic workloads and the per-layer cost model (MACs, compulsory bytes).

Shapes follow the networks the paper measures (WideResNet-40-2 on 32x32 images, ResNet-34 on
224x224 images, Section IV-A) with every 3x3 convolution read as a grouped 3x3 convolution, plus a
ResNeXt-50-32x4d-shaped family and a group-count sweep down to depthwise.  The MAC count is
Eq. (2) of the paper.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import List


@dataclass(frozen=True)
class Layer:
    name: str
    N: int
    C_in: int
    H: int
    W: int
    C_out: int
    KH: int = 3
    KW: int = 3
    stride: int = 1
    pad: int = 1
    dilation: int = 1
    groups: int = 1
    x_dist: str = "uniform"
    repeat: int = 1  # how many times the layer occurs in its stack

    @property
    def Cg(self) -> int:
        return self.C_in // self.groups

    @property
    def Kg(self) -> int:
        return self.C_out // self.groups

    @property
    def H_out(self) -> int:
        return (self.H + 2 * self.pad - self.dilation * (self.KH - 1) - 1) // self.stride + 1

    @property
    def W_out(self) -> int:
        return (self.W + 2 * self.pad - self.dilation * (self.KW - 1) - 1) // self.stride + 1

    @property
    def macs(self) -> int:
        """Eq. (2): N*C_in*C_out*KH*KW*H_out*W_out / g."""
        return self.N * self.C_in * self.C_out * self.KH * self.KW * self.H_out * self.W_out // self.groups

    @property
    def flops(self) -> int:
        return 2 * self.macs

    @property
    def x_elems(self) -> int:
        return self.N * self.C_in * self.H * self.W

    @property
    def y_elems(self) -> int:
        return self.N * self.C_out * self.H_out * self.W_out

    @property
    def w_elems(self) -> int:
        return self.C_out * self.Cg * self.KH * self.KW

    @property
    def compulsory_bytes(self) -> int:
        """x read once + y written once + w read once, fp32."""
        return 4 * (self.x_elems + self.y_elems + self.w_elems)

    def desc_args(self):
        return (self.N, self.C_in, self.H, self.W, self.C_out, self.KH, self.KW, self.stride, self.pad,
                self.dilation, self.groups)

    def with_(self, **kw) -> "Layer":
        return replace(self, **kw)


def config0() -> List[Layer]:
    """Single small layer: 64->64 @16x16, 3x3, groups 4, N=1."""
    return [Layer("cfg0_64x16_g4", 1, 64, 16, 16, 64, groups=4)]


def wrn_stack(groups: int, N: int) -> List[Layer]:
    """WideResNet-40-2-shaped stack: channels 32/64/128 at 32/16/8, six 3x3 layers per stage, the
    first layer of stages 2 and 3 has stride 2 and widens the channel count."""
    g = groups
    return [
        Layer("wrn_s1_32@32", N, 32, 32, 32, 32, groups=g, repeat=6),
        Layer("wrn_s2t_32-64@32s2", N, 32, 32, 32, 64, stride=2, groups=g, repeat=1),
        Layer("wrn_s2_64@16", N, 64, 16, 16, 64, groups=g, repeat=5),
        Layer("wrn_s3t_64-128@16s2", N, 64, 16, 16, 128, stride=2, groups=g, repeat=1),
        Layer("wrn_s3_128@8", N, 128, 8, 8, 128, groups=g, repeat=5),
    ]


WRN_GROUPS = (1, 2, 4, 8, 16)
WRN_BATCHES = (1, 128)


def resnet34_layers(groups: int, N: int) -> List[Layer]:
    """ResNet-34-shaped 3x3 layers at 224x224 input: 64/128/256/512 channels at 56/28/14/7."""
    g = groups
    return [
        Layer("r34_64@56", N, 64, 56, 56, 64, groups=g),
        Layer("r34_64-128@56s2", N, 64, 56, 56, 128, stride=2, groups=g),
        Layer("r34_128@28", N, 128, 28, 28, 128, groups=g),
        Layer("r34_128-256@28s2", N, 128, 28, 28, 256, stride=2, groups=g),
        Layer("r34_256@14", N, 256, 14, 14, 256, groups=g),
        Layer("r34_256-512@14s2", N, 256, 14, 14, 512, stride=2, groups=g),
        Layer("r34_512@7", N, 512, 7, 7, 512, groups=g),
    ]


R34_GROUPS = (1, 2, 4, 8, 16, 32)
R34_BATCHES = (1, 64)


def resnext_layers(N: int = 64) -> List[Layer]:
    """ResNeXt-50-32x4d-shaped bottleneck middle convs: 3x3, 32 groups, N(0,1) inputs."""
    mk = lambda name, C, HW, s: Layer(name, N, C, HW, HW, C, stride=s, groups=32, x_dist="normal")
    return [
        mk("rx_128@56", 128, 56, 1), mk("rx_256@56s2", 256, 56, 2), mk("rx_256@28", 256, 28, 1),
        mk("rx_512@28s2", 512, 28, 2), mk("rx_512@14", 512, 14, 1), mk("rx_1024@14s2", 1024, 14, 2),
        mk("rx_1024@7", 1024, 7, 1),
    ]


SWEEP_GROUPS = (1, 2, 4, 8, 16, 32, 64, 128, 256)


def sweep_layers(N: int = 32) -> List[Layer]:
    """Group-count sweep to depthwise: 256->256 @56x56, 3x3, stride 1, pad 1."""
    return [Layer("sweep_256@56_g%d" % g, N, 256, 56, 56, 256, groups=g) for g in SWEEP_GROUPS]


def mobilenetv2_dw_layers(N: int = 64) -> List[Layer]:
    """MobileNetV2-shaped depthwise 3x3 layers at 224x224 input (the paper's third network, whose default
    architecture is the G(N) model): expansion widths 32...960 at spatial 112...7, stride 1 and 2."""
    mk = lambda C, HW, s: Layer("mbv2_dw_%d@%d%s" % (C, HW, "s2" if s == 2 else ""), N, C, HW, HW, C, stride=s, groups=C)
    return [mk(32, 112, 1), mk(96, 112, 2), mk(144, 56, 1), mk(144, 56, 2), mk(192, 28, 1), mk(192, 28, 2),
            mk(384, 14, 1), mk(576, 14, 1), mk(576, 14, 2), mk(960, 7, 1)]


def depthwise5x5_layers(N: int = 64) -> List[Layer]:
    """Depthwise 5x5 layers (pad 2, stride 1 and 2) at the sizes later mobile networks use them: 56x56 down to 7x7,
    widths 72...960.  The second depthwise family of the follow-up items."""
    mk = lambda C, HW, s: Layer("dw5_%d@%d%s" % (C, HW, "s2" if s == 2 else ""), N, C, HW, HW, C, 5, 5, s, 2, 1, C)
    return [mk(72, 56, 2), mk(120, 28, 1), mk(240, 28, 2), mk(672, 14, 1), mk(672, 14, 2), mk(960, 7, 1)]


def fused_blocks(N: int = 128):
    """(grouped 3x3 layer, pointwise output channels) pairs of the paper's G(g) block -- a grouped 3x3 followed by a
    pointwise convolution (Section II) -- at the three stages of the WRN-40-2-shaped stack, plus two ResNeXt-shaped
    blocks (56x56 and 28x28 planes, 4-channel groups)."""
    out = []
    for g in (2, 4, 8, 16):
        out.append((Layer("blk32@32", N, 32, 32, 32, 32, groups=g), 32))
    out.append((Layer("blk64@16", N, 64, 16, 16, 64, groups=4), 64))
    out.append((Layer("blk128@8", N, 128, 8, 8, 128, groups=8), 128))
    out.append((Layer("blk64@56", N // 2, 64, 56, 56, 64, groups=16), 64))
    out.append((Layer("blk128@28", N // 2, 128, 28, 28, 128, groups=32), 64))
    return out


def pointwise_layers(N: int = 64) -> List[Layer]:
    """Pointwise (1x1, pad 0, groups = 1) layers: the second half of the paper's G(g) block at the three stages of the
    WRN-40-2-shaped stack (batch 2N), and the 1x1 layers around a ResNeXt-shaped grouped 3x3 (56x56, 28x28, 14x14)."""
    mk = lambda n, ci, hw, co, s=1: Layer("pw_%d-%d@%d%s" % (ci, co, hw, "s2" if s == 2 else ""), n, ci, hw, hw, co, 1, 1, s, 0, 1, 1)
    return [mk(2 * N, 32, 32, 32), mk(2 * N, 64, 16, 64), mk(2 * N, 128, 8, 128), mk(N, 256, 56, 128), mk(N, 128, 56, 256),
            mk(N, 512, 28, 256), mk(N, 512, 14, 512), mk(N, 256, 56, 512, 2)]

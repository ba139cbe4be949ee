"""Layer shapes of the paper's three CIFAR-10 networks (Section 3): ResNet-20, VGG-19 and the
two-layer CNN, as lists of convolution geometries.  Only shapes live here; no arithmetic of the
method.  Every convolution is described by ConvLayer (batch n, input c x h x w, k filters of r x s,
stride, zero padding)."""
from __future__ import annotations

from dataclasses import dataclass, replace


@dataclass(frozen=True)
class ConvLayer:
    name: str
    n: int
    c: int
    h: int
    w: int
    k: int
    r: int
    s: int
    stride: int = 1
    pad: int = 0
    x_dist: str = "relu_normal"   # value recipe for X: "relu_normal" or "uniform_pm1"
    dy_std: float = 0.01          # dY ~ N(0, dy_std^2)

    @property
    def p(self) -> int:
        return (self.h + 2 * self.pad - self.r) // self.stride + 1

    @property
    def q(self) -> int:
        return (self.w + 2 * self.pad - self.s) // self.stride + 1

    def with_batch(self, n: int) -> "ConvLayer":
        return replace(self, n=n)

    # algorithmic work of one filter-gradient evaluation
    def flops_exact(self) -> int:
        return 2 * self.n * self.k * self.c * self.r * self.s * self.p * self.q

    def bytes_exact(self, elem_bytes: int) -> int:
        return (self.n * self.c * self.h * self.w + self.n * self.k * self.p * self.q) * elem_bytes \
            + self.k * self.c * self.r * self.s * 4

    def bytes_top1(self, elem_bytes: int) -> int:
        patches = self.n * self.k * self.r * self.s * self.c * elem_bytes
        x_all = self.n * self.c * self.h * self.w * elem_bytes
        return self.n * self.k * self.p * self.q * elem_bytes + min(patches, x_all) \
            + self.k * self.c * self.r * self.s * 4

    def fma_top1(self) -> int:
        return self.n * self.k * self.c * self.r * self.s


def _c3(name, n, c, k, hw, stride=1, **kw):
    return ConvLayer(name, n, c, hw, hw, k, 3, 3, stride, 1, **kw)


def config1_layer() -> ConvLayer:
    """Single 3x3 layer, 16 -> 16 channels at 32x32, batch 8, dY ~ N(0,1)."""
    return ConvLayer("c1 16->16@32", 8, 16, 32, 32, 16, 3, 3, 1, 1, dy_std=1.0)


def resnet20_layers(n: int = 128) -> list[ConvLayer]:
    """The 19 3x3 convolutions of ResNet-20 for CIFAR-10 (no projection shortcuts)."""
    ls = [_c3("stem 3->16@32", n, 3, 16, 32)]
    ls += [_c3("16->16@32", n, 16, 16, 32) for _ in range(6)]
    ls += [_c3("16->32@32s2", n, 16, 32, 32, 2)]
    ls += [_c3("32->32@16", n, 32, 32, 16) for _ in range(5)]
    ls += [_c3("32->64@16s2", n, 32, 64, 16, 2)]
    ls += [_c3("64->64@8", n, 64, 64, 8) for _ in range(5)]
    return ls


def vgg19_layers(n: int = 128) -> list[ConvLayer]:
    """The 16 3x3 convolutions of VGG-19 on 32x32 inputs."""
    spec = [(3, 64, 32), (64, 64, 32), (64, 128, 16), (128, 128, 16), (128, 256, 8)] \
        + [(256, 256, 8)] * 3 + [(256, 512, 4)] + [(512, 512, 4)] * 3 + [(512, 512, 2)] * 4
    return [_c3("%d->%d@%d" % (c, k, hw), n, c, k, hw) for c, k, hw in spec]


def cnn2_layers(n: int = 128) -> list[ConvLayer]:
    """The two 5x5 convolutions of the two-layer CIFAR-10 CNN (a 3x3 stride-2 max-pool sits between)."""
    return [ConvLayer("conv1 5x5 3->64@32", n, 3, 32, 32, 64, 5, 5, 1, 2, x_dist="uniform_pm1"),
            ConvLayer("conv2 5x5 64->64@16", n, 64, 16, 16, 64, 5, 5, 1, 2)]


def layer_set(config: int, n: int | None = None) -> list[ConvLayer]:
    """Layer list of workload `config`: 1 single layer, 2 ResNet-20, 3 two-layer CNN, 4 VGG-19."""
    if config == 1:
        return [config1_layer() if n is None else config1_layer().with_batch(n)]
    if config == 2:
        return resnet20_layers(128 if n is None else n)
    if config == 3:
        return cnn2_layers(128 if n is None else n)
    if config == 4:
        return vgg19_layers(128 if n is None else n)
    raise ValueError("config must be 1..4")

"""Seeded synthetic inputs and the workload table.

Holds none of the method's arithmetic: only a counter-based random generator
(the splitmix64 finaliser applied to seed, tensor id and flat index),
bf16 rounding of inputs, and the shapes of the workloads.  Both the CPU
checker and the CUDA path are fed from here; neither is imported here.

The paper measures on no dataset; the convolution shapes are ResNet-50 layer
shapes used as shapes only, with random activations and He-style random
weights standing in for a trained network.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _splitmix64(x: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = x + np.uint64(0x9E3779B97F4A7C15)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        return z ^ (z >> np.uint64(31))


def _bits(seed: int, tensor_id: int, count: int, lane: int = 0) -> np.ndarray:
    base = (int(seed) * 0x9E3779B97F4A7C15 + (int(tensor_id) << 40) + (int(lane) << 36)) & 0xFFFFFFFFFFFFFFFF
    idx = np.arange(count, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _splitmix64(_splitmix64(np.uint64(base) + idx))


def _unit(seed, tensor_id, count, lane=0) -> np.ndarray:
    """Uniform in [0,1) from the top 24 bits."""
    return (_bits(seed, tensor_id, count, lane) >> np.uint64(40)).astype(np.float64) / float(1 << 24)


def uniform(seed: int, tensor_id: int, shape, lo: float, hi: float) -> np.ndarray:
    n = int(np.prod(shape, dtype=np.int64))
    return (lo + (hi - lo) * _unit(seed, tensor_id, n)).astype(np.float32).reshape(shape)


def uniform_int(seed: int, tensor_id: int, shape, lo: int, hi: int) -> np.ndarray:
    """Integers uniform in [lo, hi], returned as float32."""
    n = int(np.prod(shape, dtype=np.int64))
    span = np.uint64(hi - lo + 1)
    vals = (_bits(seed, tensor_id, n) >> np.uint64(11)) % span
    return (vals.astype(np.int64) + lo).astype(np.float32).reshape(shape)


def normal(seed: int, tensor_id: int, shape, std: float = 1.0) -> np.ndarray:
    """N(0, std^2) by Box-Muller on two uniform streams."""
    n = int(np.prod(shape, dtype=np.int64))
    u1 = 1.0 - _unit(seed, tensor_id, n, lane=1)       # (0,1]
    u2 = _unit(seed, tensor_id, n, lane=2)
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)
    return (std * z).astype(np.float32).reshape(shape)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_round(x: np.ndarray) -> np.ndarray:
    """float32 -> nearest bf16, returned as float32."""
    return (bf16_bits(x).astype(np.uint32) << np.uint32(16)).view(np.float32).reshape(np.shape(x))


# --------------------------------------------------------------------------
# Workloads
# --------------------------------------------------------------------------

BASE_SEED = 20210509


@dataclass(frozen=True)
class ConvCase:
    name: str
    n: int
    c: int
    h: int
    w: int
    o: int
    kh: int
    kw: int
    stride: int
    pad: int
    integer: bool = False

    @property
    def ho(self):
        return (self.h + 2 * self.pad - self.kh) // self.stride + 1

    @property
    def wo(self):
        return (self.w + 2 * self.pad - self.kw) // self.stride + 1

    @property
    def m(self):
        return self.n * self.ho * self.wo

    @property
    def kd(self):
        return self.c * self.kh * self.kw

    @property
    def flops(self):
        return 2.0 * self.m * self.o * self.kd

    @property
    def algorithmic_bytes(self):
        """bf16 activations (only the rows and columns some window touches) and weights read
        once, fp32 result written once."""
        def touched(extent, out, k):
            return min(extent, out * k if k < self.stride else (out - 1) * self.stride + k)
        cells = touched(self.h, self.ho, self.kh) * touched(self.w, self.wo, self.kw)
        return 2 * self.n * self.c * cells + 2 * self.o * self.kd + 4 * self.m * self.o

    def inputs(self, seed: int):
        """(activations NCHW, weights OCKhKw) as float32 arrays of bf16 values."""
        if self.integer:
            x = uniform_int(seed, 1, (self.n, self.c, self.h, self.w), -3, 3)
            wt = uniform_int(seed, 2, (self.o, self.c, self.kh, self.kw), -3, 3)
        else:
            x = normal(seed, 1, (self.n, self.c, self.h, self.w), 1.0)
            wt = normal(seed, 2, (self.o, self.c, self.kh, self.kw), math.sqrt(2.0 / self.kd))
        return bf16_round(x), bf16_round(wt)


CONV_TINY = ConvCase("conv_tiny_1x3x8x8_k3", 1, 3, 8, 8, 4, 3, 3, 1, 0, integer=True)

CONV_SWEEP_3X3 = (
    ConvCase("conv3x3_56x56x64", 32, 64, 56, 56, 64, 3, 3, 1, 1),
    ConvCase("conv3x3_28x28x128", 32, 128, 28, 28, 128, 3, 3, 1, 1),
    ConvCase("conv3x3_14x14x256", 32, 256, 14, 14, 256, 3, 3, 1, 1),
    ConvCase("conv3x3_7x7x512", 32, 512, 7, 7, 512, 3, 3, 1, 1),
)

CONV_STRIDED_1X1 = (
    ConvCase("conv7x7s2_224x224x3", 32, 3, 224, 224, 64, 7, 7, 2, 3),
    ConvCase("conv1x1s2_56x56x256", 32, 256, 56, 56, 128, 1, 1, 2, 0),
    ConvCase("conv1x1_14x14x1024", 32, 1024, 14, 14, 256, 1, 1, 1, 0),
)


@dataclass(frozen=True)
class DenseCase:
    name: str
    m: int
    o: int
    k: int

    @property
    def flops(self):
        return 2.0 * self.m * self.o * self.k

    @property
    def algorithmic_bytes(self):
        return 2 * self.m * self.k + 2 * self.o * self.k + 4 * self.m * self.o

    def inputs(self, seed: int):
        a = bf16_round(normal(seed, 1, (self.m, self.k)))
        b = bf16_round(normal(seed, 2, (self.o, self.k)))
        return a, b


DENSE_4096 = DenseCase("dense_4096x4096x4096_relu", 4096, 4096, 4096)


@dataclass(frozen=True)
class MemCase:
    name: str
    kind: str                 # "im2col" | "transpose" | "maxpool" | "relu" | "pad"
    shape: tuple              # NCHW
    window: tuple = ()
    stride: int = 1
    pad: int = 0
    perm: tuple = ()

    def inputs(self, seed: int):
        return uniform(seed, 1, self.shape, -1.0, 1.0)

    @property
    def out_hw(self):
        n, c, h, w = self.shape
        kh, kw = self.window
        return (h + 2 * self.pad - kh) // self.stride + 1, (w + 2 * self.pad - kw) // self.stride + 1

    @property
    def algorithmic_bytes(self):
        n, c, h, w = self.shape
        src = 4 * n * c * h * w
        if self.kind in ("transpose", "relu"):
            return 2 * src
        if self.kind == "pad":        # one border cell on each side of the last dimension
            return src + 4 * n * c * h * (w + 2 * self.pad)
        ho, wo = self.out_hw
        if self.kind == "im2col":
            return src + 4 * n * ho * wo * c * self.window[0] * self.window[1]
        return src + 4 * n * c * ho * wo


MEM_IM2COL = MemCase("im2col_32x64x56x56_k3p1", "im2col", (32, 64, 56, 56), (3, 3), 1, 1)
MEM_TRANSPOSE = MemCase("transpose_nchw_nhwc_32x256x56x56", "transpose", (32, 256, 56, 56), perm=(0, 2, 3, 1))
MEM_RELU = MemCase("relu_4096x4096", "relu", (1, 1, 4096, 4096))
MEM_PAD = MemCase("pad_w1_32x64x56x56", "pad", (32, 64, 56, 56), pad=1)
MEM_MAXPOOL = MemCase("maxpool3x3s2p1_32x64x112x112", "maxpool", (32, 64, 112, 112), (3, 3), 2, 1)


@dataclass(frozen=True)
class ChainCase:
    """The kernels of Fig. 2 composed into one program at the scale of a ResNet stem:
    conv 7x7 stride 2 pad 3 (3 -> c1) + relu, max pool 3x3 stride 2 pad 1, conv 3x3 pad 1 (c1 -> c2) + relu,
    max pool `pool2` x `pool2` with that stride, flatten per image, dense layer to `units` outputs.
    Layer results are stored as bf16 (the next layer's operand type); the dense layer's result is fp32."""
    name: str
    n: int
    h: int
    w: int
    c1: int
    c2: int
    pool2: int
    units: int
    integer: bool = False

    def dims(self):
        h1, w1 = (self.h + 6 - 7) // 2 + 1, (self.w + 6 - 7) // 2 + 1          # conv 7x7 s2 p3
        h2, w2 = (h1 + 2 - 3) // 2 + 1, (w1 + 2 - 3) // 2 + 1                  # pool 3x3 s2 p1
        h3, w3 = (h2 - self.pool2) // self.pool2 + 1, (w2 - self.pool2) // self.pool2 + 1
        return (h1, w1), (h2, w2), (h3, w3)

    @property
    def features(self):
        return self.c2 * self.dims()[2][0] * self.dims()[2][1]

    @property
    def flops(self):
        (h1, w1), (h2, w2), _ = self.dims()
        return 2.0 * self.n * (h1 * w1 * self.c1 * 147 + h2 * w2 * self.c2 * 9 * self.c1 + self.units * self.features)

    @property
    def algorithmic_bytes(self):
        """Every layer reads its operands once and writes its result once (bf16 between layers, fp32 at the end)."""
        (h1, w1), (h2, w2), (h3, w3) = self.dims()
        acts = (self.h * self.w * 3, h1 * w1 * self.c1, h2 * w2 * self.c1, h2 * w2 * self.c2, h3 * w3 * self.c2)
        moved = acts[0] + 2 * sum(acts[1:])                       # each intermediate written once and read once
        weights = self.c1 * 147 + self.c2 * 9 * self.c1 + self.units * self.features
        return 2 * (self.n * moved + weights) + 4 * self.n * self.units

    def inputs(self, seed: int):
        """(image NCHW, conv1 weights, conv2 weights, dense weights [units, (c2, h3, w3)]) as float32 arrays of
        bf16 values.  The integer variant draws from {-1, 0, 1}: every layer's sums are then exact in fp32."""
        (h3, w3) = self.dims()[2]
        shapes = ((self.n, 3, self.h, self.w), (self.c1, 3, 7, 7), (self.c2, self.c1, 3, 3), (self.units, self.c2, h3, w3))
        if self.integer:
            return tuple(uniform_int(seed, i + 1, shp, -1, 1) for i, shp in enumerate(shapes))
        fan = (1.0, 147.0, 9.0 * self.c1, float(self.features))
        return tuple(bf16_round(normal(seed, i + 1, shp, 1.0 if i == 0 else math.sqrt(2.0 / fan[i])))
                     for i, shp in enumerate(shapes))


CHAIN_STEM = ChainCase("chain_stem_32x224x224", 32, 224, 224, 64, 64, 8, 1000)


def config_seed(config_index: int) -> int:
    return BASE_SEED + config_index

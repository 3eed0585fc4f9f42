"""Seeded synthetic inputs shaped like the paper's CNN workloads.

This module only draws random tensors and picks the quantizer parameters the
paper's experiments start from (Sec. VI-B.3: step sizes from the mean absolute
value, b bits).  It holds none of the quantizer's or the layer's arithmetic
and is the one module used both by the CUDA path's callers and by the tests
that drive the CPU oracle, so that both sides always see the same bits.

Everything is generated on the host with numpy's PCG64 from an explicit seed.
The tensors stand in for CIFAR-100 / ImageNet layer tensors (Sec. VI-C, VI-D):
He-normal weights, post-ReLU (half-normal or rectified-normal) activations,
N(0,1) / Laplace(0,1) mixtures for the bandwidth sweep.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


def _rng(seed: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([int(seed), int(stream)]))


def normal(shape, std: float, seed: int, stream: int = 0) -> np.ndarray:
    return (_rng(seed, stream).standard_normal(shape, dtype=np.float32) * np.float32(std)).astype(np.float32)


def relu_normal(shape, seed: int, stream: int = 0) -> np.ndarray:
    """max(0, N(0,1)): about half of the entries are exactly 0."""
    return np.maximum(_rng(seed, stream).standard_normal(shape, dtype=np.float32), np.float32(0))


def half_normal(shape, seed: int, stream: int = 0) -> np.ndarray:
    """|N(0,1)|."""
    return np.abs(_rng(seed, stream).standard_normal(shape, dtype=np.float32))


def he_normal(fan_in: int, shape, seed: int, stream: int = 0) -> np.ndarray:
    return normal(shape, float(np.sqrt(2.0 / fan_in)), seed, stream)


def laplace(shape, seed: int, stream: int = 0) -> np.ndarray:
    return _rng(seed, stream).laplace(0.0, 1.0, shape).astype(np.float32)


def normal_laplace_mixture(shape, seed: int, stream: int = 0) -> np.ndarray:
    """Element-wise 50/50 mixture of N(0,1) and Laplace(0,1)."""
    r = _rng(seed, stream)
    a = r.standard_normal(shape, dtype=np.float32)
    b = r.laplace(0.0, 1.0, shape).astype(np.float32)
    pick = r.random(shape, dtype=np.float32) < np.float32(0.5)
    return np.where(pick, a, b).astype(np.float32)


def step_from_mean_abs(t: np.ndarray, bits: int) -> float:
    """Initial step size of Sec. VI-B.3: 2 * mean|t| / sqrt(2^(bits-1)), as a binary32 value."""
    m = float(np.mean(np.abs(t.astype(np.float64))))
    return float(np.float32(2.0 * m / np.sqrt(2.0 ** (bits - 1))))


def indices_from_histogram(shape, hist: np.ndarray, lo: int, seed: int, stream: int = 0) -> np.ndarray:
    """Index matrix (int8 if lo < 0 else uint8) whose entries follow the level histogram `hist`."""
    p = hist.astype(np.float64) / float(hist.sum())
    cdf = np.cumsum(p)
    cdf[-1] = 1.0
    u = _rng(seed, stream).random(shape, dtype=np.float32)
    k = np.searchsorted(cdf, u, side="right").astype(np.int64)
    k = np.minimum(k, hist.size - 1) + lo
    return k.astype(np.int8 if lo < 0 else np.uint8)


def uniform_indices(shape, lo: int, hi: int, seed: int, stream: int = 0) -> np.ndarray:
    k = _rng(seed, stream).integers(lo, hi + 1, size=shape)
    return k.astype(np.int8 if lo < 0 else np.uint8)


@dataclass
class Quantizer:
    """(q, lo, hi, alpha) of one tensor in the paper's notation, plus the rate weight."""
    q: float
    lo: int
    hi: int
    alpha: float
    rate_weight: float = 0.0
    window: int = 0

    @property
    def nlev(self) -> int:
        return self.hi - self.lo + 1


@dataclass
class LayerCase:
    """One quantized layer: tensors to quantize and the GEMM (M, K, N) it feeds."""
    name: str
    M: int
    K: int
    N: int
    w_shape: tuple
    a_shape: tuple
    wq: Quantizer
    aq: Quantizer
    seed: int
    g_std: float = 1e-2
    notes: dict = field(default_factory=dict)


def tiny_layer(seed: int = 0):
    """Tiny layer: W 256x128 ~ N(0, 0.05^2), A 64x256 = ReLU(N(0,1)); 15 signed / 16 unsigned levels."""
    case = LayerCase("tiny", M=64, K=256, N=128, w_shape=(256, 128), a_shape=(64, 256),
                     wq=Quantizer(q=0.02, lo=-7, hi=7, alpha=50.0, rate_weight=0.01),
                     aq=Quantizer(q=0.25, lo=0, hi=15, alpha=50.0, rate_weight=0.01), seed=seed)
    w = normal(case.w_shape, 0.05, seed, 1)
    a = relu_normal(case.a_shape, seed, 2)
    return case, w, a


def cifar_resnet20_conv(seed: int = 2):
    """ResNet-20 style 3x3 conv, batch 128, 32x32, 16->16: GEMM (131072, 144, 16); L=1 weights, 4-bit acts."""
    M, K, N = 128 * 32 * 32, 144, 16
    w = he_normal(K, (K, N), seed, 1)
    a = half_normal((128, 32, 32, 16), seed, 2)
    case = LayerCase("cifar_resnet20_conv", M, K, N, (K, N), a.shape,
                     wq=Quantizer(step_from_mean_abs(w, 2), -1, 1, 20.0, 0.005),
                     aq=Quantizer(step_from_mean_abs(a, 4), 0, 15, 20.0, 0.005, window=5), seed=seed)
    return case, w, a


def resnet18_layer3_conv(seed: int = 3):
    """ResNet-18 layer3 3x3 conv, batch 256, 14x14, 256->256: GEMM (50176, 2304, 256); L=7, 4-bit acts."""
    M, K, N = 256 * 14 * 14, 2304, 256
    w = he_normal(K, (K, N), seed, 1)
    a = half_normal((256, 14, 14, 256), seed, 2)
    case = LayerCase("resnet18_layer3_conv", M, K, N, (K, N), a.shape,
                     wq=Quantizer(step_from_mean_abs(w, 4), -7, 7, 100.0, 0.01),
                     aq=Quantizer(step_from_mean_abs(a, 4), 0, 15, 100.0, 0.01, window=5), seed=seed)
    return case, w, a


def resnet18_layers(batch: int = 256):
    """ResNet-18 at 224x224: every conv and the FC layer as (name, M, K, N, n_x): the im2col GEMM it runs
    (M = batch x output pixels, K = kernel area x input channels, N = output channels) and the number of elements
    n_x of its input activation tensor (batch x input pixels x input channels, what the quantizer sees)."""
    b = batch
    L = [("conv1", b * 112 * 112, 147, 64, b * 224 * 224 * 3)]
    L += [(f"layer1.{i}", b * 56 * 56, 576, 64, b * 56 * 56 * 64) for i in range(4)]
    L += [("layer2.0", b * 28 * 28, 576, 128, b * 56 * 56 * 64)]
    L += [(f"layer2.{i}", b * 28 * 28, 1152, 128, b * 28 * 28 * 128) for i in range(1, 4)]
    L += [("layer2.ds", b * 28 * 28, 64, 128, b * 56 * 56 * 64)]
    L += [("layer3.0", b * 14 * 14, 1152, 256, b * 28 * 28 * 128)]
    L += [(f"layer3.{i}", b * 14 * 14, 2304, 256, b * 14 * 14 * 256) for i in range(1, 4)]
    L += [("layer3.ds", b * 14 * 14, 128, 256, b * 28 * 28 * 128)]
    L += [("layer4.0", b * 7 * 7, 2304, 512, b * 14 * 14 * 256)]
    L += [(f"layer4.{i}", b * 7 * 7, 4608, 512, b * 7 * 7 * 512) for i in range(1, 4)]
    L += [("layer4.ds", b * 7 * 7, 256, 512, b * 14 * 14 * 256)]
    L += [("fc", b, 512, 1000, b * 512)]
    return L


def resnet18_conv_geometry(name: str):
    """(H, W, C, R, S, stride, padding) of a ResNet-18 layer as a convolution on its NHWC input tensor, for the layers
    the convolution form of the products covers: every 3 x 3 layer (the first of stages 2-4 with stride 2) and the
    1 x 1 stride-2 shortcuts.  None for conv1 (3 input channels) and the fully connected layer."""
    side = {"layer1": (56, 64), "layer2": (28, 128), "layer3": (14, 256), "layer4": (7, 512)}
    stage, _, idx = name.partition(".")
    if stage not in side:
        return None
    hw, c = side[stage]
    if idx in ("1", "2", "3") or (stage == "layer1" and idx == "0"):
        return hw, hw, c, 3, 3, 1, 1
    if idx == "0":                      # opens the stage: input of the previous stage's size, stride 2
        return 2 * hw, 2 * hw, c // 2, 3, 3, 2, 1
    if idx == "ds":
        return 2 * hw, 2 * hw, c // 2, 1, 1, 2, 0
    return None

"""Seeded synthetic inputs shaped like the paper's workloads (numpy only).

This module is the one piece shared by the CUDA path's tests, the benchmark and the
CPU oracle's tests.  It holds none of the method's arithmetic: it only produces int8
operand bytes together with the (scale, zero_point) metadata that describes them.
Any int8 bytes are valid layer inputs, so nothing downstream depends on how the
samples were placed on the 8-bit grid here.

Value recipes (Sec. 5 of the paper trains ResNet18 / VGG16 / MobileNetV2 on Tiny
ImageNet and ImageNet; no dataset is used here, only the layer shapes and the kind
of distribution each tensor has there):
  * post-ReLU activations : |N(0,1)|, grid from 0 to the sample maximum  (zero_point -128)
  * signed activations    : N(0,1), grid from sample min to sample max
  * activation gradients  : Student-t(nu=3) times a per-iteration lognormal(0,0.3)
                            factor, grid from sample min to sample max (heavy tails, so
                            most codes sit within a few levels of the zero point)
  * weights               : N(0,0.05), symmetric grid, zero_point 0
  * raw int8              : uniform on -128..127
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

BASE_SEED = 0x2105_04246


def rng(*keys: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([BASE_SEED, *[int(k) for k in keys]]))


@dataclass
class QTensor:
    """int8 codes plus the metadata a layer needs to interpret them."""
    q: np.ndarray          # int8
    scale: float           # real value of one code step
    zero_point: int        # code that represents real 0


def _place_on_grid(x: np.ndarray, lo: float, hi: float) -> QTensor:
    lo, hi = min(float(lo), 0.0), max(float(hi), 0.0)
    scale = np.float32((hi - lo) / 255.0) if hi > lo else np.float32(1.0)
    z = int(np.clip(-128 - np.rint(lo / scale), -128, 127))
    q = np.clip(np.rint(x / scale) + z, -128, 127).astype(np.int8)
    return QTensor(q, float(scale), z)


def uniform_int8(g: np.random.Generator, shape, scale: float = 1.0, zero_point: int = 0) -> QTensor:
    return QTensor(g.integers(-128, 128, size=shape, dtype=np.int8), float(scale), int(zero_point))


def relu_activations(g: np.random.Generator, shape) -> QTensor:
    x = np.abs(g.standard_normal(shape, dtype=np.float32))
    return _place_on_grid(x, 0.0, float(x.max()))


def signed_activations(g: np.random.Generator, shape) -> QTensor:
    x = g.standard_normal(shape, dtype=np.float32)
    return _place_on_grid(x, float(x.min()), float(x.max()))


def image_like(g: np.random.Generator, shape) -> QTensor:
    """Normalised-image-like input: uniform codes on an asymmetric grid."""
    return QTensor(g.integers(-128, 128, size=shape, dtype=np.int8), 1.0 / 58.0, -14)


def gradients(g: np.random.Generator, shape, drift: float | None = None) -> QTensor:
    x = g.standard_t(3.0, size=shape).astype(np.float32)
    f = float(np.exp(g.normal(0.0, 0.3))) if drift is None else float(drift)
    x *= np.float32(1e-3 * f)
    return _place_on_grid(x, float(x.min()), float(x.max()))


def weights(g: np.random.Generator, shape, std: float = 0.05) -> QTensor:
    w = (g.standard_normal(shape, dtype=np.float32) * np.float32(std))
    s = np.float32(np.abs(w).max() / 127.0)
    q = np.clip(np.rint(w / s), -127, 127).astype(np.int8)
    return QTensor(q, float(s), 0)


def tiled(make, g: np.random.Generator, shape, block_elems: int = 1 << 22) -> QTensor:
    """Large tensors: draw `block_elems` samples once and repeat them with a rolling
    offset, which keeps host time bounded while no two rows of the tensor are equal."""
    n = int(np.prod(shape))
    if n <= block_elems:
        return make(g, shape)
    base = make(g, (block_elems,))
    reps = -(-n // block_elems)
    parts = [np.roll(base.q, 7919 * i) for i in range(reps)]
    return QTensor(np.concatenate(parts)[:n].reshape(shape), base.scale, base.zero_point)

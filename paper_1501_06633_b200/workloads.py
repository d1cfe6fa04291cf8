"""Seeded synthetic inputs for the FPROP convolution workloads.

This module only *draws numbers and names shapes*; it holds none of the
method's arithmetic and is the one module that both the CUDA path's callers
and the CPU checker's tests may import.  Arrays come out in the storage layout
of the library: maps ``[Nc][Hi][Wi][Nb]``, filters ``[Nc][Sk][Sk][No]`` (fp32,
batch / filter index innermost).

The five named workloads have the layer structure the paper measures
(a large-kernel strided first layer, a 5x5 mid layer, a wide small-map 3x3
layer; Table 1) plus one larger 3x3 layer; values are synthetic because the
paper's efficiency metric is value-independent.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Tuple

import numpy as np

BASE_SEED = 150106633


@dataclass(frozen=True)
class Workload:
    name: str
    Nb: int
    Wi: int
    Hi: int
    Nc: int
    No: int
    Sk: int
    stride: int
    pad: int
    alpha: float
    in_dist: Tuple[str, float, float]      # ("uniform", lo, hi)
    filt_dist: Tuple[str, float, float]    # ("uniform", lo, hi) or ("normal", mean, sigma)
    seed: int

    @property
    def dims(self):
        """(Nb, Wi, Hi, Nc, No, Sk, stride, pad, alpha) — the descriptor's field order."""
        return (self.Nb, self.Wi, self.Hi, self.Nc, self.No, self.Sk, self.stride, self.pad,
                self.alpha)

    def scaled(self, **kw) -> "Workload":
        """Same recipe with some dimensions replaced (reduced-size parity cases)."""
        return replace(self, **kw)


WORKLOADS = {
    "tiny3x3": Workload("tiny3x3", 32, 16, 16, 16, 32, 3, 1, 1, 1.0,
                        ("uniform", -1.0, 1.0), ("uniform", -1.0, 1.0), BASE_SEED + 10),
    "first11x11s4": Workload("first11x11s4", 128, 227, 227, 3, 96, 11, 4, 0, 1.0,
                             ("uniform", 0.0, 1.0), ("normal", 0.0, 0.01), BASE_SEED + 20),
    "mid5x5": Workload("mid5x5", 128, 27, 27, 96, 256, 5, 1, 2, 1.0,
                       ("uniform", 0.0, 1.0), ("normal", 0.0, 0.01), BASE_SEED + 30),
    "wide3x3": Workload("wide3x3", 128, 13, 13, 256, 384, 3, 1, 1, 0.5,
                        ("uniform", 0.0, 1.0), ("normal", 0.0, 0.01), BASE_SEED + 40),
    "large3x3": Workload("large3x3", 64, 56, 56, 128, 256, 3, 1, 1, 1.0,
                         ("uniform", -1.0, 1.0), ("normal", 0.0, (1.0 / (9 * 128)) ** 0.5),
                         BASE_SEED + 50),
}
ORDER = ["tiny3x3", "first11x11s4", "mid5x5", "wide3x3", "large3x3"]


def _table1(name, k, Wi, Nc, No, Sk, stride, pad):
    return Workload(name, 128, Wi, Wi, Nc, No, Sk, stride, pad, 1.0, ("uniform", 0.0, 1.0),
                    ("normal", 0.0, 0.01), BASE_SEED + 100 + 10 * k)


# The ten layer shapes of the paper's Table 1 (minibatch 128; padding chosen so that the
# printed output size results).  Shapes only: values follow the same synthetic recipe.
TABLE1 = {w.name: w for w in [
    _table1("alexnet_conv1", 0, 224, 3, 64, 11, 4, 2),      # 224x224x3  -> 55x55x64
    _table1("alexnet_conv2", 1, 27, 64, 192, 5, 1, 2),      # 27x27x64   -> 27x27x192
    _table1("alexnet_conv3", 2, 13, 192, 384, 3, 1, 1),     # 13x13x192  -> 13x13x384
    _table1("alexnet_conv4", 3, 13, 384, 256, 3, 1, 1),     # 13x13x384  -> 13x13x256
    _table1("alexnet_conv5", 4, 13, 256, 256, 3, 1, 1),     # 13x13x256  -> 13x13x256
    _table1("overfeat_L1", 5, 231, 3, 96, 11, 4, 0),        # 231x231x3  -> 56x56x96
    _table1("overfeat_L2", 6, 24, 96, 256, 5, 1, 0),        # 24x24x96   -> 20x20x256
    _table1("overfeat_L3", 7, 12, 256, 512, 3, 1, 1),       # 12x12x256  -> 12x12x512
    _table1("overfeat_L4", 8, 12, 512, 1024, 3, 1, 1),      # 12x12x512  -> 12x12x1024
    _table1("overfeat_L5", 9, 12, 1024, 1024, 3, 1, 1),     # 12x12x1024 -> 12x12x1024
]}
TABLE1_ORDER = list(TABLE1)
ALL = dict(WORKLOADS, **TABLE1)


def _draw(rng: np.random.Generator, dist, shape) -> np.ndarray:
    kind, a, b = dist
    if kind == "uniform":
        return rng.uniform(a, b, size=shape).astype(np.float32)
    if kind == "normal":
        return (a + b * rng.standard_normal(size=shape)).astype(np.float32)
    raise ValueError("unknown distribution %r" % (kind,))


def make_inputs(w: Workload, seed_offset: int = 0):
    """(maps, filters) as fp32 numpy arrays in storage layout; PCG64, maps from
    ``seed``, filters from ``seed + 1``.  ``seed_offset`` gives other ranks /
    repetitions their own independent draw of the same recipe."""
    rng_in = np.random.default_rng(w.seed + 1000 * seed_offset)
    rng_f = np.random.default_rng(w.seed + 1000 * seed_offset + 1)
    maps = _draw(rng_in, w.in_dist, (w.Nc, w.Hi, w.Wi, w.Nb))
    filt = _draw(rng_f, w.filt_dist, (w.Nc, w.Sk, w.Sk, w.No))
    return maps, filt


def make_dout(w: Workload, seed_offset: int = 0):
    """Output gradient for the backward-propagation entry points: uniform [-1, 1) in the
    output's storage layout [No][Ho][Wo][Nb], PCG64 from ``seed + 2``."""
    Ho = (w.Hi + 2 * w.pad - w.Sk) // w.stride + 1
    Wo = (w.Wi + 2 * w.pad - w.Sk) // w.stride + 1
    rng = np.random.default_rng(w.seed + 1000 * seed_offset + 2)
    return rng.uniform(-1.0, 1.0, size=(w.No, Ho, Wo, w.Nb)).astype(np.float32)


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 storage (uint16), round-to-nearest-even; finite inputs."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    """bf16 storage (uint16) -> the fp32 values it represents."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def truncate_to_tf32(a: np.ndarray) -> np.ndarray:
    """fp32 values with the low 13 mantissa bits cleared (what a TF32 tensor
    core reads from an fp32 word)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    return (u & np.uint32(0xFFFFE000)).view(np.float32)

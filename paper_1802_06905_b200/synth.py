"""Seeded synthetic inputs for the seven-nested-loop CNN, shared by the CUDA path and its checkers.

This module holds no arithmetic of the method: it only draws numbers and rounds them to bf16.
Values are produced on the host as float32 from ``numpy.random.Generator(PCG64(seed))``, rounded
once to bf16 (round-to-nearest-even) and handed out as ``uint16`` bit patterns, so that every
consumer sees the same bits.

Array conventions (dense, last subscript fastest), following Eq. 1 and Section 2:
    Image  [Wi][Hi][C][B], Wi = sw*(W-1)+R, Hi = sh*(H-1)+S   (valid-window extent)
    Filter [K][R][S][C]
    Out    [K][H][W][B]
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

SEED_BASE = 0x18020690


@dataclass(frozen=True)
class ConvShape:
    """The seven loop bounds and two strides of Eq. 1, plus the input recipe."""

    name: str
    B: int
    C: int
    K: int
    W: int
    H: int
    R: int
    S: int
    sw: int = 1
    sh: int = 1
    image_dist: str = "normal"      # "normal" N(0,1) | "uniform_pm1" U[-1,1] | "uniform_01" U[0,1]
    filter_dist: str = "normal_fan"  # "normal_fan" N(0, var=1/(C*R*S)) | "uniform_pm1"
    seed: int = SEED_BASE

    @property
    def Wi(self) -> int:
        return self.sw * (self.W - 1) + self.R

    @property
    def Hi(self) -> int:
        return self.sh * (self.H - 1) + self.S

    @property
    def image_shape(self):
        return (self.Wi, self.Hi, self.C, self.B)

    @property
    def filter_shape(self):
        return (self.K, self.R, self.S, self.C)

    @property
    def out_shape(self):
        return (self.K, self.H, self.W, self.B)

    @property
    def macs(self) -> int:
        return self.B * self.C * self.K * self.W * self.H * self.R * self.S

    @property
    def flops(self) -> int:
        return 2 * self.macs

    @property
    def image_words(self) -> int:
        return self.Wi * self.Hi * self.C * self.B

    @property
    def filter_words(self) -> int:
        return self.K * self.R * self.S * self.C

    @property
    def out_words(self) -> int:
        return self.K * self.H * self.W * self.B

    def dims(self):
        return (self.B, self.C, self.K, self.W, self.H, self.R, self.S, self.sw, self.sh)


# The five benchmark shapes.  Index 0 is the small case a CPU finishes at once; index 1 is the one
# the headline metric is quoted on.
CONFIGS = (
    ConvShape("cfg1_tiny_3x3", B=2, C=8, K=16, W=14, H=14, R=3, S=3,
              image_dist="uniform_pm1", filter_dist="uniform_pm1", seed=SEED_BASE + 1),
    ConvShape("cfg2_resnet_3x3", B=32, C=256, K=256, W=14, H=14, R=3, S=3, seed=SEED_BASE + 2),
    ConvShape("cfg3_stem_7x7_s2", B=64, C=3, K=64, W=112, H=112, R=7, S=7, sw=2, sh=2,
              image_dist="uniform_01", seed=SEED_BASE + 3),
    ConvShape("cfg4_pointwise_1x1", B=64, C=1024, K=256, W=14, H=14, R=1, S=1, seed=SEED_BASE + 4),
    ConvShape("cfg5_large_3x3", B=128, C=512, K=512, W=28, H=28, R=3, S=3, seed=SEED_BASE + 5),
)

# Pooling shapes (Section 6) timed by the benchmark: (name, B, C, K, W, H, R, S, sw, sh).  The first
# is the usual per-channel layer behind a stem convolution (64 channels folded into b); the second
# the paper's seven-loop form with a channel reduction and K equal planes; the third writes many
# planes from a small Image.
POOL_SHAPES = (
    ("pool_per_channel_3x3_s2", 4096, 1, 1, 55, 55, 3, 3, 2, 2),
    ("pool_seven_loop_c64_k256", 64, 64, 256, 27, 27, 3, 3, 2, 2),
    ("pool_many_planes_2x2_s2", 64, 16, 1024, 28, 28, 2, 2, 2, 2),
)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even); returns uint16 bit patterns.  Finite inputs."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _draw(rng, dist, shape, fan):
    if dist == "normal":
        return rng.standard_normal(shape, dtype=np.float32)
    if dist == "normal_fan":
        return rng.standard_normal(shape, dtype=np.float32) * np.float32(fan ** -0.5)
    if dist == "uniform_pm1":
        return rng.random(shape, dtype=np.float32) * np.float32(2.0) - np.float32(1.0)
    if dist == "uniform_01":
        return rng.random(shape, dtype=np.float32)
    raise ValueError(dist)


def make_inputs(shp: ConvShape, seed: int | None = None):
    """Return (image_bits, filter_bits): uint16 arrays of shapes ``image_shape``/``filter_shape``."""
    rng = np.random.Generator(np.random.PCG64(shp.seed if seed is None else seed))
    fan = shp.C * shp.R * shp.S
    image = _draw(rng, shp.image_dist, shp.image_shape, fan)
    filt = _draw(rng, shp.filter_dist, shp.filter_shape, fan)
    return f32_to_bf16_bits(image), f32_to_bf16_bits(filt)

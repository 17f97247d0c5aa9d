"""Seeded synthetic tensors shared by the tests, the benchmark and the CPU checker.

This module holds data generation only: counter-based random streams keyed by
(seed, tensor name), the usual initialisation distributions, and conversion of
float32 arrays to and from bfloat16 bit patterns.  None of the method's
arithmetic (convolution, folding, pooling, normalisation, filter merging) lives
here, so both the CUDA library's callers and the checker can import it.

Every float array returned is already exactly representable in bfloat16
(round-to-nearest-even applied once), so the CPU side can widen it to double
and the GPU side can narrow it to 16 bits without either changing a value.
"""
from __future__ import annotations

import hashlib

import numpy as np

__all__ = [
    "stream", "to_bf16_bits", "from_bf16_bits", "round_bf16",
    "normal", "uniform", "he_normal", "INCEPTION_V1", "RESNET50_STAGES",
]


def stream(seed: int, name: str) -> np.random.Generator:
    """Independent Philox stream for one named tensor.

    The key is a hash of (seed, name), so a tensor's values do not depend on
    the order in which tensors are generated.
    """
    h = hashlib.sha256(f"{seed}:{name}".encode()).digest()
    key = int.from_bytes(h[:16], "little")
    return np.random.Generator(np.random.Philox(key=key))


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> uint16 bfloat16 bit patterns, round-to-nearest-even."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounding = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + rounding) >> 16).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    """uint16 bfloat16 bit patterns -> float32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def round_bf16(a: np.ndarray) -> np.ndarray:
    """float32 array rounded once to the nearest bfloat16 value, kept as float32."""
    return from_bf16_bits(to_bf16_bits(a)).reshape(np.shape(a))


def normal(seed: int, name: str, shape, std: float = 1.0, mean: float = 0.0) -> np.ndarray:
    g = stream(seed, name)
    return round_bf16((g.standard_normal(shape, dtype=np.float32) * np.float32(std) + np.float32(mean)))


def uniform(seed: int, name: str, shape, lo: float, hi: float) -> np.ndarray:
    g = stream(seed, name)
    return round_bf16((g.random(shape, dtype=np.float32) * np.float32(hi - lo) + np.float32(lo)))


def he_normal(seed: int, name: str, cout: int, k: int, cin: int) -> np.ndarray:
    """He-normal filter bank in [Cout][k][k][Cin] order, std = sqrt(2 / (k*k*Cin))."""
    std = float(np.sqrt(2.0 / (k * k * cin)))
    return normal(seed, name, (cout, k, k, cin), std=std)


# Inception-v1 channel table: module -> (Cin, c1, c3r, c3, c5r, c5, pp).
# Architecture facts of the published network; the checker and the CUDA library
# each keep their own topology code, this table only sizes the random tensors.
INCEPTION_V1 = {
    "3a": (192, 64, 96, 128, 16, 32, 32),
    "3b": (256, 128, 128, 192, 32, 96, 64),
    "4a": (480, 192, 96, 208, 16, 48, 64),
    "4b": (512, 160, 112, 224, 24, 64, 64),
    "4c": (512, 128, 128, 256, 24, 64, 64),
    "4d": (512, 112, 144, 288, 32, 64, 64),
    "4e": (528, 256, 160, 320, 32, 128, 128),
    "5a": (832, 256, 160, 320, 32, 128, 128),
    "5b": (832, 384, 192, 384, 48, 128, 128),
}

# ResNet-50 stages: (bottleneck width, number of blocks); output channels are 4x the width.
RESNET50_STAGES = ((64, 3), (128, 4), (256, 6), (512, 3))


# AlexNet (the grouped two-tower form): (name, Cout, k, stride, pad, groups, Cin of the whole layer).
# fc6 is written as a 6x6 convolution over the 6x6x256 plane that pool5 leaves for a 227x227 image.
ALEXNET_CONVS = (
    ("conv1", 96, 11, 4, 0, 1, 3), ("conv2", 256, 5, 1, 2, 2, 96), ("conv3", 384, 3, 1, 1, 1, 256),
    ("conv4", 384, 3, 1, 1, 2, 384), ("conv5", 256, 3, 1, 1, 2, 384),
    ("fc6", 4096, 6, 1, 0, 1, 256), ("fc7", 4096, 1, 1, 0, 1, 4096), ("fc8", 1000, 1, 1, 0, 1, 4096),
)

"""Seeded synthetic inputs (numpy only; none of the method's arithmetic lives here).

Every tensor is drawn from a Philox counter-based stream keyed by (seed, stream
id), so a given (seed, stream, shape) regenerates the same values on any
machine.  The distributions follow the workloads of the EOQ paper's networks:
uniform int8 codes for the single-layer case, half-rectified codes for
post-ReLU activations, standard normal draws for images, weights and errors.
"""
from __future__ import annotations

import numpy as np

BASE_SEED = 20210528


def rng(seed: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(stream) & (2**64 - 1)]))


def int8_uniform(shape, seed: int, stream: int = 0, lo: int = -127, hi: int = 127) -> np.ndarray:
    """Integer codes uniform in [lo, hi]."""
    return rng(seed, stream).integers(lo, hi + 1, size=shape, dtype=np.int64).astype(np.int8)


def normal_f32(shape, seed: int, stream: int = 0, std: float = 1.0) -> np.ndarray:
    """fp32 N(0, std^2) draws."""
    return (rng(seed, stream).standard_normal(size=shape) * std).astype(np.float32)


def normal_f64(shape, seed: int, stream: int = 0) -> np.ndarray:
    """float64 N(0, 1) draws (raw material for weight initialisation)."""
    return rng(seed, stream).standard_normal(size=shape)


def relu_codes(shape, seed: int, stream: int = 0, std_codes: float = 48.0) -> np.ndarray:
    """Codes shaped like a post-ReLU activation: about half zeros, the rest half-normal, capped at 127."""
    v = rng(seed, stream).standard_normal(size=shape) * std_codes
    return np.clip(np.rint(np.maximum(v, 0.0)), 0, 127).astype(np.int8)


def normal_codes(shape, seed: int, stream: int = 0, std_codes: float = 32.0) -> np.ndarray:
    """Signed codes shaped like a back-propagated error: rounded normal, capped at +-127."""
    v = rng(seed, stream).standard_normal(size=shape) * std_codes
    return np.clip(np.rint(v), -127, 127).astype(np.int8)


def bits(shape, seed: int, stream: int = 0, p_one: float = 0.5) -> np.ndarray:
    """0/1 bytes (a stand-in ReLU mask)."""
    return (rng(seed, stream).random(size=shape) < p_one).astype(np.uint8)


def labels(n: int, classes: int, seed: int, stream: int = 0) -> np.ndarray:
    return rng(seed, stream).integers(0, classes, size=(n,), dtype=np.int64)

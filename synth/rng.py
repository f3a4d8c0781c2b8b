"""Counter-based random numbers for the synthetic inputs.

SplitMix64 (Steele, Lea, Flood 2014) used as a counter-based generator: the
i-th output of a stream is ``mix(key + (i + 1) * GAMMA)`` with the published
finaliser, so any element of any stream can be produced independently and
the values do not depend on the numpy or torch version.

Only input generation lives here. Nothing in this module knows what the
masking path computes.
"""
from __future__ import annotations

import numpy as np

GAMMA = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_S30, _S27, _S31 = np.uint64(30), np.uint64(27), np.uint64(31)

SEED_BASE = 20260529


def _mix(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> _S30)) * _M1
    z = (z ^ (z >> _S27)) * _M2
    return z ^ (z >> _S31)


def stream_key(*ids: int) -> np.uint64:
    """Fold a tuple of small integers (seed, config, purpose, step, row ...) into a stream key."""
    with np.errstate(over="ignore"):
        k = np.uint64(0x243F6A8885A308D3)
        for v in ids:
            k = _mix(np.asarray(k ^ np.uint64(int(v) & 0xFFFFFFFFFFFFFFFF)) + GAMMA)
        return np.uint64(k)


def u64(key: np.uint64, n: int, offset: int = 0) -> np.ndarray:
    """Outputs ``offset .. offset+n-1`` of the stream ``key`` as uint64."""
    with np.errstate(over="ignore"):
        ctr = np.arange(offset + 1, offset + n + 1, dtype=np.uint64)
        return _mix(np.uint64(key) + ctr * GAMMA)


def uniform(key: np.uint64, n: int, offset: int = 0) -> np.ndarray:
    """Uniform doubles in (0, 1): the top 53 bits, shifted half a step off zero."""
    return ((u64(key, n, offset) >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal_f32(key: np.uint64, n: int, sigma: float = 1.0) -> np.ndarray:
    """N(0, sigma^2) float32 samples by the Box-Muller transform (both branches used)."""
    h = (n + 1) // 2
    u1 = uniform(key, h, 0)
    u2 = uniform(key, h, h)
    rad = np.sqrt(-2.0 * np.log(u1))
    ang = (2.0 * np.pi) * u2
    out = np.empty(2 * h, dtype=np.float32)
    out[0::2] = rad * np.cos(ang) * sigma
    out[1::2] = rad * np.sin(ang) * sigma
    return out[:n]


def permutation(key: np.uint64, n: int) -> np.ndarray:
    """A permutation of 0..n-1: stable argsort of n stream outputs."""
    return np.argsort(u64(key, n), kind="stable").astype(np.int64)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns the 16-bit patterns as uint16."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (b >> np.uint32(16)) & np.uint32(1)
    rounded = b + np.uint32(0x7FFF) + lsb
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns (uint16) to float32."""
    return (np.ascontiguousarray(h, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)

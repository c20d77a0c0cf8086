"""Counter-based random numbers for the synthetic workloads.

Every value is a pure function of (seed, stream, index): a SplitMix64 finaliser
applied to a 64-bit counter, as published by Steele, Lea and Flood ("Fast
splittable pseudorandom number generators", OOPSLA 2014).  Normal deviates use
the Box-Muller transform on two such uniforms.  Nothing here belongs to the
rollout method itself; the module only makes reproducible test data.
"""
from __future__ import annotations

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _mix(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def bits64(seed: int, stream: int, n: int, offset: int = 0) -> np.ndarray:
    """n 64-bit words for counters offset .. offset+n-1 of (seed, stream)."""
    with np.errstate(over="ignore"):
        key = _mix(np.array([(seed * 0x632BE59BD9B4E019 + stream * 0xD1342543DE82EF95 + 0x1234567) % (1 << 64)],
                            dtype=np.uint64))
        ctr = np.arange(offset, offset + n, dtype=np.uint64)
        return _mix(key + (ctr + np.uint64(1)) * _GOLDEN)


def uniform(seed: int, stream: int, n: int, offset: int = 0) -> np.ndarray:
    """n doubles in [0, 1) with 53 random bits each."""
    return (bits64(seed, stream, n, offset) >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))


def normal(seed: int, stream: int, n: int) -> np.ndarray:
    """n standard normal doubles (Box-Muller, both branches used)."""
    m = (n + 1) // 2
    u = uniform(seed, stream, 2 * m)
    u1 = 1.0 - u[:m]            # (0, 1]
    u2 = u[m:]
    r = np.sqrt(-2.0 * np.log(u1))
    out = np.concatenate([r * np.cos(2.0 * np.pi * u2), r * np.sin(2.0 * np.pi * u2)])
    return out[:n]


def integers(seed: int, stream: int, n: int, high: int) -> np.ndarray:
    """n integers in [0, high)."""
    return np.minimum((uniform(seed, stream, n) * high).astype(np.int64), high - 1)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result stays float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    r = ((u + bias) & np.uint32(0xFFFF0000)).astype(np.uint32)
    return r.view(np.float32).reshape(x.shape)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of values that are already exactly representable in bfloat16."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16).reshape(x.shape)

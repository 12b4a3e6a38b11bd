"""Counter-based random numbers: SplitMix64 addressed by (seed, stream, index).

Element i of a stream depends only on (seed, stream, i), so any slice of any
tensor can be regenerated without producing what precedes it.
"""
from __future__ import annotations

import numpy as np

_GAMMA = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

# stream identifiers; a layer l of a network adds 16*l
STREAM_X, STREAM_W, STREAM_BIAS, STREAM_MASK = 0, 1, 2, 3


def _mix(z: np.ndarray) -> np.ndarray:
    """SplitMix64 output function (Steele, Lea, Flood 2014) on uint64 arrays."""
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def u64_stream(seed: int, stream: int, n: int, start: int = 0) -> np.ndarray:
    """n consecutive 64-bit outputs of stream (seed, stream), beginning at index start."""
    with np.errstate(over="ignore"):
        key = np.array([(int(seed) << 32) + int(stream)], dtype=np.uint64)
        s0 = _mix(key * _GAMMA + _GAMMA)
        i = np.arange(start + 1, start + n + 1, dtype=np.uint64)
        return _mix(s0 + i * _GAMMA)


def uniform01(seed: int, stream: int, n: int, start: int = 0) -> np.ndarray:
    """U[0,1) on a 2^-24 grid, so every value is exact in fp32."""
    bits = u64_stream(seed, stream, n, start)
    return ((bits >> np.uint64(40)).astype(np.float64) * 2.0 ** -24).astype(np.float32)


def normal(seed: int, stream: int, n: int, sigma: float) -> np.ndarray:
    """N(0, sigma^2) by Box-Muller in fp64 on pairs of 53-bit uniforms, cast to fp32."""
    m = (n + 1) // 2
    bits = u64_stream(seed, stream, 2 * m)
    u = ((bits >> np.uint64(11)).astype(np.float64) + 0.5) * 2.0 ** -53
    r = np.sqrt(-2.0 * np.log(u[0::2]))
    t = 2.0 * np.pi * u[1::2]
    z = np.empty(2 * m, dtype=np.float64)
    z[0::2] = r * np.cos(t)
    z[1::2] = r * np.sin(t)
    return (z[:n] * sigma).astype(np.float32)

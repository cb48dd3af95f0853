"""Counter-based random numbers for the synthetic workloads.

Every value is a pure function of (seed, stream, index), so the result does not
depend on chunking, threading or library versions.  This module produces input
data only; it contains none of the method's arithmetic.

The mixer is the public splitmix64 finaliser applied to a 64-bit counter.
"""
from __future__ import annotations

import numpy as np

_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_GOLD = np.uint64(0x9E3779B97F4A7C15)


def _mix(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def key(seed: int, stream: int) -> np.uint64:
    """64-bit key of a (seed, stream) pair."""
    with np.errstate(over="ignore"):
        k = _mix(np.asarray([np.uint64(seed & 0xFFFFFFFFFFFFFFFF) * _GOLD + _GOLD], dtype=np.uint64))
        k = _mix(k ^ (np.uint64(stream & 0xFFFFFFFFFFFFFFFF) * _M2 + _GOLD))
    return k[0]


def bits(seed: int, stream: int, idx) -> np.ndarray:
    """uint64 random bits for every counter value in ``idx`` (any integer array)."""
    idx = np.asarray(idx).astype(np.uint64, copy=False)
    with np.errstate(over="ignore"):
        return _mix(_mix((idx + np.uint64(1)) * _GOLD ^ key(seed, stream)))


def uniform(seed: int, stream: int, idx) -> np.ndarray:
    """float64 uniform in [0, 1) with 53 random bits."""
    return (bits(seed, stream, idx) >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def randint(seed: int, stream: int, idx, lo: int, hi: int) -> np.ndarray:
    """int64 uniform in [lo, hi) (multiply-shift on the top 32 bits; hi-lo < 2**31)."""
    span = np.uint64(hi - lo)
    top = bits(seed, stream, idx) >> np.uint64(32)
    return ((top * span) >> np.uint64(32)).astype(np.int64) + lo


def normal(seed: int, stream: int, start: int, count: int, std: float, out_dtype=np.float32) -> np.ndarray:
    """``count`` normal deviates N(0, std^2) for counters start .. start+count-1.

    Box-Muller in float64 on counter pairs: elements 2j and 2j+1 come from the
    uniforms drawn at counter j (cosine and sine branch).
    """
    first_pair = start // 2
    last_pair = (start + count - 1) // 2
    j = np.arange(first_pair, last_pair + 1, dtype=np.uint64)
    b = bits(seed, stream, j)
    # two 32-bit uniforms from one 64-bit word; u1 in (0, 1]
    u1 = ((b >> np.uint64(32)).astype(np.float64) + 1.0) * (1.0 / 4294967296.0)
    u2 = (b & np.uint64(0xFFFFFFFF)).astype(np.float64) * (1.0 / 4294967296.0)
    r = np.sqrt(-2.0 * np.log(u1)) * std
    t = (2.0 * np.pi) * u2
    z = np.empty(2 * j.size, dtype=np.float64)
    z[0::2] = r * np.cos(t)
    z[1::2] = r * np.sin(t)
    off = start - 2 * first_pair
    return z[off:off + count].astype(out_dtype)

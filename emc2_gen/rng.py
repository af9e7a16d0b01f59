"""Counter-based random streams for the synthetic frame generator.

Every random quantity is a pure function of (seed, stream name, counter), so a
frame can be regenerated piecewise and in any order.  The 64-bit mixer is the
public splitmix64 finaliser; uniform, normal and order-statistic transforms are
written here so that results do not depend on numpy's own generators.

This module only makes inputs.  It holds none of the bridge's arithmetic.
"""
from __future__ import annotations

import zlib

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_TWO_M53 = 1.0 / 9007199254740992.0


def _mix(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


class Stream:
    """One independent random stream: value i is mix(key + (i + 1) * golden)."""

    def __init__(self, seed: int, name: str):
        tag = zlib.crc32(name.encode("utf-8")) & 0xFFFFFFFF
        k = np.array([(int(seed) & 0xFFFFFFFFFFFFFFFF)], dtype=np.uint64)
        with np.errstate(over="ignore"):
            k = _mix(k * _GOLDEN + np.uint64(tag))
            k = _mix(k + np.uint64(tag) * _M1)
        self.key = k[0]
        self.pos = 0

    def u64(self, n: int) -> np.ndarray:
        i = np.arange(self.pos + 1, self.pos + n + 1, dtype=np.uint64)
        self.pos += n
        with np.errstate(over="ignore"):
            return _mix(self.key + i * _GOLDEN)

    def uniform(self, n: int, lo: float = 0.0, hi: float = 1.0) -> np.ndarray:
        """float64 in [lo, hi) from the top 53 bits."""
        u = (self.u64(n) >> np.uint64(11)).astype(np.float64) * _TWO_M53
        return lo + (hi - lo) * u

    def normal(self, n: int) -> np.ndarray:
        """Standard normal float64 by Box-Muller (two uniforms per value pair)."""
        m = (n + 1) // 2
        u1 = 1.0 - self.uniform(m)  # (0, 1]
        u2 = self.uniform(m)
        r = np.sqrt(-2.0 * np.log(u1))
        out = np.empty(2 * m, dtype=np.float64)
        out[0::2] = r * np.cos(2.0 * np.pi * u2)
        out[1::2] = r * np.sin(2.0 * np.pi * u2)
        return out[:n]

    def normal_f32(self, n: int, chunk: int = 1 << 22) -> np.ndarray:
        """Standard normal float32, generated in chunks to bound host memory."""
        out = np.empty(n, dtype=np.float32)
        for s in range(0, n, chunk):
            e = min(n, s + chunk)
            out[s:e] = self.normal(e - s)
        return out

    def beta25(self, n: int) -> np.ndarray:
        """Beta(2, 5): the 2nd smallest of 6 uniforms."""
        u = self.uniform(6 * n).reshape(n, 6)
        u.sort(axis=1)
        return u[:, 1].copy()

    def integers(self, n: int, k: int) -> np.ndarray:
        """Integers in [0, k) (k small, modulo bias negligible for 64-bit draws)."""
        return (self.u64(n) % np.uint64(k)).astype(np.int64)

    def permutation(self, n: int) -> np.ndarray:
        return np.argsort(self.u64(n), kind="stable")

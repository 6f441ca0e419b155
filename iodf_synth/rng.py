"""Counter-based random streams (splitmix64 finaliser over a 64-bit counter).

Element i of a stream is a pure function of (seed, stream name, i), so any slice can be drawn on
any machine in any order and the result does not depend on a library's generator state.
"""
import hashlib

import numpy as np

_MASK = np.uint64(0xFFFFFFFFFFFFFFFF)
_GOLDEN = np.uint64(0x9E3779B97F4A7C15)


def _mix(x):
    """splitmix64 output function, vectorised over uint64 arrays."""
    with np.errstate(over="ignore"):
        x = (x + _GOLDEN) & _MASK
        x = ((x ^ (x >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _MASK
        x = ((x ^ (x >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _MASK
        return x ^ (x >> np.uint64(31))


class Stream:
    """One named sub-stream of a seed. Draws advance an internal counter."""

    def __init__(self, seed, name):
        h = hashlib.sha256(("%d/%s" % (int(seed), name)).encode()).digest()
        self._key = np.uint64(int.from_bytes(h[:8], "little"))
        self._ctr = 0

    def bits(self, n):
        idx = np.arange(self._ctr, self._ctr + n, dtype=np.uint64)
        self._ctr += n
        with np.errstate(over="ignore"):
            return _mix(_mix(idx * _GOLDEN + self._key) ^ self._key)

    def uniform(self, n):
        """float64 in [0, 1) with 53 random bits."""
        return (self.bits(n) >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)

    def normal(self, n):
        """Standard normals by Box-Muller (two uniforms per pair)."""
        m = (n + 1) // 2
        u1 = 1.0 - self.uniform(m)            # (0, 1]
        u2 = self.uniform(m)
        r = np.sqrt(-2.0 * np.log(u1))
        out = np.empty(2 * m, dtype=np.float64)
        out[0::2] = r * np.cos(2.0 * np.pi * u2)
        out[1::2] = r * np.sin(2.0 * np.pi * u2)
        return out[:n]

    def integers(self, lo, hi, n):
        """Integers uniform in [lo, hi) (hi - lo < 2**53), as int64."""
        return (lo + np.floor(self.uniform(n) * float(hi - lo))).astype(np.int64)

    def permutation(self, n):
        """Fisher-Yates shuffle of 0..n-1."""
        p = np.arange(n, dtype=np.int64)
        u = self.uniform(max(n - 1, 0))
        for i in range(n - 1, 0, -1):
            j = int(u[n - 1 - i] * (i + 1))
            p[i], p[j] = p[j], p[i]
        return p

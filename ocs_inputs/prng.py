"""Counter-based seeded random streams for the synthetic workloads.

Every tensor is drawn from its own sub-stream of a SplitMix64 generator (Steele, Lea &
Flood, "Fast splittable pseudorandom number generators", OOPSLA 2014): element i of
stream (seed, stream_id) is mix64(base + (i + 1) * GOLDEN), so any slice can be produced
independently and in chunks.  All transforms run in float64 and are rounded to float32
once at the end.  Nothing in this module knows about channel splitting or quantization:
it only manufactures inputs, which the CPU checker and the CUDA library both receive as
plain arrays.
"""
from __future__ import annotations

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_MASK64 = (1 << 64) - 1
_CHUNK = 1 << 22


def _mix64(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def _mix64_int(z: int) -> int:
    z &= _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


class Stream:
    """One independent random stream, addressed by element index."""

    def __init__(self, seed: int, stream_id: int):
        # two rounds of mixing decorrelate (seed, stream_id) pairs that differ in one bit
        self.base = _mix64_int(_mix64_int(seed * 0x9E3779B97F4A7C15 + 0x1234567) ^
                               ((stream_id + 1) * 0xD1342543DE82EF95))

    def bits(self, start: int, count: int) -> np.ndarray:
        """uint64 outputs for element indices [start, start + count)."""
        with np.errstate(over="ignore"):
            idx = np.arange(start + 1, start + count + 1, dtype=np.uint64)
            return _mix64(np.uint64(self.base) + idx * _GOLDEN)

    def uniform(self, start: int, count: int) -> np.ndarray:
        """float64 uniforms strictly inside (0, 1)."""
        return ((self.bits(start, count) >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / (1 << 53))


def _chunks(n: int):
    for s in range(0, n, _CHUNK):
        yield s, min(_CHUNK, n - s)


def normal64(seed: int, stream_id: int, n: int) -> np.ndarray:
    """Standard normal draws (Box-Muller, cosine branch; two sub-streams)."""
    s1, s2 = Stream(seed, 2 * stream_id), Stream(seed, 2 * stream_id + 1)
    out = np.empty(n, dtype=np.float64)
    for s, c in _chunks(n):
        u1, u2 = s1.uniform(s, c), s2.uniform(s, c)
        out[s:s + c] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return out


def normal(seed, stream_id, shape, std=1.0, absolute=False) -> np.ndarray:
    n = int(np.prod(shape))
    x = normal64(seed, stream_id, n) * std
    if absolute:
        np.abs(x, out=x)
    return x.astype(np.float32).reshape(shape)


def uniform(seed, stream_id, shape, lo=0.0, hi=1.0) -> np.ndarray:
    n = int(np.prod(shape))
    st = Stream(seed, 2 * stream_id)
    out = np.empty(n, dtype=np.float32)
    for s, c in _chunks(n):
        out[s:s + c] = (lo + (hi - lo) * st.uniform(s, c)).astype(np.float32)
    return out.reshape(shape)


def laplace(seed, stream_id, shape, scale) -> np.ndarray:
    """Laplace(0, scale) by inverse CDF."""
    n = int(np.prod(shape))
    st = Stream(seed, 2 * stream_id)
    out = np.empty(n, dtype=np.float32)
    for s, c in _chunks(n):
        u = st.uniform(s, c) - 0.5
        out[s:s + c] = (-scale * np.sign(u) * np.log1p(-2.0 * np.abs(u))).astype(np.float32)
    return out.reshape(shape)


def student_t3(seed, stream_id, shape, scale) -> np.ndarray:
    """scale * Z / sqrt(chi2_3 / 3): Student-t with three degrees of freedom."""
    n = int(np.prod(shape))
    z = normal64(seed, 4 * stream_id, n)
    chi = np.zeros(n, dtype=np.float64)
    for k in range(1, 4):
        g = normal64(seed, 4 * stream_id + k, n)
        chi += g * g
    return (scale * z / np.sqrt(chi / 3.0)).astype(np.float32).reshape(shape)


def distinct_positions(seed, stream_id, n_total: int, count: int) -> np.ndarray:
    """`count` distinct flat indices in [0, n_total), in draw order."""
    if count <= 0:
        return np.zeros(0, dtype=np.int64)
    if count > n_total:
        raise ValueError("more positions than elements")
    st = Stream(seed, 2 * stream_id)
    got = np.zeros(0, dtype=np.int64)
    start = 0
    while got.size < count:
        need = max(16, int((count - got.size) * 1.25) + 8)
        cand = (st.bits(start, need) % np.uint64(n_total)).astype(np.int64)
        start += need
        allc = np.concatenate([got, cand])
        _, first = np.unique(allc, return_index=True)
        got = allc[np.sort(first)]
    return got[:count]


def signs(seed, stream_id, count: int) -> np.ndarray:
    st = Stream(seed, 2 * stream_id)
    return np.where(st.bits(0, count) >> np.uint64(63), -1.0, 1.0)


def zipf_tokens(seed, stream_id, shape, vocab: int, exponent: float) -> np.ndarray:
    """Token ids in [0, vocab): rank k (1-based) has probability k**-exponent / H, by inverse CDF
    on the exact finite normaliser."""
    n = int(np.prod(shape))
    w = np.arange(1, vocab + 1, dtype=np.float64) ** (-exponent)
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    u = Stream(seed, 2 * stream_id).uniform(0, n)
    ids = np.minimum(np.searchsorted(cdf, u, side="left"), vocab - 1)
    return ids.astype(np.int32).reshape(shape)

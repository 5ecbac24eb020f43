"""Counter-based random numbers: value = f(seed, stream, index).

Every draw is a pure function of its coordinates, so any consumer (the oracle,
the GPU tests, the benchmark) can regenerate exactly the same tensor without
sharing generator state.  The mixer is the 64-bit finaliser of SplitMix64
applied to a Weyl sequence; normals come from Box-Muller on two uniforms.
"""
import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_STREAM_MUL = np.uint64(0xD1342543DE82EF95)


def _mix64(x):
    x = np.asarray(x, dtype=np.uint64)
    with np.errstate(over="ignore"):
        x = (x ^ (x >> np.uint64(30))) * _M1
        x = (x ^ (x >> np.uint64(27))) * _M2
        x = x ^ (x >> np.uint64(31))
    return x


def _bits(seed, stream, index):
    """64 random bits for each entry of the uint64 array `index`."""
    with np.errstate(over="ignore"):
        key = _mix64(np.uint64(seed) * _GOLDEN + np.uint64(stream) * _STREAM_MUL + np.uint64(1))
        return _mix64(key + (np.asarray(index, dtype=np.uint64) + np.uint64(1)) * _GOLDEN)


def uniform01(seed, stream, n, offset=0):
    """n doubles in (0, 1), element j drawn at counter offset + j."""
    idx = np.arange(offset, offset + n, dtype=np.uint64)
    b = _bits(seed, stream, idx)
    return ((b >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(seed, stream, n, offset=0):
    """n standard normal doubles (Box-Muller; element j uses counters 2j and 2j+1)."""
    idx = np.arange(offset, offset + n, dtype=np.uint64)
    b1 = _bits(seed, stream, idx * np.uint64(2))
    b2 = _bits(seed, stream, idx * np.uint64(2) + np.uint64(1))
    scale = 1.0 / 9007199254740992.0
    u1 = ((b1 >> np.uint64(11)).astype(np.float64) + 0.5) * scale
    u2 = ((b2 >> np.uint64(11)).astype(np.float64) + 0.5) * scale
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def randint(seed, stream, n, high, offset=0):
    """n integers uniform on [0, high)."""
    u = uniform01(seed, stream, n, offset)
    return np.minimum((u * high).astype(np.int64), high - 1)


def zipf_ranks(seed, stream, n, vocab, exponent, offset=0):
    """n ranks in [0, vocab) with P(rank r) proportional to (r+1)^-exponent (inverse CDF)."""
    w = np.arange(1, vocab + 1, dtype=np.float64) ** (-exponent)
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    u = uniform01(seed, stream, n, offset)
    return np.minimum(np.searchsorted(cdf, u, side="left"), vocab - 1).astype(np.int64)

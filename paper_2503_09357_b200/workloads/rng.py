"""Counter-based random numbers for the synthetic workloads.

Every draw is a pure function of (seed, stream, a, b), so any graph parameter or
any candidate can be regenerated on its own and in any order.  The mixing
function is the SplitMix64 output finaliser (Steele, Lea, Flood 2014); the C++
candidate generator in ``candgen.cpp`` implements the same definition.
"""
import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_STREAM = np.uint64(0xD1B54A32D192ED03)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def mix64(z):
    z = np.asarray(z, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def rand64(seed, stream, a, b=0):
    """64 random bits keyed by (seed, stream, a, b); ``a`` and ``b`` may be arrays."""
    a = np.asarray(a, dtype=np.uint64)
    b = np.asarray(b, dtype=np.uint64)
    with np.errstate(over="ignore"):
        h = mix64(np.uint64(seed) ^ (np.uint64(stream) * _STREAM))
        h = mix64(h + (a + np.uint64(1)) * _GOLDEN)
        h = mix64(h + (b + np.uint64(1)) * _GOLDEN)
    return h


def randint(seed, stream, a, b, lo, hi):
    """Integers uniform on {lo..hi} (inclusive) by multiply-shift of the high 32 bits."""
    n = np.uint64(hi - lo + 1)
    hi32 = rand64(seed, stream, a, b) >> np.uint64(32)
    return (lo + ((hi32 * n) >> np.uint64(32)).astype(np.int64)).astype(np.int64)


def uniform01(seed, stream, a, b=0):
    """Doubles in (0, 1): 53 random bits, offset by half an ulp so 0 never occurs."""
    bits = rand64(seed, stream, a, b) >> np.uint64(11)
    return (bits.astype(np.float64) + 0.5) / float(1 << 53)

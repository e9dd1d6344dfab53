"""Counter-based random numbers, identical on every host and numpy version.

Every draw is a pure function of (seed, stream, index): the 64-bit counter
``seed * GOLDEN + stream * ODD + index`` is mixed with the published SplitMix64
finaliser (Steele, Lea, Flood 2014) and the top 53 bits become a double in [0, 1).
Normals come from the Box-Muller transform of two such uniforms.
"""
import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_ODD = np.uint64(0xD1B54A32D192ED03)


def _mix(z):
    z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
    z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
    return z ^ (z >> np.uint64(31))


def _unit(seed, stream, n, lane):
    """n doubles in [0,1); ``lane`` separates the two Box-Muller inputs."""
    with np.errstate(over="ignore"):
        base = np.uint64(seed) * _GOLDEN + np.uint64(2 * stream + lane) * _ODD
        ctr = base + np.arange(1, n + 1, dtype=np.uint64) * _GOLDEN
        bits = _mix(ctr)
    return (bits >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def uniform(seed, stream, shape, lo=0.0, hi=1.0):
    n = int(np.prod(shape))
    u = _unit(seed, stream, n, 0)
    return (lo + (hi - lo) * u).astype(np.float32).reshape(shape)


def normal(seed, stream, shape, mean=0.0, std=1.0):
    n = int(np.prod(shape))
    u1 = 1.0 - _unit(seed, stream, n, 0)          # (0, 1]
    u2 = _unit(seed, stream, n, 1)
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return (mean + std * z).astype(np.float32).reshape(shape)


def round_to_bf16(a):
    """float32 array -> nearest bf16-representable float32 (ties to even)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) & np.uint64(0xFFFF0000)
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def bf16_bits(a):
    """bf16-representable float32 array -> uint16 bit patterns (exact)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    if np.any(u & np.uint32(0xFFFF)):
        raise ValueError("array holds values that are not bf16-representable")
    return (u >> np.uint32(16)).astype(np.uint16).reshape(a.shape)


def from_bf16_bits(b):
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).reshape(b.shape)

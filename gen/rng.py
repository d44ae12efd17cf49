"""Counter-based random streams for the synthetic TSVD inputs.

Every element of every tensor is a pure function of (seed, tensor id, element
index), so any slice can be generated anywhere, in any order, and the CPU
checker and the GPU harness see bit-identical inputs.  The generator is the
SplitMix64 output function (Steele, Lea & Flood, "Fast splittable pseudorandom
number generators", OOPSLA 2014) applied to a Weyl sequence; normals come from
the Box-Muller transform evaluated in float64.

This module holds input generation only: none of the TSVD arithmetic lives here.
"""
from __future__ import annotations

import numpy as np

_GOLD = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 22


def _mix(z: np.ndarray) -> np.ndarray:
    """SplitMix64 finaliser on a uint64 array (wraps modulo 2**64)."""
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def _key(seed: int, tensor_id: int, lane: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = _mix(np.array([np.uint64(seed) * _GOLD + np.uint64(tensor_id)], dtype=np.uint64))
        k = _mix(k * _GOLD + np.uint64(lane))
    return k[0]


def raw_u64(seed: int, tensor_id: int, lane: int, start: int, count: int) -> np.ndarray:
    """`count` 64-bit words of stream (seed, tensor_id, lane), elements start..start+count."""
    idx = np.arange(start, start + count, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _mix(_key(seed, tensor_id, lane) + (idx + np.uint64(1)) * _GOLD)


def uniform01(seed: int, tensor_id: int, lane: int, start: int, count: int) -> np.ndarray:
    """float64 uniform on (0,1): top 53 bits, offset by half a step so 0 never occurs."""
    w = raw_u64(seed, tensor_id, lane, start, count) >> np.uint64(11)
    return (w.astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def _chunks(n: int):
    for s in range(0, n, _CHUNK):
        yield s, min(_CHUNK, n - s)


def ternary(seed: int, tensor_id: int, n: int, density: float) -> np.ndarray:
    """int8 array of n i.i.d. entries: nonzero w.p. `density`, sign +-1 equiprobable."""
    out = np.empty(n, dtype=np.int8)
    for s, c in _chunks(n):
        nz = uniform01(seed, tensor_id, 0, s, c) < density
        neg = (raw_u64(seed, tensor_id, 1, s, c) >> np.uint64(63)).astype(bool)
        out[s:s + c] = np.where(nz, np.where(neg, -1, 1), 0).astype(np.int8)
    return out


def normal(seed: int, tensor_id: int, n: int) -> np.ndarray:
    """float64 standard normals (Box-Muller, cosine branch, one normal per index)."""
    out = np.empty(n, dtype=np.float64)
    for s, c in _chunks(n):
        u1 = uniform01(seed, tensor_id, 0, s, c)
        u2 = uniform01(seed, tensor_id, 1, s, c)
        out[s:s + c] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return out


def laplace(seed: int, tensor_id: int, n: int) -> np.ndarray:
    """float64 standard Laplace variates (density exp(-|x|)/2) by inversion of the distribution."""
    out = np.empty(n, dtype=np.float64)
    for s, c in _chunks(n):
        u = uniform01(seed, tensor_id, 0, s, c) - 0.5
        out[s:s + c] = -np.sign(u) * np.log1p(-2.0 * np.abs(u))
    return out


def uniform(seed: int, tensor_id: int, n: int, lo: float, hi: float) -> np.ndarray:
    out = np.empty(n, dtype=np.float64)
    for s, c in _chunks(n):
        out[s:s + c] = lo + (hi - lo) * uniform01(seed, tensor_id, 0, s, c)
    return out


def int8_uniform(seed: int, tensor_id: int, n: int, lo: int = -127, hi: int = 127) -> np.ndarray:
    """int8 uniform on the integers lo..hi inclusive."""
    span = hi - lo + 1
    out = np.empty(n, dtype=np.int8)
    for s, c in _chunks(n):
        v = np.floor(uniform01(seed, tensor_id, 0, s, c) * span).astype(np.int64)
        out[s:s + c] = (np.minimum(v, span - 1) + lo).astype(np.int8)
    return out


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns the uint16 bit patterns."""
    b = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns to float32."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)

"""Seeded, counter-based synthetic tensor generator shared by the oracle tests and the CUDA tests.

This module holds no arithmetic of the fused-chain method itself: it only draws numbers and rounds
them to the storage type.  Both sides of every parity test receive the *same stored bits*.

Recipe (every tensor): stream key = splitmix64-hash(seed, tensor_tag); element i uses counters
2i and 2i+1 of that stream; two 53-bit uniforms -> Box-Muller (cosine branch) in fp64 -> scale and
shift -> round to fp32 (RNE) -> for bf16 storage round the fp32 value to bf16 (RNE) and keep the
16-bit pattern.  Uniform tensors use counter 2i only.

bf16 tensors are carried as numpy uint16 bit patterns, fp32 tensors as numpy float32.
"""
from __future__ import annotations

import zlib
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 21


def _mix(z: np.ndarray) -> np.ndarray:
    """splitmix64 output function on a uint64 array (wrap-around arithmetic)."""
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def stream_key(seed: int, tag: str) -> np.uint64:
    """A 64-bit key for (seed, tensor tag)."""
    h = zlib.crc32(tag.encode()) & 0xFFFFFFFF
    base = np.array([(int(seed) & 0xFFFFFFFF) << 32 | h], dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _mix(base * _GOLDEN + _GOLDEN)[0]


def _bits(key: np.uint64, start: int, count: int, lane: int) -> np.ndarray:
    """64 random bits for counters 2*(start+i)+lane, i in [0,count)."""
    with np.errstate(over="ignore"):
        ctr = (np.arange(start, start + count, dtype=np.uint64) * np.uint64(2) + np.uint64(lane))
        return _mix(key + (ctr + np.uint64(1)) * _GOLDEN)


def _uniform53(bits: np.ndarray, open_low: bool) -> np.ndarray:
    """(0,1] when open_low else [0,1), 53-bit resolution."""
    k = (bits >> np.uint64(11)).astype(np.float64)
    if open_low:
        k = k + 1.0
    return k * (1.0 / 9007199254740992.0)


def _chunks(n: int):
    for s in range(0, n, _CHUNK):
        yield s, min(_CHUNK, n - s)


def _parallel_fill(n: int, fn) -> np.ndarray:
    out = np.empty(n, dtype=np.float32)

    def work(sc):
        s, c = sc
        out[s:s + c] = fn(s, c)

    jobs = list(_chunks(n))
    if len(jobs) <= 1:
        for j in jobs:
            work(j)
    else:
        with ThreadPoolExecutor(max_workers=8) as ex:
            list(ex.map(work, jobs))
    return out


def normal_f32(seed: int, tag: str, shape, mean: float = 0.0, std: float = 1.0) -> np.ndarray:
    """N(mean, std) samples rounded to fp32."""
    key = stream_key(seed, tag)
    n = int(np.prod(shape, dtype=np.int64))

    def fn(s, c):
        u1 = _uniform53(_bits(key, s, c, 0), True)
        u2 = _uniform53(_bits(key, s, c, 1), False)
        z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
        return (z * std + mean).astype(np.float32)

    return _parallel_fill(n, fn).reshape(shape)


def uniform_f32(seed: int, tag: str, shape, lo: float, hi: float) -> np.ndarray:
    """U[lo, hi) samples rounded to fp32."""
    key = stream_key(seed, tag)
    n = int(np.prod(shape, dtype=np.int64))

    def fn(s, c):
        u = _uniform53(_bits(key, s, c, 0), False)
        return (lo + (hi - lo) * u).astype(np.float32)

    return _parallel_fill(n, fn).reshape(shape)


def integers_f32(seed: int, tag: str, shape, lo: int, hi: int) -> np.ndarray:
    """Integers in [lo, hi] as fp32 (exactly representable in bf16 when |v| <= 256)."""
    key = stream_key(seed, tag)
    n = int(np.prod(shape, dtype=np.int64))
    span = np.uint64(hi - lo + 1)

    def fn(s, c):
        b = _bits(key, s, c, 0) >> np.uint64(16)
        return ((b % span).astype(np.int64) + lo).astype(np.float32)

    return _parallel_fill(n, fn).reshape(shape)


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to bf16 (round to nearest even) and return the uint16 patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    nan = (u & np.uint32(0x7FFFFFFF)) > np.uint32(0x7F800000)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    with np.errstate(over="ignore"):
        r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    r = np.where(nan, (u >> np.uint32(16)) | np.uint32(0x40), r)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32 (used by generators and by test comparisons)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _e4m3_table():
    """Value of each of the 127 non-negative finite E4M3 patterns (finite-only variant), ascending."""
    b = np.arange(127)
    e, f = b >> 3, b & 7
    return np.where(e == 0, f * 2.0 ** -9, (8 + f) * 2.0 ** (e.astype(np.float64) - 10))


def f32_to_e4m3_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to 8-bit E4M3 (nearest, ties to the even pattern, magnitudes beyond 448 saturate)
    and return the uint8 patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32).astype(np.float64)
    tab = _e4m3_table()
    mag = np.minimum(np.abs(a), tab[-1])
    hi = np.clip(np.searchsorted(tab, mag, side="left"), 1, 126)
    lo = hi - 1
    dlo, dhi = mag - tab[lo], tab[hi] - mag
    pick_hi = (dhi < dlo) | ((dhi == dlo) & (hi % 2 == 0))
    code = np.where(pick_hi, hi, lo).astype(np.uint8)
    return np.where(np.signbit(a), code | np.uint8(0x80), code).astype(np.uint8)


def store(a_f32: np.ndarray, dtype: str) -> np.ndarray:
    """Round an fp32 array to the storage type: 'f32' -> float32, 'bf16' -> uint16 patterns, 'f16' -> float16,
    'f8e4m3' -> uint8 patterns, 'e8m0' -> scale bytes (biased exponents) tagged int8."""
    if dtype == "f32":
        return np.ascontiguousarray(a_f32, dtype=np.float32)
    if dtype == "bf16":
        return f32_to_bf16_bits(a_f32)
    if dtype == "f16":
        return np.ascontiguousarray(a_f32, dtype=np.float32).astype(np.float16)   # IEEE half, round to nearest even
    if dtype == "f8e4m3":
        return f32_to_e4m3_bits(a_f32)
    if dtype == "e8m0":
        # the values are exponents x: the stored byte is x + 127 (scale 2^x), clipped to the finite patterns 0..254.
        # The array is tagged int8 so that consumers can tell scale bytes from E4M3 elements (both are one byte).
        return np.clip(np.rint(np.asarray(a_f32, dtype=np.float64)) + 127, 0, 254).astype(np.uint8).view(np.int8)
    raise ValueError(dtype)

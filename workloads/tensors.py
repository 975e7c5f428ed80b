"""Counter-based seeded tensors.

Element ``i`` of stream ``stream`` under ``seed`` depends only on
``(seed, stream, i)``: a splitmix64 finaliser over a Weyl sequence gives 64
random bits, the top 53 make a uniform in [0, 1), and a Box-Muller pair of
uniforms makes a standard normal.  Values are produced in float64 and rounded
once to the storage type (float32, or bfloat16 kept as its 16-bit pattern).
"""
from __future__ import annotations

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _mix(z: np.ndarray) -> np.ndarray:
    z = z.copy()
    z ^= z >> np.uint64(30)
    z *= _M1
    z ^= z >> np.uint64(27)
    z *= _M2
    z ^= z >> np.uint64(31)
    return z


def _key(seed: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = _mix(np.array([(seed & 0xFFFFFFFF) | ((stream & 0xFFFFFFFF) << 32)], dtype=np.uint64))
        return _mix(k + _GOLDEN)[0]


def _bits(seed: int, stream: int, start: int, count: int, lane: int, lanes: int) -> np.ndarray:
    """64 random bits for counters ``lanes*(start+j)+lane``, j < count."""
    with np.errstate(over="ignore"):
        idx = np.arange(start, start + count, dtype=np.uint64) * np.uint64(lanes) + np.uint64(lane)
        return _mix(_key(seed, stream) + (idx + np.uint64(1)) * _GOLDEN)


_CHUNK = 1 << 22


def uniform(seed: int, stream: int, n: int, lo: float = 0.0, hi: float = 1.0) -> np.ndarray:
    """``n`` float64 draws, uniform on [lo, hi)."""
    out = np.empty(n, dtype=np.float64)
    for s in range(0, n, _CHUNK):
        c = min(_CHUNK, n - s)
        u = (_bits(seed, stream, s, c, 0, 2) >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))
        out[s:s + c] = lo + (hi - lo) * u
    return out


def normal(seed: int, stream: int, n: int, mean: float = 0.0, std: float = 1.0) -> np.ndarray:
    """``n`` float64 draws from N(mean, std^2) by Box-Muller on two uniforms per element."""
    out = np.empty(n, dtype=np.float64)
    for s in range(0, n, _CHUNK):
        c = min(_CHUNK, n - s)
        u1 = (_bits(seed, stream, s, c, 0, 2) >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))
        u2 = (_bits(seed, stream, s, c, 1, 2) >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))
        r = np.sqrt(-2.0 * np.log1p(-u1))  # 1-u1 is in (0, 1]
        out[s:s + c] = mean + std * r * np.cos(2.0 * np.pi * u2)
    return out


def integers(seed: int, stream: int, n: int, lo: int, hi: int) -> np.ndarray:
    """``n`` float64 draws of integers uniform on [lo, hi]."""
    span = hi - lo + 1
    out = np.empty(n, dtype=np.float64)
    for s in range(0, n, _CHUNK):
        c = min(_CHUNK, n - s)
        b = _bits(seed, stream, s, c, 0, 2) >> np.uint64(33)
        out[s:s + c] = (b % np.uint64(span)).astype(np.float64) + lo
    return out


def round_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32/float64 values to bfloat16 (nearest, ties to even); returns uint16 patterns."""
    f = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (f >> np.uint32(16)) & np.uint32(1)
    r = (f + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def make_tensor(law: dict, shape, dtype: str, seed: int, stream: int) -> np.ndarray:
    """Draw one tensor.

    ``law`` is ``{"kind": "normal", "mean": m, "std": s}``, ``{"kind": "uniform",
    "lo": a, "hi": b}`` or ``{"kind": "int", "lo": a, "hi": b}``.  Returns a
    float32 array for ``dtype == "f32"`` and a uint16 array of bfloat16 bit
    patterns for ``dtype == "bf16"``.
    """
    n = int(np.prod(shape)) if len(shape) else 1
    kind = law["kind"]
    if kind == "normal":
        v = normal(seed, stream, n, law.get("mean", 0.0), law.get("std", 1.0))
    elif kind == "uniform":
        v = uniform(seed, stream, n, law.get("lo", 0.0), law.get("hi", 1.0))
    elif kind == "int":
        v = integers(seed, stream, n, law["lo"], law["hi"])
    else:
        raise ValueError(f"unknown law {kind!r}")
    v32 = v.astype(np.float32).reshape(shape)
    if dtype == "f32":
        return v32
    if dtype == "bf16":
        return round_to_bf16_bits(v32).reshape(shape)
    raise ValueError(f"unknown dtype {dtype!r}")


def as_float64(arr: np.ndarray, dtype: str) -> np.ndarray:
    """Widen a stored tensor (float32, or bfloat16 bit patterns) exactly to float64."""
    if dtype == "bf16":
        return bf16_bits_to_f32(arr).astype(np.float64)
    return arr.astype(np.float64)

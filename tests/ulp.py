"""Error metrics shared by the parity tests (host-side numpy; no method arithmetic).

ord(v): the IEEE bit pattern of a stored value mapped onto the signed integer
line, so that adjacent representable values differ by 1, +0 and -0 coincide and
subnormals need no special case.  The ulp distance in a storage type is the
absolute difference of two such ordinals.

fp32 results are judged against the fp64 oracle value o itself:
  strict  E  = |got - o| / ulp32(o),    ulp32 = spacing of fp32 at |o| (>= 2^-149)
  scaled  Ec = |got - o| / ulp32(T),    T = |h| + |x h'|, the size of the two
             addends whose difference forms f' for x < 0.  T >= |o|, T == |o| for x >= 0.
16-bit results are judged against the oracle value rounded once to the type.
"""
from __future__ import annotations

import numpy as np

TINY32 = 2.0 ** -149
MIN_NORMAL32 = 2.0 ** -126


def ulp32(o: np.ndarray) -> np.ndarray:
    """Spacing of fp32 numbers at |o| (o in fp64), floored at the subnormal spacing."""
    a = np.abs(np.asarray(o, np.float64))
    a = np.minimum(a, np.finfo(np.float32).max)
    with np.errstate(over="ignore", invalid="ignore"):
        # exponent of |o| in fp64 -> spacing of a 24-bit significand there
        e = np.floor(np.log2(np.maximum(a, MIN_NORMAL32)))
        e = np.where(2.0 ** e > np.maximum(a, MIN_NORMAL32), e - 1, e)
        e = np.where(2.0 ** (e + 1) <= np.maximum(a, MIN_NORMAL32), e + 1, e)
    return np.maximum(2.0 ** (e - 23), TINY32)


def err_strict32(got: np.ndarray, o: np.ndarray) -> np.ndarray:
    return np.abs(got.astype(np.float64) - o) / ulp32(o)


def err_scaled32(got: np.ndarray, o: np.ndarray, scale: np.ndarray) -> np.ndarray:
    return np.abs(got.astype(np.float64) - o) / ulp32(np.maximum(np.abs(scale), np.abs(o)))


def ord16(bits: np.ndarray) -> np.ndarray:
    """Ordinal of a 16-bit pattern (bf16 or fp16): sign-magnitude -> signed integer line."""
    b = np.asarray(bits).view(np.uint16).astype(np.int64)
    mag = b & 0x7FFF
    return np.where(b & 0x8000, -mag, mag)


def ord32(vals: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(vals, np.float32).view(np.uint32).astype(np.int64)
    mag = b & 0x7FFFFFFF
    return np.where(b & 0x80000000, -mag, mag)


def ulp_distance16(a_bits: np.ndarray, b_bits: np.ndarray) -> np.ndarray:
    return np.abs(ord16(a_bits) - ord16(b_bits))


def is_nan16(bits: np.ndarray, dtype: str) -> np.ndarray:
    b = np.asarray(bits).view(np.uint16).astype(np.int64) & 0x7FFF
    return b > (0x7F80 if dtype == "bf16" else 0x7C00)


def same_bits_or_both_nan(a: np.ndarray, b: np.ndarray, dtype: str) -> np.ndarray:
    """Equality of the raw bit patterns (so +0 and -0 differ: a single rounding of the exact product fixes the
    sign of a zero too), any NaN equal to any NaN (backward parity)."""
    if dtype == "f32":
        a32 = np.ascontiguousarray(a, np.float32)
        b32 = np.ascontiguousarray(b, np.float32)
        return (a32.view(np.uint32) == b32.view(np.uint32)) | (np.isnan(a32) & np.isnan(b32))
    a16, b16 = np.asarray(a).view(np.uint16), np.asarray(b).view(np.uint16)
    return (a16 == b16) | (is_nan16(a, dtype) & is_nan16(b, dtype))

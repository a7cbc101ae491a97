"""TEST INFRASTRUCTURE -- plain restatement of the prediction compression used before the exchange of
Section 3 (fewer bits per prediction: b_pred halves when 32-bit logits are sent as bfloat16).

Only ``tests/`` may import this module.  bfloat16 is the upper half of an IEEE binary32; packing rounds to
nearest, ties to even, written out here on the integer bit patterns one element at a time (pure Python for
the pins, vectorised numpy with the same integer arithmetic for larger arrays).  NaN stays NaN (quiet),
infinities stay infinities; unpacking is exact.
"""
from __future__ import annotations

import struct

import numpy as np


def pack_one(x: float) -> int:
    """bf16 bit pattern of one binary32 value, round-to-nearest-even (the definition, element-wise)."""
    (u,) = struct.unpack("<I", struct.pack("<f", x))
    if (u & 0x7F800000) == 0x7F800000 and (u & 0x007FFFFF):      # NaN: keep it a NaN
        return ((u >> 16) | 0x0040) & 0xFFFF
    upper, lower = u >> 16, u & 0xFFFF
    if lower > 0x8000 or (lower == 0x8000 and (upper & 1)):       # above the half-way point, or a tie towards even
        upper += 1                                                  # may carry into the exponent: that is the rounding to the next binade / infinity
    return upper & 0xFFFF


def unpack_one(b: int) -> float:
    return struct.unpack("<f", struct.pack("<I", (b & 0xFFFF) << 16))[0]


def pack(x: np.ndarray) -> np.ndarray:
    """Vectorised form of pack_one (same integer arithmetic); returns uint16."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    upper, lower = u >> np.uint64(16), u & np.uint64(0xFFFF)
    up = (lower > 0x8000) | ((lower == 0x8000) & ((upper & np.uint64(1)) == 1))
    out = (upper + up.astype(np.uint64)) & np.uint64(0xFFFF)
    nan = ((u & np.uint64(0x7F800000)) == np.uint64(0x7F800000)) & ((u & np.uint64(0x007FFFFF)) != 0)
    out = np.where(nan, ((u >> np.uint64(16)) | np.uint64(0x0040)) & np.uint64(0xFFFF), out)
    return out.astype(np.uint16)


def unpack(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)

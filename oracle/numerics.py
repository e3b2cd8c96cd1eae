"""Rounding helpers of the oracle (test infrastructure; not used by the product)."""
from __future__ import annotations

import numpy as np


def round_bf16(a):
    """Nearest-even rounding of float64/float32 values to bf16, returned as float64.

    A bf16 number is a float32 whose low 16 mantissa bits are zero.  The value is
    first rounded to float32 (as the hardware converts an fp32 result), then the
    low half is rounded away, ties to even.
    """
    a32 = np.asarray(a, dtype=np.float32)
    bits = np.ascontiguousarray(a32).view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    bits = (bits + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    out = bits.astype(np.uint32).view(np.float32).reshape(a32.shape)
    return out.astype(np.float64)

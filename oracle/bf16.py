"""ORACLE — TEST INFRASTRUCTURE ONLY.

bfloat16 storage rounding (round to nearest, ties to even) written with integer
arithmetic on the IEEE bit patterns.  The paper counts stored elements (Eq. 3)
and sizes caches "under BF16" (Section 1), so factors are stored in the same
type as dense pages; this module lets the oracle apply that storage step to its
fp64 factors.  Values pass through fp32 first (the type the factors are
produced in on the GPU), then lose the low 16 mantissa bits.
"""
import numpy as np


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """fp64 array -> nearest bf16 values, returned as fp64."""
    f32 = np.asarray(x, dtype=np.float64).astype(np.float32)
    bits = f32.view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    rounded = (bits + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    out = rounded.astype(np.uint32).view(np.float32)
    nan = np.isnan(f32)
    if nan.any():
        out = np.where(nan, np.float32(np.nan), out)
    return out.astype(np.float64).reshape(np.shape(x))

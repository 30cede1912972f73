"""bfloat16 <-> float32, written out from the format definition.

Test infrastructure (see the package header).  bfloat16 is the upper 16 bits of
an IEEE binary32 value.  Widening is exact.  Narrowing rounds to nearest, ties
to even; Inf stays Inf, NaN stays NaN (quietened).

Pinned by tests/test_oracle_quantizers.py against torch's own conversion on all
65536 bit patterns and on random floats including exact ties.
"""
import numpy as np


def bf16_bits_to_f32(bits):
    """uint16 bit patterns -> float32 values (exact)."""
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32)


def f32_to_bf16_bits(x):
    """float32 -> uint16 bfloat16 bit patterns, round-to-nearest-even."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    # adding 0x7FFF + lsb carries into bit 16 exactly when the discarded half is
    # above one half, or equal to one half with an odd kept mantissa
    rounded = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    is_nan = (u & np.uint32(0x7FFFFFFF)) > np.uint32(0x7F800000)
    nan_bits = (u >> np.uint32(16)) | np.uint32(0x0040)
    return np.where(is_nan, nan_bits, rounded).astype(np.uint16)


def round_to_bf16(x):
    """float32 -> the float32 value of its nearest bfloat16."""
    return bf16_bits_to_f32(f32_to_bf16_bits(x))

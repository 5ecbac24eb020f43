"""bfloat16 rounding for the oracle (round to nearest, ties to even).

Pin: exhaustive comparison against the definition (nearest of the two
neighbouring 8-bit-mantissa values, even mantissa on ties) on hand-picked
bit patterns in the CPU tests.
"""
import numpy as np


def bf16_round(x):
    """Return float64 array holding `x` rounded to bfloat16-representable values.

    The value is first rounded to float32 (the GPU holds it in fp32 before the
    cast), then to bfloat16: add 0x7FFF plus the lowest kept bit to the float32
    bit pattern and clear the low 16 bits.  Finite inputs only (no overflow of
    the 32-bit pattern can occur below infinity).
    """
    a = np.ascontiguousarray(np.asarray(x, dtype=np.float64).astype(np.float32))
    bits = a.view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    bits = (bits + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return bits.view(np.float32).reshape(a.shape).astype(np.float64)

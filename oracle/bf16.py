"""Round-to-nearest-even conversion of binary32 values to bfloat16 precision.

TEST INFRASTRUCTURE ONLY (see the package docstring).

bfloat16 keeps the sign, the 8 exponent bits and the top 7 mantissa bits of a
binary32 number.  Rounding to nearest with ties to even therefore has a closed
form on the bit pattern: add 0x7FFF plus the lowest kept bit, then clear the
low 16 bits.  NaNs are passed through quietly (the add could otherwise carry a
NaN payload into the exponent).  The paper fixes no precision; the rounding
points at which this function is applied are listed in the module docstring
of ``layerpipe_oracle`` (mirror mode) and applied by
``DelayedGradientTrainer._Q``.
"""
import numpy as np


def rn_bf16(x):
    """Return ``x`` rounded to the nearest bfloat16 value, as float32.

    Pinned in tests against an exhaustive sweep of bit patterns converted by
    torch's own float32 -> bfloat16 cast.
    """
    x32 = np.ascontiguousarray(x, dtype=np.float32)
    bits = x32.view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    rounded = (bits + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    is_nan = (bits & np.uint32(0x7FFFFFFF)) > np.uint32(0x7F800000)
    rounded = np.where(is_nan, bits | np.uint32(0x00400000), rounded)
    rounded = (rounded & np.uint32(0xFFFF0000)).astype(np.uint32)
    return rounded.view(np.float32).reshape(x32.shape)

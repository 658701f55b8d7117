"""BF16 helpers for the oracle (test infrastructure; numpy only).

BF16 is the upper half of an IEEE-754 binary32, so widening is exact and
narrowing is a rounding of the binary32/binary64 value to 8 significant bits.
The paper keeps activations and the layer output in BF16 (Abstract; Section 3.1).
"""
import numpy as np


def bits_to_float(bits):
    """uint16 BF16 bit patterns -> float32 values (exact)."""
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32)


def float_to_bits(x):
    """float32 values that are already BF16-representable -> uint16 bit patterns."""
    u = np.ascontiguousarray(np.asarray(x, dtype=np.float32)).view(np.uint32)
    if np.any(u & np.uint32(0xFFFF)):
        raise ValueError("value is not BF16-representable")
    return (u >> np.uint32(16)).astype(np.uint16)


def round_to_bf16(x):
    """Round float64 values to the nearest BF16 (ties to even), returned as float64.

    Done in one step from the binary64 value (no intermediate binary32 rounding):
    x = m * 2**e with 0.5 <= |m| < 1; keep 8 significant bits of m.
    Values below the BF16 normal range are rounded on the subnormal grid 2**-133.
    """
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)
    # exponent of the least significant kept bit: e-8 for normals, -133 floor for subnormals
    lsb = np.maximum(e - 8, -133)
    r = np.rint(np.ldexp(x, -lsb))          # np.rint rounds half to even
    out = np.ldexp(r, lsb)
    out = np.where(np.isfinite(x), out, x)
    # overflow to infinity beyond the largest finite BF16
    big = np.float64(np.float32(3.3895313892515355e38))
    out = np.where(np.abs(out) > big, np.sign(out) * np.inf, out)
    return out

"""Number formats of the method (oracle side, test infrastructure only).

E2M1 payload       : Section "Problem 2", codebook {0, 1/2, 1, 3/2, 2, 3, 4, 6};
                     rounding boundaries Eq. "e2m1-boundaries" {1/4, 3/4, 5/4, 7/4, 5/2, 7/2, 5};
                     ties go to the code with an even (zero) mantissa bit.
E8M0 scale byte    : Section "Fix 1": u = e + 127, alpha = 2**e.
E4M3 scale byte    : Table "fp4-formats" / Eq. "nv-scale": 1-4-3 float, bias 7, max 448,
                     subnormals kept (smallest 2**-9), unsigned use (sign bit 0).
"""
from __future__ import annotations

import numpy as np

# magnitude of nibble codes 0..7 (bit 3 of the nibble is the sign)
E2M1_VALUES = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0], dtype=np.float64)
E2M1_BOUNDARIES = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0], dtype=np.float64)
# at a boundary the neighbour with mantissa bit 0 wins: codes 0,2,4,6 -> boundary k is
# "inclusive upward" exactly when code k+1 is even.
_TIE_GOES_UP = np.array([(k + 1) % 2 == 0 for k in range(7)])


def e2m1_encode_mag(v) -> np.ndarray:
    """Code index 0..7 of |v| rounded to nearest E2M1 magnitude, ties to even, saturating at 6."""
    a = np.abs(np.asarray(v, dtype=np.float64))
    code = np.zeros(a.shape, dtype=np.uint8)
    for k in range(7):
        t = E2M1_BOUNDARIES[k]
        code += (a >= t) if _TIE_GOES_UP[k] else (a > t)
    return code


def e2m1_encode(v) -> np.ndarray:
    """Signed nibble (sign in bit 3).  Zero results keep sign bit 0."""
    v = np.asarray(v, dtype=np.float64)
    mag = e2m1_encode_mag(v)
    sign = ((v < 0) & (mag > 0)).astype(np.uint8)
    return (mag | (sign << 3)).astype(np.uint8)


def e2m1_decode(nib) -> np.ndarray:
    nib = np.asarray(nib, dtype=np.uint8)
    mag = E2M1_VALUES[nib & 7]
    return np.where((nib & 8) != 0, -mag, mag)


def ceil_log2(a) -> np.ndarray:
    """ceil(log2(a)) for a > 0, exact (from the binary exponent, no logarithm)."""
    m, e = np.frexp(np.asarray(a, dtype=np.float64))   # a = m * 2**e, m in [0.5, 1)
    return np.where(m == 0.5, e - 1, e).astype(np.int64)


def e8m0_decode(u) -> np.ndarray:
    """alpha = 2**(u - 127) as float64 (exact for every byte 0..254)."""
    return np.ldexp(1.0, np.asarray(u, dtype=np.int64) - 127)


def e4m3_decode(byte) -> np.ndarray:
    b = np.asarray(byte, dtype=np.int64)
    e = (b >> 3) & 0xF
    m = b & 7
    mag = np.where(e == 0, np.ldexp(m.astype(np.float64), -9), np.ldexp(1.0 + m / 8.0, e - 7))
    return np.where((b & 0x80) != 0, -mag, mag)


def e4m3_encode_unsigned(t) -> np.ndarray:
    """Byte of the E4M3 value nearest to t >= 0: ties to even mantissa, saturate at 448."""
    t = np.asarray(t, dtype=np.float64)
    out = np.zeros(t.shape, dtype=np.uint8)
    tt = np.minimum(t, 448.0)
    _, e = np.frexp(tt)                 # tt in [2**(e-1), 2**e)
    exp = np.maximum(e - 1, -6)         # subnormals share the exponent of the smallest normal
    step = np.ldexp(1.0, exp - 3)       # spacing of representable values at this exponent
    k = np.rint(tt / step)              # numpy rint is round-half-even; tt/step is exact
    val = k * step
    # re-derive the byte from the rounded value (rounding may carry into the next binade)
    _, e2 = np.frexp(val)
    exp2 = np.maximum(e2 - 1, -6)
    is_sub = val < np.ldexp(1.0, -6)
    mant = np.where(is_sub, np.rint(val * 512.0), np.rint((val / np.ldexp(1.0, exp2) - 1.0) * 8.0))
    ebits = np.where(is_sub, 0, exp2 + 7)
    out = (ebits.astype(np.int64) << 3 | mant.astype(np.int64)).astype(np.uint8)
    out = np.where(t > 0, out, 0).astype(np.uint8)
    return out


def e4m3_encode(t) -> np.ndarray:
    """Signed E4M3 byte of the value nearest to t (ties to even mantissa, saturating at +-448); a result that rounds
    to zero keeps sign bit 0."""
    t = np.asarray(t, dtype=np.float64)
    mag = e4m3_encode_unsigned(np.abs(t))
    sign = ((t < 0) & (mag > 0)).astype(np.uint8)
    return (mag | (sign << 7)).astype(np.uint8)

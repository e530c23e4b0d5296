"""TEST INFRASTRUCTURE, NOT PRODUCT CODE.

The paper's dynamic floating-point data type (Section 2.1), written out bit by
bit in exact Python integers so the integer special case used by the
convolution path can be checked against the general definition.

A value is alpha * beta (Eq. 1); beta is an n-bit pattern b_{n-1} .. b_0 with p
significand bits, decoded by sign and magnitude (Eq. 2) with the exponent field
of Eq. 4.  Eq. 5 gives the largest beta in closed form.

Pinned in tests/test_oracle_format.py: the closed form of Eq. 5 equals the
enumerated maximum; (n=8, p=6) and (n=8, p=7) are the integers -127..127 (the
discussion section calls p = 6 "int8"); (n=8, p=2) scaled by 2^-16 equals the
IEEE binary16 value of the byte placed in the top half (the discussion section
calls p = 2 truncated half precision).
"""
from fractions import Fraction


def bit(pattern: int, i: int) -> int:
    return (pattern >> i) & 1


def exponent_field(pattern: int, n: int, p: int) -> int:
    """Eq. 4: 0 if p = n-1, else the integer held in bits p .. n-2."""
    if p == n - 1:
        return 0
    return sum(bit(pattern, i) << (i - p) for i in range(p, n - 1))


def significand_field(pattern: int, p: int) -> int:
    return sum(bit(pattern, i) << i for i in range(p))


def decode_sign_magnitude(pattern: int, n: int, p: int) -> Fraction:
    """Eq. 2.  Subnormal (exponent field 0): +-significand.  Normal: hidden bit
    2^p added and the whole scaled by 2^(exponent field - 1)."""
    e_hat = exponent_field(pattern, n, p)
    sign = -1 if bit(pattern, n - 1) else 1
    m = significand_field(pattern, p)
    if e_hat == 0:
        return Fraction(sign * m)
    return Fraction(2) ** (e_hat - 1) * sign * ((1 << p) + m)


def decode_twos_complement_as_printed(pattern: int, n: int, p: int) -> Fraction:
    """Eq. 3 exactly as printed: the sign bit subtracts 2^p + 2^(p+1).  Kept only
    to document that the printed form is not ordinary two's complement (-1 is not
    representable for n = 8); the build stores the Eq. 2 value set in ordinary
    two's-complement bytes instead."""
    e_hat = exponent_field(pattern, n, p)
    neg = bit(pattern, n - 1) * ((1 << p) + (1 << (p + 1)))
    m = significand_field(pattern, p)
    if e_hat == 0:
        return Fraction(-neg + m)
    return Fraction(2) ** (e_hat - 1) * (-neg + (1 << p) + m)


def beta_max_closed_form(n: int, p: int) -> int:
    """Eq. 5 with equality (Inf/NaN patterns reused as numbers)."""
    if p == n - 1:
        return (1 << (n - 1)) - 1
    return (1 << ((1 << (n - p - 1)) - 2)) * ((1 << (p + 1)) - 1)


def value_set(n: int, p: int):
    """All values beta can take (as exact Fractions), one per bit pattern."""
    return [decode_sign_magnitude(b, n, p) for b in range(1 << n)]


def mac_accumulator_bits(N: int, b_x: int, eps_x: int, b_y: int, eps_y: int) -> int:
    """Eq. 8 (with the second factor read as b_y + eps_y, as Eq. 9 has it):
    smallest two's-complement width q that holds any sum of N products with
    beta_x in [-b_x-eps_x, b_x] and beta_y in [-b_y-eps_y, b_y].
    Evaluated in exact integers: ceil(log2(v + 1) + 1) for integer v >= 1 is
    (v).bit_length() + 1."""
    v = N * (b_x + eps_x) * (b_y + eps_y)
    return v.bit_length() + 1


def mac_max_terms(q: int, b_x: int, eps_x: int, b_y: int, eps_y: int) -> int:
    """Eq. 9: the largest N a q-bit accumulator holds without loss."""
    return ((1 << (q - 1)) - 1) // ((b_x + eps_x) * (b_y + eps_y))


def add_accumulator_bits(N: int, b_x: int, eps_x: int) -> int:
    """Eq. 12: width for a sum of N values in [-b_x-eps_x, b_x]."""
    if eps_x == 0:
        return (N * b_x).bit_length() + 1          # ceil(log2(N b + 1) + 1)
    v = N * b_x + N * eps_x                        # ceil(log2(v) + 1)
    return (v - 1).bit_length() + 1


def add_max_terms(q: int, b_x: int, eps_x: int) -> int:
    """Eq. 13."""
    if eps_x == 0:
        return ((1 << (q - 1)) - 1) // b_x
    return (1 << (q - 1)) // (b_x + eps_x)


# ---------------------------------------------------------------------------------------------
# float <-> (n, p) codes (Section 3: clamp to the threshold range, divide by the scale, round to
# the desired beta; back by multiplying with the scale).  The scale is alpha = 2^e.  A code is the
# n-bit sign-and-magnitude pattern of Eq. 2 held in one byte.  Rounding is to the nearest
# representable value, ties to the even pattern (the reading taken for the integer path as well);
# values beyond beta_max saturate; NaN maps to 0; a zero magnitude always gets the pattern 0.
#
# Pinned in tests/test_oracle_format.py: brute force over the enumerated value set in exact
# rationals; (8, 2) with e = -16 against torch's float32 -> float8_e5m2 conversion and (8, 3) with
# e = -9 against float8_e4m3fn (same grids below those types' Inf/NaN codes); decode(encode(v)) = v
# for every representable v.
# ---------------------------------------------------------------------------------------------
def nonneg_values_f64(n: int, p: int):
    import numpy as np
    vals = [decode_sign_magnitude(b, n, p) for b in range(1 << (n - 1))]
    assert all(vals[i] < vals[i + 1] for i in range(len(vals) - 1))
    return np.array([float(v) for v in vals], dtype=np.float64)      # exact: at most p+1 significant bits


def quantize_np(x, e: int, n: int, p: int):
    """float32 array -> uint8 codes.  All arithmetic in float64, which holds x / 2^e, every
    representable value and every midpoint between neighbours exactly."""
    import numpy as np
    x = np.asarray(x, dtype=np.float32)
    vals = nonneg_values_f64(n, p)
    a = np.abs(x.astype(np.float64)) * (2.0 ** -e)
    nan = np.isnan(a)
    a = np.where(nan, 0.0, a)
    a = np.minimum(a, vals[-1])                                   # clamp to the threshold range
    hi = np.searchsorted(vals, a, side="left")                    # first value >= a
    hi = np.minimum(hi, len(vals) - 1)
    lo = np.maximum(hi - 1, 0)
    d_lo, d_hi = a - vals[lo], vals[hi] - a
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))    # nearest; ties to the even pattern
    mag = np.where(pick_hi, hi, lo).astype(np.uint8)
    sign = ((np.signbit(x) & (mag != 0) & ~nan).astype(np.uint8)) << (n - 1)
    return (sign | mag).astype(np.uint8)


def dequantize_np(codes, e: int, n: int, p: int):
    """uint8 codes -> float32 (value * 2^e; exact whenever the result is a finite binary32 number)."""
    import numpy as np
    codes = np.asarray(codes, dtype=np.uint8)
    vals = nonneg_values_f64(n, p)
    mag = vals[codes & ((1 << (n - 1)) - 1)]
    sgn = np.where((codes >> (n - 1)) & 1, -1.0, 1.0)
    return (sgn * mag * (2.0 ** e)).astype(np.float32)

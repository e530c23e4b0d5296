"""TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Convolution on dynamic floating-point operands (Section 2.1 data type, Eq. 6 contraction, Section 3
conversion), for the formats the paper's discussion singles out for 8 bits (p = 4 and p = 3) and any
other (n, p) whose values are integers: every operand is alpha * beta with alpha = 2^e and beta the
value of an n-bit sign-and-magnitude pattern (Eq. 2, exponent field per Eq. 4).  Because alpha is
factored out, the sum of Eq. 6 runs over the betas alone, and those are integers (up to beta_max of
Eq. 5: 1984 for (8, 4), 245760 for (8, 3)), so the contraction is an exact integer sum.

Steps, in the order of the integer oracle (oracle/qconv_ref.c) and of Section 3:
  1. decode the input and weight patterns to integers (Eq. 2),
  2. acc[n, p, q, k] = sum over taps and channels of beta_x * beta_w, zero outside the image (Eq. 6),
     in Python / int64 integers (the bound of Eq. 8-9 with b = beta_max is asserted),
  3. add the integer bias (held at the scale 2^(e_x + e_w[k]) of the sum),
  4. ReLU on the wide value,
  5. convert to the output type: the real number acc / 2^s[k] (s[k] = e_z - e_x - e_w[k] >= 0) goes to the
     nearest value of the (n_out, p_out) type, ties to the even pattern, magnitudes beyond beta_max
     saturate, a zero magnitude is pattern 0 -- the rule of dynfloat.quantize_np, applied here to an
     exact rational instead of a float.

Pinned in tests/test_oracle_fpconv.py: for p = n - 1 on every operand the result equals the integer
oracle's (nearest-even, symmetric saturation); the wide value equals a float64 convolution of the
decoded operands (exact below 2^53); the conversion of step 5 equals dynfloat.quantize_np wherever the
rational is a float; all-beta_max operands reach N * beta_max^2 and the width formula of Eq. 8.
"""
import numpy as np

from oracle import dynfloat


def magnitudes(n: int, p: int):
    """Values of the non-negative patterns 0 .. 2^(n-1)-1 as Python integers, ascending."""
    vals = [dynfloat.decode_sign_magnitude(b, n, p) for b in range(1 << (n - 1))]
    assert all(v.denominator == 1 for v in vals), "the (n, p) type has non-integer values"
    out = [int(v) for v in vals]
    assert all(out[i] < out[i + 1] for i in range(len(out) - 1))
    return out


def decode_codes(codes, n: int, p: int):
    """uint8 patterns -> int64 betas (Eq. 2)."""
    codes = np.asarray(codes, dtype=np.uint8)
    mags = np.array(magnitudes(n, p), dtype=np.int64)
    v = mags[codes & ((1 << (n - 1)) - 1)]
    return np.where((codes >> (n - 1)) & 1, -v, v)


def encode_exact(acc, shift, n: int, p: int):
    """acc: integer array; shift: integer array broadcastable to it.  Pattern of the (n, p) value nearest
    to acc / 2^shift; ties go to the even pattern; beyond beta_max saturates; zero magnitude is pattern 0.
    Brute force over the value list in exact integers: |value * 2^shift - |acc|| is minimised."""
    acc = np.asarray(acc)
    shift = np.broadcast_to(np.asarray(shift), acc.shape)
    mags = magnitudes(n, p)
    out = np.zeros(acc.shape, dtype=np.uint8)
    flat_a, flat_s, flat_o = acc.reshape(-1), shift.reshape(-1), out.reshape(-1)
    for i in range(flat_a.size):
        a, s = int(flat_a[i]), int(flat_s[i])
        mag = abs(a)
        best, best_d = 0, None
        for c, v in enumerate(mags):
            d = abs(v * (1 << s) - mag)
            if best_d is None or d < best_d or (d == best_d and c % 2 == 0 and best % 2 == 1):
                best, best_d = c, d
        flat_o[i] = best | ((1 << (n - 1)) if (a < 0 and best != 0) else 0)
    return out


def encode_exact_fast(acc, shift, n: int, p: int):
    """The same function vectorised (binary search in the ascending value list, int64 throughout; the
    caller keeps |acc| and beta_max * 2^shift below 2^62).  tests check it against encode_exact."""
    acc = np.asarray(acc, dtype=np.int64)
    shift = np.broadcast_to(np.asarray(shift, dtype=np.int64), acc.shape)
    mags = np.array(magnitudes(n, p), dtype=np.int64)
    mag = np.abs(acc)
    hi = np.zeros(acc.shape, dtype=np.int64)                       # first pattern with value * 2^s >= mag
    for c in range(len(mags)):
        hi += (mags[c] << shift) < mag
    hi = np.minimum(hi, len(mags) - 1)
    lo = np.maximum(hi - 1, 0)
    d_lo, d_hi = mag - (mags[lo] << shift), (mags[hi] << shift) - mag
    d_hi = np.where(d_hi < 0, np.int64(2**62), d_hi)               # beyond the last value: saturate to it
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0)) | (lo == hi)
    beyond = mag >= (mags[-1] << shift)
    code = np.where(beyond, len(mags) - 1, np.where(pick_hi, hi, lo))
    sign = np.where((acc < 0) & (code != 0), 1 << (n - 1), 0)
    return (code | sign).astype(np.uint8)


def wide_value(x_codes, w_codes, bias, fmt_in, fmt_w, *, R, S, stride=(1, 1), pad=(0, 0), relu=0):
    """Steps 1-4: int64 [N, P, Q, K].  x_codes [N, H, W, C], w_codes [K, R, S, C] (uint8 patterns)."""
    x = decode_codes(x_codes, *fmt_in)
    w = decode_codes(w_codes, *fmt_w)
    N, H, W, C = x.shape
    K = w.shape[0]
    P = (H + 2 * pad[0] - R) // stride[0] + 1
    Q = (W + 2 * pad[1] - S) // stride[1] + 1
    bx, bw = magnitudes(*fmt_in)[-1], magnitudes(*fmt_w)[-1]
    bmax = int(np.max(np.abs(bias))) if bias is not None else 0
    assert R * S * C * bx * bw + bmax < 2 ** 62, "Eq. 9: the sum may not fit a 64-bit accumulator"
    xp = np.zeros((N, H + 2 * pad[0], W + 2 * pad[1], C), dtype=np.int64)
    xp[:, pad[0]:pad[0] + H, pad[1]:pad[1] + W, :] = x
    acc = np.zeros((N, P, Q, K), dtype=np.int64)
    for r in range(R):
        for s in range(S):
            patch = xp[:, r:r + (P - 1) * stride[0] + 1:stride[0], s:s + (Q - 1) * stride[1] + 1:stride[1], :]
            acc += np.tensordot(patch, w[:, r, s, :], axes=([3], [1]))
    if bias is not None:
        acc += np.asarray(bias, dtype=np.int64)[None, None, None, :]
    if relu:
        acc = np.maximum(acc, 0)
    return acc


def qconv_np(x_codes, w_codes, bias, shift, fmt_in, fmt_w, fmt_out, *, R, S, stride=(1, 1), pad=(0, 0), relu=0):
    """The whole layer: uint8 patterns of the (n_out, p_out) type, [N, P, Q, K]."""
    acc = wide_value(x_codes, w_codes, bias, fmt_in, fmt_w, R=R, S=S, stride=stride, pad=pad, relu=relu)
    K = acc.shape[3]
    sh = np.zeros(K, dtype=np.int64) if shift is None else np.asarray(shift, dtype=np.int64)
    return encode_exact_fast(acc, sh[None, None, None, :], *fmt_out)

"""Pins of the oracle for convolution on dynamic floating-point operands (oracle/fpconv_ref.py):
it must reduce to the integer oracle when p = n - 1, its wide value must be the plain float64
convolution of the decoded operands, its conversion must be the pinned float conversion wherever the
rational is a float, and the accumulator widths must follow Eq. 8-9 with b = beta_max (Eq. 5)."""
import numpy as np
import pytest
import torch

from oracle import dynfloat, fpconv_ref, ref

FORMATS = [(8, 4), (8, 3), (8, 5), (6, 2), (7, 3), (5, 4), (4, 0)]


def _to_sign_magnitude(v, n):
    v = np.asarray(v, dtype=np.int64)
    return (np.abs(v) | np.where(v < 0, 1 << (n - 1), 0)).astype(np.uint8)


def _rand_codes(rng, shape, n):
    c = rng.integers(0, 1 << n, size=shape).astype(np.uint8)
    c[c == (1 << (n - 1))] = 0                      # "minus zero" is not a pattern the encoder produces
    return c


@pytest.mark.parametrize("p", [7, 6])
def test_integer_formats_reduce_to_the_integer_oracle(p):
    """(8, 7) and (8, 6) hold exactly the integers -127 .. 127 (the discussion section calls p = 6 int8), so
    the layer must equal the int8 oracle with nearest-even rounding and symmetric saturation."""
    rng = np.random.default_rng(1)
    for (N, H, W, C, K, R, S, stride, pad, relu) in [(2, 7, 9, 5, 6, 3, 3, (1, 1), (1, 1), 1),
                                                       (1, 8, 6, 4, 3, 3, 2, (2, 1), (0, 1), 0),
                                                       (2, 5, 5, 16, 8, 1, 1, (1, 1), (0, 0), 0)]:
        x = rng.integers(-127, 128, size=(N, H, W, C)).astype(np.int8)
        w = rng.integers(-127, 128, size=(K, R, S, C)).astype(np.int8)
        bias = rng.integers(-2**14, 2**14, size=K).astype(np.int32)
        shift = rng.integers(0, 14, size=K).astype(np.int32)
        want = ref.qconv(x, w, bias, shift, R=R, S=S, stride=stride, pad=pad, relu=relu)
        got = fpconv_ref.qconv_np(_to_sign_magnitude(x, 8), _to_sign_magnitude(w, 8), bias, shift, (8, p), (8, p), (8, p),
                                  R=R, S=S, stride=stride, pad=pad, relu=relu)
        assert (fpconv_ref.decode_codes(got, 8, p) == want.astype(np.int64)).all()
        assert not ((got == 0x80).any())             # a zero magnitude is always pattern 0


@pytest.mark.parametrize("fmt", FORMATS)
def test_wide_value_is_the_float64_convolution_of_the_decoded_operands(fmt):
    n, p = fmt
    rng = np.random.default_rng(n * 10 + p)
    for (N, H, W, C, K, R, S, stride, pad) in [(2, 6, 7, 3, 4, 3, 2, (1, 2), (1, 0)), (1, 9, 5, 6, 5, 2, 3, (2, 1), (0, 1))]:
        xc, wc = _rand_codes(rng, (N, H, W, C), n), _rand_codes(rng, (K, R, S, C), n)
        bias = rng.integers(-1000, 1000, size=K).astype(np.int64)
        acc = fpconv_ref.wide_value(xc, wc, bias, fmt, fmt, R=R, S=S, stride=stride, pad=pad)
        xf = torch.from_numpy(fpconv_ref.decode_codes(xc, n, p).astype(np.float64)).permute(0, 3, 1, 2)
        wf = torch.from_numpy(fpconv_ref.decode_codes(wc, n, p).astype(np.float64)).permute(0, 3, 1, 2)
        y = torch.nn.functional.conv2d(xf, wf, torch.from_numpy(bias.astype(np.float64)), stride=stride, padding=pad)
        assert np.abs(acc).max() < 2.0 ** 53
        assert (y.permute(0, 2, 3, 1).numpy() == acc.astype(np.float64)).all()
        relu = fpconv_ref.wide_value(xc, wc, bias, fmt, fmt, R=R, S=S, stride=stride, pad=pad, relu=1)
        assert (relu == np.maximum(acc, 0)).all()


@pytest.mark.parametrize("fmt", FORMATS)
def test_conversion_is_nearest_value_ties_to_even_pattern(fmt):
    n, p = fmt
    mags = fpconv_ref.magnitudes(n, p)
    assert mags[-1] == dynfloat.beta_max_closed_form(n, p)                     # Eq. 5
    rng = np.random.default_rng(3)
    for s in (0, 1, 3, 7):
        # every value, every midpoint between neighbours, one unit either side, both signs, and beyond the range
        pts = set()
        for a, b in zip(mags[:-1], mags[1:]):
            mid2 = (a + b) << s                                                 # twice the midpoint, scaled
            for d in (-1, 0, 1):
                if mid2 % 2 == 0:
                    pts.add(mid2 // 2 + d)
                pts.add((a << s) + d)
        pts.update([(mags[-1] << s) + k for k in (-1, 0, 1, 1000)])
        pts.update(int(v) for v in rng.integers(0, (mags[-1] << s) + 50, size=300))
        acc = np.array(sorted(pts) + [-v for v in sorted(pts)], dtype=np.int64)
        slow = fpconv_ref.encode_exact(acc, s, n, p)
        fast = fpconv_ref.encode_exact_fast(acc, s, n, p)
        assert (slow == fast).all()
        # the pinned float conversion on the same rationals (exact in binary32 below 2^24)
        small = np.abs(acc) < 2 ** 24
        assert (dynfloat.quantize_np(acc[small].astype(np.float32), s, n, p) == fast[small]).all()
        # nearest: no other value is strictly closer; the result never exceeds the range
        dec = fpconv_ref.decode_codes(fast, n, p)
        err = np.abs(dec * (1 << s) - acc)
        for v in mags:
            assert (err <= np.abs(np.abs(acc) - (v << s))).all()
    # shift 0 is the identity on representable values
    vals = np.array(mags + [-m for m in mags[1:]], dtype=np.int64)
    assert (fpconv_ref.decode_codes(fpconv_ref.encode_exact_fast(vals, 0, n, p), n, p) == vals).all()


def test_accumulator_width_follows_eq8_with_beta_max():
    """All-beta_max operands reach N * beta_max^2; the width Eq. 8 gives for b = beta_max (eps = 0: the
    sign-magnitude range is symmetric) holds that sum and one bit less does not."""
    for (n, p) in [(8, 4), (8, 3)]:
        b = dynfloat.beta_max_closed_form(n, p)
        C, R, S = 32, 3, 3
        top = (1 << (n - 1)) - 1                                           # pattern of +beta_max
        x = np.full((1, R, S, C), top, np.uint8)
        w = np.full((1, R, S, C), top | (1 << (n - 1)), np.uint8)          # -beta_max
        acc = fpconv_ref.wide_value(x, w, None, (n, p), (n, p), R=R, S=S)
        N = R * S * C
        assert int(acc[0, 0, 0, 0]) == -N * b * b
        q = dynfloat.mac_accumulator_bits(N, b, 0, b, 0)
        assert -(1 << (q - 1)) <= -N * b * b and N * b * b > (1 << (q - 2)) - 1
        assert dynfloat.mac_max_terms(q, b, 0, b, 0) >= N
        # the 8-bit formats the discussion section recommends need far more than the 32 bits of the integer path
        assert q > 32 if (n, p) == (8, 3) else q > 31
        out = fpconv_ref.qconv_np(x, w, None, np.array([3]), (n, p), (n, p), (n, p), R=R, S=S)
        assert int(out[0, 0, 0, 0]) == (top | (1 << (n - 1)))              # saturates to -beta_max

"""Pins for the data-type part of the oracle (Section 2.1, Eq. 2-5; Eq. 8-9, 12-13)."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import dynfloat as df

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [tuple(int(t) for t in ln.split()) for ln in f if ln.strip() and not ln.startswith("#")]


def test_beta_max_closed_form_matches_hand_evaluated_table():
    for n, p, bmax in _rows("beta_max_eq5.txt"):
        assert df.beta_max_closed_form(n, p) == bmax


@pytest.mark.parametrize("n", range(2, 9))
def test_beta_max_closed_form_equals_enumerated_maximum(n):
    # Eq. 5 says equality holds when every pattern (Inf/NaN included) is a number.
    for p in range(0, n):
        vals = df.value_set(n, p)
        assert max(vals) == df.beta_max_closed_form(n, p), (n, p)
        assert min(vals) == -df.beta_max_closed_form(n, p), (n, p)      # strictly symmetric


def test_p6_and_p7_are_int8_symmetric_integers():
    # Discussion: "p = 6, a.k.a. int8"; one exponent bit is dynamic fixed point by definition.
    want = set(Fraction(v) for v in range(-127, 128))
    assert set(df.value_set(8, 7)) == want
    assert set(df.value_set(8, 6)) == want
    # the (8,7) pattern is plain sign-magnitude
    for b in range(256):
        m = b & 0x7F
        assert df.decode_sign_magnitude(b, 8, 7) == (-m if b & 0x80 else m)


def test_p2_is_truncated_half_precision():
    # Discussion: "p = 2, a.k.a. truncated half-precision": the byte is the top half of a
    # binary16 word (1 sign, 5 exponent, 2 of 10 fraction bits); beta * 2^-16 is its value.
    # numpy's float16 decoding is the independent routine; exponent field 31 is Inf/NaN in
    # IEEE but a number here, so it is checked against the extended formula only.
    for b in range(256):
        e_hat = df.exponent_field(b, 8, 2)
        beta = df.decode_sign_magnitude(b, 8, 2)
        if e_hat == 31:
            assert abs(beta) >= Fraction(2) ** 30 * 4
            continue
        half = np.array([b << 8], dtype=np.uint16).view(np.float16)[0]
        assert Fraction(float(half)) == beta * Fraction(1, 2 ** 16), b


def test_subnormals_and_normals_meet_without_gap():
    # Eq. 2: the largest subnormal is 2^p - 1 and the smallest normal is 2^p.
    for n, p in [(8, 4), (8, 3), (7, 4), (6, 3)]:
        pos = sorted(set(v for v in df.value_set(n, p) if v >= 0))
        assert pos[: (1 << (p + 1))] == [Fraction(i) for i in range(1 << (p + 1))]
        # spacing doubles with each exponent step
        for e_hat in range(1, (1 << (n - p - 1))):
            lo = Fraction(2) ** (e_hat - 1) * (1 << p)
            assert lo in pos and lo + Fraction(2) ** (e_hat - 1) in pos


def test_eq3_as_printed_is_not_twos_complement():
    # The printed Eq. 3 subtracts 2^p + 2^(p+1) for the sign bit; for n = 8 it cannot
    # represent -1, which is why the build stores Eq. 2's value set in ordinary bytes.
    for p, lo in [(7, -384), (6, -192)]:
        vals = [df.decode_twos_complement_as_printed(b, 8, p) for b in range(256)]
        assert min(vals) == lo and max(vals) == 127
        assert Fraction(-1) not in vals


def test_accumulator_bounds_eq9_table():
    for q, bx, ex, by, ey, N in _rows("accumulator_eq9.txt"):
        assert df.mac_max_terms(q, bx, ex, by, ey) == N


@pytest.mark.parametrize("bx,ex,by,ey", [(127, 0, 127, 0), (127, 1, 127, 1), (127, 1, 127, 0),
                                         (7, 0, 127, 0), (1, 0, 1, 0), (3, 2, 5, 0)])
def test_eq8_eq9_against_the_range_condition(bx, ex, by, ey):
    # Definition (text before Eq. 8): lossless iff -2^(q-1) <= N a_y b_x (taking the more
    # negative cross product) and N a_x a_y <= 2^(q-1) - 1.
    ax, ay = -bx - ex, -by - ey

    def fits(N, q):
        lo = N * min(ay * bx, ax * by)
        hi = N * max(ax * ay, bx * by)
        return -(1 << (q - 1)) <= lo and hi <= (1 << (q - 1)) - 1

    for q in range(12, 40):
        N = df.mac_max_terms(q, bx, ex, by, ey)
        if N >= 1:
            assert fits(N, q)
        assert not fits(N + 1, q)
    for N in [1, 2, 27, 144, 147, 2048, 4608, 131071, 133144, 133145]:
        q = df.mac_accumulator_bits(N, bx, ex, by, ey)
        assert fits(N, q) and not fits(N, q - 1)


def test_conv_configs_fit_int32():
    # K_gemm = 4608 (3x3x512) needs 28 bits; every configured layer is far below N_max(32).
    assert df.mac_accumulator_bits(4608, 127, 0, 127, 0) == 28
    assert df.mac_accumulator_bits(4608, 127, 1, 127, 1) == 28
    assert df.mac_max_terms(32, 127, 1, 127, 1) == 131071 > 4608


@pytest.mark.parametrize("bx,ex", [(127, 0), (127, 1), (1, 0), (5, 3)])
def test_eq12_eq13_against_the_range_condition(bx, ex):
    ax = -bx - ex

    def fits(N, q):
        return -(1 << (q - 1)) <= N * ax and N * bx <= (1 << (q - 1)) - 1

    for q in range(9, 34):
        N = df.add_max_terms(q, bx, ex)
        if N >= 1:
            assert fits(N, q)
        assert not fits(N + 1, q)
    for N in [1, 2, 3, 64, 1000, 16909320]:
        q = df.add_accumulator_bits(N, bx, ex)
        assert fits(N, q) and not fits(N, q - 1)


# ---------------------------------------------------------------------------------- float <-> (n, p) codes
def _brute_force_code(x, e, n, p):
    """Nearest representable value in exact rationals; ties to the even pattern; saturating."""
    if x != x:
        return 0
    vals = [df.decode_sign_magnitude(b, n, p) for b in range(1 << (n - 1))]
    a = vals[-1] + 1 if np.isinf(x) else abs(Fraction(float(x))) / Fraction(2) ** e
    best = min(range(len(vals)), key=lambda b: (abs(vals[b] - a), b % 2))
    if best == 0:
        return 0
    return best | ((1 << (n - 1)) if x < 0 else 0)


@pytest.mark.parametrize("n,p,e", [(8, 7, -3), (8, 6, 0), (8, 4, -6), (8, 3, -9), (8, 2, -16), (8, 0, -20), (6, 3, 2),
                                   (5, 4, -1), (4, 1, 0), (2, 1, 0), (3, 0, -2)])
def test_quantize_np_against_exact_brute_force(n, p, e):
    rng = np.random.default_rng(n * 10 + p)
    top = float(df.beta_max_closed_form(n, p)) * 2.0 ** e
    x = np.concatenate([rng.normal(size=300) * top / 3, rng.uniform(-1.2, 1.2, 200) * top,
                        [0.0, -0.0, top, -top, top * 4, np.inf, -np.inf, np.nan, 2.0 ** e / 2, -(2.0 ** e) / 2,
                         1.5 * 2.0 ** e, 2.5 * 2.0 ** e]]).astype(np.float32)
    # every midpoint between neighbours (the ties) and one float either side of it
    vals = df.nonneg_values_f64(n, p) * 2.0 ** e
    mids = ((vals[:-1] + vals[1:]) / 2).astype(np.float32)
    x = np.concatenate([x, mids, -mids, np.nextafter(mids, np.float32(0)), np.nextafter(mids, np.float32(np.inf))])
    got = df.quantize_np(x, e, n, p)
    want = np.array([_brute_force_code(v, e, n, p) for v in x], dtype=np.uint8)
    assert np.array_equal(got, want)


def test_quantize_np_matches_torch_float8_types_on_their_finite_range():
    import torch
    rng = np.random.default_rng(0)
    for (p, e, dt, lim) in ((2, -16, torch.float8_e5m2, 57000.0), (3, -9, torch.float8_e4m3fn, 440.0)):
        x = np.concatenate([rng.normal(size=20000) * lim / 4, rng.uniform(-lim, lim, 20000),
                            rng.normal(size=5000) * 2.0 ** (e + 2)]).astype(np.float32)
        x = x[np.abs(x) <= lim]
        bits = torch.from_numpy(x).to(dt).view(torch.uint8).numpy()
        got = df.quantize_np(x, e, 8, p)
        # the IEEE-style types keep a signed zero; the paper's type has one zero
        bits = np.where((bits & 0x7F) == 0, 0, bits)
        assert np.array_equal(got, bits), (p, e)


@pytest.mark.parametrize("n,p", [(8, 7), (8, 4), (8, 3), (8, 2), (6, 2), (4, 3), (3, 1)])
def test_codes_round_trip(n, p):
    codes = np.arange(1 << n, dtype=np.uint8)
    e = -5
    v = df.dequantize_np(codes, e, n, p)
    want = np.array([float(df.decode_sign_magnitude(int(c), n, p)) * 2.0 ** e for c in codes], dtype=np.float32)
    assert np.array_equal(v, want)
    back = df.quantize_np(v, e, n, p)
    keep = (codes & ((1 << (n - 1)) - 1)) != 0                   # negative zero folds into code 0
    assert np.array_equal(back[keep], codes[keep]) and np.all(back[~keep] == 0)

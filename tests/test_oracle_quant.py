"""Pins for conversion, scale selection and calibration statistics (Section 3,
relation gamma = alpha * beta_max before Eq. 5, first step of Algorithm 1)."""
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import ref


def test_scale_exponent_brute_force():
    # e = min { e : beta_max * 2^e >= gamma }, checked with exact rationals around every
    # boundary gamma = beta_max * 2^e, one float ulp either side.
    for n in [2, 4, 7, 8]:
        bmax = 2 ** (n - 1) - 1
        for e in range(-24, 25):
            g0 = np.float32(bmax * 2.0 ** e)
            for g in [g0, np.nextafter(g0, np.float32(0)), np.nextafter(g0, np.float32(np.inf)),
                      np.float32(g0 * 0.75), np.float32(g0 * 1.5)]:
                got = ref.scale_exponent(float(g), n)
                assert Fraction(bmax) * Fraction(2) ** got >= Fraction(float(g))
                assert Fraction(bmax) * Fraction(2) ** (got - 1) < Fraction(float(g))
    assert ref.scale_exponent(127.0, 8) == 0 and ref.scale_exponent(127.00001, 8) == 1
    assert ref.scale_exponent(1.0, 8) == -6 and ref.scale_exponent(0.0, 8) == 0
    assert ref.scale_exponent(float("inf"), 8) == 0 and ref.scale_exponent(float("nan"), 8) == 0


def test_quantize_matches_exact_definition():
    rng = np.random.default_rng(1)
    x = (rng.standard_normal(4000) * 3).astype(np.float32)
    x[:8] = [0.0, -0.0, 1e-30, -1e30, np.inf, -np.inf, np.nan, 2.5]
    for n, e in [(8, -5), (8, -3), (8, 2), (4, -1), (6, -4)]:
        bmax = 2 ** (n - 1) - 1
        got = ref.quantize_f32(x, e, n)
        for v, g in zip(x[:600], got[:600]):
            if math.isnan(v):
                want = 0
            elif math.isinf(v):
                want = bmax if v > 0 else -bmax
            else:
                want = max(-bmax, min(bmax, round(Fraction(float(v)) / Fraction(2) ** e)))
            assert int(g) == want, (v, e, n)
        assert got.min() >= -bmax and got.max() <= bmax
    # ties go to even: 2.5 / 2^0 -> 2, 3.5 -> 4, -2.5 -> -2
    assert list(ref.quantize_f32(np.array([2.5, 3.5, -2.5, 0.5, 1.5], np.float32), 0, 8)) == [2, 4, -2, 0, 2]
    # clamp-then-round equals round-then-clamp
    big = np.array([126.4, 126.5, 127.49, 127.5, 500.0, -127.5, -900.0], np.float32)
    assert list(ref.quantize_f32(big, 0, 8)) == [126, 126, 127, 127, 127, -127, -127]


def test_weight_and_bias_quantization():
    rng = np.random.default_rng(2)
    K, R, S, Cg = 5, 3, 2, 4
    w = (rng.standard_normal((K, R, S, Cg)) * np.array([0.01, 0.1, 1, 10, 0])[:, None, None, None]).astype(np.float32)
    wq, e_w = ref.quantize_weights(w, K=K, R=R, S=S, Cg=Cg, per_channel=1)
    for k in range(K):
        g = float(np.abs(w[k]).max())
        assert e_w[k] == ref.scale_exponent(g)
        if g > 0:
            assert 64 <= np.abs(wq[k]).max() <= 127             # the channel uses its top bit
            assert np.abs(wq[k].astype(np.float64) * 2.0 ** e_w[k] - w[k]).max() <= 2.0 ** e_w[k] / 2
    assert (wq[4] == 0).all() and e_w[4] == 0
    wq1, e1 = ref.quantize_weights(w, K=K, R=R, S=S, Cg=Cg, per_channel=0)
    assert (e1 == ref.scale_exponent(float(np.abs(w).max()))).all()
    # layout 1 is the transpose
    wt = np.ascontiguousarray(w.transpose(1, 2, 3, 0))
    wq2, e2 = ref.quantize_weights(wt, K=K, R=R, S=S, Cg=Cg, layout=1, per_channel=1)
    assert (e2 == e_w).all() and (wq2 == wq.transpose(1, 2, 3, 0)).all()
    b = np.array([0.0, 0.3, -0.3, 1e9, -1e9], np.float32)
    bq = ref.quantize_bias(b, -4, e_w)
    for k in range(K):
        want = round(Fraction(float(b[k])) / Fraction(2) ** (-4 + int(e_w[k])))
        assert bq[k] == max(-2**31, min(2**31 - 1, want))


def test_histogram_on_dyadic_data_equals_numpy_histogram():
    # hi a power of two and data on a grid of hi/8192: every fp32 step is exact, so the
    # result must equal numpy's histogram of |x| bit for bit.
    rng = np.random.default_rng(4)
    hi = 4.0
    x = (rng.integers(-8192, 8193, size=50000).astype(np.float32) * np.float32(hi / 8192))
    x[0] = hi                                              # the maximum itself lands in the last bin
    st = ref.calib_stats(x, 2048)
    assert st["maxabs"] == np.float32(hi)
    want, _ = np.histogram(np.abs(x), bins=2048, range=(0.0, hi))
    assert (st["hist"] == want.astype(np.uint64)).all()
    assert st["hist"].sum() == st["count"] == x.size and st["nonfinite"] == 0
    # explicit range below the maximum: the overflow collects in the last bin
    st2 = ref.calib_stats(x, 64, 2.0)
    want2, _ = np.histogram(np.minimum(np.abs(x), np.float32(1.999)), bins=64, range=(0.0, 2.0))
    assert (st2["hist"] == want2.astype(np.uint64)).all()


def test_stats_sums_and_nonfinite():
    rng = np.random.default_rng(6)
    x = rng.standard_normal(30000).astype(np.float32) * 5
    x[[5, 77, 900]] = [np.nan, np.inf, -np.inf]
    st = ref.calib_stats(x, 2048)
    fin = x[np.isfinite(x)]
    assert st["nonfinite"] == 3 and st["count"] == fin.size
    assert st["maxabs"] == np.abs(fin).max()
    assert st["hist"].sum() == fin.size
    s, ss = math.fsum(float(v) for v in fin), math.fsum(float(v) * float(v) for v in fin)
    assert abs(st["sum"] - s) <= 1e-6 * max(1.0, abs(s)) and abs(st["sumsq"] - ss) <= 1e-6 * ss
    # bin index definition: one fp32 multiply, truncated
    inv_w = np.float32(2048) / st["maxabs"]
    bins = np.minimum((np.abs(fin) * inv_w).astype(np.int64), 2047)
    assert (st["hist"] == np.bincount(bins, minlength=2048).astype(np.uint64)).all()
    z = ref.calib_stats(np.zeros(10, np.float32), 16)
    assert z["maxabs"] == 0 and z["hist"][0] == 10 and z["hist"].sum() == 10


def test_packed_bit_fields_of_the_oracle():
    """n-bit two's-complement fields, little-endian bit order.  Hand-worked: the 5-bit values 1, -1, 2 are the
    fields 00001, 11111, 00010; laid out from bit 0 upwards they read 0b11100001, 0b00001011."""
    assert ref.pack_bits([1, -1, 2], 5).tolist() == [0b11100001, 0b00001011]
    assert ref.pack_bits([-4, 3], 3).tolist() == [0b00011100]
    for n in range(2, 9):
        vals = np.arange(-(1 << (n - 1)), 1 << (n - 1))
        vals = np.concatenate([vals, vals[::-1], vals[::3]])
        packed = ref.pack_bits(vals, n)
        assert packed.size == (vals.size * n + 7) // 8
        assert (ref.unpack_bits(packed, vals.size, n) == vals).all()
    assert (ref.pack_bits(np.arange(-128, 128), 8) == np.arange(-128, 128).astype(np.int8).view(np.uint8)).all()

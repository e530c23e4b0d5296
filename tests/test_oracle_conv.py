"""Pins for the convolution / requantization part of the oracle (Eq. 6, Eq. 10,
Section 3): every check compares against something other than the oracle's own
formula -- exact rationals, an independent im2col product, a float64 library
convolution, or an invariant the scheme fixes."""
import decimal
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import ref
from paper_1805_07941_b200 import workloads as wl


# ----------------------------------------------------------------- rounding
def _exact_round(acc, s, mode):
    v = Fraction(acc, 2 ** s)
    if mode == 0:
        return round(v)                       # Python rounds exact rationals half-to-even
    d = decimal.Decimal(v.numerator) / decimal.Decimal(v.denominator)   # exact: denominator 2^s
    rule = {1: decimal.ROUND_HALF_UP, 3: decimal.ROUND_FLOOR}.get(mode)
    if mode == 2:                             # ties toward +infinity
        return int((d + decimal.Decimal("0.5")).to_integral_value(rounding=decimal.ROUND_FLOOR))
    return int(d.to_integral_value(rounding=rule))   # decimal's HALF_UP is half-away-from-zero


@pytest.mark.parametrize("mode", [0, 1, 2, 3])
def test_round_shift_matches_exact_rationals(mode):
    decimal.getcontext().prec = 60
    rng = np.random.default_rng(7)
    accs = list(range(-70, 71)) + [int(v) for v in rng.integers(-2**31, 2**31, size=300)]
    accs += [2**31 - 1, -2**31, 2**40 + 1, -(2**40) - 1]
    for s in [0, 1, 2, 3, 5, 7, 12, 20, 31]:
        for acc in accs:
            assert ref.round_shift(acc, s, mode) == _exact_round(acc, s, mode), (acc, s, mode)


@pytest.mark.parametrize("mode", [0, 1, 2, 3])
def test_round_shift_ties(mode):
    # acc = (2m+1) * 2^(s-1) sits exactly between m and m+1.
    for s in [1, 4, 7, 15]:
        for m in range(-6, 7):
            acc = (2 * m + 1) << (s - 1)
            want = {0: m if m % 2 == 0 else m + 1, 1: m + 1 if acc > 0 else m, 2: m + 1, 3: m}[mode]
            assert ref.round_shift(acc, s, mode) == want


def test_round_shift_zero_is_identity_and_float64_rint_agrees():
    rng = np.random.default_rng(3)
    acc = rng.integers(-2**31, 2**31, size=2000)
    for a in acc[:200]:
        for mode in range(4):
            assert ref.round_shift(int(a), 0, mode) == int(a)
    for s in [1, 6, 7, 13]:
        want = np.rint(acc.astype(np.float64) / 2.0 ** s).astype(np.int64)   # exact below 2^53
        got = np.array([ref.round_shift(int(a), s, 0) for a in acc])
        assert (got == want).all()


# ----------------------------------------------------------------- contraction
def _im2col_conv(x, w_krsc, bias, stride, pad, groups):
    """Independent statement: gather patches into a matrix, int64 matrix product."""
    N, H, W, C = x.shape
    K, R, S, Cg = w_krsc.shape
    P, Q = ref.out_hw(H, W, R, S, stride[0], stride[1], pad[0], pad[1])
    xp = np.zeros((N, H + 2 * pad[0], W + 2 * pad[1], C), dtype=np.int64)
    xp[:, pad[0]:pad[0] + H, pad[1]:pad[1] + W, :] = x
    out = np.zeros((N, P, Q, K), dtype=np.int64)
    Kg = K // groups
    for g in range(groups):
        cols = np.zeros((N, P, Q, R, S, Cg), dtype=np.int64)
        for r in range(R):
            for s in range(S):
                cols[:, :, :, r, s, :] = xp[:, r:r + stride[0] * P:stride[0], s:s + stride[1] * Q:stride[1],
                                            g * Cg:(g + 1) * Cg]
        A = cols.reshape(N * P * Q, R * S * Cg)
        B = w_krsc[g * Kg:(g + 1) * Kg].reshape(Kg, R * S * Cg).astype(np.int64)
        out[..., g * Kg:(g + 1) * Kg] = (A @ B.T).reshape(N, P, Q, Kg)
    if bias is not None:
        out += bias.astype(np.int64)
    return out


CASES = [
    # N  H   W   C   K  R  S  stride  pad     groups
    (1, 5, 5, 4, 3, 3, 3, (1, 1), (1, 1), 1),
    (2, 9, 7, 6, 10, 3, 2, (2, 1), (1, 0), 2),
    (1, 8, 11, 5, 7, 1, 1, (1, 1), (0, 0), 1),
    (2, 10, 6, 8, 8, 3, 3, (2, 2), (1, 1), 8),      # depthwise
    (1, 12, 9, 3, 5, 7, 7, (2, 2), (3, 3), 1),
    (1, 6, 13, 4, 6, 5, 3, (1, 2), (2, 1), 2),
    (3, 4, 4, 16, 4, 1, 1, (2, 2), (0, 0), 1),
]


@pytest.mark.parametrize("case", CASES)
def test_conv_raw_accumulator_vs_im2col_and_float64_library(case):
    N, H, W, C, K, R, S, stride, pad, groups = case
    rng = np.random.default_rng(hash(case) % 2**32)
    x = rng.integers(-128, 128, size=(N, H, W, C), dtype=np.int8)
    w = rng.integers(-128, 128, size=(K, R, S, C // groups), dtype=np.int8)
    bias = rng.integers(-5000, 5000, size=(K,), dtype=np.int32)
    got = ref.qconv(x, w, bias, None, R=R, S=S, stride=stride, pad=pad, groups=groups, out_mode=1)
    want = _im2col_conv(x, w, bias, stride, pad, groups)
    assert (got.astype(np.int64) == want).all()
    # float64 library convolution: exact while |acc| < 2^53
    tx = torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2)
    tw = torch.from_numpy(w.astype(np.float64)).permute(0, 3, 1, 2)
    ty = torch.nn.functional.conv2d(tx, tw, torch.from_numpy(bias.astype(np.float64)), stride=stride,
                                    padding=pad, groups=groups).permute(0, 2, 3, 1).numpy()
    assert (got.astype(np.float64) == ty).all()


def test_weight_layouts_agree():
    rng = np.random.default_rng(11)
    x = rng.integers(-128, 128, size=(1, 6, 7, 4), dtype=np.int8)
    w = rng.integers(-128, 128, size=(6, 3, 2, 4), dtype=np.int8)          # KRSC
    a = ref.qconv(x, w, R=3, S=2, pad=(1, 1), out_mode=1, weight_layout=0)
    b = ref.qconv(x, np.ascontiguousarray(w.transpose(1, 2, 3, 0)), R=3, S=2, pad=(1, 1), out_mode=1,
                  weight_layout=1, K=6)
    assert (a == b).all()


def test_shift_zero_is_identity_and_outputs_stay_in_bounds():
    rng = np.random.default_rng(5)
    x = rng.integers(-3, 4, size=(1, 6, 6, 4), dtype=np.int8)
    w = rng.integers(-3, 4, size=(5, 3, 3, 4), dtype=np.int8)
    raw = ref.qconv(x, w, R=3, S=3, pad=(1, 1), out_mode=1)
    assert np.abs(raw).max() <= 127                 # small enough that nothing saturates
    y = ref.qconv(x, w, None, np.zeros(5, np.int32), R=3, S=3, pad=(1, 1), out_mode=0)
    assert (y.astype(np.int32) == raw).all()
    # large values: every output inside the symmetric bound, for every n_out and mode
    x = rng.integers(-128, 128, size=(1, 6, 6, 8), dtype=np.int8)
    w = rng.integers(-128, 128, size=(5, 3, 3, 8), dtype=np.int8)
    for n_out in [2, 4, 7, 8]:
        for mode in range(4):
            for sym in [0, 1]:
                y = ref.qconv(x, w, None, np.full(5, 3, np.int32), R=3, S=3, pad=(1, 1), n_out=n_out,
                              symmetric=sym, rounding=mode)
                hi = 2 ** (n_out - 1) - 1
                lo = -hi if sym else -hi - 1
                assert y.min() >= lo and y.max() <= hi
                if n_out == 8 and mode == 0:
                    assert y.min() == lo and y.max() == hi      # the clamp really was reached


def test_equals_float_convolution_when_everything_is_representable():
    # Values alpha * beta with power-of-two alpha; if the exact result is itself representable
    # at the output scale, quantized conv followed by beta -> float equals the float conv.
    rng = np.random.default_rng(9)
    e_x, e_w, e_z = -3, -4, -5
    bx = rng.integers(-4, 5, size=(1, 5, 5, 3), dtype=np.int8)
    bw = rng.integers(-3, 4, size=(4, 3, 3, 3), dtype=np.int8)
    bw[:, :, :, :] = (bw // 2) * 2                                  # even weights ...
    bx[:, :, :, :] = (bx // 2) * 2                                  # ... and inputs: acc % 4 == 0
    shift = np.full(4, e_z - e_x - e_w, np.int32)                   # = 2
    y = ref.qconv(bx, bw, None, shift, R=3, S=3, pad=(1, 1))
    assert np.abs(y).max() < 127
    xf = torch.from_numpy(bx.astype(np.float64) * 2.0 ** e_x).permute(0, 3, 1, 2)
    wf = torch.from_numpy(bw.astype(np.float64) * 2.0 ** e_w).permute(0, 3, 1, 2)
    zf = torch.nn.functional.conv2d(xf, wf, padding=1).permute(0, 2, 3, 1).numpy()
    assert (y.astype(np.float64) * 2.0 ** e_z == zf).all()


def test_bias_residual_relu_round_clamp_order():
    rng = np.random.default_rng(13)
    N, H, W, C, K = 2, 5, 6, 8, 6
    x = rng.integers(-128, 128, size=(N, H, W, C), dtype=np.int8)
    w = rng.integers(-128, 128, size=(K, 3, 3, C), dtype=np.int8)
    bias = rng.integers(-2**15, 2**15, size=(K,), dtype=np.int32)
    res = rng.integers(-128, 128, size=(N, H, W, K), dtype=np.int8)
    t = rng.integers(0, 9, size=(K,), dtype=np.int32)
    s = rng.integers(0, 12, size=(K,), dtype=np.int32)
    raw = _im2col_conv(x, w, bias, (1, 1), (1, 1), 1) + res.astype(np.int64) * (2 ** t.astype(np.int64))
    for relu in [0, 1]:
        wide = np.maximum(raw, 0) if relu else raw
        assert (ref.qconv(x, w, bias, s, res, t, R=3, S=3, pad=(1, 1), relu=relu, out_mode=1) == wide).all()
        for mode in range(4):
            want = np.empty_like(wide)
            for k in range(K):
                want[..., k] = [[[_exact_round(int(v), int(s[k]), mode) for v in row] for row in img]
                                for img in wide[..., k]]
            want = np.clip(want, -127, 127)
            got = ref.qconv(x, w, bias, s, res, t, R=3, S=3, pad=(1, 1), relu=relu, rounding=mode)
            assert (got == want).all()
            if relu:
                # ReLU before or after the monotone round+clamp gives the same codes.
                late = np.maximum(ref.qconv(x, w, bias, s, res, t, R=3, S=3, pad=(1, 1), relu=0,
                                            rounding=mode), 0)
                assert (got == late).all()


def test_float_out_is_wide_value_times_scale():
    rng = np.random.default_rng(17)
    x = rng.integers(-128, 128, size=(1, 4, 4, 16), dtype=np.int8)
    w = rng.integers(-128, 128, size=(3, 3, 3, 16), dtype=np.int8)
    acc_exp = np.array([-9, -12, 3], np.int32)
    raw = ref.qconv(x, w, R=3, S=3, pad=(1, 1), out_mode=1)
    f = ref.qconv(x, w, None, None, None, None, acc_exp, R=3, S=3, pad=(1, 1), out_mode=2)
    want = raw.astype(np.float32) * (2.0 ** acc_exp.astype(np.float64)).astype(np.float32)
    assert (f == want).all()
    # above 2^24 the int -> float conversion rounds to nearest even
    big = np.full((1, 1, 1, 2048), 127, np.int8)
    wb = np.full((1, 1, 1, 2048), 127, np.int8)
    wb[0, 0, 0, 0] = 126
    rawb = int(ref.qconv(big, wb, R=1, S=1, out_mode=1)[0, 0, 0, 0])
    assert rawb == 2047 * 16129 + 127 * 126 and rawb > 2 ** 24 and rawb % 2 == 1
    fb = ref.qconv(big, wb, None, None, None, None, np.zeros(1, np.int32), R=1, S=1, out_mode=2)
    assert float(fb[0, 0, 0, 0]) == float(np.float32(rawb))


def test_concat_offset_pitch_and_points():
    rng = np.random.default_rng(19)
    x = rng.integers(-128, 128, size=(2, 5, 4, 8), dtype=np.int8)
    w1 = rng.integers(-128, 128, size=(3, 1, 1, 8), dtype=np.int8)
    w2 = rng.integers(-128, 128, size=(5, 3, 3, 8), dtype=np.int8)
    s1, s2 = np.full(3, 6, np.int32), np.full(5, 9, np.int32)
    buf = np.full((2, 5, 4, 10), 77, np.int8)
    ref.qconv(x, w1, None, s1, R=1, S=1, out=buf, out_c_offset=0)
    ref.qconv(x, w2, None, s2, R=3, S=3, pad=(1, 1), out=buf, out_c_offset=3)
    assert (buf[..., :3] == ref.qconv(x, w1, None, s1, R=1, S=1)).all()
    assert (buf[..., 3:8] == ref.qconv(x, w2, None, s2, R=3, S=3, pad=(1, 1))).all()
    assert (buf[..., 8:] == 77).all()
    full = ref.qconv(x, w2, None, s2, R=3, S=3, pad=(1, 1))
    pts = np.array([[n, p, q, k] for n in range(2) for p in range(5) for q in range(4) for k in range(5)],
                   np.int32)
    got = ref.qconv_points(x, w2, pts, None, s2, R=3, S=3, pad=(1, 1))
    assert (got == full.reshape(-1)).all()


def test_extreme_inputs_at_longest_configured_dot_product():
    # K_gemm = 3*3*512 = 4608 with every product at its extreme: 4608 * 128 * 128 < 2^31 (Eq. 9).
    for xv, wv in [(-128, -128), (127, -128), (-128, 127)]:
        x = np.full((1, 3, 3, 512), xv, np.int8)
        w = np.full((1, 3, 3, 512), wv, np.int8)
        raw = ref.qconv(x, w, R=3, S=3, pad=(1, 1), out_mode=1)
        assert int(raw[0, 1, 1, 0]) == 4608 * xv * wv            # centre pixel sees all 9 taps
        assert int(raw[0, 0, 0, 0]) == 4 * 512 * xv * wv         # corner sees 4


def test_single_conv_config_statistics():
    c = wl.single_conv_cfg()
    y = ref.qconv(c["x"], c["w"], c["bias"], c["shift"], R=3, S=3, stride=c["stride"], pad=c["pad"],
                  relu=1, weight_layout=1, K=16)
    assert y.shape == (1, 32, 32, 16) and y.min() == 0 and y.max() == 127
    raw = ref.qconv(c["x"], c["w"], c["bias"], None, R=3, S=3, pad=c["pad"], out_mode=1, weight_layout=1,
                    K=16)
    want = np.clip(np.rint(np.maximum(raw, 0).astype(np.float64) / 128.0), 0, 127)
    assert (y == want).all()


def test_maxpool_vs_library():
    rng = np.random.default_rng(23)
    for (H, W, R, stride, pad) in [(8, 8, 2, 2, 0), (9, 7, 3, 2, 1), (6, 6, 3, 1, 1), (7, 10, 3, 2, 0)]:
        x = rng.integers(-128, 128, size=(2, H, W, 5), dtype=np.int8)
        y = ref.maxpool_i8(x, R, R, stride, pad)
        t = torch.from_numpy(x.astype(np.float32)).permute(0, 3, 1, 2)
        ty = torch.nn.functional.max_pool2d(t, R, stride, pad).permute(0, 2, 3, 1).numpy()
        assert (y.astype(np.float32) == ty).all()


def test_eltwise_add_against_exact_rationals_and_float_addition():
    # Eq. 10: z = sum_i x_i with x_i = 2^e_i * beta_i, output at scale 2^e_z >= every 2^e_i.
    rng = np.random.default_rng(29)
    e = [-6, -4, -5]
    e_min, e_z = min(e), -3
    xs = [rng.integers(-128, 128, size=500, dtype=np.int8) for _ in e]
    lshift = [ei - e_min for ei in e]
    for mode in range(4):
        for relu in (0, 1):
            got = ref.eltwise_add(xs, lshift, e_z - e_min, relu=relu, rounding=mode)
            for j in range(500):
                wide = sum(int(x[j]) << l for x, l in zip(xs, lshift))
                if relu:
                    wide = max(wide, 0)
                want = max(-127, min(127, _exact_round(wide, e_z - e_min, mode)))
                assert int(got[j]) == want
    # when the exact sum is representable at the output scale, it equals the float sum
    xs2 = [(x // 8) * 8 for x in xs]                    # multiples of 8 at every input scale
    got = ref.eltwise_add(xs2, lshift, e_z - e_min)
    fsum = sum(x.astype(np.float64) * 2.0 ** ei for x, ei in zip(xs2, e))
    inside = np.abs(fsum) <= 127 * 2.0 ** e_z
    assert inside.any() and (got[inside].astype(np.float64) * 2.0 ** e_z == fsum[inside]).all()
    assert (np.abs(got[~inside]) == 127).all()          # outside the range it saturates symmetrically
    # a single input with no shift is the identity (up to the symmetric clamp)
    one = ref.eltwise_add([xs[0]], [0], 0)
    assert (one == np.maximum(xs[0], -127)).all()

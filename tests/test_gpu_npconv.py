"""GPU parity of the convolution on dynamic floating-point operands (qconv_np_*) against
oracle/fpconv_ref.py: every output pattern must be identical.  Formats: the 8-bit types the paper's
discussion recommends, (8, 4) and (8, 3), the integer type (8, 7) as the degenerate case, narrower
types, and mixed input / weight / output types; flat, box and halo forms of the inner GEMM, strides,
ragged sizes; exact ties of the conversion driven through the bias."""
import numpy as np
import pytest

from oracle import fpconv_ref
from paper_1805_07941_b200 import binding

pytestmark = pytest.mark.gpu


def _codes(rng, shape, n, p, spread=1.0):
    """Random patterns, magnitudes drawn so that large exponents are rarer (activation-like)."""
    top = (1 << (n - 1)) - 1
    mag = np.minimum(np.abs(rng.standard_normal(shape)) * spread * top / 3.0, top).astype(np.uint8)
    sign = (rng.integers(0, 2, size=shape).astype(np.uint8) << (n - 1)) * (mag != 0)
    return (mag | sign).astype(np.uint8)


def _run(x, w, bias, shift, fi, fw, fo, **kw):
    import torch
    N, H, W, C = x.shape
    K, R, S, _ = w.shape
    st, pad = kw.get("stride", (1, 1)), kw.get("pad", (0, 0))
    conv = binding.QConvNP(w, bias, shift, N=N, H=H, W=W, C=C, K=K, R=R, S=S, stride_h=st[0], stride_w=st[1],
                           pad_h=pad[0], pad_w=pad[1], n_in=fi[0], p_in=fi[1], n_w=fw[0], p_w=fw[1],
                           n_out=fo[0], p_out=fo[1], relu=kw.get("relu", 0))
    y = torch.full((N, conv.P, conv.Q, K), 0x55, dtype=torch.uint8, device="cuda")
    conv.run(torch.from_numpy(x).cuda(), y)
    assert conv.status() == 0, conv.describe()
    desc = conv.describe()
    conv.destroy()
    return y.cpu().numpy(), desc


CASES = [
    # N, H, W, C, K, R, stride, pad
    (2, 9, 11, 32, 48, 1, (1, 1), (0, 0)),          # flat
    (3, 14, 14, 64, 40, 3, (1, 1), (1, 1)),         # box, K not a multiple of 16
    (2, 14, 14, 128, 64, 3, (1, 1), (1, 1)),        # halo form of the inner GEMM
    (1, 17, 13, 16, 24, 5, (1, 1), (2, 2)),
    (2, 12, 12, 32, 32, 1, (2, 2), (0, 0)),         # strided view
    (1, 15, 15, 16, 16, 3, (2, 2), (1, 1)),         # 3x3 stride 2
    (40, 7, 7, 64, 128, 3, (1, 1), (1, 1)),         # several images per tile, several tiles
]
FMTS = [((8, 4), (8, 4), (8, 4)), ((8, 3), (8, 3), (8, 3)), ((8, 7), (8, 7), (8, 7)), ((8, 4), (8, 3), (8, 5)),
        ((6, 2), (5, 4), (8, 4)), ((8, 3), (8, 7), (7, 3))]


@pytest.mark.parametrize("fmts", FMTS, ids=lambda f: "-".join("%d.%d" % t for t in f))
@pytest.mark.parametrize("case", CASES)
def test_np_convolution_matches_the_oracle(case, fmts):
    N, H, W, C, K, R, stride, pad = case
    fi, fw, fo = fmts
    rng = np.random.default_rng(sum(case[:6]) + 7 * fi[1] + fw[1])
    x = _codes(rng, (N, H, W, C), *fi)
    w = _codes(rng, (K, R, R, C), *fw, spread=0.7)
    bias = rng.integers(-2**20, 2**20, size=K).astype(np.int32)
    # a shift that lands typical sums inside the output range, varied per channel
    acc = fpconv_ref.wide_value(x[:1], w, bias, fi, fw, R=R, S=R, stride=stride, pad=pad)
    scale = max(1.0, float(np.abs(acc).mean()) * 4 / fpconv_ref.magnitudes(*fo)[-1])
    shift = (int(np.log2(scale)) + rng.integers(-2, 3, size=K)).clip(0, 40).astype(np.int32)
    for relu in (0, 1):
        want = fpconv_ref.qconv_np(x, w, bias, shift, fi, fw, fo, R=R, S=R, stride=stride, pad=pad, relu=relu)
        got, desc = _run(x, w, bias, shift, fi, fw, fo, stride=stride, pad=pad, relu=relu)
        bad = np.argwhere(got != want)
        assert bad.size == 0, (desc, bad[:5], got[tuple(bad[0])], want[tuple(bad[0])])
        assert len(np.unique(want)) > 8, "degenerate case: outputs barely vary"


@pytest.mark.parametrize("fo", [(8, 4), (8, 3), (8, 7), (4, 0)])
def test_np_conversion_ties_and_saturation_through_the_kernel(fo):
    """Rows of zero input leave the bias as the wide value: place it on every midpoint between neighbouring
    output values (scaled by 2^s), one unit either side, and beyond the range, both signs."""
    mags = fpconv_ref.magnitudes(*fo)
    for s in (0, 2, 5):
        pts = []
        for a, b in zip(mags[:-1], mags[1:]):
            mid2 = (a + b) << s
            if mid2 % 2 == 0:
                pts += [mid2 // 2 - 1, mid2 // 2, mid2 // 2 + 1]
        pts += [(mags[-1] << s) - 1, mags[-1] << s, (mags[-1] << s) + 5, 2**31 - 1]
        pts = [v for v in pts if v < 2**31]
        vals = np.array(pts + [-v for v in pts], dtype=np.int64)
        K = int(np.ceil(len(vals) / 16) * 16)
        bias = np.zeros(K, np.int32)
        bias[:len(vals)] = vals
        x = np.zeros((1, 4, 4, 16), np.uint8)
        w = np.full((K, 1, 1, 16), 3, np.uint8)
        shift = np.full(K, s, np.int32)
        want = fpconv_ref.qconv_np(x, w, bias, shift, (8, 4), (8, 4), fo, R=1, S=1)
        got, desc = _run(x, w, bias, shift, (8, 4), (8, 4), fo)
        assert (got == want).all(), desc
        assert (fpconv_ref.encode_exact(vals, s, *fo) == want[0, 0, 0, :len(vals)]).all()


def test_np_create_rejects_what_it_cannot_hold():
    w = np.zeros((16, 1, 1, 16), np.uint8)
    base = dict(N=1, H=4, W=4, C=16, K=16, R=1, S=1, n_in=8, p_in=4, n_w=8, p_w=4, n_out=8, p_out=4)
    with pytest.raises(binding.QconvError) as e:
        binding.QConvNP(w, **dict(base, p_in=2))             # (8, 2): beta_max 7 * 2^30 needs five digit planes
    assert e.value.code == binding.ERR_UNSUPPORTED_SHAPE
    with pytest.raises(binding.QconvError) as e:
        binding.QConvNP(w, **dict(base, p_out=8))
    assert e.value.code == binding.ERR_BAD_ARG
    with pytest.raises(binding.QconvError) as e:
        binding.QConvNP(w, None, np.full(16, 41, np.int32), **base)
    assert e.value.code == binding.ERR_BAD_SHIFT
    with pytest.raises(binding.QconvError) as e:
        binding.QConvNP(np.zeros((16, 1, 1, 24), np.uint8), **dict(base, C=24))
    assert e.value.code == binding.ERR_UNSUPPORTED_SHAPE
    # Eq. 9 with b = beta_max of (8, 3): 245760^2 * terms must stay below 2^62
    big = dict(base, C=1 << 20, p_in=3, p_w=3, H=1, W=1)
    with pytest.raises(binding.QconvError) as e:
        binding.QConvNP(np.zeros((16, 1, 1, 1 << 20), np.uint8), **big)
    assert e.value.code in (binding.ERR_OVERFLOW_RISK, binding.ERR_UNSUPPORTED_SHAPE)

"""GPU parity: every kernel, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Integer outputs must be bit-exact; float statistics within 1e-6 relative."""
import numpy as np
import pytest

from oracle import ref
from paper_1805_07941_b200 import binding
from paper_1805_07941_b200 import workloads as wl
from tests.helpers import gpu_conv, oracle_conv, rand_layer

pytestmark = pytest.mark.gpu

ALGO = dict(auto=0, direct=1, igemm=2, dw=3)


def _compare(args, kw, algo, expect_desc=None):
    want = oracle_conv(*args, **kw)
    got, desc = gpu_conv(*args, algo=algo, **kw)
    if expect_desc:
        assert expect_desc in desc, desc
    if kw.get("out_mode", 0) == 2:
        assert (got == want).all(), desc            # float-out is an exact function of the integer
    else:
        bad = np.argwhere(got != want)
        assert bad.size == 0, (desc, bad[:5], got[tuple(bad[0])], want[tuple(bad[0])])
    return got, desc


# ------------------------------------------------------------------ small kernels
def test_quantize_f32():
    import torch
    from paper_1805_07941_b200 import binding
    rng = np.random.default_rng(0)
    for count in (1, 15, 16, 17, 4099, 1 << 20):
        x = (rng.standard_normal(count) * 4).astype(np.float32)
        x[:min(count, 7)] = np.float32([0.5, 1.5, 2.5, -2.5, np.nan, np.inf, -np.inf])[:min(count, 7)]
        for e, n in [(-5, 8), (0, 8), (-3, 4), (2, 6)]:
            y = binding.qquantize_f32(torch.from_numpy(x).cuda(), e, n).cpu().numpy()
            assert (y == ref.quantize_f32(x, e, n)).all()
    x = torch.from_numpy((rng.standard_normal(1001) * 4).astype(np.float32)).cuda()
    y = binding.qquantize_f32(x[1:], -4).cpu().numpy()                      # unaligned pointer
    assert (y == ref.quantize_f32(x[1:].cpu().numpy(), -4)).all()


def test_maxpool():
    import torch
    from paper_1805_07941_b200 import binding
    rng = np.random.default_rng(1)
    for (N, H, W, C, R, stride, pad) in [(2, 8, 8, 16, 2, 2, 0), (1, 9, 7, 32, 3, 2, 1), (2, 6, 6, 48, 3, 1, 1),
                                         (1, 7, 10, 5, 3, 2, 0), (1, 112, 112, 64, 3, 2, 1), (3, 28, 28, 192, 3, 1, 1),
                                         (2, 14, 14, 480, 3, 1, 1), (1, 37, 23, 32, 3, 1, 0), (2, 45, 31, 16, 2, 2, 0),
                                         (1, 33, 35, 64, 3, 2, 0), (1, 5, 5, 16, 3, 1, 2), (2, 19, 19, 32, 5, 1, 2)]:
        x = rng.integers(-128, 128, size=(N, H, W, C), dtype=np.int8)
        y = binding.qmaxpool_i8(torch.from_numpy(x).cuda(), R, R, stride, pad).cpu().numpy()
        assert (y == ref.maxpool_i8(x, R, R, stride, pad)).all()


def test_calibration_statistics():
    import torch
    from paper_1805_07941_b200 import binding
    rng = np.random.default_rng(2)
    for count, relu_like in [(1, False), (1000, False), (1 << 20, True), ((1 << 21) + 3, False)]:
        x = (rng.standard_normal(count) * 3).astype(np.float32)
        if relu_like:
            x = np.maximum(x, 0)
        if count > 100:
            x[[3, 50, 99]] = [np.nan, np.inf, -np.inf]
        for nbins, hi in [(2048, 0.0), (64, 2.0), (4096, 0.0)]:
            got = binding.qcalib_collect(torch.from_numpy(x).cuda(), nbins, hi)
            want = ref.calib_stats(x, nbins, hi)
            assert got["maxabs"] == want["maxabs"]                          # exact
            assert (got["hist"] == want["hist"]).all()                      # exact integer counts
            assert got["count"] == want["count"] and got["nonfinite"] == want["nonfinite"]
            assert abs(got["sum"] - want["sum"]) <= 1e-6 * max(1.0, abs(want["sum"]))
            assert abs(got["sumsq"] - want["sumsq"]) <= 1e-6 * max(1.0, want["sumsq"])
    z = binding.qcalib_collect(torch.zeros(100, device="cuda"), 16)
    assert z["maxabs"] == 0 and z["hist"][0] == 100


# ------------------------------------------------------------------ direct kernel
DIRECT_CASES = [
    (1, 5, 5, 4, 3, 3, 3, (1, 1), (1, 1), 1),
    (2, 9, 7, 6, 10, 3, 2, (2, 1), (1, 0), 2),
    (2, 10, 6, 8, 8, 3, 3, (2, 2), (1, 1), 8),
    (1, 12, 9, 3, 5, 7, 7, (2, 2), (3, 3), 1),
    (1, 6, 13, 4, 6, 5, 3, (1, 2), (2, 1), 2),
    (1, 9, 9, 32, 32, 3, 3, (2, 2), (1, 1), 1),        # strided 3x3: not taken by the tensor-core path
]


@pytest.mark.parametrize("case", DIRECT_CASES)
def test_direct_conv(case):
    N, H, W, C, K, R, S, stride, pad, groups = case
    rng = np.random.default_rng(sum(case[:7]))
    x, w, bias, shift, res, t = rand_layer(rng, N, H, W, C, K, R, S, groups, with_res=True, stride=stride, pad=pad)
    for rounding in range(4):
        for relu in (0, 1):
            _compare((x, w, bias, shift, res, t), dict(R=R, S=S, stride=stride, pad=pad, groups=groups, relu=relu,
                                                      rounding=rounding), ALGO["direct"], "direct")
    _compare((x, w, bias, shift, res, t), dict(R=R, S=S, stride=stride, pad=pad, groups=groups, out_mode=1),
             ALGO["direct"])
    _compare((x, w, bias, None, res, t, np.arange(K, dtype=np.int32) - 9),
             dict(R=R, S=S, stride=stride, pad=pad, groups=groups, out_mode=2), ALGO["direct"])


# ------------------------------------------------------------------ depthwise kernel
@pytest.mark.parametrize("case", [(2, 9, 11, 8, 1), (1, 14, 14, 32, 2), (2, 13, 10, 64, 2), (1, 28, 28, 128, 1),
                                  (3, 7, 7, 1024, 1), (1, 5, 3, 4, 1)])
def test_depthwise(case):
    N, H, W, C, st = case
    rng = np.random.default_rng(C + H)
    x, w, bias, shift, res, t = rand_layer(rng, N, H, W, C, C, 3, 3, groups=C, with_res=True, stride=(st, st),
                                           pad=(1, 1))
    shift = (shift - 5).clip(0, 31)
    kw = dict(R=3, S=3, stride=(st, st), pad=(1, 1), groups=C)
    for rounding in range(4):
        _compare((x, w, bias, shift, None, None), dict(relu=1, rounding=rounding, **kw), ALGO["auto"], "depthwise")
    _compare((x, w, bias, shift, res, t), dict(relu=0, **kw), ALGO["auto"], "depthwise")
    _compare((x, w, bias, shift), dict(out_mode=1, **kw), ALGO["dw"])
    _compare((x, w, bias, None, None, None, rng.integers(-12, -3, C).astype(np.int32)), dict(out_mode=2, **kw),
             ALGO["dw"])
    _compare((x, w, bias, shift), dict(out_c_pitch=C + 8, out_c_offset=4, **kw), ALGO["dw"])
    # shifts over the whole range (0, the largest that scales exactly in binary32, beyond it) with biases up to the
    # float-rounding path's limit, then past it (general kernel)
    shift2 = np.resize(np.array([0, 1, 22, 23, 31, 7, 12, 3], np.int32), C)
    bias2 = rng.integers(-4_000_000, 4_000_001, C).astype(np.int32)
    for relu in (0, 1):
        _compare((x, w, bias2, shift2), dict(relu=relu, **kw), ALGO["auto"], "depthwise")
        _compare((x, w, bias2 * 2, shift2), dict(relu=relu, **kw), ALGO["auto"], "depthwise")


# ------------------------------------------------------------------ tensor-core implicit GEMM
FLAT_CASES = [  # N, H, W, C, K
    (2, 9, 7, 32, 48), (3, 20, 20, 64, 64), (1, 16, 16, 16, 16), (2, 14, 14, 48, 24), (1, 28, 28, 144, 100),
    (2, 13, 13, 128, 208), (1, 31, 17, 256, 300), (4, 7, 7, 512, 128), (1, 1, 1, 2048, 512), (1, 40, 40, 112, 8),
]


@pytest.mark.parametrize("case", FLAT_CASES)
def test_igemm_1x1(case):
    N, H, W, C, K = case
    rng = np.random.default_rng(sum(case))
    x, w, bias, shift, res, t = rand_layer(rng, N, H, W, C, K, 1, 1, with_res=True)
    _compare((x, w, bias, shift), dict(R=1, S=1, relu=1), ALGO["auto"], "igemm/flat")
    _compare((x, w, bias, shift, res, t), dict(R=1, S=1, relu=1, rounding=1), ALGO["igemm"])
    _compare((x, w, bias, shift, res, t), dict(R=1, S=1, out_mode=1), ALGO["igemm"])
    _compare((x, w, None, None, None, None, rng.integers(-14, -4, K).astype(np.int32)), dict(R=1, S=1, out_mode=2),
             ALGO["igemm"])


@pytest.mark.parametrize("case", [(256, 1024, 1000), (32, 2048, 1000), (7, 512, 10), (128, 4096, 4096)])
def test_inner_product_layer(case):
    """An inner-product (fully connected) layer is Eq. 6 with a 1 x 1 image: batch rows against a
    K x C weight matrix, same bias / shift / saturation.  Classifier widths that are no multiple of
    16 take the general epilogue; logits are also read wide (int32)."""
    N, C, K = case
    rng = np.random.default_rng(N + C + K)
    x, w, bias, shift, _, _ = rand_layer(rng, N, 1, 1, C, K, 1, 1)
    _compare((x, w, bias, shift), dict(R=1, S=1), ALGO["auto"], "igemm/flat")
    _compare((x, w, bias, shift), dict(R=1, S=1, relu=1, out_mode=1), ALGO["auto"], "igemm/flat")


BOX_CASES = [  # N, H, W, C, K, R, S, pad
    (1, 32, 32, 16, 16, 3, 3, (1, 1)), (2, 7, 7, 64, 32, 3, 3, (1, 1)), (3, 14, 14, 32, 48, 3, 3, (1, 1)),
    (1, 28, 28, 96, 128, 3, 3, (1, 1)), (1, 56, 56, 64, 64, 3, 3, (1, 1)), (2, 14, 14, 32, 64, 5, 5, (2, 2)),
    (1, 19, 23, 48, 40, 3, 3, (1, 1)), (1, 12, 15, 16, 24, 7, 7, (3, 3)), (2, 10, 9, 32, 16, 3, 5, (0, 2)),
    (1, 9, 130, 16, 16, 3, 3, (1, 1)), (5, 5, 5, 160, 64, 3, 3, (1, 1)), (1, 8, 8, 32, 32, 2, 2, (0, 0)),
]


@pytest.mark.parametrize("case", BOX_CASES)
def test_igemm_box(case):
    N, H, W, C, K, R, S, pad = case
    rng = np.random.default_rng(sum(case[:7]))
    x, w, bias, shift, res, t = rand_layer(rng, N, H, W, C, K, R, S, with_res=True, pad=pad)
    # filters at least four taps wide on at most 64 channels read a filter row as one wide window
    name = "igemm/wrow" if (S >= 4 and C <= 64) else "igemm/box"
    for rounding in range(4):
        _compare((x, w, bias, shift), dict(R=R, S=S, pad=pad, relu=1, rounding=rounding), ALGO["auto"], name)
    _compare((x, w, bias, shift, res, t), dict(R=R, S=S, pad=pad), ALGO["igemm"])
    _compare((x, w, bias, shift, res, t), dict(R=R, S=S, pad=pad, symmetric=0, n_out=6), ALGO["igemm"])
    _compare((x, w, bias, shift), dict(R=R, S=S, pad=pad, out_mode=1), ALGO["igemm"])
    # the in-library CUDA-core kernel agrees too
    a, _ = gpu_conv(x, w, bias, shift, res, t, R=R, S=S, pad=pad, algo=ALGO["direct"])
    b, _ = gpu_conv(x, w, bias, shift, res, t, R=R, S=S, pad=pad, algo=ALGO["igemm"])
    assert (a == b).all()


# window rows (stride 1, wide filters, few channels): every fold factor, one and two chunks per
# filter row, residual, concat window, ragged images, several tiles; the plain box form must agree
WROW_CASES = [  # N, H, W, C, K, R, S, pad
    (2, 28, 28, 16, 32, 5, 5, (2, 2)), (1, 28, 28, 32, 96, 5, 5, (2, 2)), (3, 14, 14, 48, 128, 5, 5, (2, 2)),
    (1, 20, 24, 16, 16, 5, 5, (2, 2)), (2, 13, 17, 32, 64, 7, 7, (3, 3)), (1, 9, 40, 64, 32, 3, 4, (1, 2)),
    (1, 30, 30, 16, 48, 5, 5, (0, 0)), (2, 11, 16, 32, 24, 1, 5, (0, 1)), (1, 16, 64, 16, 8, 5, 8, (2, 4)),
]


@pytest.mark.parametrize("case", WROW_CASES)
def test_igemm_window_rows(case):
    N, H, W, C, K, R, S, pad = case
    rng = np.random.default_rng(sum(case[:7]) + 1)
    x, w, bias, shift, res, t = rand_layer(rng, N, H, W, C, K, R, S, with_res=True, pad=pad)
    kw = dict(R=R, S=S, pad=pad)
    got, _ = _compare((x, w, bias, shift), dict(relu=1, **kw), ALGO["auto"], "igemm/wrow")
    _compare((x, w, bias, shift, res, t), dict(relu=1, **kw), ALGO["auto"], "igemm/wrow")
    _compare((x, w, bias, shift), dict(out_mode=1, **kw), ALGO["auto"], "igemm/wrow")
    _compare((x, w, bias, shift), dict(relu=1, out_c_offset=16, out_c_pitch=K + 48, **kw), ALGO["auto"], "igemm/wrow")
    with binding.plan_hints(window_rows=0):
        _compare((x, w, bias, shift), dict(relu=1, **kw), ALGO["auto"], "igemm/box")


@pytest.mark.parametrize("case", [(2, 14, 14, 64, 128, 2), (1, 15, 9, 32, 48, 2), (3, 28, 28, 256, 512, 2),
                                  (1, 10, 10, 16, 16, 3)])
def test_igemm_strided_1x1(case):
    N, H, W, C, K, st = case
    rng = np.random.default_rng(sum(case))
    x, w, bias, shift, _, _ = rand_layer(rng, N, H, W, C, K, 1, 1)
    _compare((x, w, bias, shift), dict(R=1, S=1, stride=(st, st)), ALGO["auto"], "igemm/view")
    _compare((x, w, bias, shift), dict(R=1, S=1, stride=(st, 1)), ALGO["igemm"], "igemm/view")


@pytest.mark.parametrize("case", [(2, 32, 32, 3, 64, 7, (2, 2), (3, 3)), (1, 20, 24, 3, 64, 3, (1, 1), (1, 1)),
                                  (2, 17, 17, 3, 32, 3, (2, 2), (1, 1)), (1, 9, 9, 1, 16, 5, (1, 1), (2, 2)),
                                  (1, 8, 8, 4, 24, 3, (1, 2), (1, 0))])
def test_igemm_stem(case):
    N, H, W, C, K, R, stride, pad = case
    rng = np.random.default_rng(sum(case[:6]))
    x, w, bias, shift, _, _ = rand_layer(rng, N, H, W, C, K, R, R, stride=stride, pad=pad)
    name = "igemm/s2d" if stride == (2, 2) else ("igemm/wrow" if stride == (1, 1) else "igemm/stem")
    _compare((x, w, bias, shift), dict(R=R, S=R, stride=stride, pad=pad, relu=1), ALGO["auto"], name)
    _compare((x, w, bias, shift), dict(R=R, S=R, stride=stride, pad=pad, out_mode=1), ALGO["igemm"])
    if stride == (1, 1):
        with binding.plan_hints(window_rows=0):              # the patch-matrix form of the same layer
            _compare((x, w, bias, shift), dict(R=R, S=R, stride=stride, pad=pad, relu=1), ALGO["auto"], "igemm/stem")


# stride-1 layers on at most 4 channels read padded rows of 8- or 16-byte pixels: folded (K <= 64) and
# unfolded, 1 to 4 channels, non-square filters, every padding, odd widths (the row pitch is rounded up
# to 16 bytes), several tiles with ragged tails, a batch smaller than planned
ROW_STEM_CASES = [(2, 32, 32, 3, 64, 3, 3, (1, 1)), (1, 21, 19, 3, 32, 3, 3, (1, 1)), (1, 20, 26, 1, 16, 5, 5, (2, 2)),
                  (2, 15, 17, 4, 128, 3, 3, (1, 1)), (1, 12, 40, 2, 48, 2, 4, (0, 3)), (3, 9, 9, 3, 80, 3, 2, (2, 0)),
                  (1, 64, 224, 3, 64, 3, 3, (1, 1)), (1, 10, 13, 3, 8, 7, 7, (3, 3)), (2, 11, 11, 3, 24, 1, 16, (0, 8))]


@pytest.mark.parametrize("case", ROW_STEM_CASES)
def test_igemm_stem_padded_rows(case):
    import torch
    N, H, W, C, K, R, S, pad = case
    rng = np.random.default_rng(sum(case[:7]) + 11)
    x, w, bias, shift, _, _ = rand_layer(rng, N, H, W, C, K, R, S, pad=pad)
    kw = dict(R=R, S=S, pad=pad)
    _compare((x, w, bias, shift), dict(relu=1, **kw), ALGO["auto"], "igemm/wrow")
    _compare((x, w, bias, shift), dict(out_mode=1, **kw), ALGO["auto"], "igemm/wrow")
    _compare((x, w, bias, shift), dict(out_mode=2, **kw), ALGO["auto"], "igemm/wrow")
    _compare((x, w, bias, shift), dict(relu=1, out_c_offset=16, out_c_pitch=K + 48, **kw), ALGO["auto"], "igemm/wrow")
    # the float image through the same packing kernel, and a partial batch
    e_x = -4
    xf = (rng.standard_normal((N, H, W, C)) * (40.0 * 2.0 ** e_x)).astype(np.float32)
    xf.flat[:6] = np.float32([np.nan, np.inf, -np.inf, 0.5 * 2.0 ** e_x, 1.5 * 2.0 ** e_x, -2.5 * 2.0 ** e_x])
    xq = ref.quantize_f32(xf, e_x, 8)
    conv = binding.QConv(w, bias, shift, N=N, H=H, W=W, C=C, K=K, R=R, S=S, pad_h=pad[0], pad_w=pad[1], relu=1)
    for n_run in sorted({N, 1}):
        want = oracle_conv(xq[:n_run], w, bias, shift, R=R, S=S, pad=pad, relu=1)
        y = torch.full(want.shape, 77, dtype=torch.int8, device="cuda")
        conv.run_f32(torch.from_numpy(xf[:n_run]).cuda(), e_x, y, n_run=n_run)
        assert conv.status() == 0
        assert (y.cpu().numpy() == want).all()
        y2 = torch.full(want.shape, 78, dtype=torch.int8, device="cuda")
        conv.run(torch.from_numpy(xq[:n_run]).cuda(), y2, n_run=n_run)
        assert (y2.cpu().numpy() == want).all()
    conv.destroy()


# stride-2 stems run in space-to-depth form: odd and even image sizes, every pad parity, filters
# from 1 to 7 taps (also non-square), 1 to 4 channels, several tiles with a ragged tail
S2D_CASES = [(2, 32, 32, 3, 64, 7, 7, (3, 3)), (1, 33, 31, 3, 32, 3, 3, (1, 1)), (2, 17, 19, 3, 32, 3, 3, (0, 0)),
             (1, 21, 16, 1, 16, 5, 5, (2, 2)), (1, 16, 23, 4, 24, 3, 5, (1, 2)), (1, 12, 12, 2, 48, 2, 2, (0, 0)),
             (3, 30, 28, 3, 64, 7, 3, (2, 1)), (1, 11, 13, 3, 16, 1, 1, (0, 0)), (1, 40, 300, 3, 32, 3, 3, (1, 1)),
             (2, 9, 9, 3, 80, 4, 6, (3, 3))]


@pytest.mark.parametrize("case", S2D_CASES)
def test_igemm_stem_space_to_depth(case):
    N, H, W, C, K, R, S, pad = case
    rng = np.random.default_rng(sum(case[:7]))
    x, w, bias, shift, _, _ = rand_layer(rng, N, H, W, C, K, R, S, stride=(2, 2), pad=pad)
    kw = dict(R=R, S=S, stride=(2, 2), pad=pad)
    got, _ = _compare((x, w, bias, shift), dict(relu=1, **kw), ALGO["auto"], "igemm/s2d")
    _compare((x, w, bias, shift), dict(out_mode=1, **kw), ALGO["auto"], "igemm/s2d")
    # the patch-matrix form of the same layer stays available and must agree too
    with binding.plan_hints(space_to_depth=0):
        _compare((x, w, bias, shift), dict(relu=1, **kw), ALGO["auto"], "igemm/stem")


# 2 x 2 max-pool taken inside the layer: image widths that give tile rows of 16, 8, 4 and 2 pixels, ragged last
# tiles along both axes, several images per tile, 64 to 512 output channels, per-channel and per-layer shifts,
# with and without ReLU, integer and float-rounding epilogues, concat window, 256-wide and SM-pair tiles
POOL_CASES = [(2, 32, 32, 64, 64, 3), (1, 20, 24, 32, 128, 3), (3, 28, 28, 64, 96, 3), (4, 14, 14, 128, 64, 3),
              (1, 12, 56, 16, 48, 5), (2, 6, 6, 64, 32, 3), (1, 16, 36, 32, 80, 3), (5, 2, 2, 16, 16, 3)]


@pytest.mark.parametrize("case", POOL_CASES)
def test_igemm_fused_max_pool(case):
    N, H, W, C, K, R = case
    rng = np.random.default_rng(sum(case) + 17)
    pad = (R // 2, R // 2)
    stride, Hc, Wc = (1, 1), H, W
    for per_channel in (True, False):
        x, w, bias, shift, _, _ = rand_layer(rng, N, Hc, Wc, C, K, R, R, stride=stride, pad=pad, per_channel_shift=per_channel)
        for relu in (1, 0):
            kw = dict(R=R, S=R, stride=stride, pad=pad, relu=relu)
            want = ref.maxpool_i8(oracle_conv(x, w, bias, shift, **kw), 2, 2, 2, 0)
            got, desc = gpu_conv(x, w, bias, shift, pool=2, **kw)
            assert "pool=2" in desc and "igemm/box" in desc, desc
            assert (got == want).all(), (desc, np.argwhere(got != want)[:5])
        # weights small enough for the float-rounding epilogue
        ws = (w // 16).astype(np.int8)
        bs = (bias // 8).astype(np.int32)
        ss = np.maximum(shift - 4, 0).astype(np.int32)
        kw = dict(R=R, S=R, stride=stride, pad=pad, relu=1)
        want = ref.maxpool_i8(oracle_conv(x, ws, bs, ss, **kw), 2, 2, 2, 0)
        got, desc = gpu_conv(x, ws, bs, ss, pool=2, **kw)
        assert "flt=1" in desc or C * R * R > 1024, desc
        assert (got == want).all(), desc
    # into a concat buffer
    kw = dict(R=R, S=R, stride=stride, pad=pad, relu=1)
    full = oracle_conv(x, w, bias, shift, **kw)
    got, _ = gpu_conv(x, w, bias, shift, pool=2, out_c_offset=16, out_c_pitch=K + 48, **kw)
    assert (got[..., 16:16 + K] == ref.maxpool_i8(full, 2, 2, 2, 0)).all()
    assert (got[..., :16] == 77).all() and (got[..., 16 + K:] == 77).all()


def test_igemm_fused_max_pool_wide_and_pair_tiles():
    rng = np.random.default_rng(91)
    for (N, H, W, C, K) in [(2, 28, 28, 128, 256), (1, 14, 14, 256, 512), (2, 56, 24, 64, 256)]:
        x, w, bias, shift, _, _ = rand_layer(rng, N, H, W, C, K, 3, 3, pad=(1, 1), per_channel_shift=False)
        kw = dict(R=3, S=3, pad=(1, 1), relu=1)
        want = ref.maxpool_i8(oracle_conv(x, w, bias, shift, **kw), 2, 2, 2, 0)
        with binding.plan_hints(bn_max=256):
            got, desc = gpu_conv(x, w, bias, shift, pool=2, **kw)
            assert "BN=256" in desc and "pool=2" in desc, desc
            assert (got == want).all(), desc
        with binding.plan_hints(bn_max=256, pair_tiles=1):
            got, desc = gpu_conv(x, w, bias, shift, pool=2, **kw)
            assert "pair=1" in desc and "pool=2" in desc, desc
            assert (got == want).all(), desc


def test_fused_max_pool_refuses_what_it_cannot_take():
    rng = np.random.default_rng(92)
    x, w, bias, shift, res, t = rand_layer(rng, 1, 8, 8, 32, 32, 3, 3, pad=(1, 1), with_res=True)
    for bad in (dict(out_mode=1), dict(n_out=6), dict(rounding=1)):
        with pytest.raises(binding.QconvError) as err:
            gpu_conv(x, w, bias, shift, R=3, S=3, pad=(1, 1), pool=2, **bad)
        assert err.value.code == binding.ERR_UNSUPPORTED_SHAPE
    with pytest.raises(binding.QconvError) as err:
        gpu_conv(x, w, bias, shift, res, t, R=3, S=3, pad=(1, 1), pool=2)
    assert err.value.code == binding.ERR_UNSUPPORTED_SHAPE
    with pytest.raises(binding.QconvError) as err:                  # odd output size
        gpu_conv(x[:, :7], w, bias, shift, R=3, S=3, pad=(1, 1), pool=2)
    assert err.value.code == binding.ERR_UNSUPPORTED_SHAPE
    with pytest.raises(binding.QconvError) as err:                  # 1x1 stride 1 runs as a flat GEMM
        gpu_conv(x, w[:, :1, :1], bias, shift, R=1, S=1, pool=2)
    assert err.value.code == binding.ERR_UNSUPPORTED_SHAPE
    with pytest.raises(binding.QconvError) as err:
        gpu_conv(x, w, bias, shift, R=3, S=3, pad=(1, 1), pool=3)
    assert err.value.code == binding.ERR_BAD_ARG


def test_concat_written_in_place():
    rng = np.random.default_rng(5)
    x, w, bias, shift, _, _ = rand_layer(rng, 2, 14, 14, 64, 48, 3, 3, pad=(1, 1))
    for off, pitch in [(0, 112), (64, 112), (16, 80), (3, 57)]:
        for algo in ("igemm", "direct"):
            _compare((x, w, bias, shift), dict(R=3, S=3, pad=(1, 1), out_c_offset=off, out_c_pitch=pitch),
                     ALGO[algo])


def test_weight_layout_rsck_and_single_conv_config():
    c = wl.single_conv_cfg()
    args = (c["x"], c["w"], c["bias"], c["shift"])
    kw = dict(R=3, S=3, stride=c["stride"], pad=c["pad"], relu=1, weight_layout=1, K=16)
    got, desc = _compare(args, kw, ALGO["auto"], "igemm")
    assert got.min() == 0 and got.max() == 127
    _compare(args, kw, ALGO["direct"])


def test_extreme_values_fill_the_accumulator():
    # Eq. 9: 4608 products of -128 * -128 still fit int32; the GPU's 32-bit accumulator must agree with
    # the oracle's 64-bit one.
    for xv, wv in [(-128, -128), (127, -128), (-128, 127)]:
        x = np.full((1, 6, 6, 512), xv, np.int8)
        w = np.full((16, 3, 3, 512), wv, np.int8)
        got, _ = _compare((x, w), dict(R=3, S=3, pad=(1, 1), out_mode=1), ALGO["igemm"])
        assert abs(int(got[0, 2, 2, 0])) == 4608 * abs(xv * wv)
        _compare((x, w, None, np.full(16, 19, np.int32)), dict(R=3, S=3, pad=(1, 1)), ALGO["igemm"])


def test_rounding_ties_through_the_kernels():
    # one input channel carrying value v times weight 1 gives acc = v exactly; shifts make ties
    vals = np.arange(-128, 128, dtype=np.int8)
    x = np.zeros((1, 16, 16, 16), np.int8)
    x[0, :, :, 0] = vals.reshape(16, 16)
    w = np.zeros((16, 1, 1, 16), np.int8)
    w[:, 0, 0, 0] = 1
    shift = (np.arange(16) % 8).astype(np.int32)
    for rounding in range(4):
        for algo in ("igemm", "direct"):
            _compare((x, w, None, shift), dict(R=1, S=1, rounding=rounding), ALGO[algo])


# Layers on at most 64 channels put the taps of a filter row into one ring stage (one activation box per
# tap, side by side): filters 2 to 4 taps wide, non-square, padded and unpadded, resident and streamed weights.
@pytest.mark.parametrize("case", [(2, 20, 20, 16, 16, 3, 3, (1, 1)), (1, 33, 17, 32, 48, 3, 3, (1, 1)), (3, 14, 14, 64, 64, 3, 3, (1, 1)),
                                  (2, 16, 18, 48, 32, 2, 2, (0, 0)), (1, 19, 23, 64, 128, 5, 4, (2, 1)), (2, 12, 40, 32, 200, 1, 3, (0, 1)),
                                  (1, 64, 64, 64, 64, 3, 3, (1, 1))])
def test_igemm_grouped_taps(case):
    N, H, W, C, K, R, S, pad = case
    rng = np.random.default_rng(sum(case[:7]) + 3)
    x, w, bias, shift, res, t = rand_layer(rng, N, H, W, C, K, R, S, with_res=True, pad=pad)
    kw = dict(R=R, S=S, pad=pad)
    with binding.plan_hints(window_rows=0, halo=0, group_taps=1):
        _, desc = _compare((x, w, bias, shift), dict(relu=1, **kw), ALGO["igemm"], "grp=%d" % S)
        _compare((x, w, bias, shift, res, t), dict(relu=1, **kw), ALGO["igemm"], "grp=%d" % S)
        _compare((x, w, bias, shift), dict(out_mode=1, **kw), ALGO["igemm"], "grp=%d" % S)
        if K % 16 == 0:
            _compare((x, w, bias, shift), dict(relu=1, out_c_offset=16, out_c_pitch=K + 32, **kw), ALGO["igemm"], "grp=%d" % S)
    for rw in (0, 1):
        with binding.plan_hints(window_rows=0, halo=0, group_taps=1, resident_weights=rw):
            _compare((x, w, bias, shift), dict(relu=1, **kw), ALGO["igemm"], "b_res=%d" % rw if rw == 0 else "grp=%d" % S)
    with binding.plan_hints(window_rows=0, halo=0, group_taps=0):
        _compare((x, w, bias, shift), dict(relu=1, **kw), ALGO["igemm"], "grp=0")


# Tiles 256 channels wide (one CTA per SM, MMAs of N = 256): the planner takes them for tensor-bound
# layers; here they are forced on small shapes -- several channel tiles, a ragged last one, flat /
# strided-view / box forms, per-layer and per-channel shifts, float-rounding and integer epilogues.
@pytest.mark.parametrize("case", [(2, 14, 14, 128, 256, 3, 1), (1, 28, 28, 64, 512, 3, 1), (3, 9, 11, 128, 320, 3, 1),
                                  (2, 16, 16, 256, 256, 1, 1), (2, 16, 16, 128, 784, 1, 2), (1, 30, 30, 32, 272, 5, 1),
                                  (70, 14, 14, 128, 256, 3, 1)])
def test_igemm_wide_tiles(case):
    N, H, W, C, K, R, st = case
    rng = np.random.default_rng(sum(case) + 77)
    pad = (R // 2, R // 2)
    for per_channel in (False, True):
        x, w, bias, shift, _, _ = rand_layer(rng, N, H, W, C, K, R, R, stride=(st, st), pad=pad,
                                             per_channel_shift=per_channel)
        kw = dict(R=R, S=R, stride=(st, st), pad=pad)
        with binding.plan_hints(bn_max=256, window_rows=0):
            _, desc = _compare((x, w, bias, shift), dict(relu=1, **kw), ALGO["igemm"])
            bn = int(desc.split("BN=")[1].split()[0])
            assert bn > 128 and "ctas/sm=1" in desc, desc
            _compare((x, w, bias, shift), dict(relu=0, **kw), ALGO["igemm"], "BN=%d" % bn)
            _compare((x, w, bias, shift), dict(relu=1, out_c_offset=32, out_c_pitch=K + 64, **kw), ALGO["igemm"], "BN=%d" % bn)
            # small weights: the float-rounding epilogue in this width
            ws = (w.astype(np.int32) % 3 - 1).astype(np.int8)
            _compare((x, ws, (bias // 8).astype(np.int32), np.minimum(shift, 6)), dict(relu=1, **kw), ALGO["igemm"], "flt=1")
            _compare((x, ws, (bias // 8).astype(np.int32), np.minimum(shift, 6)), dict(relu=0, **kw), ALGO["igemm"], "flt=1")


# Tiles of 256 pixels x 256 channels on pairs of SMs (tcgen05.mma.cta_group::2, each CTA loading its own
# halves of the operands): forced on small shapes -- an odd number of pixel boxes (the last pair has one box),
# several channel tiles with a ragged last one, flat / strided-view / box / strided-box forms, more pair tiles
# than SM pairs (ring and accumulator phases wrap), both epilogue families, per-layer and per-channel shifts.
@pytest.mark.parametrize("case", [(2, 14, 14, 128, 256, 3, 1), (3, 9, 11, 128, 320, 3, 1), (1, 28, 28, 64, 512, 3, 1),
                                  (2, 16, 16, 256, 256, 1, 1), (2, 16, 16, 128, 784, 1, 2), (1, 31, 31, 64, 272, 3, 2),
                                  (90, 14, 14, 128, 256, 3, 1)])
def test_igemm_sm_pairs(case):
    N, H, W, C, K, R, st = case
    rng = np.random.default_rng(sum(case) + 177)
    pad = (R // 2, R // 2)
    for per_channel in (False, True):
        x, w, bias, shift, _, _ = rand_layer(rng, N, H, W, C, K, R, R, stride=(st, st), pad=pad,
                                             per_channel_shift=per_channel)
        kw = dict(R=R, S=R, stride=(st, st), pad=pad)
        with binding.plan_hints(bn_max=256, pair_tiles=1, window_rows=0):
            _, desc = _compare((x, w, bias, shift), dict(relu=1, **kw), ALGO["igemm"], "pair=1")
            _compare((x, w, bias, shift), dict(relu=0, **kw), ALGO["igemm"], "pair=1")
            _compare((x, w, bias, shift), dict(relu=1, out_c_offset=32, out_c_pitch=K + 64, **kw), ALGO["igemm"], "pair=1")
            ws = (w.astype(np.int32) % 3 - 1).astype(np.int8)
            _compare((x, ws, (bias // 8).astype(np.int32), np.minimum(shift, 6)), dict(relu=1, **kw), ALGO["igemm"], "flt=1")
            _compare((x, ws, (bias // 8).astype(np.int32), np.minimum(shift, 6)), dict(relu=0, **kw), ALGO["igemm"], "flt=1")


# The tensor-core path rounds in fp32 when the wide value provably stays below 2^22 (one FMA with the
# constants 2^-s and M(1 - 2^-s), M = 1.5 * 2^23).  s = 22 is the last shift whose constants are exact;
# beyond it the kernel switches to scale 0.  Wide values are driven to +-2^20, +-2^21, +-3 * 2^20 (the
# ties and their neighbours at s = 21 and 22) by the bias; rows of zero input hit the ties exactly.
@pytest.mark.parametrize("per_channel", [False, True])
@pytest.mark.parametrize("geom", [(1, 1, 32, 32), (1, 1, 64, 160), (3, 3, 64, 64), (3, 3, 128, 64)])
def test_float_rounding_epilogue_at_large_shifts(geom, per_channel):
    R, S, C, K = geom
    rng = np.random.default_rng(100 * R + C + K + int(per_channel))
    N, H, W = 3, 12, 20
    x = rng.integers(-128, 128, size=(N, H, W, C), dtype=np.int8)
    x[0, :3] = 0                                             # accumulator == bias exactly on these rows
    w = np.zeros((K, R, S, C), np.int8)
    for k in range(K):                                       # eight taps of +-1 per channel: |sum| <= 1024
        idx = rng.choice(R * S * C, size=8, replace=False)
        w[k].reshape(-1)[idx] = rng.choice(np.int8([-1, 1]), size=8)
    anchors = np.int64([1 << 20, 1 << 21, 3 << 20, (1 << 20) + (1 << 19), 1 << 19])
    bias = (rng.choice(anchors, size=K) * rng.choice([-1, 1], size=K)).astype(np.int64)
    bias[K // 2:] += rng.integers(-600, 600, size=K - K // 2)
    bias = bias.astype(np.int32)
    pad = (R // 2, S // 2)
    P, Q = H, W
    res = rng.integers(-128, 128, size=(N, P, Q, K), dtype=np.int8)
    for s_base in (21, 22, 23, 31):
        if per_channel:
            shift = np.int32([21, 22, 23, 31, 20, 24])[(np.arange(K) + s_base) % 6]
            t = rng.integers(0, 13, size=K).astype(np.int32)
        else:
            shift = np.full(K, s_base, np.int32)
            t = np.full(K, 12, np.int32)
        for relu in (0, 1):
            kw = dict(R=R, S=S, pad=pad, relu=relu)
            _, desc = _compare((x, w, bias, shift), kw, ALGO["igemm"], "flt=1")
            assert ("uni=0" if per_channel else "uni=1") in desc, desc
            _, desc = _compare((x, w, bias, shift, res, t), kw, ALGO["igemm"], "flt=1")
            # both store paths: tiles staged for TMA stores (short contractions) and 16-byte register stores
            with binding.plan_hints(tma_store=0):
                _compare((x, w, bias, shift, res, t), kw, ALGO["igemm"], "tma_store=0")
            with binding.plan_hints(tma_store=1):
                _, desc = _compare((x, w, bias, shift), kw, ALGO["igemm"], "flt=1")
                assert "tma_store=0" not in desc, desc
    # the same data through the integer-rounding instantiation must agree as well
    with binding.plan_hints(float_rounding=0):
        _compare((x, w, bias, np.full(K, 22, np.int32)), dict(R=R, S=S, pad=pad), ALGO["igemm"], "flt=0")


# An expired wait must end the kernel cleanly: status raised, every role out, copies landed, tensor
# memory freed, the context and the handle usable afterwards.  Limit 0 makes every wait expire at once
# (nothing faults or hangs: each role gives up on its first poll).  Cases: constants staged once /
# per tile (more than 512 channels, per-channel shifts), tiles stored from registers / by TMA, residual
# tiles fetched by TMA, resident weights, and the TMA-staged depthwise kernel.
@pytest.mark.parametrize("case", [
    dict(g=(1, 14, 14, 32, 32, 3), hints={}),
    dict(g=(2, 14, 14, 64, 1024, 1), hints=dict(tma_store=0)),
    dict(g=(2, 14, 14, 64, 1024, 1), hints={}),
    dict(g=(4, 28, 28, 64, 256, 1), hints={}, res=True),
    dict(g=(40, 28, 28, 128, 64, 3), hints=dict(resident_weights=1)),
    dict(g=(2, 28, 28, 64, 64, 3), hints={}, dw=True),
])
def test_bounded_wait_reports_timeout_and_context_survives(case):
    import torch
    N, H, W, C, K, R = case["g"]
    rng = np.random.default_rng(8 + K)
    dw = case.get("dw", False)
    x, w, bias, shift, res, t = rand_layer(rng, N, H, W, C, K, R, R, groups=C if dw else 1,
                                           with_res=case.get("res", False), pad=(R // 2, R // 2))
    if dw:
        bias = (bias // 64).astype(np.int32)
    kw = dict(R=R, S=R, pad=(R // 2, R // 2), groups=C if dw else 1, relu=1)
    with binding.plan_hints(**case["hints"]):
        got, conv = gpu_conv(x, w, bias, shift, res, t, algo=ALGO["dw" if dw else "igemm"], want_handle=True, **kw)
    want = oracle_conv(x, w, bias, shift, res, t, **kw)
    assert (got == want).all(), conv.describe()
    if dw:
        assert "tma" in conv.describe()
    xd = torch.from_numpy(x).cuda()
    rd = torch.from_numpy(res).cuda() if res is not None else None
    y = torch.zeros((N, H, W, K), dtype=torch.int8, device="cuda")
    conv.set_wait_limit(0)                   # every device-side wait gives up at once
    conv.run(xd, y, rd)
    assert conv.status() == binding.ERR_TIMEOUT
    assert conv.status() == 0                # status is cleared once read
    conv.set_wait_limit(1 << 22)
    conv.run(xd, y, rd)
    assert conv.status() == 0
    assert (y.cpu().numpy() == want).all()
    conv.destroy()


def test_run_time_argument_errors():
    import torch
    from paper_1805_07941_b200 import binding
    w = np.ones((16, 1, 1, 16), np.int8)
    conv = binding.QConv(w, N=2, H=4, W=4, C=16, K=16, R=1, S=1)
    x = torch.zeros(2 * 4 * 4 * 16 + 16, dtype=torch.int8, device="cuda")
    y = torch.zeros(2 * 4 * 4 * 16, dtype=torch.int8, device="cuda")
    with pytest.raises(binding.QconvError) as e:
        conv.run(x[1:], y, n_run=2)
    assert e.value.code == binding.ERR_ALIGNMENT
    with pytest.raises(binding.QconvError) as e:
        conv.run(x, y, n_run=3)
    assert e.value.code == binding.ERR_BAD_ARG
    with pytest.raises(binding.QconvError) as e:
        conv.run(x, y, residual=y, n_run=2)
    assert e.value.code == binding.ERR_BAD_ARG
    conv.run(x, y, n_run=1)                  # a smaller batch than the maximum is fine
    assert conv.status() == 0


def test_eltwise_add_layer():
    import torch
    from paper_1805_07941_b200 import binding
    rng = np.random.default_rng(31)
    for count in (1, 15, 4096 + 7, 1 << 20):
        for n_in, lshift, rshift in [(2, [0, 3], 4), (3, [2, 0, 1], 2), (1, [0], 0), (4, [0, 0, 5, 1], 7)]:
            xs = [rng.integers(-128, 128, size=count, dtype=np.int8) for _ in range(n_in)]
            ts = [torch.from_numpy(x).cuda() for x in xs]
            for mode in range(4):
                for relu, sym, n_out in [(0, 1, 8), (1, 1, 8), (0, 0, 6)]:
                    got = binding.qeltwise_add_i8(ts, lshift, rshift, relu, mode, n_out, sym).cpu().numpy()
                    want = ref.eltwise_add(xs, lshift, rshift, relu, mode, n_out, sym)
                    assert (got == want).all(), (count, n_in, mode, relu)
    t = torch.zeros(64, dtype=torch.int8, device="cuda")
    with pytest.raises(binding.QconvError) as e:
        binding.qeltwise_add_i8([t, t], [0, 24], 3)
    assert e.value.code == binding.ERR_RESIDUAL_SCALE
    with pytest.raises(binding.QconvError) as e:
        binding.qeltwise_add_i8([t, t], [0, 1], 32)
    assert e.value.code == binding.ERR_BAD_SHIFT
    with pytest.raises(binding.QconvError) as e:
        binding.qeltwise_add_i8([t] * 8, [23] * 8, 3)
    assert e.value.code == binding.ERR_OVERFLOW_RISK


def test_identity_conv_splice_rescales_an_edge():
    """Section 3's splice for an edge whose consumer wants a coarser scale: a 1 x 1 convolution with
    identity weights and a right shift s multiplies the tensor by 2^-s in (0, 1].  Each output must
    be the rounded, saturated shift of its input (checked against exact rationals, not the oracle's
    own convolution), in every rounding mode, through the tensor-core path."""
    from fractions import Fraction
    import math
    rng = np.random.default_rng(77)
    C = 64
    x = rng.integers(-128, 128, size=(2, 9, 11, C), dtype=np.int8)
    w = np.zeros((C, 1, 1, C), np.int8)
    w[np.arange(C), 0, 0, np.arange(C)] = 1
    for s in (0, 1, 3):
        shift = np.full(C, s, np.int32)
        for rounding in range(4):
            got, desc = gpu_conv(x, w, None, shift, R=1, S=1, rounding=rounding)
            assert "igemm" in desc
            want = np.empty_like(x)
            for v in range(-128, 128):
                q = Fraction(v, 2 ** s)
                fl = math.floor(q)
                if rounding == 0:
                    r = round(q)                                   # exact rationals: ties to even
                elif rounding == 1:
                    r = fl + 1 if q - fl > Fraction(1, 2) or (q - fl == Fraction(1, 2) and v > 0) else fl
                elif rounding == 2:
                    r = math.floor(q + Fraction(1, 2))
                else:
                    r = fl
                want[x == v] = max(-127, min(127, r))
            assert (got == want).all(), (s, rounding)


@pytest.mark.parametrize("case", [(2, 32, 32, 3, 64, 7, (3, 3), -5), (1, 33, 31, 3, 32, 3, (1, 1), -6),
                                  (2, 17, 20, 1, 16, 5, (2, 2), -4), (1, 16, 23, 4, 24, 3, (1, 1), 1)])
def test_stem_on_float_input(case):
    """qconv_run_f32: the input conversion fused into the stem's packing kernel must give what
    qquantize_f32 followed by qconv_run gives, i.e. the oracle's quantize + convolution."""
    import torch
    from paper_1805_07941_b200 import binding
    N, H, W, C, K, R, pad, e_x = case
    rng = np.random.default_rng(sum(case[:6]) + 3)
    _, w, bias, shift, _, _ = rand_layer(rng, N, H, W, C, K, R, R, stride=(2, 2), pad=pad)
    xf = (rng.standard_normal((N, H, W, C)) * (40.0 * 2.0 ** e_x)).astype(np.float32)
    xf.flat[:6] = np.float32([np.nan, np.inf, -np.inf, 0.5 * 2.0 ** e_x, 1.5 * 2.0 ** e_x, -2.5 * 2.0 ** e_x])
    xq = ref.quantize_f32(xf, e_x, 8)
    want = oracle_conv(xq, w, bias, shift, R=R, S=R, stride=(2, 2), pad=pad, relu=1)
    conv = binding.QConv(w, bias, shift, N=N, H=H, W=W, C=C, K=K, R=R, S=R, stride_h=2, stride_w=2,
                         pad_h=pad[0], pad_w=pad[1], relu=1)
    assert "igemm/s2d" in conv.describe()
    y = torch.full(want.shape, 77, dtype=torch.int8, device="cuda")
    conv.run_f32(torch.from_numpy(xf).cuda(), e_x, y)
    assert conv.status() == 0
    assert (y.cpu().numpy() == want).all()
    # a second call on other data through the int8 entry: the handle is not left in the fused state
    y2 = torch.empty_like(y)
    conv.run(torch.from_numpy(xq).cuda(), y2)
    assert (y2.cpu().numpy() == want).all()
    conv.destroy()
    # layers that do not repack in space-to-depth form refuse
    other = binding.QConv(np.ones((16, 1, 1, 16), np.int8), N=1, H=4, W=4, C=16, K=16, R=1, S=1)
    with pytest.raises(binding.QconvError) as err:
        other.run_f32(torch.zeros((1, 4, 4, 16), device="cuda"), 0, torch.zeros((1, 4, 4, 16), dtype=torch.int8, device="cuda"))
    assert err.value.code == binding.ERR_UNSUPPORTED_SHAPE
    other.destroy()


# 3x3 stride-1 layers on a multiple of 128 channels load one activation box per filter row (with its
# horizontal halo) and read it shifted by one pixel per tap: image widths with one to many image rows
# per tile, several images per tile, residual, concat window, partial last tiles
HALO_CASES = [(2, 14, 14, 128, 64), (1, 28, 28, 256, 128), (3, 7, 7, 512, 100), (1, 56, 56, 128, 256),
              (1, 9, 126, 128, 32), (5, 5, 6, 128, 48), (2, 13, 17, 256, 64), (4, 56, 56, 64, 64),
              (2, 30, 30, 64, 32), (40, 28, 28, 128, 64), (1, 20, 100, 64, 200),
              # images wider than 126 pixels: equal column segments, each with its own halo
              (2, 6, 224, 64, 64), (1, 5, 127, 128, 48), (1, 3, 300, 64, 32), (3, 4, 130, 64, 80), (1, 3, 253, 128, 16)]


@pytest.mark.parametrize("case", HALO_CASES)
def test_igemm_halo_rows(case):
    N, H, W, C, K = case
    rng = np.random.default_rng(sum(case) + 5)
    x, w, bias, shift, res, t = rand_layer(rng, N, H, W, C, K, 3, 3, with_res=True, pad=(1, 1))
    kw = dict(R=3, S=3, pad=(1, 1))
    with binding.plan_hints(halo=1):                        # also where the planner would keep per-tap boxes
        _, desc = _compare((x, w, bias, shift), dict(relu=1, **kw), ALGO["auto"], "igemm/box")
        assert "halo=3" in desc, desc
        _compare((x, w, bias, shift, res, t), dict(relu=1, **kw), ALGO["auto"], "halo=3")
        _compare((x, w, bias, shift), dict(out_mode=1, **kw), ALGO["auto"], "halo=3")
        _compare((x, w, bias, shift), dict(pad=(0, 1), R=3, S=3), ALGO["auto"], "halo=3")          # no vertical padding
        if K % 16 == 0:
            _compare((x, w, bias, shift), dict(relu=1, out_c_offset=16, out_c_pitch=K + 48, **kw), ALGO["auto"], "halo=3")
    if C <= 128:                                            # one chunk per tap: the weights may stay resident
        with binding.plan_hints(halo=1, resident_weights=1):
            _, desc = _compare((x, w, bias, shift, res, t), dict(relu=1, **kw), ALGO["auto"], "halo=3")
            assert C > 64 or "b_res=1" in desc, desc        # (at 128 channels they need not fit beside the ring)
    with binding.plan_hints(halo=0):
        _compare((x, w, bias, shift), dict(relu=1, **kw), ALGO["auto"], "halo=0")

"""GPU parity on seeded random layer shapes: every planner branch of the tensor-core path
(flat / strided view / box / window rows / space-to-depth and patch-row stems; folded rows,
resident weights, staged TMA stores with and without a residual, concat windows, partial
batches) against the CPU oracle, bit for bit."""
import numpy as np
import pytest

from oracle import ref
from tests.helpers import oracle_conv, rand_layer

pytestmark = pytest.mark.gpu


def _random_case(rng):
    kind = rng.choice(["1x1", "1x1s2", "3x3", "5x5", "wide", "stem2", "stem1"])
    N = int(rng.integers(1, 5))
    H, W = int(rng.integers(5, 41)), int(rng.integers(5, 41))
    C = int(rng.choice([16, 32, 48, 64, 96, 128, 256]))
    K = int(rng.choice([8, 16, 24, 32, 64, 100, 128, 200, 256]))
    stride, R, S = (1, 1), 1, 1
    if kind == "1x1s2":
        stride = (2, 2)
    elif kind == "3x3":
        R = S = 3
    elif kind == "5x5":
        R = S = 5
        C = int(rng.choice([16, 32, 48, 64, 96]))
    elif kind == "wide":
        R, S = int(rng.choice([1, 3])), int(rng.choice([4, 5, 7]))
        C = int(rng.choice([16, 32, 64]))
    elif kind == "stem2":
        C, R, stride = int(rng.integers(1, 5)), int(rng.choice([3, 5, 7])), (2, 2)
        S = R
    elif kind == "stem1":
        C, R = int(rng.integers(1, 5)), int(rng.choice([3, 5]))
        S = R
    pad = (int(rng.integers(0, R // 2 + 1)), int(rng.integers(0, S // 2 + 1)))
    if H + 2 * pad[0] < R or W + 2 * pad[1] < S:
        H, W = H + R, W + S
    return kind, N, H, W, C, K, R, S, stride, pad


def _strided_case(rng):
    """3x3 / 5x5 (also non-square) filters with stride 2 in one or both directions on C % 16 == 0."""
    N = int(rng.integers(1, 5))
    H, W = int(rng.integers(6, 41)), int(rng.integers(6, 41))
    C = int(rng.choice([16, 32, 64, 128, 256]))
    K = int(rng.choice([16, 24, 64, 128, 200, 256]))
    R, S = int(rng.choice([2, 3, 5])), int(rng.choice([2, 3, 5]))
    stride = [(2, 2), (2, 2), (1, 2), (2, 1)][int(rng.integers(0, 4))]
    pad = (int(rng.integers(0, R // 2 + 1)), int(rng.integers(0, S // 2 + 1)))
    return "3x3s2", N, H, W, C, K, R, S, stride, pad


@pytest.mark.parametrize("seed", range(72))
def test_random_layer_matches_the_oracle(seed):
    import torch
    from paper_1805_07941_b200 import binding
    rng = np.random.default_rng(1000 + seed)
    kind, N, H, W, C, K, R, S, stride, pad = _random_case(rng) if seed < 48 else _strided_case(rng)
    with_res = bool(rng.integers(0, 2))
    per_channel = bool(rng.integers(0, 2))
    relu = int(rng.integers(0, 2))
    x, w, bias, shift, res, t = rand_layer(rng, N, H, W, C, K, R, S, with_res=with_res, stride=stride, pad=pad,
                                          per_channel_shift=per_channel)
    if with_res and not per_channel:
        t = np.full(K, int(t[0]), np.int32)
    if rng.integers(0, 3) == 0:                              # small weights: the float-rounding epilogue
        w = (w // 16).astype(np.int8)
        shift = np.maximum(shift - 4, 0).astype(np.int32)
        if with_res:
            t = np.minimum(t, 5).astype(np.int32)
    concat = K % 16 == 0 and rng.integers(0, 3) == 0
    off, pitch = (16, K + 48) if concat else (0, 0)
    n_run = N if rng.integers(0, 3) else max(1, N - 1)
    kw = dict(R=R, S=S, stride=stride, pad=pad, relu=relu, out_c_offset=off, out_c_pitch=pitch)
    want = oracle_conv(x[:n_run], w, bias, shift, None if res is None else res[:n_run], t, **kw)
    n_w, packed = 8, False
    if seed % 4 == 3:
        # kind "w5bit": weights of 5 to 7 bits (Section 4.3), handed over as a packed bit stream
        n_w, packed = int(5 + seed % 3), True
        w = (w.astype(np.int32) >> (8 - n_w)).astype(np.int8)
        want = oracle_conv(x[:n_run], w, bias, shift, None if res is None else res[:n_run], t, **kw)
    conv = binding.QConv(binding.qpack_weights(w, n_w) if packed else w, bias, shift, t, None, packed=packed, n_w=n_w,
                         N=N, H=H, W=W, C=C, K=K, R=R, S=S, stride_h=stride[0],
                         stride_w=stride[1], pad_h=pad[0], pad_w=pad[1], relu=relu, out_c_offset=off,
                         out_c_pitch=pitch, has_residual=int(res is not None))
    P, Q = ref.out_hw(H, W, R, S, stride[0], stride[1], pad[0], pad[1])
    y = torch.full((N, P, Q, pitch or K), 77, dtype=torch.int8, device="cuda")
    rd = None if res is None else torch.from_numpy(res).cuda()
    for _ in range(2):                                       # twice: cached tensor maps, ring phases
        conv.run(torch.from_numpy(x).cuda(), y, rd, n_run=n_run)
    assert conv.status() == 0, conv.describe()
    got = y.cpu().numpy()
    assert (got[:n_run] == want).all(), (kind, conv.describe(), (N, H, W, C, K, R, S, stride, pad, n_run))
    if kind == "3x3s2":
        assert "igemm/box" in conv.describe(), conv.describe()
    assert (got[n_run:] == 77).all(), "images beyond n_run were written"
    conv_desc = conv.describe()
    conv.destroy()
    # kind "pool": the same layer with the 2 x 2 max-pool behind it taken inside the layer, where the library offers that
    if "igemm/box" in conv_desc and not with_res and not packed and P % 2 == 0 and Q % 2 == 0 and K % 16 == 0:
        pc = binding.QConv(w, bias, shift, None, None, N=N, H=H, W=W, C=C, K=K, R=R, S=S, stride_h=stride[0],
                           stride_w=stride[1], pad_h=pad[0], pad_w=pad[1], relu=relu, out_c_offset=off, out_c_pitch=pitch, pool=2)
        assert "pool=2" in pc.describe()
        yp = torch.full((N, P // 2, Q // 2, pitch or K), 77, dtype=torch.int8, device="cuda")
        pc.run(torch.from_numpy(x).cuda(), yp, n_run=n_run)
        assert pc.status() == 0, pc.describe()
        gp = yp.cpu().numpy()
        wp = ref.maxpool_i8(np.ascontiguousarray(want[..., off:off + K]), 2, 2, 2, 0)
        assert (gp[:n_run, :, :, off:off + K] == wp).all(), (pc.describe(), (N, H, W, C, K, R, S, stride, pad, n_run))
        if pitch:
            assert (gp[..., :off] == 77).all() and (gp[..., off + K:] == 77).all()
        assert (gp[n_run:] == 77).all()
        pc.destroy()

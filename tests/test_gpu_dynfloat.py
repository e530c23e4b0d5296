"""float <-> (n, p) dynamic floating-point codes on the GPU against the oracle (bit-exact)."""
import numpy as np
import pytest

from oracle import dynfloat as df
from paper_1805_07941_b200 import binding

pytestmark = pytest.mark.gpu

FORMATS = [(8, 7, -3), (8, 6, 0), (8, 4, -6), (8, 3, -9), (8, 2, -16), (8, 1, -30), (8, 0, -40), (6, 3, 2), (5, 4, -1),
           (4, 1, 0), (2, 1, 0), (3, 0, -2), (8, 4, 100), (8, 3, -120)]


def _inputs(n, p, e, count, seed):
    rng = np.random.default_rng(seed)
    top = float(df.beta_max_closed_form(n, p)) * 2.0 ** e
    x = np.concatenate([rng.normal(size=count) * top / 3, rng.uniform(-1.3, 1.3, count) * top,
                        rng.normal(size=count // 4) * 2.0 ** (e + 1)]).astype(np.float32)
    vals = df.nonneg_values_f64(n, p) * 2.0 ** e
    mids = ((vals[:-1] + vals[1:]) / 2).astype(np.float32)          # every tie, and one float either side
    special = np.array([0.0, -0.0, np.inf, -np.inf, np.nan, top, -top, np.float32(top) * 2], dtype=np.float32)
    return np.concatenate([x, mids, -mids, np.nextafter(mids, np.float32(0)), np.nextafter(mids, np.float32(np.inf)),
                           special]).astype(np.float32)


@pytest.mark.parametrize("n,p,e", FORMATS)
def test_encode_matches_oracle(n, p, e):
    import torch
    x = _inputs(n, p, e, 40000, n * 100 + p)
    want = df.quantize_np(x, e, n, p)
    got = binding.qquantize_f32_np(torch.from_numpy(x).cuda(), e, n, p).cpu().numpy()
    assert np.array_equal(got, want)
    # ragged length and a misaligned view take the scalar path
    got2 = binding.qquantize_f32_np(torch.from_numpy(x).cuda()[3:1000], e, n, p).cpu().numpy()
    assert np.array_equal(got2, want[3:1000])


@pytest.mark.parametrize("n,p,e", FORMATS)
def test_decode_matches_oracle_and_round_trips(n, p, e):
    import torch
    codes = np.tile(np.arange(1 << n, dtype=np.uint8), 9)[:-5]
    want = df.dequantize_np(codes, e, n, p)
    got = binding.qdequantize_np(torch.from_numpy(codes).cuda(), e, n, p)
    assert np.array_equal(got.cpu().numpy(), want)
    back = binding.qquantize_f32_np(got, e, n, p).cpu().numpy()
    keep = (codes & ((1 << (n - 1)) - 1)) != 0
    assert np.array_equal(back[keep], codes[keep]) and np.all(back[~keep] == 0)


def test_int8_special_case_agrees_with_the_integer_quantizer():
    # (8, 7) codes are sign-magnitude; the convolution path's quantizer writes the same values as two's complement
    import torch
    x = torch.randn(1 << 16, device="cuda") * 3
    e = -5
    sm = binding.qquantize_f32_np(x, e, 8, 7).cpu().numpy()
    tc = binding.qquantize_f32(x, e, 8).cpu().numpy()
    val = np.where(sm & 0x80, -(sm & 0x7F).astype(np.int32), (sm & 0x7F).astype(np.int32))
    assert np.array_equal(val, tc.astype(np.int32))


def test_argument_errors():
    import torch
    x = torch.zeros(16, device="cuda")
    y = torch.zeros(16, dtype=torch.uint8, device="cuda")
    L = binding.lib()
    assert L.qquantize_f32_np(x.data_ptr(), 16, 0, 9, 3, y.data_ptr(), None) == binding.ERR_BAD_ARG
    assert L.qquantize_f32_np(x.data_ptr(), 16, 0, 8, 8, y.data_ptr(), None) == binding.ERR_BAD_ARG
    assert L.qquantize_f32_np(x.data_ptr(), 16, 200, 8, 4, y.data_ptr(), None) == binding.ERR_BAD_ARG
    assert L.qdequantize_np(None, 16, 0, 8, 4, x.data_ptr(), None) == binding.ERR_BAD_ARG

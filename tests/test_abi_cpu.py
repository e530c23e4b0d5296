"""CPU-only checks of the boundary: the CUDA library loads, exports every symbol the
header declares, and its pure-host helpers agree with the oracle bit for bit.  No compute
call that needs a GPU is made here."""
import ctypes
import re

import numpy as np
import pytest

from oracle import ref
from paper_1805_07941_b200 import binding


@pytest.fixture(scope="module")
def lib():
    binding.build_library()
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    text = open(binding.HEADER_PATH).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(q[a-z0-9_]+)\s*\(", text)
    assert set(names) >= {"qconv_create", "qconv_run", "qcalib_collect", "qconv_status", "qconv_destroy",
                          "qquantize_f32", "qmaxpool_i8", "qscale_exponent", "qquantize_weights"}
    for n in set(names):
        assert hasattr(lib, n), n


def test_descriptor_struct_matches_header():
    text = open(binding.HEADER_PATH).read()
    body = re.search(r"typedef struct \{(.*?)\} qconv_desc;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = [f.strip() for decl in re.findall(r"int ([^;]+);", body) for f in decl.split(",")]
    assert fields == [f for f, _ in binding.qconv_desc._fields_]


def test_plan_hints_struct_matches_header(lib):
    text = open(binding.HEADER_PATH).read()
    body = re.search(r"typedef struct \{((?:(?!typedef).)*?)\} qconv_plan_hints;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = [f.strip() for decl in re.findall(r"int ([^;]+);", body) for f in decl.split(",")]
    assert fields == [f for f, _ in binding.qconv_plan_hints._fields_]
    with binding.plan_hints(halo=0, bn_max=64):
        pass
    with pytest.raises(TypeError):
        binding.plan_hints(no_such_form=1)


def test_exponent_bookkeeping_helpers_against_exact_integers(lib):
    """Section 3 with alpha = 2^e: s[k] = e_z - (e_x + e_w[k]) in [0, 31], t[k] = e_res - (e_x + e_w[k])
    in [0, 23], and a join takes the largest exponent any branch needs."""
    rng = np.random.default_rng(3)
    for _ in range(50):
        K = int(rng.integers(1, 40))
        e_x = int(rng.integers(-12, 4))
        e_w = rng.integers(-14, -2, K).astype(np.int32)
        acc = binding.qacc_exponents(e_x, e_w)
        assert acc.tolist() == [e_x + int(v) for v in e_w]
        e_z = int(acc.max()) + int(rng.integers(0, 10))
        assert binding.qrequant_shifts(e_z, acc).tolist() == [e_z - int(a) for a in acc]
        e_res = int(acc.max()) + int(rng.integers(0, 6))
        assert binding.qresidual_shifts(e_res, acc).tolist() == [e_res - int(a) for a in acc]
        # powers of two: alpha_x alpha_w / alpha_z = 2^-s exactly, and alpha_res / (alpha_x alpha_w) = 2^t
        for a, sft in zip(acc, binding.qrequant_shifts(e_z, acc)):
            assert 2.0 ** int(a) / 2.0 ** e_z == 2.0 ** -int(sft)
        nb = int(rng.integers(1, 5))
        accs = [rng.integers(-20, -5, int(rng.integers(1, 9))).astype(np.int32) for _ in range(nb)]
        own = rng.integers(-22, -3, nb).astype(np.int32)
        want = max(int(own.max()), max(int(a.max()) for a in accs))
        assert binding.qjoin_exponent(own, accs) == want
    acc = np.int32([-10, -12])
    with pytest.raises(binding.QconvError) as e:
        binding.qrequant_shifts(-11, acc)                   # a factor above 1: negative shift
    assert e.value.code == binding.ERR_BAD_SHIFT
    with pytest.raises(binding.QconvError) as e:
        binding.qrequant_shifts(21, acc)                    # 21 - (-12) = 33 > 31
    assert e.value.code == binding.ERR_BAD_SHIFT
    with pytest.raises(binding.QconvError) as e:
        binding.qresidual_shifts(-11, acc)                  # residual finer than the accumulator
    assert e.value.code == binding.ERR_RESIDUAL_SCALE
    with pytest.raises(binding.QconvError) as e:
        binding.qresidual_shifts(14, acc)                   # 14 + 12 = 26 > 23
    assert e.value.code == binding.ERR_RESIDUAL_SCALE


def test_argument_errors_without_gpu(lib):
    h = ctypes.c_void_p()
    d = binding.qconv_desc(N=1, H=4, W=4, C=6, K=4, R=3, S=3, stride_h=1, stride_w=1, groups=4, n_in=8,
                           n_w=8, n_out=8)
    w = np.zeros(1000, np.int8)
    wp = ctypes.c_void_p(w.ctypes.data)
    assert lib.qconv_create(ctypes.byref(h), ctypes.byref(d), wp, None, None, None, None) == \
        binding.ERR_UNSUPPORTED_SHAPE
    assert b"groups" in lib.qconv_last_error_string()
    d.groups = 1
    assert lib.qconv_create(ctypes.byref(h), None, wp, None, None, None, None) == binding.ERR_BAD_ARG
    d.n_out = 9
    assert lib.qconv_create(ctypes.byref(h), ctypes.byref(d), wp, None, None, None, None) == binding.ERR_BAD_ARG
    d.n_out = 8
    bad = np.array([0, 32, 0, 0], np.int32)
    assert lib.qconv_create(ctypes.byref(h), ctypes.byref(d), wp, None, ctypes.c_void_p(bad.ctypes.data),
                            None, None) == binding.ERR_BAD_SHIFT
    neg = np.array([0, -1, 0, 0], np.int32)
    assert lib.qconv_create(ctypes.byref(h), ctypes.byref(d), wp, None, ctypes.c_void_p(neg.ctypes.data),
                            None, None) == binding.ERR_BAD_SHIFT      # factors must stay in (0, 1]
    d.has_residual = 1
    t = np.array([0, 0, 24, 0], np.int32)
    assert lib.qconv_create(ctypes.byref(h), ctypes.byref(d), wp, None, None,
                            ctypes.c_void_p(t.ctypes.data), None) == binding.ERR_RESIDUAL_SCALE
    d.has_residual = 0
    # Eq. 9: a dot product longer than floor((2^31 - 1) / 128^2) = 131071 terms may overflow int32
    big = binding.qconv_desc(N=1, H=1, W=1, C=131072, K=1, R=1, S=1, stride_h=1, stride_w=1, groups=1,
                             n_in=8, n_w=8, n_out=8)
    wbig = np.zeros(131072, np.int8)
    assert lib.qconv_create(ctypes.byref(h), ctypes.byref(big), ctypes.c_void_p(wbig.ctypes.data), None, None,
                            None, None) == binding.ERR_OVERFLOW_RISK
    assert not h.value


def test_scale_exponent_matches_oracle_exactly():
    rng = np.random.default_rng(0)
    gammas = np.concatenate([np.exp(rng.uniform(-30, 30, 3000)).astype(np.float32),
                             np.float32([0, 127, 1, 63.5, 254, 1e-38, 3e38, np.inf, np.nan, -1])])
    for n in (2, 5, 8):
        bm = 2 ** (n - 1) - 1
        edge = [np.float32(bm * 2.0 ** e) for e in range(-30, 31)]
        edge += [np.nextafter(v, np.float32(0)) for v in edge] + [np.nextafter(v, np.float32(np.inf)) for v in edge]
        for g in list(gammas) + edge:
            assert binding.qscale_exponent(float(g), n) == ref.scale_exponent(float(g), n), (g, n)


def test_weight_and_bias_quantization_match_oracle_exactly():
    rng = np.random.default_rng(1)
    for layout in (0, 1):
        for per_channel in (0, 1):
            K, R, S, Cg = 7, 3, 2, 5
            w = (rng.standard_normal(K * R * S * Cg) * np.exp(rng.uniform(-6, 3, K * R * S * Cg))).astype(np.float32)
            w[3] = np.nan
            w[5] = np.inf
            a, ea = binding.qquantize_weights(w, K, R, S, Cg, layout, per_channel, 8)
            b, eb = ref.quantize_weights(w, K=K, R=R, S=S, Cg=Cg, layout=layout, per_channel=per_channel, n=8)
            assert (a == b).all() and (ea == eb).all()
    b = (rng.standard_normal(64) * 10).astype(np.float32)
    e_w = rng.integers(-12, -2, 64).astype(np.int32)
    assert (binding.qquantize_bias(b, -5, e_w) == ref.quantize_bias(b, -5, e_w)).all()


def test_fpspace_helper_equals_the_oracle_value_set(lib):
    from oracle import threshold_ref
    for n in range(2, 9):
        for p in range(0, n):
            got = binding.qfpspace(n, p)
            want = threshold_ref.fpspace(0.0, 1.0, n, p)
            assert got.shape == want.shape and np.array_equal(got, want), (n, p)


def test_threshold_search_argument_errors_without_gpu(lib):
    g, d, i = ctypes.c_double(), ctypes.c_double(), ctypes.c_int()
    h = np.ones(200, np.uint64)
    hp = ctypes.c_void_p(h.ctypes.data)
    call = lambda *a: lib.qthreshold_search(*a, ctypes.byref(g), ctypes.byref(d), ctypes.byref(i), None, None)
    assert call(None, 200, 1.0, 8, 7, 0) == binding.ERR_BAD_ARG
    assert call(hp, 128, 1.0, 8, 7, 0) == binding.ERR_BAD_ARG          # fewer bins than the first candidate
    assert call(hp, 5000, 1.0, 8, 7, 0) == binding.ERR_BAD_ARG
    assert call(hp, 200, 0.0, 8, 7, 0) == binding.ERR_BAD_ARG
    assert call(hp, 200, 1.0, 8, 8, 0) == binding.ERR_BAD_ARG          # p <= n-1
    assert call(hp, 200, 1.0, 8, 7, 4) == binding.ERR_BAD_ARG
    z = np.zeros(200, np.uint64)
    assert call(ctypes.c_void_p(z.ctypes.data), 200, 1.0, 8, 7, 0) == binding.ERR_BAD_ARG
    assert b"empty" in lib.qconv_last_error_string()


def test_packed_weight_helpers_match_the_oracle(lib):
    rng = np.random.default_rng(9)
    for n in range(2, 9):
        w = rng.integers(-(1 << (n - 1)), 1 << (n - 1), size=1237).astype(np.int8)
        packed = binding.qpack_weights(w, n)
        assert np.array_equal(packed, ref.pack_bits(w, n))
        assert np.array_equal(binding.qunpack_weights(packed, w.size, n), w)
        assert np.array_equal(binding.qunpack_weights(packed, w.size, n), ref.unpack_bits(packed, w.size, n))
    with pytest.raises(binding.QconvError) as e:
        binding.qpack_weights(np.int8([0, 16]), 5)           # 16 needs six bits
    assert e.value.code == binding.ERR_BAD_ARG

"""TEST INFRASTRUCTURE, NOT PRODUCT CODE.

numpy-facing wrapper around the plain C oracle in qconv_ref.c.  It builds the
shared object with gcc on first use and marshals arrays; it adds no arithmetic.
Only tests, the smoke check and the CPU-baseline timing may import this module.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qconv_ref.c")
_LIB = os.path.join(_HERE, "libqconv_oracle.so")
_lib = None

_i8p = ctypes.POINTER(ctypes.c_int8)
_i32p = ctypes.POINTER(ctypes.c_int32)
_f32p = ctypes.POINTER(ctypes.c_float)
_u64p = ctypes.POINTER(ctypes.c_uint64)
_f64p = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile qconv_ref.c into libqconv_oracle.so beside it (gcc, OpenMP)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
                               _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_round_shift.restype = ctypes.c_int64
        _lib.oracle_round_shift.argtypes = [ctypes.c_int64, ctypes.c_int, ctypes.c_int]
        _lib.oracle_scale_exponent.restype = ctypes.c_int
        _lib.oracle_scale_exponent.argtypes = [ctypes.c_float, ctypes.c_int]
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def _ptr(a, typ):
    if a is None:
        return ctypes.cast(None, typ)
    return a.ctypes.data_as(typ)


def _c(a, dtype):
    if a is None:
        return None
    return np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def round_shift(acc: int, s: int, mode: int = 0) -> int:
    return int(lib().oracle_round_shift(int(acc), int(s), int(mode)))


def out_hw(H, W, R, S, stride_h, stride_w, pad_h, pad_w):
    return (H + 2 * pad_h - R) // stride_h + 1, (W + 2 * pad_w - S) // stride_w + 1


_OUT_DTYPES = {0: np.int8, 1: np.int32, 2: np.float32}


def qconv(x, w, bias=None, shift=None, res=None, res_lshift=None, acc_exp=None, *,
          R, S, stride=(1, 1), pad=(0, 0), groups=1, n_out=8, symmetric=1, relu=0,
          rounding=0, out_mode=0, weight_layout=0, K=None, out=None, out_c_offset=0):
    """x int8 [N,H,W,C]; w int8 in layout 0 [K,R,S,C/g] or 1 [R,S,C/g,K].
    Returns y [N,P,Q,K] (or writes the K channels into `out` at out_c_offset)."""
    x = _c(x, np.int8)
    w = _c(w, np.int8)
    N, H, W, C = x.shape
    if K is None:
        K = w.shape[0] if weight_layout == 0 else w.shape[3]
    assert w.size == K * R * S * (C // groups)
    P, Q = out_hw(H, W, R, S, stride[0], stride[1], pad[0], pad[1])
    bias = _c(bias, np.int32)
    shift = _c(shift, np.int32)
    res = _c(res, np.int8)
    res_lshift = _c(res_lshift, np.int32)
    acc_exp = _c(acc_exp, np.int32)
    if res is not None:
        assert res.shape == (N, P, Q, K) and res_lshift is not None
    if out is None:
        y = np.zeros((N, P, Q, K), dtype=_OUT_DTYPES[out_mode])
    else:
        y = out
        assert y.flags.c_contiguous and y.dtype == _OUT_DTYPES[out_mode] and y.shape[:3] == (N, P, Q)
    pitch = y.shape[3]
    lib().oracle_qconv(
        _ptr(x, _i8p), _ptr(w, _i8p), _ptr(bias, _i32p), _ptr(shift, _i32p), _ptr(res, _i8p),
        _ptr(res_lshift, _i32p), _ptr(acc_exp, _i32p), ctypes.c_void_p(y.ctypes.data),
        *[ctypes.c_int(int(v)) for v in (N, H, W, C, K, R, S, stride[0], stride[1], pad[0], pad[1],
                                         groups, n_out, symmetric, relu, rounding, out_mode,
                                         out_c_offset, pitch, weight_layout)])
    return y


def qconv_points(x, w, points, bias=None, shift=None, res=None, res_lshift=None, acc_exp=None, *,
                 R, S, stride=(1, 1), pad=(0, 0), groups=1, n_out=8, symmetric=1, relu=0,
                 rounding=0, out_mode=0, weight_layout=0, K=None):
    """The layer evaluated only at `points` (int32 [npoints, 4] rows n, p, q, k)."""
    x = _c(x, np.int8)
    w = _c(w, np.int8)
    N, H, W, C = x.shape
    if K is None:
        K = w.shape[0] if weight_layout == 0 else w.shape[3]
    points = _c(points, np.int32)
    out = np.zeros(points.shape[0], dtype=_OUT_DTYPES[out_mode])
    bias = _c(bias, np.int32)
    shift = _c(shift, np.int32)
    res = _c(res, np.int8)
    res_lshift = _c(res_lshift, np.int32)
    acc_exp = _c(acc_exp, np.int32)
    lib().oracle_qconv_points(
        _ptr(x, _i8p), _ptr(w, _i8p), _ptr(bias, _i32p), _ptr(shift, _i32p), _ptr(res, _i8p),
        _ptr(res_lshift, _i32p), _ptr(acc_exp, _i32p), ctypes.c_void_p(out.ctypes.data),
        _ptr(points, _i32p), ctypes.c_size_t(points.shape[0]),
        *[ctypes.c_int(int(v)) for v in (N, H, W, C, K, R, S, stride[0], stride[1], pad[0], pad[1],
                                         groups, n_out, symmetric, relu, rounding, out_mode,
                                         weight_layout)])
    return out


def scale_exponent(gamma: float, n: int = 8) -> int:
    return int(lib().oracle_scale_exponent(ctypes.c_float(float(gamma)), int(n)))


def quantize_f32(x, e: int, n: int = 8):
    x = _c(x, np.float32)
    y = np.zeros(x.shape, dtype=np.int8)
    lib().oracle_quantize_f32(_ptr(x, _f32p), ctypes.c_size_t(x.size), ctypes.c_int(int(e)),
                              ctypes.c_int(int(n)), _ptr(y, _i8p))
    return y


def quantize_weights(w, *, K, R, S, Cg, layout=0, per_channel=1, n=8):
    w = _c(w, np.float32)
    assert w.size == K * R * S * Cg
    wq = np.zeros(w.shape, dtype=np.int8)
    e_w = np.zeros(K, dtype=np.int32)
    lib().oracle_quantize_weights(_ptr(w, _f32p), *[ctypes.c_int(int(v)) for v in
                                                     (K, R, S, Cg, layout, per_channel, n)],
                                  _ptr(wq, _i8p), _ptr(e_w, _i32p))
    return wq, e_w


def quantize_bias(b, e_x: int, e_w):
    b = _c(b, np.float32)
    e_w = _c(e_w, np.int32)
    bq = np.zeros(b.shape, dtype=np.int32)
    lib().oracle_quantize_bias(_ptr(b, _f32p), ctypes.c_int(b.size), ctypes.c_int(int(e_x)),
                               _ptr(e_w, _i32p), _ptr(bq, _i32p))
    return bq


def calib_stats(x, nbins: int = 2048, range_hi: float = 0.0):
    x = _c(x, np.float32).reshape(-1)
    hist = np.zeros(nbins, dtype=np.uint64)
    maxabs = ctypes.c_float(0)
    finite = ctypes.c_uint64(0)
    nonfinite = ctypes.c_uint64(0)
    s = ctypes.c_double(0)
    ss = ctypes.c_double(0)
    lib().oracle_calib_stats(_ptr(x, _f32p), ctypes.c_size_t(x.size), ctypes.c_int(nbins),
                             ctypes.c_float(float(range_hi)), ctypes.byref(maxabs),
                             _ptr(hist, _u64p), ctypes.byref(finite), ctypes.byref(nonfinite),
                             ctypes.byref(s), ctypes.byref(ss))
    return dict(maxabs=np.float32(maxabs.value), hist=hist, count=int(finite.value),
                nonfinite=int(nonfinite.value), sum=float(s.value), sumsq=float(ss.value))


def maxpool_i8(x, R, S, stride, pad):
    x = _c(x, np.int8)
    N, H, W, C = x.shape
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    y = np.zeros((N, P, Q, C), dtype=np.int8)
    lib().oracle_maxpool_i8(_ptr(x, _i8p), _ptr(y, _i8p), *[ctypes.c_int(int(v)) for v in
                                                             (N, H, W, C, R, S, stride, pad)])
    return y


def eltwise_add(inputs, lshift, rshift, relu=0, rounding=0, n_out=8, symmetric=1):
    """Sum of int8 tensors with per-input scales (Eq. 10); inputs: list of equal-shape int8 arrays."""
    arrs = [_c(a, np.int8) for a in inputs]
    ptrs = (_i8p * len(arrs))(*[_ptr(a, _i8p) for a in arrs])
    lshift = _c(lshift, np.int32)
    y = np.zeros(arrs[0].shape, dtype=np.int8)
    lib().oracle_eltwise_add(ptrs, ctypes.c_int(len(arrs)), _ptr(lshift, _i32p), ctypes.c_int(int(rshift)),
                             ctypes.c_int(int(relu)), ctypes.c_int(int(rounding)), ctypes.c_int(int(n_out)),
                             ctypes.c_int(int(symmetric)), ctypes.c_size_t(arrs[0].size), _ptr(y, _i8p))
    return y


# ---------------------------------------------------------------------------------------------
# Packed storage of n-bit betas (Section 4.3 scales the weights down to 5 bits): value i occupies bits
# [i*n, (i+1)*n) of a little-endian bit stream, as an n-bit two's-complement field.  Plain loops.
# Pinned in tests/test_oracle_quant.py: a hand-written byte string, the round trip over every value of
# every width, and the length ceil(count * n / 8).
# ---------------------------------------------------------------------------------------------
def pack_bits(values, n: int):
    values = np.asarray(values, dtype=np.int64).reshape(-1)
    assert 2 <= n <= 8 and ((values >= -(1 << (n - 1))) & (values < (1 << (n - 1)))).all()
    out = np.zeros((values.size * n + 7) // 8, dtype=np.uint8)
    for i, v in enumerate(values):
        field = int(v) & ((1 << n) - 1)
        for b in range(n):
            if (field >> b) & 1:
                pos = i * n + b
                out[pos // 8] |= 1 << (pos % 8)
    return out


def unpack_bits(packed, count: int, n: int):
    packed = np.asarray(packed, dtype=np.uint8).reshape(-1)
    out = np.zeros(count, dtype=np.int8)
    for i in range(count):
        field = 0
        for b in range(n):
            pos = i * n + b
            field |= ((int(packed[pos // 8]) >> (pos % 8)) & 1) << b
        out[i] = field - (1 << n) if field >> (n - 1) else field
    return out

"""Thin ctypes binding of the C ABI in include/qconv.h.

Argument marshalling only: every function forwards torch tensors' device
pointers (or numpy host arrays) to the CUDA library; no arithmetic of the
method happens here.  The shared object is built in-tree by `build_library()`
(nvcc, sm_100a) and loading fails loudly if it is missing -- there is no CPU
fallback.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_HERE, "csrc")
LIB_PATH = os.path.join(_HERE, "libqconv_b200.so")
CHECKED_LIB_PATH = os.path.join(_HERE, "libqconv_b200_checked.so")     # -DQCONV_CHECKED build (index tests in the CUDA-core kernels)
HEADER_PATH = os.path.join(os.path.dirname(_HERE), "include", "qconv.h")

QCONV_OK = 0
ERR_BAD_ARG, ERR_UNSUPPORTED_SHAPE, ERR_OVERFLOW_RISK, ERR_BAD_SHIFT = -1, -2, -3, -4
ERR_RESIDUAL_SCALE, ERR_ALIGNMENT, ERR_CUDA, ERR_TIMEOUT = -5, -6, -7, -8
ALGO_AUTO, ALGO_DIRECT, ALGO_IGEMM, ALGO_DEPTHWISE = 0, 1, 2, 3
OUT_INT8, OUT_INT32, OUT_FLOAT = 0, 1, 2


class QconvError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__("qconv error %d: %s" % (code, msg))
        self.code = code


class qconv_desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in (
        "N", "H", "W", "C", "K", "R", "S", "stride_h", "stride_w", "pad_h", "pad_w", "groups",
        "n_in", "n_w", "n_out", "symmetric", "relu", "rounding", "out_mode", "out_c_offset",
        "out_c_pitch", "has_residual", "weight_layout", "algo", "pool")]


class qconv_plan_hints(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in (
        "halo", "window_rows", "space_to_depth", "resident_weights", "fold", "fast_epilogue",
        "float_rounding", "uniform_shift", "tma_store", "tma_residual", "depthwise_form", "pdl",
        "group_taps", "pair_tiles", "bn_max", "ctas_per_sm")]


class qconv_np_desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in (
        "N", "H", "W", "C", "K", "R", "S", "stride_h", "stride_w", "pad_h", "pad_w",
        "n_in", "p_in", "n_w", "p_w", "n_out", "p_out", "relu")]


class qcalib_stats(ctypes.Structure):
    _fields_ = [("maxabs", ctypes.c_float), ("range_hi", ctypes.c_float),
                ("count", ctypes.c_uint64), ("nonfinite", ctypes.c_uint64),
                ("sum", ctypes.c_double), ("sumsq", ctypes.c_double),
                ("hist", ctypes.POINTER(ctypes.c_uint64))]


def sources():
    return [os.path.join(_CSRC, f) for f in sorted(os.listdir(_CSRC)) if f.endswith((".cu", ".cuh"))] + \
        [HEADER_PATH]


def build_library(force=False, verbose=False, checked=False):
    """Compile csrc/qconv_api.cu for sm_100a into libqconv_b200.so beside this file (checked=True: the
    -DQCONV_CHECKED variant, libqconv_b200_checked.so; load it by setting LIB_PATH before the first lib())."""
    srcs = sources()
    path = CHECKED_LIB_PATH if checked else LIB_PATH
    stale = (not os.path.exists(path)) or any(os.path.getmtime(s) > os.path.getmtime(path) for s in srcs)
    if not (force or stale):
        return path
    tmp = path + ".tmp%d" % os.getpid()
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-o", tmp, os.path.join(_CSRC, "qconv_api.cu")]
    if checked:
        cmd.insert(1, "-DQCONV_CHECKED")
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.check_call(cmd)
    os.replace(tmp, path)
    return path


_lib = None


def lib():
    """The loaded CUDA library.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("CUDA library %s is missing: run paper_1805_07941_b200.binding."
                              "build_library() (needs nvcc); there is no CPU fallback" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, ci, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        L.qconv_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(qconv_desc), vp, vp, vp, vp, vp]
        L.qconv_run.argtypes = [vp, vp, vp, vp, ci, vp]
        L.qconv_run_f32.argtypes = [vp, vp, ci, vp, vp, ci, vp]
        L.qconv_run_f32.restype = ci
        L.qconv_status.argtypes = [vp]
        L.qconv_set_wait_limit.argtypes = [vp, ctypes.c_uint]
        L.qconv_describe.argtypes = [vp, ctypes.c_char_p, sz]
        L.qconv_destroy.argtypes = [vp]
        L.qcalib_collect.argtypes = [vp, sz, ci, ctypes.c_float, ctypes.POINTER(qcalib_stats), vp]
        L.qcalib_collect_static.argtypes = [vp, sz, ci, ctypes.c_float, ctypes.POINTER(qcalib_stats), vp]
        L.qcalib_collect_static.restype = ci
        L.qeltwise_add_i8.argtypes = [vp, ci, vp, ci, ci, ci, ci, ci, sz, vp, vp]
        L.qeltwise_add_i8.restype = ci
        L.qthreshold_search.argtypes = [vp, ci, ctypes.c_float, ci, ci, ci, ctypes.POINTER(ctypes.c_double),
                                        ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ci), vp, vp]
        L.qthreshold_search.restype = ci
        L.qfpspace.argtypes = [ci, ci, vp, ctypes.POINTER(ci)]
        L.qfpspace.restype = ci
        L.qquantize_f32.argtypes = [vp, sz, ci, ci, vp, vp]
        L.qquantize_f32_np.argtypes = [vp, sz, ci, ci, ci, vp, vp]
        L.qquantize_f32_np.restype = ci
        L.qdequantize_np.argtypes = [vp, sz, ci, ci, ci, vp, vp]
        L.qdequantize_np.restype = ci
        L.qmaxpool_i8.argtypes = [vp, ci, ci, ci, ci, ci, ci, ci, ci, vp, vp]
        L.qscale_exponent.argtypes = [ctypes.c_float, ci, ctypes.POINTER(ci)]
        L.qquantize_weights.argtypes = [vp, ci, ci, ci, ci, ci, ci, ci, vp, vp]
        L.qquantize_bias.argtypes = [vp, ci, ci, vp, vp]
        L.qconv_set_plan_hints.argtypes = [ctypes.POINTER(qconv_plan_hints)]
        L.qconv_set_plan_hints.restype = ci
        L.qacc_exponents.argtypes = [ci, vp, ci, vp]
        L.qrequant_shifts.argtypes = [ci, vp, ci, vp]
        L.qresidual_shifts.argtypes = [ci, vp, ci, vp]
        L.qjoin_exponent.argtypes = [vp, vp, vp, ci, ctypes.POINTER(ci)]
        for name in ("qacc_exponents", "qrequant_shifts", "qresidual_shifts", "qjoin_exponent"):
            getattr(L, name).restype = ci
        L.qbench_mma_i8.argtypes = [ci, ci, ci, ci, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_double),
                                    ctypes.POINTER(ci), vp]
        L.qbench_mma_i8.restype = ci
        L.qconv_np_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(qconv_np_desc), vp, vp, vp]
        L.qconv_np_run.argtypes = [vp, vp, vp, ci, vp]
        L.qconv_np_status.argtypes = [vp]
        L.qconv_np_describe.argtypes = [vp, ctypes.c_char_p, sz]
        L.qconv_np_destroy.argtypes = [vp]
        for name in ("qconv_np_create", "qconv_np_run", "qconv_np_status", "qconv_np_describe", "qconv_np_destroy"):
            getattr(L, name).restype = ci
        L.qpack_weights.argtypes = [vp, sz, ci, vp]
        L.qunpack_weights.argtypes = [vp, sz, ci, vp]
        L.qconv_create_packed.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(qconv_desc), vp, vp, vp, vp, vp]
        for name in ("qpack_weights", "qunpack_weights", "qconv_create_packed"):
            getattr(L, name).restype = ci
        L.qconv_checked_faults.argtypes = [ctypes.POINTER(ci)]
        L.qconv_checked_faults.restype = ci
        L.qconv_last_error_string.restype = ctypes.c_char_p
        for name in ("qconv_create", "qconv_run", "qconv_status", "qconv_set_wait_limit", "qconv_describe",
                     "qconv_destroy", "qcalib_collect", "qquantize_f32", "qmaxpool_i8", "qscale_exponent",
                     "qquantize_weights", "qquantize_bias"):
            getattr(L, name).restype = ci
        _lib = L
    return _lib


def _check(code):
    if code != QCONV_OK:
        raise QconvError(code, lib().qconv_last_error_string().decode())


def _host(a, dtype):
    if a is None:
        return None, None
    a = np.ascontiguousarray(a, dtype=dtype)
    return a, ctypes.c_void_p(a.ctypes.data)


def _stream():
    import torch
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else None


class plan_hints:
    """Context manager around qconv_set_plan_hints: layers created inside the block (by this thread)
    are planned with the given overrides, e.g. `with plan_hints(halo=0): conv = QConv(...)`."""

    def __init__(self, **kw):
        vals = {n: (0 if n in ("bn_max", "ctas_per_sm") else -1) for n, _ in qconv_plan_hints._fields_}
        for k in kw:
            if k not in vals:
                raise TypeError("unknown plan hint %r" % k)
        vals.update(kw)
        self.h = qconv_plan_hints(**vals)

    def __enter__(self):
        _check(lib().qconv_set_plan_hints(ctypes.byref(self.h)))
        return self

    def __exit__(self, *exc):
        _check(lib().qconv_set_plan_hints(None))
        return False


class QConv:
    """One layer handle (qconv_create / qconv_run / qconv_status / qconv_destroy)."""

    def __init__(self, w, bias=None, shift=None, res_lshift=None, acc_exp=None, packed=False, **desc):
        """packed=True: w is the packed n_w-bit stream of qpack_weights (qconv_create_packed)."""
        d = dict(stride_h=1, stride_w=1, pad_h=0, pad_w=0, groups=1, n_in=8, n_w=8, n_out=8,
                 symmetric=1, relu=0, rounding=0, out_mode=0, out_c_offset=0, out_c_pitch=0,
                 has_residual=0, weight_layout=0, algo=0, pool=0)
        d.update(desc)
        self.desc = qconv_desc(**d)
        self._keep = [_host(w, np.uint8 if packed else np.int8), _host(bias, np.int32), _host(shift, np.int32),
                      _host(res_lshift, np.int32), _host(acc_exp, np.int32)]
        self.handle = ctypes.c_void_p()
        if packed:
            self._keep[0] = _host(w, np.uint8)
            _check(lib().qconv_create_packed(ctypes.byref(self.handle), ctypes.byref(self.desc),
                                             *[p for _, p in self._keep]))
        else:
            _check(lib().qconv_create(ctypes.byref(self.handle), ctypes.byref(self.desc),
                                      *[p for _, p in self._keep]))
        self._keep = None
        dd = self.desc
        self.P = (dd.H + 2 * dd.pad_h - dd.R) // dd.stride_h + 1
        self.Q = (dd.W + 2 * dd.pad_w - dd.S) // dd.stride_w + 1
        self.K = dd.K
        self.pitch = dd.out_c_pitch or dd.K

    def run(self, x, y, residual=None, n_run=None):
        """x, y, residual: torch CUDA tensors (contiguous).  Asynchronous on the current stream."""
        n = x.shape[0] if n_run is None else n_run
        _check(lib().qconv_run(self.handle, _dev(x), _dev(residual), _dev(y), int(n), _stream()))
        return y

    def run_f32(self, x_f32, e_x, y, residual=None, n_run=None):
        """Float input converted (exponent e_x) inside the layer's packing kernel; stems only."""
        n = x_f32.shape[0] if n_run is None else n_run
        _check(lib().qconv_run_f32(self.handle, _dev(x_f32), int(e_x), _dev(residual), _dev(y), int(n), _stream()))
        return y

    def status(self):
        return lib().qconv_status(self.handle)

    def set_wait_limit(self, polls):
        _check(lib().qconv_set_wait_limit(self.handle, int(polls)))

    def describe(self):
        buf = ctypes.create_string_buffer(256)
        _check(lib().qconv_describe(self.handle, buf, 256))
        return buf.value.decode()

    def destroy(self):
        if self.handle:
            lib().qconv_destroy(self.handle)
            self.handle = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


class QConvNP:
    """One layer on dynamic floating-point operands (qconv_np_create / run / status / destroy): uint8 patterns
    in, uint8 patterns out."""

    def __init__(self, w_codes, bias=None, shift=None, **desc):
        d = dict(stride_h=1, stride_w=1, pad_h=0, pad_w=0, relu=0)
        d.update(desc)
        self.desc = qconv_np_desc(**d)
        keep = [_host(w_codes, np.uint8), _host(bias, np.int32), _host(shift, np.int32)]
        self.handle = ctypes.c_void_p()
        _check(lib().qconv_np_create(ctypes.byref(self.handle), ctypes.byref(self.desc), *[p for _, p in keep]))
        dd = self.desc
        self.P = (dd.H + 2 * dd.pad_h - dd.R) // dd.stride_h + 1
        self.Q = (dd.W + 2 * dd.pad_w - dd.S) // dd.stride_w + 1

    def run(self, x, y, n_run=None):
        n = x.shape[0] if n_run is None else n_run
        _check(lib().qconv_np_run(self.handle, _dev(x), _dev(y), int(n), _stream()))
        return y

    def status(self):
        return lib().qconv_np_status(self.handle)

    def describe(self):
        buf = ctypes.create_string_buffer(400)
        _check(lib().qconv_np_describe(self.handle, buf, 400))
        return buf.value.decode()

    def destroy(self):
        if self.handle:
            lib().qconv_np_destroy(self.handle)
            self.handle = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def qcalib_collect(x, nbins=2048, range_hi=0.0):
    """x: float32 CUDA tensor.  Returns dict(maxabs, range_hi, count, nonfinite, sum, sumsq, hist)."""
    hist = np.zeros(nbins, dtype=np.uint64)
    st = qcalib_stats()
    st.hist = hist.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64))
    _check(lib().qcalib_collect(_dev(x), x.numel(), int(nbins), float(range_hi), ctypes.byref(st), _stream()))
    return dict(maxabs=np.float32(st.maxabs), range_hi=np.float32(st.range_hi), count=int(st.count),
                nonfinite=int(st.nonfinite), sum=float(st.sum), sumsq=float(st.sumsq), hist=hist)


def qcalib_collect_static(x, nbins=2048, range_hi=0.0):
    """qcalib_collect for callers that may not allocate device memory: same arguments and result,
    scratch taken from a fixed array inside the library (nbins <= 4096, count <= 2^40; calls on one
    device must not overlap)."""
    hist = np.zeros(max(int(nbins), 1), dtype=np.uint64)
    st = qcalib_stats()
    st.hist = hist.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64))
    _check(lib().qcalib_collect_static(_dev(x), x.numel(), int(nbins), float(range_hi), ctypes.byref(st),
                                       _stream()))
    return dict(maxabs=np.float32(st.maxabs), range_hi=np.float32(st.range_hi), count=int(st.count),
                nonfinite=int(st.nonfinite), sum=float(st.sum), sumsq=float(st.sumsq), hist=hist)


def qquantize_f32(x, e, n=8, out=None):
    import torch
    y = torch.empty(x.shape, dtype=torch.int8, device=x.device) if out is None else out
    _check(lib().qquantize_f32(_dev(x), x.numel(), int(e), int(n), _dev(y), _stream()))
    return y


def qquantize_f32_np(x, e, n, p, out=None):
    """float32 CUDA tensor -> uint8 codes of the (n, p) dynamic floating-point type at scale 2^e."""
    import torch
    y = torch.empty(x.shape, dtype=torch.uint8, device=x.device) if out is None else out
    _check(lib().qquantize_f32_np(_dev(x), x.numel(), int(e), int(n), int(p), _dev(y), _stream()))
    return y


def qdequantize_np(codes, e, n, p, out=None):
    import torch
    y = torch.empty(codes.shape, dtype=torch.float32, device=codes.device) if out is None else out
    _check(lib().qdequantize_np(_dev(codes), codes.numel(), int(e), int(n), int(p), _dev(y), _stream()))
    return y


def qmaxpool_i8(x, R, S, stride, pad, out=None):
    import torch
    N, H, W, C = x.shape
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    y = torch.empty((N, P, Q, C), dtype=torch.int8, device=x.device) if out is None else out
    _check(lib().qmaxpool_i8(_dev(x), N, H, W, C, R, S, stride, pad, _dev(y), _stream()))
    return y


def qeltwise_add_i8(inputs, lshift, rshift, relu=0, rounding=0, n_out=8, symmetric=1, out=None):
    """Eltwise addition layer: inputs is a list of equal-shape int8 CUDA tensors; lshift[i] aligns input i
    to the finest input scale, rshift takes the sum to the output scale."""
    import torch
    y = torch.empty_like(inputs[0]) if out is None else out
    ptrs = (ctypes.c_void_p * len(inputs))(*[t.data_ptr() for t in inputs])
    ls, lp = _host(lshift, np.int32)
    _check(lib().qeltwise_add_i8(ctypes.cast(ptrs, ctypes.c_void_p), len(inputs), lp, int(rshift), int(relu),
                                 int(rounding), int(n_out), int(symmetric), inputs[0].numel(), _dev(y), _stream()))
    return y


MEASURES = {"l1": 0, "ks": 1, "cvm": 2, "kl": 3}


def qthreshold_search(hist, range_hi, n=8, p=7, measure="l1", return_all=False):
    """Algorithm 1 on a histogram of abs(x) (numpy uint64, equal bins on [0, range_hi]).
    Returns (gamma, delta), or (gamma, delta, index, deltas) with return_all."""
    h, hp = _host(hist, np.uint64)
    gamma, delta, index = ctypes.c_double(0), ctypes.c_double(0), ctypes.c_int(0)
    deltas = np.zeros(h.size + 1, dtype=np.float64) if return_all else None
    _check(lib().qthreshold_search(hp, h.size, float(range_hi), int(n), int(p), MEASURES[measure],
                                   ctypes.byref(gamma), ctypes.byref(delta), ctypes.byref(index),
                                   ctypes.c_void_p(deltas.ctypes.data) if return_all else None, _stream()))
    if return_all:
        return gamma.value, delta.value, index.value, deltas
    return gamma.value, delta.value


def qfpspace(n, p):
    out = np.zeros(1 << (n - 1), dtype=np.float64)
    cnt = ctypes.c_int(0)
    _check(lib().qfpspace(int(n), int(p), ctypes.c_void_p(out.ctypes.data), ctypes.byref(cnt)))
    return out[:cnt.value]


def qscale_exponent(gamma, n=8):
    e = ctypes.c_int(0)
    _check(lib().qscale_exponent(float(gamma), int(n), ctypes.byref(e)))
    return int(e.value)


def qconv_checked_faults():
    """(failed index tests since the last call, source line of the first); (-1, 0) unless the checked build is loaded."""
    line = ctypes.c_int(0)
    n = lib().qconv_checked_faults(ctypes.byref(line))
    return int(n), int(line.value)


def qbench_mma_i8(bn=128, mmas_per_cta=8192, row_bytes=128, commit_every=0):
    """Tensor-pipe ceiling of the int8 MMA (no loads, no epilogue): dict(tops, cycles_per_mma, ms, ctas)."""
    ms, cyc, ctas = ctypes.c_float(0), ctypes.c_double(0), ctypes.c_int(0)
    _check(lib().qbench_mma_i8(int(bn), int(mmas_per_cta), int(row_bytes), int(commit_every), ctypes.byref(ms), ctypes.byref(cyc), ctypes.byref(ctas),
                               _stream()))
    ops = 2.0 * 128 * bn * 32 * mmas_per_cta * ctas.value
    return dict(tops=ops / (ms.value * 1e-3) / 1e12, cycles_per_mma=cyc.value, ms=ms.value, ctas=ctas.value,
                macs_per_clk_per_sm=128.0 * bn * 32 / cyc.value)


def qacc_exponents(e_x, e_w):
    e_w, ep = _host(e_w, np.int32)
    out = np.zeros(e_w.size, dtype=np.int32)
    _check(lib().qacc_exponents(int(e_x), ep, e_w.size, ctypes.c_void_p(out.ctypes.data)))
    return out


def qrequant_shifts(e_z, acc_exp):
    a, ap = _host(acc_exp, np.int32)
    out = np.zeros(a.size, dtype=np.int32)
    _check(lib().qrequant_shifts(int(e_z), ap, a.size, ctypes.c_void_p(out.ctypes.data)))
    return out


def qresidual_shifts(e_res, acc_exp):
    a, ap = _host(acc_exp, np.int32)
    out = np.zeros(a.size, dtype=np.int32)
    _check(lib().qresidual_shifts(int(e_res), ap, a.size, ctypes.c_void_p(out.ctypes.data)))
    return out


def qjoin_exponent(e_own, acc_exps):
    """e_own: one exponent per branch; acc_exps: one int32 array per branch."""
    arrs = [np.ascontiguousarray(a, dtype=np.int32) for a in acc_exps]
    own, op = _host(e_own, np.int32)
    ks, kp = _host([a.size for a in arrs], np.int32)
    ptrs = (ctypes.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])
    e_z = ctypes.c_int(0)
    _check(lib().qjoin_exponent(op, ctypes.cast(ptrs, ctypes.c_void_p), kp, len(arrs), ctypes.byref(e_z)))
    return int(e_z.value)


def qpack_weights(wq, n):
    wq, wp = _host(wq, np.int8)
    out = np.zeros((wq.size * n + 7) // 8, dtype=np.uint8)
    _check(lib().qpack_weights(wp, wq.size, int(n), ctypes.c_void_p(out.ctypes.data)))
    return out


def qunpack_weights(packed, count, n):
    packed, pp = _host(packed, np.uint8)
    out = np.zeros(count, dtype=np.int8)
    _check(lib().qunpack_weights(pp, int(count), int(n), ctypes.c_void_p(out.ctypes.data)))
    return out


def qquantize_weights(w, K, R, S, Cg, layout=0, per_channel=1, n=8):
    w, wp = _host(w, np.float32)
    assert w.size == K * R * S * Cg
    wq = np.zeros(w.shape, dtype=np.int8)
    e_w = np.zeros(K, dtype=np.int32)
    _check(lib().qquantize_weights(wp, K, R, S, Cg, layout, per_channel, n,
                                   ctypes.c_void_p(wq.ctypes.data), ctypes.c_void_p(e_w.ctypes.data)))
    return wq, e_w


def qquantize_bias(b, e_x, e_w):
    b, bp = _host(b, np.float32)
    e_w, ep = _host(e_w, np.int32)
    bq = np.zeros(b.shape, dtype=np.int32)
    _check(lib().qquantize_bias(bp, b.size, int(e_x), ep, ctypes.c_void_p(bq.ctypes.data)))
    return bq

"""qcalib_collect_static: the calibration statistics for callers that may not allocate on the device
(a server that froze its memory layout at start-up, a host that gives plug-ins no memory budget).
It must return what qcalib_collect returns and what the CPU oracle computes -- exact maximum, counts
and histogram, fp64 sums within the suite's 1e-6 -- on consecutive calls that reuse its single
built-in scratch array, allocate nothing on the device, and refuse sizes its scratch cannot hold.
Collected last on purpose: a failure here stops nothing else."""
import ctypes

import numpy as np
import pytest

from oracle import ref
from paper_1805_07941_b200 import binding


def _same(a, b):
    assert a["maxabs"] == b["maxabs"]
    if "range_hi" in b:                                  # (the oracle returns no range: it is an input there)
        assert a["range_hi"] == b["range_hi"]
    assert a["count"] == b["count"] and a["nonfinite"] == b["nonfinite"]
    assert (a["hist"] == b["hist"]).all()
    assert abs(a["sum"] - b["sum"]) <= 1e-6 * max(1.0, abs(b["sum"]))
    assert abs(a["sumsq"] - b["sumsq"]) <= 1e-6 * max(1.0, b["sumsq"])


@pytest.mark.gpu
def test_static_scratch_matches_allocating_entry_point_on_consecutive_calls():
    import torch
    rng = np.random.default_rng(11)
    # two calls in a row on different data and shapes: the second must not see the first's counters
    x1 = (rng.standard_normal((1 << 20) + 5) * 3).astype(np.float32)
    x1[[7, 99]] = [np.nan, -np.inf]
    x2 = np.maximum(rng.standard_normal(300_001) * 0.2, 0).astype(np.float32)      # smaller, ReLU-like
    t1, t2 = torch.from_numpy(x1).cuda(), torch.from_numpy(x2).cuda()
    got1 = binding.qcalib_collect_static(t1, 2048)
    got2 = binding.qcalib_collect_static(t2, 2048)
    got3 = binding.qcalib_collect_static(t2, 64, 0.5)                              # fixed range, fewer bins
    _same(got1, binding.qcalib_collect(t1, 2048))
    _same(got2, binding.qcalib_collect(t2, 2048))
    _same(got3, binding.qcalib_collect(t2, 64, 0.5))
    # ... and against the CPU oracle, not only against the sibling call
    _same(got1, ref.calib_stats(x1, 2048))
    _same(got2, ref.calib_stats(x2, 2048))
    _same(got3, ref.calib_stats(x2, 64, 0.5))
    # the property the call exists for: once the library is loaded, further calls leave the amount of
    # free device memory unchanged (nothing is allocated, nothing freed)
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for _ in range(3):
        _same(binding.qcalib_collect_static(t1, 2048), got1)
        _same(binding.qcalib_collect_static(t2, 64, 0.5), got3)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert got1["nonfinite"] == 2 and got2["nonfinite"] == 0
    assert got2["hist"].sum() == x2.size and got1["hist"].sum() == x1.size - 2


@pytest.mark.gpu
def test_static_scratch_rejects_what_it_cannot_hold():
    import torch
    x = torch.zeros(1000, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.QconvError) as e:
        binding.qcalib_collect_static(x, 4097)
    assert e.value.code == binding.ERR_BAD_ARG and "nbins" in str(e.value)
    hist = np.zeros(16, np.uint64)
    st = binding.qcalib_stats()
    st.hist = hist.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64))
    rc = binding.lib().qcalib_collect_static(ctypes.c_void_p(x.data_ptr()), (1 << 40) + 1, 16, 0.0,
                                             ctypes.byref(st), None)
    assert rc == binding.ERR_BAD_ARG and b"count" in binding.lib().qconv_last_error_string()
    ok = binding.qcalib_collect_static(x, 16)                                      # still usable afterwards
    assert ok["count"] == 1000 and ok["hist"][0] == 1000

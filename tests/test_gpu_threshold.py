"""Algorithm 1 (threshold search) on the GPU against the oracle, through the C ABI.

Both sides work in float64; they differ in the order of additions (cumsum vs exact integer prefix
sums, a tree instead of numpy's pairwise sum) and in the interpolation's operation order, so every
candidate's measure is compared to relative 1e-9 (+1e-13 absolute); the arg-min must be the
oracle's unless the two best candidates are closer than that tolerance, in which case the chosen
candidate's measure must equal the minimum within it.
"""
import numpy as np
import pytest

from oracle import threshold_ref
from paper_1805_07941_b200 import binding

pytestmark = pytest.mark.gpu


def _hist(kind, nbins, seed):
    rng = np.random.default_rng(seed)
    if kind == "halfnormal_outlier":
        x = np.abs(rng.normal(size=400000)) * 0.04
        x[0] = 1.0                                          # the maximum is a far outlier
    elif kind == "relu_spike":
        x = np.maximum(rng.normal(size=300000), 0.0) * 0.2
        x = np.minimum(x, 1.0)
        x[1] = 1.0
    elif kind == "uniform":
        x = rng.random(200000)
        x[2] = 1.0
    else:
        x = np.abs(rng.laplace(size=300000)) * 0.08
        x = np.minimum(x, 1.0)
        x[3] = 1.0
    h = np.zeros(nbins, dtype=np.uint64)
    np.add.at(h, np.minimum((x * nbins).astype(np.int64), nbins - 1), 1)
    return h


def _compare(h, hi, n, p, kind):
    g, d, idx, deltas = binding.qthreshold_search(h, hi, n, p, kind, return_all=True)
    og, od, oidx, odeltas = threshold_ref.threshold(h, hi, n, p, kind, return_all=True)
    first = 2 ** (n - 1) + 1
    assert np.isnan(deltas[:first]).all() and np.isnan(odeltas[:first]).all()
    np.testing.assert_allclose(deltas[first:], odeltas[first:], rtol=1e-9, atol=1e-13)
    tol = 1e-9 * abs(od) + 1e-13
    if idx != oidx:
        assert abs(odeltas[idx] - od) <= tol, (idx, oidx)
    assert abs(d - odeltas[idx]) <= tol
    assert g == pytest.approx(float(np.float32(hi)) * idx / len(h), rel=1e-15)
    return idx, oidx


@pytest.mark.parametrize("kind", threshold_ref.MEASURES)
@pytest.mark.parametrize("shape", ["halfnormal_outlier", "relu_spike", "uniform", "laplace"])
def test_int8_search_on_2048_bins(kind, shape):
    h = _hist(shape, 2048, 1)
    idx, oidx = _compare(h, 3.5, 8, 7, kind)
    if shape == "uniform":
        assert oidx == 2048                                  # nothing to clip


@pytest.mark.parametrize("n,p", [(8, 4), (8, 3), (8, 2), (8, 0), (6, 5), (5, 2), (2, 1)])
def test_other_formats(n, p):
    h = _hist("halfnormal_outlier", 1000, 2)                # a bin count that is not a power of two
    for kind in ("l1", "kl"):
        _compare(h, 0.75, n, p, kind)


def test_smallest_and_largest_bin_counts():
    _compare(_hist("laplace", 129, 3), 1.0, 8, 7, "l1")     # a single candidate
    _compare(_hist("laplace", 4096, 4), 1.0, 8, 7, "ks")
    _compare(_hist("relu_spike", 4095, 5), 2.0, 8, 4, "cvm")


def test_ties_keep_the_lowest_candidate():
    # all mass in bin 0: the cdf is 1 everywhere and every candidate reproduces it exactly
    h = np.zeros(300, dtype=np.uint64)
    h[0] = 1000
    g, d, idx, deltas = binding.qthreshold_search(h, 1.0, 8, 7, "l1", return_all=True)
    og, od, oidx, _ = threshold_ref.threshold(h, 1.0, 8, 7, "l1", return_all=True)
    assert oidx == 129 and idx == 129 and d == 0.0 and od == 0.0


def test_search_consumes_the_statistics_kernel_output():
    import torch
    x = torch.randn(1 << 20, device="cuda").abs_()
    x[7] = 40.0
    st = binding.qcalib_collect(x, 2048)
    g, d = binding.qthreshold_search(st["hist"], st["maxabs"], 8, 7, "l1")
    og, od = threshold_ref.threshold(st["hist"], st["maxabs"], 8, 7, "l1")
    assert g == pytest.approx(og, rel=1e-12) and d == pytest.approx(od, rel=1e-9)
    assert g < 10.0                                          # the outlier at 40 is clipped

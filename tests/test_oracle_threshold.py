"""Pins for the oracle of Algorithm 1 (threshold search, Section 3).

The choice of `measure` is a reading (the paper does not define it); what is pinned here is the
mechanics: cdf, the clipping r[i-1:] <- 1, the two interpolations through fpspace, the candidate
range, gamma = bin_edges[i], and the strict-improvement tie-break.
"""
from fractions import Fraction

import numpy as np
import pytest

from oracle import dynfloat as df
from oracle import threshold_ref as tr


# ---- an independent exact-rational restatement used only as a pin ---------------------------------

def _lerp_exact(x, xs, ys):
    """Piecewise-linear interpolation on exact rationals; xs ascending, x inside [xs[0], xs[-1]]."""
    for a in range(len(xs) - 1):
        if xs[a] <= x <= xs[a + 1]:
            if xs[a + 1] == xs[a]:
                return ys[a]
            return ys[a] + (ys[a + 1] - ys[a]) * (x - xs[a]) / (xs[a + 1] - xs[a])
    raise AssertionError("x outside the knots")


def _exact_deltas(hist, n, p, kind):
    total = sum(hist)
    nb = len(hist)
    cdf, acc = [], 0
    for h in hist:
        acc += h
        cdf.append(Fraction(acc, total))
    levels = sorted({v for v in df.value_set(n, p) if v >= 0})
    fp = [Fraction(v) / levels[-1] for v in levels]
    out = {}
    for i in range(2 ** (n - 1) + 1, nb + 1):
        r = [cdf[j] if j < i - 1 else Fraction(1) for j in range(nb)]
        grid = [Fraction(j, i - 1) for j in range(i)]
        r_at_fp = [_lerp_exact(f, grid, r[:i]) for f in fp]
        q = [_lerp_exact(grid[j], fp, r_at_fp) if j < i else r[j] for j in range(nb)]
        d = [abs(cdf[j] - q[j]) for j in range(nb)]
        if kind == "l1":
            out[i] = sum(d) / nb
        elif kind == "ks":
            out[i] = max(d)
        elif kind == "cvm":
            out[i] = sum(x * x for x in d) / nb
    return out


@pytest.mark.parametrize("n,p", [(3, 2), (4, 3), (4, 1), (5, 2)])
@pytest.mark.parametrize("kind", ["l1", "ks", "cvm"])
def test_candidate_measures_match_exact_rational_brute_force(n, p, kind):
    rng = np.random.default_rng(100 * n + p)
    nb = 2 ** (n - 1) + 14
    hist = [int(v) for v in rng.integers(0, 50, nb)]
    hist[0] += 200                                       # a spike at zero, as after a ReLU
    hist[-1] += 1                                        # the maximum sits in the last bin
    exact = _exact_deltas(hist, n, p, kind)
    gamma, delta, index, deltas = tr.threshold(hist, 3.0, n, p, kind, return_all=True)
    assert set(exact) == {i for i in range(nb + 1) if not np.isnan(deltas[i])}
    for i, v in exact.items():
        assert deltas[i] == pytest.approx(float(v), rel=1e-11, abs=1e-14), i
    best = min(exact.values())
    first = min(i for i, v in exact.items() if v == best)
    assert index == first                                # strict '>' keeps the first of equal minima
    assert gamma == pytest.approx(3.0 * first / nb, rel=1e-15)
    assert delta == pytest.approx(float(best), rel=1e-11, abs=1e-14)


def test_fpspace_int8_is_the_uniform_grid_and_fp8_is_not():
    f = tr.fpspace(0.0, 1.0, 8, 7)
    assert len(f) == 128 and np.array_equal(f, np.arange(128) / 127.0)
    g = tr.fpspace(0.0, 1.0, 8, 4)                       # 3 exponent bits, 4 significand bits
    assert g[0] == 0.0 and g[-1] == 1.0 and np.all(np.diff(g) > 0)
    assert len(g) == 128                                 # every non-negative pattern is a distinct number
    steps = np.diff(g)
    assert steps[-1] == pytest.approx(64 * steps[0])     # subnormal step 1, top binade step 2^6
    h = tr.fpspace(-2.0, 2.0, 8, 4)
    assert h[0] == -2.0 and h[-1] == 2.0


@pytest.mark.parametrize("kind", tr.MEASURES)
def test_flat_histogram_is_reproduced_exactly_at_the_last_edge(kind):
    # cdf is a straight line: both interpolations are exact at i = nbins, every smaller i clips mass
    nb = 40
    gamma, delta, index, deltas = tr.threshold([7] * nb, 5.0, 4, 3, kind, return_all=True)
    assert index == nb and gamma == 5.0
    assert abs(delta) < 1e-14
    assert np.all(deltas[9:nb] > 1e-6)


@pytest.mark.parametrize("kind", ["l1", "ks", "cvm"])
@pytest.mark.parametrize("m", [12, 17, 30])
def test_support_ending_at_bin_m_puts_gamma_on_edge_m(kind, m):
    # flat on the first m bins, nothing beyond: candidate i = m has r == cdf, a straight line up to
    # 1 -> exact; i < m clips; i > m bends at a knot that the coarse grid cannot follow
    nb = 48
    hist = [5] * m + [0] * (nb - m)
    gamma, delta, index, _ = tr.threshold(hist, 6.0, 4, 3, kind, return_all=True)
    assert index == m
    assert gamma == pytest.approx(6.0 * m / nb, rel=1e-15)
    assert abs(delta) < 1e-14


def test_scaling_the_counts_changes_nothing():
    rng = np.random.default_rng(3)
    hist = rng.integers(1, 1000, 200)
    a = tr.threshold(hist, 1.0, 6, 5, "l1", return_all=True)
    b = tr.threshold(hist * 8, 1.0, 6, 5, "l1", return_all=True)
    assert a[2] == b[2] and np.allclose(a[3][33:], b[3][33:], rtol=1e-12, atol=0)


def test_outliers_are_clipped_for_a_long_tailed_histogram():
    # bulk in the first tenth of the range + one far outlier: the search must not return the
    # maximum (that is the whole point of thresholding) and must not cut into the bulk
    nb = 2048
    hist = np.zeros(nb, dtype=np.int64)
    x = np.abs(np.random.default_rng(0).normal(size=200000)) * (0.02 * nb)
    np.add.at(hist, np.minimum(x.astype(np.int64), nb - 1), 1)
    hist[-1] += 1
    for kind in ("l1", "kl"):
        gamma, delta, index, _ = tr.threshold(hist, 1.0, 8, 7, kind, return_all=True)
        assert 0.02 * 2.0 < gamma < 0.5, (kind, gamma)


def test_kl_is_zero_for_identical_and_penalises_clipping():
    cdf = np.linspace(0.1, 1.0, 10)
    assert tr.measure(cdf, cdf, "kl") == pytest.approx(0.0, abs=1e-15)
    q = cdf.copy()
    q[5:] = 1.0                                          # bins 6..9 lose their mass, bin 5 takes it
    P = np.diff(cdf, prepend=0.0)
    want = P[5] * np.log(P[5] / (1.0 - cdf[4])) + sum(P[j] * np.log(P[j] / 2.0 ** -52) for j in range(6, 10))
    assert tr.measure(cdf, q, "kl") == pytest.approx(want, rel=1e-12)

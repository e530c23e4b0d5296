"""TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Algorithm 1, Section 3 of the paper: the search for the clamping threshold gamma over
the bin edges of a histogram of abs(x).  Stated here as three small steps per candidate
edge -- clip the cdf at the candidate, pass the kept part through the (n, p) value grid
and back, compare with the unclipped cdf -- with numpy's cumsum / linspace / interp as the
primitives, float64 throughout.

Readings (the paper leaves these open):
  * the value grid on [0, 1]: the distinct non-negative values an (n, p) pattern decodes
    to by Eq. 2, divided by beta_max (Eq. 5), ascending; first 0, last 1.
  * the histogram is normalised by its total, so the cdf ends at 1 and setting its
    entries from the candidate on to 1 is the clipping of everything past the candidate.
  * resampling is piecewise-linear interpolation (numpy.interp).
  * candidates are the edges 2^(n-1)+1 .. nbins inclusive.
  * the comparison measure is not defined by the paper; four are offered:
      "l1"  mean |cdf - q|            (Kantorovich / Wasserstein-1 on the unit range)
      "ks"  max  |cdf - q|            (Kolmogorov-Smirnov)
      "cvm" mean (cdf - q)^2          (Cramer-von Mises form)
      "kl"  sum_j P_j ln(P_j / max(Q_j, 2^-52)) over P_j > 0, P and Q the bin masses
            of cdf and q (first differences); the floor keeps clipped bins finite.
    The paper's own choice (a weighted mix of over a dozen measures) is not
    reproducible from its text: PARITY UNPINNED for the choice of measure.  The
    mechanics (cdf, clipping, the two interpolations, the arg-min and its
    tie-break) are pinned in tests/test_oracle_threshold.py: exact rational
    brute force on tiny histograms, and closed forms (a flat histogram is
    reproduced exactly at the last edge; a flat histogram on the first m bins puts
    gamma on edge m with delta 0).
"""
import numpy as np

from oracle import dynfloat

MEASURES = ("l1", "ks", "cvm", "kl")
KL_FLOOR = 2.0 ** -52


def fpspace(lo, hi, n, p):
    """Representable non-negative values of the (n, p) type mapped linearly onto [lo, hi]."""
    vals = sorted({v for v in dynfloat.value_set(n, p) if v >= 0})
    top = vals[-1]
    return np.array([lo + (hi - lo) * float(v / top) for v in vals], dtype=np.float64)


def measure(cdf, q, kind):
    if kind == "l1":
        return float(np.mean(np.abs(cdf - q)))
    if kind == "ks":
        return float(np.max(np.abs(cdf - q)))
    if kind == "cvm":
        return float(np.mean((cdf - q) ** 2))
    if kind == "kl":
        P = np.diff(cdf, prepend=0.0)
        Q = np.maximum(np.diff(q, prepend=0.0), KL_FLOOR)
        m = P > 0
        return float(np.sum(P[m] * np.log(P[m] / Q[m])))
    raise ValueError(kind)


def clip_at(cdf, i):
    """The cdf of the data clamped to the candidate edge i: everything from entry i-1 on is 1."""
    clipped = cdf.copy()
    clipped[i - 1:] = 1.0
    return clipped


def through_grid(head, grid):
    """The first len(head) cdf entries, seen as samples on a uniform axis over [0, 1], resampled
    onto the value grid of the type and from there back onto the uniform axis."""
    axis = np.linspace(0.0, 1.0, len(head))
    on_grid = np.interp(grid, axis, head)
    return np.interp(axis, grid, on_grid)


def threshold(hist, range_hi, n, p, kind="l1", return_all=False):
    """hist: counts of abs(x) in len(hist) equal bins on [0, range_hi].
    Returns (gamma, delta) or, with return_all, (gamma, delta, index, deltas) where
    deltas[i] is the measure of candidate i (NaN outside the loop's range)."""
    hist = np.asarray(hist, dtype=np.float64)
    nbins = len(hist)
    edges = np.linspace(0.0, float(range_hi), nbins + 1)
    cdf = np.cumsum(hist / hist.sum())
    grid = fpspace(0.0, 1.0, n, p)
    deltas = np.full(nbins + 1, np.nan)
    for i in range(2 ** (n - 1) + 1, nbins + 1):
        q = clip_at(cdf, i)
        q[:i] = through_grid(q[:i], grid)
        deltas[i] = measure(cdf, q, kind)
    # smallest measure; among equal ones the lowest edge; the last edge when none is finite
    index, delta = nbins, np.inf
    for i in range(2 ** (n - 1) + 1, nbins + 1):
        if deltas[i] < delta:
            index, delta = i, deltas[i]
    gamma = edges[index]
    if return_all:
        return float(gamma), float(delta), index, deltas
    return float(gamma), float(delta)

"""Pins of the oracle's sufficient statistics, level fit and symbol weights (Sec. 3.3, App. E).
CPU only."""
import itertools
import math

import numpy as np

from oracle import qgx_oracle as o


def test_histogram_by_hand():
    # bucket (1, 2, 2, 4): norm 5, u = .2 .4 .4 .8 -> bins floor(8u) = 1 3 3 6, each weighted by 25;
    # bucket (0, 0, 3, 4): norm 5, u = 0 0 .6 .8 -> bins 0 0 4 6
    v = np.array([[1, -2, 2, 4, 0, 0, -3, 4]], dtype=np.float32)
    h = o.histogram(v, 4, 8)
    exp = np.zeros(8)
    exp[[1, 3, 6]] = [25, 50, 25]
    exp[[0, 4, 6]] += [50, 25, 25]
    assert h.tolist() == exp.tolist()
    hu = o.histogram(v, 4, 8, weighted=False)
    assert hu.tolist() == [2, 1, 0, 2, 1, 0, 2, 0]
    # u = 1 falls in the last bin; L-infinity norm: u = |v| / max|v|
    assert o.histogram(np.array([[0, 5.0]], dtype=np.float32), 2, 4, weighted=False).tolist() == [1, 0, 0, 1]
    assert o.histogram(np.array([[1, -2, 4.0]], dtype=np.float32), 3, 4, o.LINF, False).tolist() == [0, 1, 1, 1]


def test_histogram_counts_and_mass():
    rng = np.random.default_rng(0)
    K, d, bucket, nbins = 3, 5000, 1024, 64
    v = rng.standard_normal((K, d)).astype(np.float32)
    norms = o.bucket_norms(v, bucket)
    h = o.histogram(v, bucket, nbins, weighted=False)
    assert h.sum() == K * d
    direct = np.zeros(nbins)
    for k in range(K):
        for i in range(d):
            u = np.float32(abs(v[k, i])) / norms[k, i // bucket]
            direct[min(int(math.floor(float(np.float32(u * np.float32(nbins))))), nbins - 1)] += 1
    assert np.array_equal(h, direct)
    hw = o.histogram(v, bucket, nbins)
    lens = np.array([1024, 1024, 1024, 1024, 904])
    mass = sum(float(norms[k, b]) ** 2 * lens[b] for k in range(K) for b in range(5))
    assert abs(hw.sum() - mass) <= 1e-12 * mass


def test_uniform_cdf_gives_equally_spaced_levels():
    # with dF = du the stationarity condition reads (l-a)^2/2 = (c-l)^2/2: each level is the midpoint
    hist = np.ones(1024)
    for nlev in (3, 5, 9, 17):
        lev = o.fit_levels(hist, nlev=nlev)
        assert np.max(np.abs(lev - np.linspace(0, 1, nlev))) < 2e-6
        skew = np.linspace(0, 1, nlev) ** 2
        # from a skewed start, 32 sweeps of coordinate descent close most of the distance
        lev2 = o.fit_levels(hist, init=skew.astype(np.float32))
        err0 = np.max(np.abs(skew - np.linspace(0, 1, nlev)))
        assert np.max(np.abs(lev2 - np.linspace(0, 1, nlev))) < (0.02 if nlev <= 9 else 0.35) * err0 + 1e-6


def _objective_by_quadrature(hist, lev, sub=64):
    # sum_i int (l_{i+1}-u)(u-l_i) dF with each bin's mass spread over `sub` equal point masses
    n = len(hist)
    u = (np.arange(n * sub) + 0.5) / (n * sub)
    w = np.repeat(np.asarray(hist, dtype=np.float64) / sub, sub)
    l = np.asarray(lev, dtype=np.float64)
    tau = np.clip(np.searchsorted(l, u, side="right") - 1, 0, len(l) - 2)
    return float(np.sum(w * (l[tau + 1] - u) * (u - l[tau])))


def test_objective_matches_quadrature_and_decreases():
    rng = np.random.default_rng(4)
    hist = rng.gamma(0.5, size=256) * np.exp(-np.arange(256) / 40.0)
    lev0 = np.linspace(0, 1, 9).astype(np.float32)
    assert abs(o.objective(hist, lev0) - _objective_by_quadrature(hist, lev0)) < 2e-4 * o.objective(hist, lev0)
    lev, trace = o.fit_levels(hist, init=lev0, return_trace=True)
    assert len(trace) >= 2 and np.all(np.diff(trace) <= 1e-15 + 1e-12 * trace[0])
    assert trace[-1] < 0.5 * trace[0]
    # at the fitted point every interior level is a root of g (or pinned by the minimum spacing)
    l64 = lev.astype(np.float64)
    scale = hist.sum()
    for j in range(1, 8):
        g = o.stationarity(hist, l64[j - 1], l64[j + 1], l64[j])
        assert abs(g) < 1e-5 * scale
    # the quantile start descends too (the objective is not convex, so the two end points may differ)
    levq, traceq = o.fit_levels(hist, nlev=9, return_trace=True)
    assert np.all(np.diff(traceq) <= 1e-15 + 1e-12 * traceq[0]) and traceq[-1] < trace[0]


def test_fit_against_brute_force_grid():
    rng = np.random.default_rng(9)
    for nlev in (3, 4):
        hist = rng.uniform(0.0, 1.0, size=32) ** 3
        lev = o.fit_levels(hist, nlev=nlev)
        grid = np.arange(1, 128) / 128.0
        best = min(_objective_by_quadrature(hist, np.r_[0.0, c, 1.0])
                   for c in itertools.combinations(grid, nlev - 2))
        got = _objective_by_quadrature(hist, lev)
        assert got <= best * (1 + 1e-3) + 1e-12      # coordinate descent reaches the grid optimum
        assert got >= best * 0.97                     # and the grid is fine enough to be comparable


def test_point_mass_attracts_a_level():
    hist = np.zeros(1024)
    hist[300] = 7.0                                   # all mass in [300/1024, 301/1024)
    hist[10] = 1e-3
    lev = o.fit_levels(hist, init=np.array([0, 0.2, 0.5, 1.0], dtype=np.float32))
    assert np.min(np.abs(lev - 300.5 / 1024)) < 1.0 / 1024
    assert o.objective(hist, lev) < 1e-3 * o.objective(hist, np.array([0, 0.2, 0.5, 1.0], dtype=np.float32))
    # an empty histogram leaves the table as it was
    keep = o.fit_levels(np.zeros(64), init=np.array([0, 0.25, 1.0], dtype=np.float32))
    assert keep.tolist() == [0.0, 0.25, 1.0]


def test_symbol_weights_sum_to_one_and_match_frequencies():
    rng = np.random.default_rng(6)
    d = 8192
    v = rng.standard_normal((8, d)).astype(np.float32)
    hist = o.histogram(v, d, 1 << 15, weighted=False)
    lev = o.fit_levels(o.histogram(v, d, 1024), nlev=9)
    p = o.symbol_pmf(hist, lev)
    assert abs(p.sum() - 1.0) < 1e-12 and np.all(p >= 0)
    norms = o.bucket_norms(v, d)
    freq = np.zeros(9)
    reps = 6
    for s in range(reps):
        idx = o.quantize(v, d, lev, norms, seed=s, xid=0) & 31
        freq += np.bincount(idx.ravel(), minlength=9)
    freq /= reps * v.size
    assert np.max(np.abs(freq - p)) < 5 * math.sqrt(0.25 / (reps * v.size)) + 2e-4
    # the fitted table beats the uniform one on the variance it was fitted to (Eq. var)
    assert o.objective(o.histogram(v, d, 1024), lev) < 0.2 * o.objective(o.histogram(v, d, 1024),
                                                                          np.linspace(0, 1, 9, dtype=np.float32))

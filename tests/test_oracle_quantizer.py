"""Pins of the oracle's quantizer (Definition 1, Theorem 1) against what the paper and the
mathematics fix.  CPU only."""
import itertools
import math

import numpy as np
import pytest

from oracle import qgx_oracle as o
from conftest import read_golden


def test_philox_known_answers():
    for row in read_golden("philox4x32_10_kat.txt"):
        w = [int(x, 16) for x in row]
        out = o.philox4x32_10(w[0:4], w[4:6])
        assert [int(x) for x in out] == w[6:10]


def test_element_word_counter_layout():
    # counter = (e/4 low, e/4 high, worker, exchange id), key = seed halves, word e mod 4
    seed = 0x0123456789ABCDEF
    for worker, xid, e in [(0, 0, 0), (3, 7, 5), (31, 2001, (1 << 34) + 6), (1, 1, 3)]:
        q = e >> 2
        blk = o.philox4x32_10([q & 0xFFFFFFFF, q >> 32, worker, xid], [seed & 0xFFFFFFFF, seed >> 32])
        assert o.element_word(seed, worker, xid, e) == int(blk[e & 3])


def test_round_up_probability_is_exact():
    # r takes the 2^24 values m*2^-24; "up" iff r < xi, so exactly ceil(xi * 2^24) of them round up
    for xi in [0.0, 1.0, 0.5, 1.0 / 3.0, 2.0 ** -24, 3.0 * 2.0 ** -25, 0.999999, 1e-9]:
        xi32 = float(np.float32(xi))
        assert o.count_up(xi32) == math.ceil(xi32 * 2 ** 24)


def test_level_search_edges():
    lev = np.array([0.0, 0.125, 0.5, 1.0], dtype=np.float32)
    assert o.level_search(0.0, lev) == 0
    assert o.level_search(0.1249999, lev) == 0
    # exactly on a level: that level, xi = 0, never rounded up
    assert o.level_search(0.125, lev) == 1
    assert o.xi(0.125, lev, 1) == 0.0
    assert o.count_up(0.0) == 0
    # u = 1 belongs to the last interval with xi = 1: always the top level
    assert o.level_search(1.0, lev) == 2
    assert o.xi(1.0, lev, 2) == 1.0
    assert o.count_up(1.0) == 2 ** 24
    assert o.check_levels(lev) == o.OK
    assert o.check_levels([0.0, 0.5, 0.5, 1.0]) == o.BAD_LEVELS
    assert o.check_levels([0.1, 0.5, 1.0]) == o.BAD_LEVELS
    assert o.check_levels([0.0, 0.5, 0.9]) == o.BAD_LEVELS


def _random_levels(rng, nlev):
    inner = np.sort(rng.uniform(0.02, 0.98, size=nlev - 2))
    return np.concatenate([[0.0], inner, [1.0]]).astype(np.float32)


@pytest.mark.parametrize("norm_type", [o.L2, o.LINF])
def test_unbiased_by_exact_enumeration(norm_type):
    """E[Q(v)] = v (Theorem 1, first claim): all 2^d outcomes of a d<=8 vector, each weighted by
    its exact probability under the 24-bit variate."""
    rng = np.random.default_rng(5)
    for d, nlev in [(3, 2), (6, 4), (8, 9)]:
        v = rng.standard_normal((1, d)).astype(np.float32)
        v[0, 0] = -abs(v[0, 0])
        lev = _random_levels(rng, nlev)
        norms = o.bucket_norms(v, d, norm_type)
        p_up = np.zeros(d)
        for i in range(d):
            u = o.normalize(float(v[0, i]), float(norms[0, 0]))
            tau = o.level_search(u, lev)
            p_up[i] = math.ceil(o.xi(u, lev, tau) * 2 ** 24) / 2 ** 24
        mean = np.zeros(d)
        total_p = 0.0
        for pattern in itertools.product([0, 1], repeat=d):
            # word 0 -> r = 0 (up unless xi = 0); word 0xffffff00 -> r = 1 - 2^-24 (down unless xi = 1)
            words = np.array([[0 if b else 0xFFFFFF00 for b in pattern]], dtype=np.uint32)
            sym = o.quantize_words(v, d, lev, norms, words)
            prob = 1.0
            for i, b in enumerate(pattern):
                prob *= p_up[i] if b else 1.0 - p_up[i]
            mean += prob * o.dequantize(norms, sym, d, lev)[0].astype(np.float64)
            total_p += prob
        assert abs(total_p - 1.0) < 1e-12
        # fp32 roundings of u, xi and of the decoded product: a few units of 2^-24 of the norm
        assert np.max(np.abs(mean - v[0])) <= 5e-7 * float(norms[0, 0])


def _per_coordinate_variance(v, norm, lev):
    # Eq. (var): ||v||^2 (l_{tau+1} - u_i)(u_i - l_tau) per coordinate, written out in fp64
    u = np.minimum(np.abs(v.astype(np.float64)) / float(norm), 1.0)
    l64 = lev.astype(np.float64)
    tau = np.clip(np.searchsorted(l64, u, side="right") - 1, 0, len(lev) - 2)
    return float(norm) ** 2 * (l64[tau + 1] - u) * (u - l64[tau])


@pytest.mark.parametrize("dist", ["gauss", "heavy"])
def test_monte_carlo_mean_and_variance(dist):
    rng = np.random.default_rng(11)
    d, trials = 4096, 1500
    if dist == "gauss":
        v = rng.standard_normal((1, d)).astype(np.float32)
    else:
        v = (rng.standard_t(3, size=(1, d)) * 0.01).astype(np.float32)
    lev = np.array([0, 0.004, 0.01, 0.02, 0.035, 0.06, 0.1, 0.3, 1.0], dtype=np.float32)
    norms = o.bucket_norms(v, d)
    acc = np.zeros(d)
    acc2 = np.zeros(d)
    err2 = np.zeros(trials)
    for s in range(trials):
        q = o.dequantize(norms, o.quantize(v, d, lev, norms, seed=1000 + s, xid=3), d, lev)[0].astype(np.float64)
        acc += q
        acc2 += q * q
        err2[s] = np.sum((q - v[0]) ** 2)
    mean = acc / trials
    # standard error from the per-coordinate variance of Eq. (var); a sample variance would be
    # zero for a coordinate whose rare outcome never showed up
    var = _per_coordinate_variance(v[0], norms[0, 0], lev)
    se = np.sqrt(var / trials) + 1e-7 * float(norms[0, 0])
    sample_var = np.maximum(acc2 / trials - mean ** 2, 0.0)
    assert abs(sample_var.sum() - var.sum()) < 0.05 * var.sum()
    z = np.abs(mean - v[0]) / se
    assert z.max() < 5.5, z.max()          # 4096 coordinates: the largest |z| is about 4
    cf = var.sum()
    se_err = err2.std(ddof=1) / math.sqrt(trials)
    assert abs(err2.mean() - cf) < 4.5 * se_err + 1e-6 * cf
    # the seeds really differ and coordinates are rounded independently
    s1 = o.quantize(v, d, lev, norms, seed=1, xid=3)
    s2 = o.quantize(v, d, lev, norms, seed=2, xid=3)
    s3 = o.quantize(v, d, lev, norms, seed=1, xid=4)
    assert (s1 != s2).mean() > 0.05 and (s1 != s3).mean() > 0.05
    assert np.array_equal(s1, o.quantize(v, d, lev, norms, seed=1, xid=3))


def _eps_q(lev, d, q=2):
    # Theorem 1: eps_Q = (lbar + 1/lbar)/4 + [l1^2 d^(2/min(q,2))/4 if d <= d_th else l1 d^(1/min(q,2)) - 1] - 1/2
    l = lev.astype(np.float64)
    lbar = np.max(l[2:] / l[1:-1]) if len(l) > 2 else 1.0
    m = min(q, 2)
    d_th = (2.0 / l[1]) ** m
    tail = 0.25 * l[1] ** 2 * d ** (2.0 / m) if d <= d_th else l[1] * d ** (1.0 / m) - 1.0
    return (lbar + 1.0 / lbar) / 4.0 + tail - 0.5


@pytest.mark.parametrize("d", [16, 512, 4096])
def test_variance_bound_theorem1(d):
    rng = np.random.default_rng(d)
    tables = [np.linspace(0, 1, 9, dtype=np.float32),
              np.array([0, 2.0 ** -6, 2.0 ** -5, 2.0 ** -4, 0.125, 0.25, 0.5, 1.0], dtype=np.float32),
              np.array([0.0, 1.0], dtype=np.float32),
              _random_levels(rng, 17)]
    inputs = [rng.standard_normal(d), rng.standard_t(3, size=d), np.r_[np.zeros(d - 1), 1.0],
              np.ones(d), rng.standard_normal(d) * (rng.uniform(size=d) < 0.05)]
    for lev in tables:
        for v in inputs:
            v = v.astype(np.float32)
            if not np.any(v):
                continue
            norm = o.bucket_norms(v[None, :], d)[0, 0]
            cf = _per_coordinate_variance(v, norm, lev).sum()
            bound = _eps_q(lev, d) * float(np.sum(v.astype(np.float64) ** 2))
            assert cf <= bound * (1 + 1e-6) + 1e-12


def test_two_level_table_is_the_ternary_scheme():
    # l = {0, 1} with L2 normalisation: each coordinate becomes sign(v)||v|| with probability |v|/||v||, else 0
    rng = np.random.default_rng(3)
    d, trials = 64, 4000
    v = rng.standard_normal((1, d)).astype(np.float32)
    lev = np.array([0.0, 1.0], dtype=np.float32)
    norms = o.bucket_norms(v, d)
    hits = np.zeros(d)
    for s in range(trials):
        sym = o.quantize(v, d, lev, norms, seed=s, xid=0)[0]
        assert set(np.unique(sym & 31)).issubset({0, 1})
        nz = (sym & 31) == 1
        assert np.array_equal((sym[nz] >> 7) == 1, v[0][nz] < 0)
        hits += nz
    p = np.abs(v[0].astype(np.float64)) / float(norms[0, 0])
    se = np.sqrt(p * (1 - p) / trials) + 1e-9
    assert np.max(np.abs(hits / trials - p) / se) < 5.0


def test_zero_bucket_signed_zero_and_nonfinite():
    lev = np.linspace(0, 1, 5, dtype=np.float32)
    v = np.zeros((1, 8), dtype=np.float32)
    v[0, 4:] = [-0.0, 1e-30, -3.0, 4.0]       # bucket 0 all zero, bucket 1 = (-0, tiny, -3, 4)
    norms = o.bucket_norms(v, 4)
    assert norms[0, 0] == 0.0 and norms[0, 1] == 5.0
    sym = o.quantize(v, 4, lev, norms, seed=9, xid=1)
    assert np.all(sym[0, :4] == 0)            # zero norm: u = 0, level 0, no sign
    assert sym[0, 4] == 0                     # -0.0 quantizes to level 0 and carries no sign
    assert (sym[0, 6] & 0x80) and not (sym[0, 7] & 0x80)
    out = o.dequantize(norms, sym, 4, lev)
    assert not np.signbit(out[0, 4]) and np.all(out[0, :4] == 0)
    bad = v.copy()
    bad[0, 1] = np.nan
    with pytest.raises(o.OracleError) as e:
        o.bucket_norms(bad, 4)
    assert e.value.status == o.NONFINITE
    bad[0, 1] = np.inf
    with pytest.raises(o.OracleError):
        o.bucket_norms(bad, 4)
    assert o.bucket_norms(np.array([[3.0, -4.0, 1.0]], dtype=np.float32), 3, o.LINF)[0, 0] == 4.0


def test_norms_tail_bucket_and_fp64_accumulation():
    rng = np.random.default_rng(21)
    v = rng.standard_normal((3, 1000)).astype(np.float32) * 1e3
    norms = o.bucket_norms(v, 384)               # 384 + 384 + 232
    assert norms.shape == (3, 3)
    for k in range(3):
        for b, (lo, hi) in enumerate([(0, 384), (384, 768), (768, 1000)]):
            ref = np.float32(math.sqrt(math.fsum(float(x) * float(x) for x in v[k, lo:hi])))
            assert abs(float(norms[k, b]) - float(ref)) <= np.spacing(ref)


def test_dequantize_and_average_by_hand():
    lev = np.array([0.0, 0.5, 1.0], dtype=np.float32)
    norms = np.array([[2.0], [3.0], [0.1]], dtype=np.float32)
    sym = np.array([[1, 0x82, 0], [2, 1, 0x81], [0x81, 2, 2]], dtype=np.uint8)
    vh = o.dequantize(norms, sym, 3, lev)
    assert vh.tolist() == [[1.0, -2.0, 0.0], [3.0, 1.5, -1.5],
                           [float(-np.float32(0.1) * np.float32(0.5)), float(np.float32(0.1)), float(np.float32(0.1))]]
    avg = o.average(norms, sym, 3, lev)
    for i in range(3):
        acc = np.float32(0.0)
        for k in range(3):
            acc = np.float32(acc + vh[k, i])     # fixed order k = 0, 1, 2 in fp32
        assert avg[i] == np.float32(acc / np.float32(3.0))
    # the mean of unbiased decoded vectors stays unbiased: K copies of one vector average back to it
    v = np.tile(np.linspace(-1, 1, 16, dtype=np.float32), (256, 1))
    nv = o.bucket_norms(v, 16)
    lev9 = np.linspace(0, 1, 9, dtype=np.float32)
    m = o.average(nv, o.quantize(v, 16, lev9, nv, seed=4, xid=0), 16, lev9)
    assert np.max(np.abs(m - v[0])) < 0.06 * float(nv[0, 0])


def test_coordinate_base_only_shifts_the_variates():
    # a tensor inside a layer-wise vector: same buckets, norms and levels; variates of coordinates base + i
    rng = np.random.default_rng(31)
    v = rng.standard_normal((2, 300)).astype(np.float32)
    lev = np.linspace(0, 1, 9, dtype=np.float32)
    whole = o.quantize(v, 100, lev, o.bucket_norms(v, 100), seed=8, xid=2)
    part = v[:, 100:300].copy()
    at = o.quantize(part, 100, lev, o.bucket_norms(part, 100), seed=8, xid=2, coord_base=100)
    assert np.array_equal(at, whole[:, 100:300])
    assert not np.array_equal(o.quantize(part, 100, lev, o.bucket_norms(part, 100), seed=8, xid=2), at)

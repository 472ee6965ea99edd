"""CPU-only checks of the library's host side: it loads, exports every symbol that include/qgx.h
declares, and its host helpers (codebooks, level fit, symbol weights, capacity) agree with the
oracle.  No kernel runs here."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import qgx_oracle as o

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def qgx():
    import paper_2308_09187_b200 as q
    q.lib()
    return q


def test_library_exports_every_declared_symbol(qgx):
    header = open(os.path.join(ROOT, "include", "qgx.h")).read()
    declared = set(re.findall(r"\b(qgx_[a-z_0-9]+)\s*\(", header))
    assert declared == set(qgx.EXPORTS)
    L = ctypes.CDLL(qgx.library_path())
    for name in declared:
        assert hasattr(L, name), name
        assert hasattr(qgx, name), name          # the binding carries the same names


def test_no_device_means_an_error_not_a_fallback(qgx):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(Exception):
        qgx.qgx_create(0)


def test_status_strings_and_level_checks(qgx):
    assert qgx.qgx_status_str(0) == "ok"
    assert "capacity" in qgx.qgx_status_str(qgx.QGX_ERR_CAPACITY)
    assert qgx.qgx_check_levels([0.0, 0.25, 1.0]) == qgx.QGX_OK
    for bad in ([0.0, 1.0, 1.0], [0.1, 1.0], [0.0, 0.6, 0.5, 1.0], [0.0], [0.0, 0.5]):
        assert qgx.qgx_check_levels(bad) == qgx.QGX_ERR_BAD_LEVELS


def test_capacity_matches_oracle(qgx):
    for d, bucket, sub, maxlen in [(5000, 1024, 128, 5), (1 << 20, 8192, 0, 12), (1728, 4096, 128, 4), (70, 64, 32, 1)]:
        assert qgx.qgx_stream_capacity_words(d, bucket, sub, maxlen) == o.capacity_words(d, bucket, sub, maxlen)


def test_codebooks_match_oracle(qgx):
    rng = np.random.default_rng(0)
    for nlev in range(2, 33):
        a, b = qgx.qgx_build_codebook_fixed(nlev, 64), o.codebook_fixed(nlev, 64)
        assert a.lengths() == b.lengths() and a.codes() == b.codes() and a.maxlen == b.maxlen
        a, b = qgx.qgx_build_codebook_elias(nlev, 32), o.codebook_elias(nlev, 32)
        assert a.lengths() == b.lengths() and a.codes() == b.codes() and a.maxlen == b.maxlen and a.subblock == 32
        for _ in range(5):
            p = rng.dirichlet(np.ones(nlev) * rng.uniform(0.05, 2.0))
            a, b = qgx.qgx_build_codebook_huffman(list(p), 0), o.codebook_huffman(p, 0)
            # two Huffman builders: equal expected length and Kraft sum (the codes may differ in ties)
            assert abs(np.dot(p, a.lengths()) - np.dot(p, b.lengths())) < 1e-12
            assert abs(sum(2.0 ** -L for L in a.lengths()) - sum(2.0 ** -L for L in b.lengths())) < 1e-12
            assert a.maxlen <= 12
    geo = np.array([2.0 ** -(j + 1) for j in range(32)])
    assert qgx.qgx_build_codebook_huffman(list(geo / geo.sum())).maxlen <= 12


def test_level_fit_and_symbol_weights_match_oracle(qgx):
    rng = np.random.default_rng(3)
    hists = [np.ones(1024), rng.gamma(0.5, size=256) * np.exp(-np.arange(256) / 40.0),
             np.exp(-0.5 * (np.arange(1024) / 12.0) ** 2) * 1e6, rng.uniform(0, 1, 32) ** 3]
    for hist in hists:
        for nlev in (3, 9, 17):
            got = np.array(qgx.qgx_fit_levels(list(hist), nlev=nlev), dtype=np.float32)
            ref = o.fit_levels(hist, nlev=nlev)
            assert o.check_levels(got) == o.OK
            assert np.max(np.abs(got - ref)) < 2e-6
            again = np.array(qgx.qgx_fit_levels(list(hist), levels=list(np.linspace(0, 1, nlev))), dtype=np.float32)
            ref2 = o.fit_levels(hist, init=np.linspace(0, 1, nlev, dtype=np.float32))
            # from a far start the table is still moving when the sweep limit ends the fit, and levels that
            # pass through regions of (numerically) no mass take slightly different paths in the two
            # solvers: compare loosely there, and by the objective reached
            assert np.max(np.abs(again - ref2)) < 5e-5
            assert abs(o.objective(hist, again) - o.objective(hist, ref2)) <= 2e-3 * o.objective(hist, ref2) + 1e-300
            p = np.array(qgx.qgx_symbol_pmf(list(hist), list(ref)))
            assert np.max(np.abs(p - o.symbol_pmf(hist, ref))) < 1e-12
    # an empty histogram keeps the table
    assert qgx.qgx_fit_levels([0.0] * 64, levels=[0.0, 0.25, 1.0]) == [0.0, 0.25, 1.0]


def test_choice_of_code_matches_oracle(qgx):
    """Cost of a code on level counts and the choice between the four candidates (App. J), host side."""
    rng = np.random.default_rng(8)
    for nlev in (3, 9, 17, 32):
        for trial in range(6):
            counts = np.zeros(32, dtype=np.uint64)
            counts[:nlev] = rng.integers(0, 10 ** rng.integers(1, 7), size=nlev)
            if trial == 0:
                counts[:] = 0
            cur_o = [o.codebook_fixed(nlev, 64), o.codebook_elias(nlev, 64), o.codebook_huffman(rng.dirichlet(np.ones(nlev)), 64)][trial % 3]
            cur = qgx.qgx_codebook()
            cur.nlev, cur.maxlen, cur.subblock = cur_o.nlev, cur_o.maxlen, cur_o.subblock
            for j in range(nlev):
                cur.len[j], cur.code[j] = cur_o.len[j], cur_o.code[j]
            assert qgx.qgx_code_bits(counts, cur) == o.code_bits(counts, cur_o)
            for allow in (False, True):
                cb = qgx.qgx_codebook.from_buffer_copy(cur)
                win, bits = qgx.qgx_choose_code_host(counts, cb, allow)
                win_o, bits_o, cb_o = o.choose_code(counts, cur_o, allow)
                # the two Huffman builders may break ties differently: equal costs, not necessarily equal codes
                assert bits == [int(b) for b in bits_o] and win == win_o
                assert qgx.qgx_code_bits(counts, cb) == min(bits) and cb.subblock == 64

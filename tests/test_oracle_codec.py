"""Pins of the oracle's codec (Sec. 3.2, App. E, App. J): hand-worked stream, loss-less round
trip, bit counts in closed form, Huffman optimality and the code-length inequalities.  CPU only."""
import itertools
import math

import numpy as np
import pytest

from oracle import qgx_oracle as o
from conftest import read_golden


def test_hand_worked_bitstream():
    cb_codes = ([1, 2, 2], [0b0, 0b10, 0b11])
    norms = np.array([[1.0]], dtype=np.float32)
    sym = np.array([[1, 0, 0x82, 2, 0]], dtype=np.uint8)
    for row in read_golden("bitstream_worked.txt"):
        sub, bits, words = int(row[0]), int(row[1]), [int(w, 16) for w in row[2:]]
        cb = o.codebook_from(*cb_codes, subblock=sub)
        stream, bbits, total = o.encode(norms, sym, 5, cb)
        assert int(bbits[0, 0]) == bits and int(total[0]) == bits
        assert stream[0, :len(words)].tolist() == words
        assert not stream[0, len(words):].any()
        n2, s2 = o.decode(stream, bbits, 5, 5, cb)
        assert np.array_equal(s2, sym) and n2[0, 0] == 1.0


def _expected_bits(sym, d, bucket, cb):
    nb = o.nbuckets(d, bucket)
    G = bucket if (cb.subblock <= 0 or cb.subblock >= bucket) else cb.subblock
    lens = np.array(cb.lengths())
    out = np.zeros((sym.shape[0], nb), dtype=np.int64)
    for k in range(sym.shape[0]):
        for b in range(nb):
            s = sym[k, b * bucket:min(d, (b + 1) * bucket)]
            nsub = -(-len(s) // G) if G < bucket else 0
            idx = s & 31
            out[k, b] = 32 + 16 * nsub + lens[idx].sum() + np.count_nonzero(idx)
    return out


def _random_symbols(rng, K, d, nlev, p=None):
    idx = rng.choice(nlev, size=(K, d), p=p).astype(np.uint8)
    sign = (rng.integers(0, 2, size=(K, d)).astype(np.uint8) << 7) * (idx != 0)
    return (idx | sign).astype(np.uint8)


@pytest.mark.parametrize("nlev", list(range(2, 33)))
def test_round_trip_every_alphabet_size(nlev):
    rng = np.random.default_rng(nlev)
    K, d, bucket = 2, 700, 256                      # buckets of 256, 256, 188
    p = rng.dirichlet(np.ones(nlev) * 0.3)
    for cb in (o.codebook_fixed(nlev, 0), o.codebook_fixed(nlev, 64), o.codebook_huffman(p, 0),
               o.codebook_huffman(p, 128), o.codebook_huffman(p, 100), o.codebook_elias(nlev, 0),
               o.codebook_elias(nlev, 64)):
        sym = _random_symbols(rng, K, d, nlev, p)
        sym[0, :256] = 0                                 # an all-zero bucket
        sym[1, 256:512] = (nlev - 1) | 0x80              # an all-top-level, all-negative bucket
        norms = rng.uniform(0.1, 10, size=(K, 3)).astype(np.float32)
        norms[0, 0] = 0.0
        stream, bbits, total = o.encode(norms, sym, bucket, cb)
        exp = _expected_bits(sym, d, bucket, cb)
        assert np.array_equal(bbits.astype(np.int64), exp)
        assert np.array_equal(total.astype(np.int64), exp.sum(axis=1))
        words_used = ((exp + 31) // 32).sum(axis=1)
        for k in range(K):
            assert not stream[k, words_used[k]:].any()
        n2, s2 = o.decode(stream, bbits, d, bucket, cb)
        assert np.array_equal(s2, sym)
        assert n2.tobytes() == norms.tobytes()


def test_fixed_length_code_closed_form():
    # every symbol costs ceil(log2 nlev) bits, nonzero ones one more
    for nlev, L in [(2, 1), (3, 2), (4, 2), (9, 4), (16, 4), (17, 5), (32, 5)]:
        cb = o.codebook_fixed(nlev)
        assert cb.lengths() == [L] * nlev and cb.maxlen == L
        assert sorted(cb.codes()) == list(range(nlev))
        d = 64
        sym = np.full((1, d), 1, dtype=np.uint8)
        _, bbits, _ = o.encode(np.ones((1, 1), dtype=np.float32), sym, d, cb)
        assert int(bbits[0, 0]) == 32 + d * (L + 1)
        assert o.capacity_words(d, d, 0, L) == (32 + d * (L + 1) + 31) // 32


def _kraft(cb):
    return sum(2.0 ** -L for L in cb.lengths())


def _is_prefix_free(cb):
    words = [format(c, "0{}b".format(L)) for c, L in zip(cb.codes(), cb.lengths())]
    return not any(i != j and b.startswith(a) for i, a in enumerate(words) for j, b in enumerate(words))


def test_huffman_textbook_example():
    for row in read_golden("huffman_textbook.txt"):
        fields = " ".join(row).split("|")
        p = [float(x) for x in fields[0].split()]
        lens = [int(x) for x in fields[1].split()]
        el = float(fields[2])
        cb = o.codebook_huffman(p)
        assert sorted(cb.lengths()) == sorted(lens)
        assert abs(sum(pi * L for pi, L in zip(p, cb.lengths())) - el) < 1e-12
        assert _is_prefix_free(cb) and abs(_kraft(cb) - 1.0) < 1e-12


def _best_expected_length_bruteforce(p):
    # all length vectors with Kraft sum <= 1 (a prefix code exists iff Kraft holds)
    n = len(p)
    best = float("inf")
    for lens in itertools.product(range(1, n), repeat=n):
        if sum(2.0 ** -L for L in lens) <= 1.0 + 1e-12:
            best = min(best, sum(pi * L for pi, L in zip(p, lens)))
    return best


def test_huffman_is_optimal_and_within_one_bit_of_entropy():
    rng = np.random.default_rng(8)
    for n in (3, 4, 5, 6):
        for _ in range(6):
            p = rng.dirichlet(np.ones(n) * rng.uniform(0.2, 2.0))
            cb = o.codebook_huffman(p)
            el = float(np.dot(p, cb.lengths()))
            assert abs(el - _best_expected_length_bruteforce(p)) < 1e-9
    assert o.codebook_huffman([0.3, 0.7]).lengths() == [1, 1]
    for n in (9, 17, 18, 32):
        for _ in range(10):
            p = rng.dirichlet(np.ones(n) * rng.uniform(0.05, 3.0))
            cb = o.codebook_huffman(p)
            assert _is_prefix_free(cb)
            if cb.maxlen < 12:                 # not flattened by the length cap
                assert abs(_kraft(cb) - 1.0) < 1e-12
                H = -np.sum(p[p > 0] * np.log2(p[p > 0]))
                el = float(np.dot(p, cb.lengths()))
                assert H - 1e-9 <= el <= H + 1 + 1e-9        # Theorem (Huffman), App. J


def test_elias_recursive_code_table_and_properties():
    """The code Psi for an unknown symbol distribution (App. J): level j is sent as Elias' recursive code of
    j + 1.  Pinned to the published table of the code, to its length recursion and to the prefix property."""
    cb = o.codebook_elias(32, 0)
    words = [format(c, "0%db" % L) for c, L in zip(cb.codes(), cb.lengths())]
    for n, w in read_golden("elias_omega.txt"):
        assert words[int(n) - 1] == w
    # length recursion: len(1) = 1, len(n) = len(floor(log2 n)) + floor(log2 n) + 1
    def length(n):
        return 1 if n == 1 else length(n.bit_length() - 1) + n.bit_length()
    assert [len(w) for w in words] == [length(n) for n in range(1, 33)]
    assert cb.maxlen == 12 and max(len(w) for w in words) == 12
    # smaller values never get longer codewords; no codeword is a prefix of another; Kraft sum below one
    assert all(len(a) <= len(b) for a, b in zip(words, words[1:]))
    assert not any(a != b and b.startswith(a) for a in words for b in words)
    assert sum(2.0 ** -len(w) for w in words) < 1.0
    # every codeword ends the recursion with a 0 and every group before it starts with a 1
    assert all(w.endswith("0") for w in words) and all(w[0] == "1" for w in words[1:])
    # a smaller alphabet takes the first codewords
    cb9 = o.codebook_elias(9, 16)
    assert cb9.codes() == cb.codes()[:9] and cb9.lengths() == cb.lengths()[:9] and cb9.subblock == 16 and cb9.maxlen == 7
    # on a distribution that decays with the level it beats the fixed-length code, as the paper says it is meant to
    p = 0.5 ** np.arange(1, 18)
    p /= p.sum()
    assert np.dot(p, o.codebook_elias(17, 0).lengths()) < np.dot(p, o.codebook_fixed(17, 0).lengths())


def test_codeword_length_cap():
    p = np.array([2.0 ** -(j + 1) for j in range(32)])
    cb = o.codebook_huffman(p / p.sum())
    assert cb.maxlen <= 12 and _is_prefix_free(cb) and _kraft(cb) <= 1.0 + 1e-12
    cb0 = o.codebook_huffman(np.r_[1.0, np.zeros(16)])
    assert cb0.maxlen <= 12 and _is_prefix_free(cb0) and cb0.lengths()[0] == 1


def test_code_length_bound_and_sparsity():
    """bits <= C_b + (1 - p0) d + (H + 1) d (App. E) with the symbol frequencies as weights, and
    the number of sign bits equals the number of nonzero coordinates (sparsity lemma)."""
    rng = np.random.default_rng(17)
    d = 4096
    v = rng.standard_normal((4, d)).astype(np.float32)
    lev = np.array([0, 0.005, 0.01, 0.015, 0.02, 0.03, 0.04, 0.06, 1.0], dtype=np.float32)
    norms = o.bucket_norms(v, d)
    sym = o.quantize(v, d, lev, norms, seed=5, xid=0)
    idx = sym & 31
    p = np.bincount(idx.ravel(), minlength=len(lev)) / idx.size
    cb = o.codebook_huffman(p)
    _, bbits, total = o.encode(norms, sym, d, cb)
    H = -np.sum(p[p > 0] * np.log2(p[p > 0]))
    mean_bits = float(total.sum()) / 4
    assert mean_bits <= 32 + (1 - p[0]) * d + (H + 1) * d + 1e-6
    sign_bits = float(total.sum()) - 4 * 32 - float(np.array(cb.lengths())[idx].sum())
    assert sign_bits == np.count_nonzero(idx)
    # expected fraction of each symbol from the symbol-weight proposition (unweighted statistics
    # of the same vectors, fine bins); in particular E||Q(v)||_0 = (1 - p0) d
    hist = o.histogram(v, d, 1 << 16, weighted=False)
    p_prop = o.symbol_pmf(hist, lev)
    assert abs(p_prop.sum() - 1.0) < 1e-12
    assert np.max(np.abs(p_prop - p)) < 4.0 * math.sqrt(0.25 / idx.size) + 1e-3


def test_corrupt_and_short_streams_are_reported():
    rng = np.random.default_rng(2)
    nlev, d, bucket = 5, 300, 128
    cb = o.codebook_fixed(nlev, 32)                  # 3-bit code, 3 of the 8 patterns unused
    sym = _random_symbols(rng, 1, d, nlev)
    norms = np.ones((1, 3), dtype=np.float32)
    stream, bbits, _ = o.encode(norms, sym, bucket, cb)
    with pytest.raises(o.OracleError) as e:
        o.encode(norms, sym, bucket, cb, cap_words=20)
    assert e.value.status == o.CAPACITY
    short = bbits.copy()
    short[0, 1] -= 9
    with pytest.raises(o.OracleError) as e:
        o.decode(stream, short, d, bucket, cb)
    assert e.value.status == o.CORRUPT
    bad = stream.copy()
    bad[0, 1] ^= 0x00010000                          # second sub-block length of bucket 0
    with pytest.raises(o.OracleError) as e:
        o.decode(bad, bbits, d, bucket, cb)
    assert e.value.status == o.CORRUPT
    huge = bbits.copy()
    huge[0, 2] = 10 ** 9
    with pytest.raises(o.OracleError) as e:
        o.decode(stream, huge, d, bucket, cb)
    assert e.value.status == o.CORRUPT


def test_choice_of_code_by_measured_bits():
    """App. J: Huffman when the level frequencies are known or estimated, Elias' recursive code when they are not.
    The cost of a code on an exchange's level counts is pinned to the encoder itself (bits of the streams minus
    the bucket headers), the choice to cases whose winner is known beforehand."""
    rng = np.random.default_rng(21)
    K, d, bucket, nlev, sub = 3, 5 * 256 + 77, 256, 17, 64
    # small levels frequent, as after quantizing a dual vector
    p_true = np.array([2.0 ** -(j + 1) for j in range(nlev)]); p_true /= p_true.sum()
    idx = rng.choice(nlev, size=(K, d), p=p_true).astype(np.uint8)
    sym = idx | ((rng.integers(0, 2, size=(K, d)).astype(np.uint8) << 7) * (idx != 0))
    norms = rng.uniform(0.5, 2.0, size=(K, o.nbuckets(d, bucket))).astype(np.float32)
    counts = o.level_counts(sym, nlev)
    assert counts.sum() == K * d and np.array_equal(counts[:nlev], np.bincount(idx.ravel(), minlength=nlev).astype(np.uint64))
    nsub = sum(-(-min(bucket, d - b * bucket) // sub) for b in range(o.nbuckets(d, bucket)))
    for cb in (o.codebook_fixed(nlev, sub), o.codebook_elias(nlev, sub), o.codebook_huffman(p_true, sub)):
        _, bb, _ = o.encode(norms, sym, bucket, cb)
        payload = int(bb.astype(np.int64).sum()) - K * (32 * o.nbuckets(d, bucket) + 16 * nsub)
        assert o.code_bits(counts, cb) == payload                     # the cost formula is what the encoder spends
    # a Huffman code fitted to frequencies that no longer hold (large levels frequent) loses to Elias' code ...
    stale = o.codebook_huffman(p_true[::-1].copy(), sub)
    win, bits, chosen = o.choose_code(counts, stale, allow_rebuild=False)
    assert win == 2 and bits[2] < bits[0] and bits[2] < bits[3]
    assert chosen.lengths() == o.codebook_elias(nlev, sub).lengths() and chosen.subblock == sub
    # ... and to a Huffman code built from the counts themselves, which no prefix code beats on those counts
    win, bits, chosen = o.choose_code(counts, stale, allow_rebuild=True)
    assert win == 1 and bits[1] <= min(bits[0], bits[2], bits[3])
    # a current code that is already the best stays (ties go to the earlier candidate)
    win, bits2, _ = o.choose_code(counts, chosen, allow_rebuild=True)
    assert win == 0 and bits2[0] == bits[1]
    # uniform levels: nothing beats the fixed-length code by more than Huffman's rounding, and Elias is worst
    flat = np.zeros(32, dtype=np.uint64); flat[:16] = 1000
    win, bits, _ = o.choose_code(flat, o.codebook_elias(16, 0), allow_rebuild=False)
    assert win == 3 and bits[3] == 16 * 1000 * 4 + 15 * 1000

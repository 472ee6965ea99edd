"""Parity of the histogram kernel and of qgx_update_levels with the oracle."""
import numpy as np
import pytest
import torch

import qgx_inputs as gen
from oracle import qgx_oracle as o

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=["one thread per sub-block", "one worker per thread", "walk, then sums"])
def q(request):
    """Every test runs with both ways of spreading the decode pass (small vectors would only see the second)."""
    import paper_2308_09187_b200 as qgx
    ctx = qgx.qgx_create(0)
    qgx.qgx_set_decode_split(ctx, {"one thread per sub-block": qgx.QGX_SPLIT_NEVER, "one worker per thread": qgx.QGX_SPLIT_ALWAYS}.get(request.param, qgx.QGX_SPLIT_SYMBOLS))
    yield qgx, ctx
    qgx.qgx_destroy(ctx)


@pytest.mark.parametrize("K,d,bucket,nbins", [(3, 5000, 1024, 64), (8, 3 * 8192 + 100, 8192, 1024), (2, 40000, 16384, 1024),
                                              (4, 2048, 512, 256), (2, 1001, 256, 32)])
def test_histogram(q, K, d, bucket, nbins):
    qgx, ctx = q
    v = gen.student_t3((K, d), seed=d, device="cuda")
    vh = v.cpu().numpy()
    hu = qgx.qgx_histogram(ctx, v, bucket, nbins, weighted=False)
    hw = qgx.qgx_histogram(ctx, v, bucket, nbins, weighted=True)
    qgx.qgx_sync_status(ctx)
    n_ref = o.bucket_norms(vh, bucket)
    ref_u = o.histogram(vh, bucket, nbins, weighted=False)
    ref_w = o.histogram(vh, bucket, nbins, weighted=True)
    assert hu.cpu().numpy().sum() == K * d
    # integer counts agree except where a norm differs in its last bit (bin edges are fp32 products)
    assert np.abs(hu.cpu().numpy() - ref_u).sum() <= max(2, 1e-6 * K * d)
    assert np.allclose(hw.cpu().numpy(), ref_w, rtol=1e-6, atol=1e-9 * ref_w.sum())
    hl = qgx.qgx_histogram(ctx, v, bucket, nbins, norm_type=qgx.QGX_NORM_LINF, weighted=False)
    qgx.qgx_sync_status(ctx)
    assert np.array_equal(hl.cpu().numpy(), o.histogram(vh, bucket, nbins, o.LINF, False))
    assert n_ref.shape == (K, o.nbuckets(d, bucket))


def test_histogram_on_bin_edges(q):
    """Coordinates that sit on, just below and just above the bin edges (u * nbins an integer, or one fp32 step
    away from one), tiny and zero coordinates, and an all-zero bucket, under the max-norm (the bucket's largest
    entry is 1, so u = |v| exactly): the counts must equal the oracle's, which takes the division and the product."""
    qgx, ctx = q
    K, bucket, nbins = 2, 4096, 64
    rng = np.random.default_rng(11)
    edges = (rng.integers(0, nbins + 1, size=(K, 2 * bucket)) / nbins).astype(np.float32)
    step = rng.integers(-2, 3, size=edges.shape)
    v = edges.copy()
    for s_ in (-2, -1, 1, 2):
        for _ in range(abs(s_)):
            v = np.where(step == s_, np.nextafter(v, np.float32(2.0 if s_ > 0 else -1.0), dtype=np.float32), v)
    v = np.clip(v, 0.0, 1.0).astype(np.float32)
    v[:, 0] = 1.0
    v[:, bucket] = 1.0
    v[:, 1:9] = [0.0, 1e-45, 1e-30, 1e-10, 0.2499 / nbins, 0.25 / nbins, 0.9999999 / nbins, 1.0 / nbins]
    v *= np.where(rng.random(v.shape) < 0.5, -1.0, 1.0).astype(np.float32)
    v = np.concatenate([v, np.zeros((K, bucket), dtype=np.float32)], axis=1)
    got = qgx.qgx_histogram(ctx, torch.from_numpy(v).cuda(), bucket, nbins, norm_type=qgx.QGX_NORM_LINF, weighted=False)
    qgx.qgx_sync_status(ctx)
    ref = o.histogram(v, bucket, nbins, o.LINF, False)
    assert ref[0] >= K * bucket and ref[nbins - 1] >= 2 * K
    assert np.array_equal(got.cpu().numpy(), ref)


def test_update_levels_matches_oracle_refit(q):
    qgx, ctx = q
    K, d, bucket, nlev = 8, 4 * 8192, 8192, 17
    v = gen.gaussian((K, d), seed=1002, device="cuda")
    vh = v.cpu().numpy()
    for code_type in (qgx.QGX_CODE_FIXED, qgx.QGX_CODE_HUFFMAN):
        cfg = qgx.make_quant_cfg(np.linspace(0, 1, nlev), bucket, qgx.qgx_build_codebook_fixed(nlev, 128), 1,
                                 code_type=code_type, nbins=1024)
        hist = qgx.qgx_update_levels(ctx, v, cfg, qgx.QGX_REFIT_FIRST)
        cbo = o.codebook_fixed(nlev, 128)
        lev_ref, hist_ref = o.refit(vh, bucket, 1024, np.linspace(0, 1, nlev, dtype=np.float32), cbo, True, code_type)
        assert np.allclose(hist, hist_ref, rtol=1e-6, atol=1e-9 * hist_ref.sum())
        lev = np.array(cfg.level_list(), dtype=np.float32)
        assert o.check_levels(lev) == o.OK
        assert np.max(np.abs(lev - lev_ref)) <= 1e-6
        # the fitted table is as good as the oracle's on the oracle's objective
        assert o.objective(hist_ref, lev) <= o.objective(hist_ref, lev_ref) * (1 + 1e-4) + 1e-12
        # same expected code length under the symbol weights; the codes themselves may differ in ties
        p = o.symbol_pmf(hist_ref, lev_ref)
        assert abs(np.dot(p, cfg.cb.lengths()) - np.dot(p, cbo.lengths())) < 1e-3
        assert cfg.cb.subblock == 128 and cfg.cb.nlev == nlev
        # a second refit continues from the fitted table and keeps it (already converged)
        qgx.qgx_update_levels(ctx, v, cfg, qgx.QGX_REFIT_CONTINUE)
        lev2 = np.array(cfg.level_list(), dtype=np.float32)
        lev_ref2, _ = o.refit(vh, bucket, 1024, lev_ref, cbo, False, code_type)
        assert np.max(np.abs(lev2 - lev_ref2)) <= 1e-6


def test_linf_normalisation_refit_and_exchange(q):
    """The max-norm variant end to end: histogram and level fit on u = |v| / max|v|, then a fused exchange
    with the fitted table.  Max norms are exact, so streams and mean are bit-identical to the oracle's."""
    qgx, ctx = q
    K, d, bucket, nlev, sub = 4, 3 * 4096 + 500, 4096, 17, 64
    v = gen.student_t3((K, d), seed=77, device="cuda") * 0.01
    vh = v.cpu().numpy()
    cfg = qgx.make_quant_cfg(np.linspace(0, 1, nlev), bucket, qgx.qgx_build_codebook_fixed(nlev, sub), 9,
                             norm_type=qgx.QGX_NORM_LINF, code_type=qgx.QGX_CODE_HUFFMAN, nbins=1024)
    hist = qgx.qgx_update_levels(ctx, v, cfg, qgx.QGX_REFIT_FIRST)
    cbo = o.codebook_fixed(nlev, sub)
    lev_ref, hist_ref = o.refit(vh, bucket, 1024, np.linspace(0, 1, nlev, dtype=np.float32), cbo, True, o.CODE_HUFFMAN,
                                norm_type=o.LINF)
    assert np.allclose(hist, hist_ref, rtol=1e-6, atol=1e-9 * hist_ref.sum())
    lev = np.array(cfg.level_list(), dtype=np.float32)
    assert o.check_levels(lev) == o.OK
    assert np.max(np.abs(lev - lev_ref)) <= 1e-6
    # the max norm spreads u over [0, 1]: the fitted table uses the upper half of the range too
    assert lev[-2] > 0.3
    # exchange with the library's table and code on both sides
    cbo = o.codebook_from(cfg.cb.lengths(), cfg.cb.codes(), subblock=sub)
    mean, total = qgx.qgx_exchange(ctx, v, cfg, 12, slot=0)
    qgx.qgx_sync_status(ctx)
    m_or, t_or = o.exchange(vh, bucket, lev, cbo, 9, 12, norm_type=o.LINF)
    assert np.array_equal(total.cpu().numpy().astype(np.uint64), t_or)
    assert np.array_equal(mean.cpu().numpy(), m_or)
    nb = o.nbuckets(d, bucket)
    stream, bbits, _ = qgx.exchange_stream_tensors(ctx, 0, K, nb)
    n_ref = o.bucket_norms(vh, bucket, o.LINF)
    st_ref, bb_ref, _ = o.encode(n_ref, o.quantize(vh, bucket, lev, n_ref, 9, 12), bucket, cbo)
    assert np.array_equal(bbits.cpu().numpy().view(np.uint32), bb_ref)
    used = ((bb_ref.astype(np.int64) + 31) // 32).sum(axis=1)
    sh = stream.cpu().numpy().view(np.uint32)
    for k in range(K):
        assert np.array_equal(sh[k, :used[k]], st_ref[k, :used[k]])

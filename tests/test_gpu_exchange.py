"""Parity of the fused exchange (quantize+encode kernel, decode+average kernel) with the oracle
and with the four separate calls, through the C ABI."""
import numpy as np
import pytest
import torch

import qgx_inputs as gen
from oracle import qgx_oracle as o

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=["one thread per sub-block", "one worker per thread", "staged encode", "walk, then sums"])
def q(request):
    """Every test runs with the three ways of spreading the decode pass (one thread per sub-block over all workers;
    one worker per thread with the values added by a second kernel; the walk alone with the sums formed from the
    symbol bytes) and with the staged encode kernel (the shapes it does not take fall back to the
    bucket-in-registers kernel)."""
    import paper_2308_09187_b200 as qgx
    ctx = qgx.qgx_create(0)
    split = {"one worker per thread": qgx.QGX_SPLIT_ALWAYS, "walk, then sums": qgx.QGX_SPLIT_SYMBOLS}
    qgx.qgx_set_decode_split(ctx, split.get(request.param, qgx.QGX_SPLIT_NEVER))
    qgx.qgx_set_encode_path(ctx, qgx.QGX_ENCODE_STAGED if request.param == "staged encode" else qgx.QGX_ENCODE_REGISTERS)
    yield qgx, ctx
    qgx.qgx_destroy(ctx)


def _levels(rng, nlev, top=0.2):
    inner = np.sort(rng.uniform(0.001, top, size=nlev - 2))
    return np.r_[0.0, inner, 1.0].astype(np.float32)


def _used_words(bbits):
    return ((bbits.astype(np.int64) + 31) // 32).sum(axis=1)


CASES = [
    # K, d, bucket, nlev, subblock, huffman
    (4, 2048, 512, 9, 128, False),        # c1 shape: 4 sub-blocks per bucket
    (8, 3 * 8192 + 1000, 8192, 17, 128, True),   # c2 shape, ragged tail
    (3, 2 * 16384 + 1728, 16384, 17, 128, True), # c5 bucket, short last bucket
    (16, 1728, 4096, 9, 128, True),       # c3's smallest tensor: one partial bucket
    (5, 40000, 4096, 17, 64, True),
    (2, 70000, 2048, 32, 32, False),
    (2, 1001, 256, 3, 32, True),          # d not a multiple of 4
    # rows a multiple of 32 floats apart: the whole buckets qualify for the staged encode kernel
    (4, 5 * 16384, 16384, 17, 64, True),
    (6, 7 * 4096 + 2048, 4096, 9, 32, True),      # short last bucket
    (3, 9 * 1024, 1024, 17, 128, False),          # sixteen buckets per group, a last group of nine
    (2, 3 * 2048 + 32, 2048, 32, 64, True),
    (5, 21 * 8192, 8192, 17, 128, True),
]


@pytest.mark.parametrize("K,d,bucket,nlev,sub,huff", CASES)
def test_fused_exchange_matches_oracle_and_steps(q, K, d, bucket, nlev, sub, huff):
    qgx, ctx = q
    rng = np.random.default_rng(K * 1000 + nlev)
    v = gen.gaussian_mixture((K, d), seed=d + 1, device="cuda")
    v[K - 1, : min(d, bucket)] = 0.0
    vh = v.cpu().numpy()
    lev = _levels(rng, nlev)
    p = rng.dirichlet(np.ones(nlev) * 0.4)
    cb = qgx.qgx_build_codebook_huffman(list(p), sub) if huff else qgx.qgx_build_codebook_fixed(nlev, sub)
    cbo = o.codebook_from(cb.lengths(), cb.codes(), subblock=sub)
    seed, xid = 1005, 41
    cfg = qgx.make_quant_cfg(lev, bucket, cb, seed)
    nb = o.nbuckets(d, bucket)

    mean, total = qgx.qgx_exchange(ctx, v, cfg, xid, slot=0)
    qgx.qgx_sync_status(ctx)
    stream, bbits, tot2 = qgx.exchange_stream_tensors(ctx, 0, K, nb)
    stream_h = stream.cpu().numpy().view(np.uint32)
    bbits_h = bbits.cpu().numpy().view(np.uint32)

    # the separate calls on the same input: same norms (same reduction), then the oracle on those norms
    norms, sym = qgx.qgx_quantize(ctx, v, bucket, lev, qgx.QGX_NORM_L2, seed, xid)
    qgx.qgx_sync_status(ctx)
    n_gpu = norms.cpu().numpy()
    assert np.all(np.abs(n_gpu - o.bucket_norms(vh, bucket)) <= np.spacing(n_gpu))
    s_ref = o.quantize(vh, bucket, lev, n_gpu, seed, xid)
    assert np.array_equal(sym.cpu().numpy(), s_ref)
    st_ref, bb_ref, tot_ref = o.encode(n_gpu, s_ref, bucket, cbo)
    assert np.array_equal(bbits_h, bb_ref)
    assert np.array_equal(total.cpu().numpy().astype(np.uint64), tot_ref)
    assert np.array_equal(tot2.cpu().numpy().astype(np.uint64), tot_ref)
    used = _used_words(bb_ref)
    for k in range(K):
        assert np.array_equal(stream_h[k, :used[k]], st_ref[k, :used[k]])      # the compact stream, bit for bit
    assert np.array_equal(mean.cpu().numpy(), o.average(n_gpu, s_ref, bucket, lev))
    m_or, t_or = o.exchange(vh, bucket, lev, cbo, seed, xid)
    flips = np.count_nonzero(o.quantize(vh, bucket, lev, o.bucket_norms(vh, bucket), seed, xid) != s_ref)
    assert flips <= max(1, int(1e-6 * K * d))
    if flips == 0 and np.array_equal(n_gpu, o.bucket_norms(vh, bucket)):
        assert np.array_equal(mean.cpu().numpy(), m_or) and np.array_equal(t_or, tot_ref)
    scale = float(n_gpu.max())
    assert np.max(np.abs(mean.cpu().numpy() - m_or)) <= 1e-5 * scale


def test_second_slot_and_repeatability(q):
    qgx, ctx = q
    K, d, bucket = 4, 50000, 4096
    v = gen.gaussian((K, d), seed=9, device="cuda")
    lev = np.linspace(0, 1, 17, dtype=np.float32) ** 2
    cfg = qgx.make_quant_cfg(lev, bucket, qgx.qgx_build_codebook_fixed(17, 128), 77)
    m0, t0 = qgx.qgx_exchange(ctx, v, cfg, 2, slot=0)
    m1, t1 = qgx.qgx_exchange(ctx, v, cfg, 3, slot=1)
    m2, t2 = qgx.qgx_exchange(ctx, v, cfg, 2, slot=1)
    qgx.qgx_sync_status(ctx)
    assert torch.equal(m0, m2) and torch.equal(t0, t2)          # same exchange id: same rounding
    assert not torch.equal(m0, m1)                              # another exchange id: fresh randomness
    # unbiased: the mean over workers of Q(v_k) is close to the mean of v_k
    err = (m0 - v.mean(0)).abs().max().item()
    assert err < 0.5 * v.abs().max().item()


def test_fused_capacity_and_nonfinite(q):
    qgx, ctx = q
    K, d, bucket = 2, 9000, 1024
    v = gen.gaussian((K, d), seed=3, device="cuda")
    v[1, 5000] = float("inf")
    lev = np.linspace(0, 1, 9, dtype=np.float32)
    cfg = qgx.make_quant_cfg(lev, bucket, qgx.qgx_build_codebook_fixed(9, 128), 5)
    qgx.qgx_exchange(ctx, v, cfg, 0, slot=0)
    assert qgx.qgx_sync_status(ctx, check=False) == qgx.QGX_ERR_NONFINITE
    v[1, 5000] = 1.0
    qgx.qgx_exchange(ctx, v, cfg, 0, slot=0)
    assert qgx.qgx_sync_status(ctx, check=False) == qgx.QGX_OK
    bad = qgx.make_quant_cfg(lev, bucket, qgx.qgx_build_codebook_fixed(9, 96), 5)      # 96 is not a fused sub-block size
    with pytest.raises(qgx.QgxError):
        qgx.qgx_exchange(ctx, v, bad, 0, slot=0)


def test_layerwise_segments_c3_shape(q):
    """c3 at reduced size: tensors of different sizes (one a partial bucket), heavy tails, per-tensor scales,
    per-tensor fitted tables and Huffman codes, K = 16, bucket 4096."""
    qgx, ctx = q
    sizes = [1728, 36864, 73728, 1728, 147456]
    lw = gen.c3_layerwise(K=16, sizes=sizes, device="cuda")
    K, d = lw.v.shape
    vh = lw.v.cpu().numpy()
    cfgs, at = [], 0
    for n in sizes:
        cfg = qgx.make_quant_cfg(np.linspace(0, 1, lw.nlev), lw.bucket, qgx.qgx_build_codebook_fixed(lw.nlev, 128), lw.seed,
                                 code_type=qgx.QGX_CODE_HUFFMAN)
        qgx.qgx_update_levels(ctx, lw.v[:, at:at + n].contiguous(), cfg, qgx.QGX_REFIT_FIRST)
        cfgs.append(cfg)
        at += n
    mean, total = qgx.qgx_exchange_segments(ctx, lw.v, sizes, cfgs, 9)
    qgx.qgx_sync_status(ctx)
    mean_h = mean.cpu().numpy()
    bits_ref = np.zeros(K, dtype=np.uint64)
    at = 0
    for n, cfg in zip(sizes, cfgs):
        part = np.ascontiguousarray(vh[:, at:at + n])
        lev = np.array(cfg.level_list(), dtype=np.float32)
        cbo = o.codebook_from(cfg.cb.lengths(), cfg.cb.codes(), subblock=128)
        norms = o.bucket_norms(part, lw.bucket)
        sym = o.quantize(part, lw.bucket, lev, norms, lw.seed, 9, coord_base=at)
        _, _, tb = o.encode(norms, sym, lw.bucket, cbo)
        bits_ref += tb
        ref = o.average(norms, sym, lw.bucket, lev)
        scale = float(norms.max())
        assert np.max(np.abs(mean_h[at:at + n] - ref)) <= 1e-5 * scale
        assert np.count_nonzero(mean_h[at:at + n] != ref) <= max(1, int(1e-6 * K * n) * K)
        at += n
    assert np.array_equal(total.cpu().numpy().astype(np.uint64), bits_ref) or \
        np.max(np.abs(total.cpu().numpy().astype(np.int64) - bits_ref.astype(np.int64))) <= 16


@pytest.mark.parametrize("K,d,bucket,nlev,sub", [(3, 2 * 4096 + 777, 4096, 17, 64), (2, 20000, 2048, 32, 128),
                                                   (4, 3000, 512, 9, 32)])
def test_elias_recursive_code(q, K, d, bucket, nlev, sub):
    """The second prefix code of App. J through the same kernels: separate calls, fused exchange and a refit that
    keeps this code, bit for bit against the oracle."""
    qgx, ctx = q
    rng = np.random.default_rng(nlev)
    v = gen.gaussian_mixture((K, d), seed=3 * d, device="cuda")
    vh = v.cpu().numpy()
    lev = _levels(rng, nlev, top=0.4)
    cb = qgx.qgx_build_codebook_elias(nlev, sub)
    cbo = o.codebook_elias(nlev, sub)
    assert cb.codes() == cbo.codes() and cb.lengths() == cbo.lengths()
    seed, xid = 31, 5
    norms, sym = qgx.qgx_quantize(ctx, v, bucket, lev, qgx.QGX_NORM_L2, seed, xid)
    qgx.qgx_sync_status(ctx)
    n_gpu = norms.cpu().numpy()
    s_ref = o.quantize(vh, bucket, lev, n_gpu, seed, xid)
    assert np.array_equal(sym.cpu().numpy(), s_ref)
    stream, bbits, total = qgx.qgx_encode(ctx, norms, sym, bucket, cb)
    qgx.qgx_sync_status(ctx)
    st_ref, bb_ref, tot_ref = o.encode(n_gpu, s_ref, bucket, cbo)
    assert np.array_equal(bbits.cpu().numpy().view(np.uint32), bb_ref)
    assert np.array_equal(stream.cpu().numpy().view(np.uint32), st_ref)
    n2, s2 = qgx.qgx_decode(ctx, stream, bbits, d, bucket, cb)
    qgx.qgx_sync_status(ctx)
    assert np.array_equal(s2.cpu().numpy(), s_ref)
    # fused
    cfg = qgx.make_quant_cfg(lev, bucket, cb, seed, code_type=qgx.QGX_CODE_ELIAS)
    mean, tot = qgx.qgx_exchange(ctx, v, cfg, xid, slot=1)
    qgx.qgx_sync_status(ctx)
    assert np.array_equal(tot.cpu().numpy().astype(np.uint64), tot_ref)
    assert np.array_equal(mean.cpu().numpy(), o.average(n_gpu, s_ref, bucket, lev))
    fs, fb, _ = qgx.exchange_stream_tensors(ctx, 1, K, o.nbuckets(d, bucket))
    used = _used_words(bb_ref)
    fsh = fs.cpu().numpy().view(np.uint32)
    for k in range(K):
        assert np.array_equal(fsh[k, :used[k]], st_ref[k, :used[k]])
    # a refit moves the levels and leaves this code in place
    qgx.qgx_update_levels(ctx, v, cfg, qgx.QGX_REFIT_FIRST)
    lev_ref, _ = o.refit(vh, bucket, 1024, lev.copy(), cbo, True, o.CODE_ELIAS)
    assert np.max(np.abs(np.array(cfg.level_list(), dtype=np.float32) - lev_ref)) <= 1e-6
    assert cfg.cb.codes() == cbo.codes() and cfg.cb.lengths() == cbo.lengths() and cfg.cb.subblock == sub


def test_choice_of_code_by_measured_bits(q):
    """App. J: the level counts of an exchange decide the code of the next ones.  Counts, costs and winner agree
    with the oracle, and the next exchange spends exactly the predicted bits."""
    qgx, ctx = q
    K, d, bucket, nlev, sub = 4, 6 * 4096 + 1000, 4096, 17, 64
    v = gen.gaussian_mixture((K, d), seed=31, device="cuda")
    vh = v.cpu().numpy()
    lev = np.r_[0.0, np.geomspace(2e-3, 0.2, nlev - 2), 1.0].astype(np.float32)
    # a code fitted to frequencies that do not hold: the large levels frequent
    stale_p = np.array([2.0 ** -(nlev - j) for j in range(nlev)])
    cb = qgx.qgx_build_codebook_huffman(list(stale_p / stale_p.sum()), sub)
    cbo = o.codebook_from(cb.lengths(), cb.codes(), subblock=sub)
    cfg = qgx.make_quant_cfg(lev, bucket, cb, 5)
    qgx.qgx_set_keep_symbols(ctx, True)
    try:
        _, total0 = qgx.qgx_exchange(ctx, v, cfg, 6, slot=0)
        counts = qgx.qgx_level_counts(ctx)
        qgx.qgx_sync_status(ctx)
        sym_ref = o.quantize(vh, bucket, lev, o.bucket_norms(vh, bucket), 5, 6)
        counts_ref = o.level_counts(sym_ref, nlev)
        got = counts.cpu().numpy().astype(np.uint64)
        flips = int(np.abs(got.astype(np.int64) - counts_ref.astype(np.int64)).sum())
        assert got.sum() == K * d and flips <= 2 * max(1, int(1e-6 * K * d))
        nsub = sum(-(-min(bucket, d - b * bucket) // sub) for b in range(o.nbuckets(d, bucket)))
        headers = K * (32 * o.nbuckets(d, bucket) + 16 * nsub)
        assert int(total0.sum().item()) == headers + qgx.qgx_code_bits(got, cfg.cb)
        for allow, want in ((False, 2), (True, 1)):          # Elias beats the stale code; a code from the counts beats both
            cfg2 = qgx.make_quant_cfg(lev, bucket, cb, 5)
            win, bits, _ = qgx.qgx_choose_code(ctx, cfg2, allow)
            win_o, bits_o, _ = o.choose_code(got, cbo, allow)
            assert win == want == win_o and bits == [int(x) for x in bits_o]
            _, total1 = qgx.qgx_exchange(ctx, v, cfg2, 6, slot=1)
            qgx.qgx_sync_status(ctx)
            assert int(total1.sum().item()) == headers + bits[win] < int(total0.sum().item())
    finally:
        qgx.qgx_set_keep_symbols(ctx, False)


def test_bounded_wait_runs_out_and_the_context_stays_usable(q):
    """A bucket waits for the word counts of its worker's earlier buckets; the wait is bounded.  With the first
    buckets left unencoded on purpose and a small limit the waiting buckets give up: QGX_ERR_TIMEOUT comes back, the
    kernel ends by itself, and the next exchange on the same context is exact again."""
    qgx, ctx = q
    K, d, bucket = 3, 12 * 1024, 1024
    v = gen.gaussian((K, d), seed=4, device="cuda")
    lev = np.linspace(0, 1, 9, dtype=np.float32)
    cfg = qgx.make_quant_cfg(lev, bucket, qgx.qgx_build_codebook_fixed(9, 64), 3)
    want, tot = qgx.qgx_exchange(ctx, v, cfg, 1, slot=0)
    qgx.qgx_sync_status(ctx)
    want, tot = want.clone(), tot.clone()
    qgx.qgx_set_wait_limit(ctx, 50)
    qgx.qgx_debug_skip_buckets(ctx, 2)
    qgx.qgx_exchange(ctx, v, cfg, 1, slot=0)
    assert qgx.qgx_sync_status(ctx, check=False) == qgx.QGX_ERR_TIMEOUT
    qgx.qgx_set_wait_limit(ctx, 1 << 22)
    again, tot2 = qgx.qgx_exchange(ctx, v, cfg, 1, slot=0)
    qgx.qgx_sync_status(ctx)
    assert torch.equal(again, want) and torch.equal(tot2, tot)


def test_decode_pass_alone_and_corrupt_streams(q):
    """The receiving side on its own reproduces the mean; streams changed behind its back are reported as corrupt
    (or decode to something else where the change happens to be a valid stream), never read out of range."""
    qgx, ctx = q
    K, d, bucket, sub = 4, 9 * 2048 + 600, 2048, 64
    v = gen.gaussian_mixture((K, d), seed=8, device="cuda")
    lev = np.r_[0.0, np.geomspace(1e-3, 0.3, 15), 1.0].astype(np.float32)
    p = np.array([2.0 ** -(j + 1) for j in range(17)])
    cfg = qgx.make_quant_cfg(lev, bucket, qgx.qgx_build_codebook_huffman(list(p / p.sum()), sub), 21)
    nb = o.nbuckets(d, bucket)
    mean, _ = qgx.qgx_exchange(ctx, v, cfg, 2, slot=1)
    qgx.qgx_sync_status(ctx)
    mean = mean.clone()
    assert torch.equal(qgx.qgx_exchange_decode(ctx, K, d, cfg, slot=1), mean)
    qgx.qgx_sync_status(ctx)
    stream, bbits, _ = qgx.exchange_stream_tensors(ctx, 1, K, nb)
    keep_s, keep_b = stream.clone(), bbits.clone()
    # 1. a sub-block length in a bucket header that disagrees with the bits that follow
    stream[1, 1] ^= 0x0004
    qgx.qgx_exchange_decode(ctx, K, d, cfg, slot=1)
    assert qgx.qgx_sync_status(ctx, check=False) == qgx.QGX_ERR_CORRUPT
    stream.copy_(keep_s)
    # 2. a bucket length beyond anything the buffers hold
    bbits[2, 3] = 0x7fffffff
    qgx.qgx_exchange_decode(ctx, K, d, cfg, slot=1)
    assert qgx.qgx_sync_status(ctx, check=False) == qgx.QGX_ERR_CORRUPT
    bbits.copy_(keep_b)
    # 3. random bits flipped all over the payload
    noise = torch.randint(0, 2 ** 31 - 1, stream.shape, dtype=torch.int32, device="cuda", generator=torch.Generator("cuda").manual_seed(1))
    stream ^= noise
    qgx.qgx_exchange_decode(ctx, K, d, cfg, slot=1)
    assert qgx.qgx_sync_status(ctx, check=False) == qgx.QGX_ERR_CORRUPT
    stream.copy_(keep_s)
    assert torch.equal(qgx.qgx_exchange_decode(ctx, K, d, cfg, slot=1), mean)
    qgx.qgx_sync_status(ctx)

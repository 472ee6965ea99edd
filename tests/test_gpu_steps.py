"""Parity of the four steps of an exchange (quantize, encode, decode, average) against the
oracle, through the C ABI, on seeded inputs that span several tiles and a ragged tail."""
import numpy as np
import pytest
import torch

import qgx_inputs as gen
from oracle import qgx_oracle as o

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def q():
    import paper_2308_09187_b200 as qgx
    ctx = qgx.qgx_create(0)
    yield qgx, ctx
    qgx.qgx_destroy(ctx)


def _u32(t):
    return t.cpu().numpy().view(np.uint32)


def _codebooks(qgx, nlev, sub, rng):
    """The same prefix code for both sides: (library struct, oracle struct)."""
    p = rng.dirichlet(np.ones(nlev) * 0.5)
    out = []
    for cb in (qgx.qgx_build_codebook_fixed(nlev, sub), qgx.qgx_build_codebook_huffman(list(p), sub)):
        out.append((cb, o.codebook_from(cb.lengths(), cb.codes(), subblock=sub)))
    return out


CASES = [
    # K, d, bucket, nlev, subblock
    (3, 2048, 512, 9, 128),
    (2, 5000, 1024, 17, 64),       # tail bucket of 904
    (4, 40000, 8192, 17, 128),     # tail bucket of 7232
    (2, 50000, 16384, 32, 256),
    (1, 1728, 4096, 9, 128),       # one partial bucket
    (2, 4100, 4096, 5, 0),         # no sub-blocks; tail bucket of 4
    (3, 1001, 256, 2, 32),         # d not a multiple of 4: scalar path
]


@pytest.mark.parametrize("K,d,bucket,nlev,sub", CASES)
def test_quantize_encode_decode_average(q, K, d, bucket, nlev, sub):
    qgx, ctx = q
    rng = np.random.default_rng(d + nlev)
    v = gen.gaussian((K, d), seed=d, device="cuda")
    v[0, : min(d, bucket)] = 0.0                       # an all-zero bucket
    vh = v.cpu().numpy()
    inner = np.sort(rng.uniform(0.001, 0.2, size=nlev - 2)) if nlev > 2 else np.array([])
    lev = np.r_[0.0, inner, 1.0].astype(np.float32)
    seed, xid = 0xABCDEF0123456789 & (2**64 - 1), 7

    norms, sym = qgx.qgx_quantize(ctx, v, bucket, lev, qgx.QGX_NORM_L2, seed, xid)
    qgx.qgx_sync_status(ctx)
    n_ref = o.bucket_norms(vh, bucket)
    n_gpu = norms.cpu().numpy()
    assert np.all(np.abs(n_gpu - n_ref) <= np.spacing(n_ref))          # within 1 ulp (fp64 sums in another order)
    # symbols are bit-exact given identical norms
    s_ref = o.quantize(vh, bucket, lev, n_gpu, seed, xid)
    assert np.array_equal(sym.cpu().numpy(), s_ref)
    # norms supplied: the same symbols again from the oracle's own norms
    n_in = torch.from_numpy(n_ref).cuda()
    _, sym2 = qgx.qgx_quantize(ctx, v, bucket, lev, qgx.QGX_NORM_L2, seed, xid, flags=qgx.QGX_NORMS_SUPPLIED, norms=n_in)
    assert np.array_equal(sym2.cpu().numpy(), o.quantize(vh, bucket, lev, n_ref, seed, xid))

    for cb, cbo in _codebooks(qgx, nlev, sub, rng):
        stream, bbits, total = qgx.qgx_encode(ctx, norms, sym, bucket, cb)
        qgx.qgx_sync_status(ctx)
        st_ref, bb_ref, tot_ref = o.encode(n_gpu, s_ref, bucket, cbo)
        assert np.array_equal(_u32(bbits), bb_ref)
        assert np.array_equal(total.cpu().numpy().astype(np.uint64), tot_ref)
        assert np.array_equal(_u32(stream), st_ref)                      # bitstream bit-exact, unused words zero
        n2, s2 = qgx.qgx_decode(ctx, stream, bbits, d, bucket, cb)
        qgx.qgx_sync_status(ctx)
        assert np.array_equal(s2.cpu().numpy(), s_ref)
        assert n2.cpu().numpy().tobytes() == n_gpu.tobytes()
        # and the library decodes what the oracle encoded
        n3, s3 = qgx.qgx_decode(ctx, torch.from_numpy(st_ref.view(np.int32)).cuda(),
                                torch.from_numpy(bb_ref.view(np.int32)).cuda(), d, bucket, cb)
        qgx.qgx_sync_status(ctx)
        assert np.array_equal(s3.cpu().numpy(), s_ref)

    out = qgx.qgx_average(ctx, norms, sym, bucket, lev)
    qgx.qgx_sync_status(ctx)
    assert np.array_equal(out.cpu().numpy(), o.average(n_gpu, s_ref, bucket, lev))


def test_supplied_norms_smaller_than_the_coordinates(q):
    """Norms handed in by the caller are used as they are: where one is smaller than a coordinate's magnitude the
    normalized coordinate is clamped to 1 (the top level), as in the oracle; nothing is read out of range."""
    qgx, ctx = q
    K, d, bucket, nlev = 3, 5 * 2048 + 100, 2048, 17
    v = gen.gaussian_mixture((K, d), seed=5, device="cuda")
    vh = v.cpu().numpy()
    lev = np.r_[0.0, np.sort(np.random.default_rng(5).uniform(0.001, 0.3, nlev - 2)), 1.0].astype(np.float32)
    for factor in (0.5, 0.01):
        n_small = (o.bucket_norms(vh, bucket) * np.float32(factor)).astype(np.float32)
        _, sym = qgx.qgx_quantize(ctx, v, bucket, lev, qgx.QGX_NORM_L2, 17, 4, flags=qgx.QGX_NORMS_SUPPLIED,
                                  norms=torch.from_numpy(n_small).cuda())
        qgx.qgx_sync_status(ctx)
        s_ref = o.quantize(vh, bucket, lev, n_small, 17, 4)
        assert np.array_equal(sym.cpu().numpy(), s_ref)
        assert np.count_nonzero((s_ref & 31) == nlev - 1) > 0          # some coordinates did exceed their norm


LEVEL_SETS = {
    "uniform17": np.linspace(0, 1, 17),
    "uniform32": np.linspace(0, 1, 32),
    "exponential": np.r_[0.0, 2.0 ** np.arange(-15, 1)],
    "below_2^-16": np.r_[0.0, 3e-6, 1.1e-5, 4e-4, 2e-2, 1.0],
    "two_levels_in_one_bin": np.r_[0.0, 0.01, 0.5, 0.5005, 0.501, 1.0],      # every coordinate takes the exact routine
    "narrow_interval": np.r_[0.0, 0.05, 0.25, 0.2500004, 0.7, 1.0],
    "two": np.r_[0.0, 1.0],
}


@pytest.mark.parametrize("name", sorted(LEVEL_SETS))
def test_rounding_agrees_with_definition_1_on_awkward_levels(q, name):
    """Symbols bit for bit on level sets that stress the kernel's rounding tables, with coordinates
    placed on the levels, next to them, at zero and at |v| = norm."""
    qgx, ctx = q
    lev = LEVEL_SETS[name].astype(np.float32)
    K, d, bucket = 2, 1 << 18, 4096
    v = gen.gaussian((K, d), seed=77, device="cuda").cpu().numpy()
    rng = np.random.default_rng(5)
    v[0, :d // 2] = (rng.random(d // 2) ** 4).astype(np.float32) * np.sign(v[0, :d // 2]) * 60.0      # spread over all octaves
    nb = d // bucket
    # second worker: buckets whose coordinates sit on multiples of the levels
    for b in range(0, nb, 2):
        seg = v[1, b * bucket:(b + 1) * bucket]
        seg[:] = 0.0
        seg[0] = 100.0                                  # dominates the norm: u = l_j reproduced closely below
        j = rng.integers(0, len(lev), bucket - 1)
        off = rng.integers(-2, 3, bucket - 1)
        val = lev[j] * np.float32(100.0)
        for _ in range(2):
            val = np.where(off > 0, np.nextafter(val, np.float32(np.inf)), np.where(off < 0, np.nextafter(val, np.float32(0)), val))
        seg[1:] = val * np.where(rng.random(bucket - 1) < 0.5, -1, 1)
    v[1, bucket:2 * bucket] = 0.0
    v[1, bucket + 5] = -3.0                             # a bucket with one nonzero coordinate: u = 1
    vd = torch.from_numpy(v).cuda()
    for norm_type in (qgx.QGX_NORM_L2, qgx.QGX_NORM_LINF):
        norms, sym = qgx.qgx_quantize(ctx, vd, bucket, lev, norm_type, 99, 4)
        qgx.qgx_sync_status(ctx)
        n_gpu = norms.cpu().numpy()
        assert np.array_equal(sym.cpu().numpy(), o.quantize(v, bucket, lev, n_gpu, 99, 4))


def test_linf_norm_and_heavy_tails(q):
    qgx, ctx = q
    K, d, bucket = 2, 9000, 4096
    v = gen.student_t3((K, d), seed=3, device="cuda") * 0.01
    vh = v.cpu().numpy()
    lev = np.linspace(0, 1, 9, dtype=np.float32)
    norms, sym = qgx.qgx_quantize(ctx, v, bucket, lev, qgx.QGX_NORM_LINF, 5, 0)
    qgx.qgx_sync_status(ctx)
    n_ref = o.bucket_norms(vh, bucket, o.LINF)
    assert np.array_equal(norms.cpu().numpy(), n_ref)
    assert np.array_equal(sym.cpu().numpy(), o.quantize(vh, bucket, lev, n_ref, 5, 0))


def test_device_side_errors_are_latched_not_fatal(q):
    qgx, ctx = q
    K, d, bucket, nlev = 2, 3000, 1024, 5
    lev = np.linspace(0, 1, nlev, dtype=np.float32)
    v = gen.gaussian((K, d), seed=1, device="cuda")
    bad = v.clone()
    bad[1, 1500] = float("nan")
    norms, sym = qgx.qgx_quantize(ctx, bad, bucket, lev, qgx.QGX_NORM_L2, 1, 0)
    assert qgx.qgx_sync_status(ctx, check=False) == qgx.QGX_ERR_NONFINITE
    assert not sym[1, 1024:2048].any()
    assert qgx.qgx_sync_status(ctx, check=False) == qgx.QGX_OK          # cleared, context still usable
    norms, sym = qgx.qgx_quantize(ctx, v, bucket, lev, qgx.QGX_NORM_L2, 1, 0)
    cb = qgx.qgx_build_codebook_fixed(nlev, 128)                          # 3-bit code with unused patterns
    cap = qgx.qgx_stream_capacity_words(d, bucket, 128, cb.maxlen)
    stream, bbits, total = qgx.qgx_encode(ctx, norms, sym, bucket, cb, cap_words=cap)
    qgx.qgx_sync_status(ctx)
    # capacity too small
    small = torch.zeros((K, 16), dtype=torch.int32, device="cuda")
    qgx.qgx_encode(ctx, norms, sym, bucket, cb, cap_words=16, stream=small)
    assert qgx.qgx_sync_status(ctx, check=False) == qgx.QGX_ERR_CAPACITY
    assert not small.any()
    # corruptions made on the host: a shortened bucket, a broken sub-block length, absurd lengths
    sh = bbits.clone(); sh[0, 1] -= 9
    qgx.qgx_decode(ctx, stream, sh, d, bucket, cb)
    assert qgx.qgx_sync_status(ctx, check=False) == qgx.QGX_ERR_CORRUPT
    bs = stream.clone(); bs[0, 1] ^= 0x00010000
    qgx.qgx_decode(ctx, bs, bbits, d, bucket, cb)
    assert qgx.qgx_sync_status(ctx, check=False) == qgx.QGX_ERR_CORRUPT
    hg = bbits.clone(); hg[1, 2] = 10 ** 9
    qgx.qgx_decode(ctx, stream, hg, d, bucket, cb)
    assert qgx.qgx_sync_status(ctx, check=False) == qgx.QGX_ERR_CORRUPT
    fl = stream.clone(); fl[:, 40:60] = -1                                 # all-ones: unassigned patterns
    qgx.qgx_decode(ctx, fl, bbits, d, bucket, cb)
    assert qgx.qgx_sync_status(ctx, check=False) == qgx.QGX_ERR_CORRUPT
    # host-side argument checks
    with pytest.raises(qgx.QgxError) as e:
        qgx.qgx_quantize(ctx, v, bucket, [0.0, 0.5, 0.5, 1.0], qgx.QGX_NORM_L2, 1, 0)
    assert e.value.status == qgx.QGX_ERR_BAD_LEVELS
    with pytest.raises(qgx.QgxError) as e:
        qgx.qgx_quantize(ctx, v, 1022, lev, qgx.QGX_NORM_L2, 1, 0)
    assert e.value.status == qgx.QGX_ERR_INVALID_ARG
    # the clean path still works afterwards
    n2, s2 = qgx.qgx_decode(ctx, stream, bbits, d, bucket, cb)
    qgx.qgx_sync_status(ctx)
    assert torch.equal(s2, sym)

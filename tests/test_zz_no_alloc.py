"""qgx_encode_noalloc against qgx_encode.

Some users of the library may not allocate device memory at the point where they encode: code that
is being recorded into a CUDA stream capture, or a service whose GPU memory is handed out once at
start-up.  For them the library has a second encode entry point whose scratch (bucket offsets and
overflow flags) is a fixed array inside the library instead of a cudaMalloc'ed workspace.  This test
calls it through the C ABI twice in a row, on different shapes so that the second call finds the
first call's leftovers in the shared scratch, and expects exactly what qgx_encode writes -- and what the
oracle's encoder writes -- (the stream is integer work: bit for bit).  The file sorts last on purpose: a run that stops at the first failure has
then already run every other test."""
import numpy as np
import pytest
import torch

import qgx_inputs as gen
from oracle import qgx_oracle as o

pytestmark = pytest.mark.gpu


def _case(qgx, ctx, K, d, bucket, nlev, sub, seed):
    v = gen.gaussian_mixture((K, d), seed=seed, device="cuda")
    lev = np.r_[0.0, np.sort(np.random.default_rng(seed).uniform(0.001, 0.3, nlev - 2)), 1.0].astype(np.float32)
    norms, sym = qgx.qgx_quantize(ctx, v, bucket, lev, qgx.QGX_NORM_L2, seed, 1)
    p = np.random.default_rng(seed + 1).dirichlet(np.ones(nlev) * 0.5)
    cb = qgx.qgx_build_codebook_huffman(list(p), sub)
    cap = qgx.qgx_stream_capacity_words(d, bucket, sub, cb.maxlen)
    nb = (d + bucket - 1) // bucket
    want = qgx.qgx_encode(ctx, norms, sym, bucket, cb, cap_words=cap)
    qgx.qgx_sync_status(ctx)
    stream = torch.zeros((K, cap), dtype=torch.int32, device="cuda")       # every buffer is the caller's
    bbits = torch.zeros((K, nb), dtype=torch.int32, device="cuda")
    total = torch.zeros((K,), dtype=torch.int64, device="cuda")
    qgx.qgx_encode_noalloc(ctx, norms, sym, bucket, cb, stream, bbits, total)
    qgx.qgx_sync_status(ctx)
    assert torch.equal(bbits, want[1])
    assert torch.equal(total, want[2])
    assert torch.equal(stream, want[0])
    # and against the oracle's encoder: lengths, totals and the used words of every worker's stream
    st_ref, bb_ref, tot_ref = o.encode(norms.cpu().numpy(), sym.cpu().numpy(), bucket, o.codebook_from(cb.lengths(), cb.codes(), subblock=sub))
    assert np.array_equal(bbits.cpu().numpy().view(np.uint32), bb_ref)
    assert np.array_equal(total.cpu().numpy().astype(np.uint64), tot_ref)
    used = ((bb_ref.astype(np.int64) + 31) // 32).sum(axis=1)
    got = stream.cpu().numpy().view(np.uint32)
    for k in range(K):
        assert np.array_equal(got[k, :used[k]], st_ref[k, :used[k]])
    return norms, sym, cb


def test_noalloc_encode_matches_encode_on_two_calls_in_a_row():
    import paper_2308_09187_b200 as qgx
    ctx = qgx.qgx_create(0)
    try:
        _case(qgx, ctx, K=6, d=5 * 4096 + 1000, bucket=4096, nlev=17, sub=128, seed=11)
        norms, sym, cb = _case(qgx, ctx, K=3, d=2 * 1024 + 52, bucket=1024, nlev=9, sub=64, seed=12)   # smaller: stale scratch beyond
        # capacity errors behave as in qgx_encode, and a later call is clean again
        small = torch.zeros((3, 8), dtype=torch.int32, device="cuda")
        bb = torch.zeros((3, 3), dtype=torch.int32, device="cuda")
        tt = torch.zeros((3,), dtype=torch.int64, device="cuda")
        qgx.qgx_encode_noalloc(ctx, norms, sym, 1024, cb, small, bb, tt)
        assert qgx.qgx_sync_status(ctx, check=False) == qgx.QGX_ERR_CAPACITY
        assert not small.any()
        _case(qgx, ctx, K=2, d=3000, bucket=512, nlev=5, sub=0, seed=13)
        # beyond the fixed scratch: refused on the host, nothing launched
        big_sym = torch.zeros((1, 4 * 70000), dtype=torch.uint8, device="cuda")
        big_norms = torch.zeros((1, 70000), dtype=torch.float32, device="cuda")
        cb4 = qgx.qgx_build_codebook_fixed(5, 0)
        out = torch.zeros((1, 16), dtype=torch.int32, device="cuda")
        before = qgx.qgx_launch_count(ctx)
        with pytest.raises(qgx.QgxError) as e:
            qgx.qgx_encode_noalloc(ctx, big_norms, big_sym, 4, cb4, out, torch.zeros((1, 70000), dtype=torch.int32, device="cuda"),
                                   torch.zeros((1,), dtype=torch.int64, device="cuda"))
        assert e.value.status == qgx.QGX_ERR_TOO_LARGE
        assert qgx.qgx_launch_count(ctx) == before
    finally:
        qgx.qgx_destroy(ctx)

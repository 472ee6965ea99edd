"""The scale workload at its full size (K = 32 workers, d = 2^26, bucket 16384), in the configuration that the
benchmark times: one extra-gradient step with a first level fit, checked against the oracle on sampled buckets --
the oracle recomputes each sampled bucket on its own (all K workers of it) from the same inputs -- and through
properties that hold at any size."""
import numpy as np
import pytest
import torch

import qgx_inputs as gen
from oracle import qgx_oracle as o

pytestmark = pytest.mark.gpu


def test_scale_workload_on_sampled_buckets():
    import paper_2308_09187_b200 as qgx
    K, d, bucket, sub, nlev = 32, 1 << 26, 16384, 64, 17
    free, _ = torch.cuda.mem_get_info()
    if free < 60 * (1 << 30):
        pytest.skip("needs about 40 GB of device memory")
    ctx = qgx.qgx_create(0)
    try:
        prob = gen.c5_diagonal(K=K, d=d, device="cuda")
        cfg = qgx.make_quant_cfg(gen.uniform_levels(nlev).numpy(), bucket, qgx.qgx_build_codebook_fixed(nlev, sub), prob.seed,
                                 code_type=qgx.QGX_CODE_HUFFMAN)
        op = qgx.make_operator(qgx.QGX_OP_DIAGONAL, prob.D)
        st = qgx.EgState(prob.x0, K)
        qgx.qgx_eg_init(ctx, st)
        bits = torch.zeros((2, K), dtype=torch.int64, device="cuda")
        qgx.qgx_eg_step(ctx, st, op, prob.noise[0], prob.noise[1], cfg, refit=qgx.QGX_REFIT_FIRST, bits=bits)
        qgx.qgx_sync_status(ctx)            # also: every sub-block of every stream decoded to exactly its stated length
        lev = np.array(cfg.level_list(), dtype=np.float32)
        assert o.check_levels(lev) == o.OK
        cbo = o.codebook_from(cfg.cb.lengths(), cfg.cb.codes(), subblock=sub)
        nb = d // bucket
        rng = np.random.default_rng(0)
        sample = sorted({0, 1, nb // 2, nb - 1} | set(int(x) for x in rng.integers(0, nb, 4)))
        sum_sq, gamma2 = st.read_scalars()
        gamma1 = np.float32(K)
        partial = 0.0
        vhat = {}
        for slot, xid, which, point in ((0, 2, 0, prob.x0), (1, 3, 1, st.Xhalf)):
            stream, bbits, tot = qgx.exchange_stream_tensors(ctx, slot, K, nb)
            words = (bbits.to(torch.int64) + 31) // 32
            offs = torch.cumsum(words, dim=1) - words                       # the streams are compact
            assert torch.equal(tot, bbits.to(torch.int64).sum(dim=1)) and torch.equal(tot, bits[slot])
            cap = stream.shape[1]
            assert int((offs[:, -1] + words[:, -1]).max()) <= cap
            # between 2 and 13 bits per coordinate, headers included
            assert 2 * d < int(tot.min()) and int(tot.max()) < 13 * d
            for b in sample:
                lo = b * bucket
                a = (prob.D[lo:lo + bucket] * point[lo:lo + bucket]).cpu().numpy()
                V = (a[None, :] + prob.noise[which, :, lo:lo + bucket].cpu().numpy()).astype(np.float32)
                first = [int(offs[k, b]) for k in range(K)]
                n_gpu = np.array([stream[k, first[k]].item() for k in range(K)], dtype=np.int32).view(np.float32).reshape(K, 1)
                n_ref = o.bucket_norms(V, bucket)
                assert np.all(np.abs(n_gpu - n_ref) <= np.spacing(n_ref))
                sym = o.quantize(V, bucket, lev, n_gpu, prob.seed, xid, coord_base=lo)
                st_ref, bb_ref, _ = o.encode(n_gpu, sym, bucket, cbo)
                for k in range(K):
                    assert int(bbits[k, b]) == int(bb_ref[k, 0])
                    nw = int(words[k, b])
                    got = stream[k, first[k]:first[k] + nw].cpu().numpy().view(np.uint32)
                    assert np.array_equal(got, st_ref[k, :nw])
                mean = o.average(n_gpu, sym, bucket, lev)
                vhat[(slot, b)] = o.dequantize(n_gpu, sym, bucket, lev)
                if slot == 0:
                    ref = prob.x0[lo:lo + bucket].cpu().numpy() - gamma1 * mean
                    assert np.array_equal(st.Xhalf[lo:lo + bucket].cpu().numpy(), ref)
                else:
                    y = (np.zeros(bucket, np.float32) - mean).astype(np.float32)
                    assert np.array_equal(st.Y[lo:lo + bucket].cpu().numpy(), y)
                    x2 = prob.x0[lo:lo + bucket].cpu().numpy() + np.float32(gamma2) * y
                    assert np.array_equal(st.X[lo:lo + bucket].cpu().numpy(), x2)
                    assert np.array_equal(st.Xbar[lo:lo + bucket].cpu().numpy(), st.Xhalf[lo:lo + bucket].cpu().numpy())
                    diff = vhat[(0, b)] - vhat[(1, b)]
                    partial += float(np.sum(diff.astype(np.float64) ** 2))
        assert abs(gamma2 - np.float32(K / np.sqrt(1.0 + sum_sq))) <= 1e-6 * gamma2
        # the sampled buckets' share of the squared differences: a part of the total, and in proportion to it
        assert 0.0 < partial < sum_sq
        share = partial / sum_sq
        assert 0.3 * len(sample) / nb < share < 3.0 * len(sample) / nb
    finally:
        qgx.qgx_destroy(ctx)


def test_microbench_config_on_sampled_buckets():
    """K = 8 vectors of 2^24 N(0, 1) coordinates, bucket 8192, 17 levels fitted on a 1024-bin histogram, Huffman code:
    one fused exchange; streams, lengths and mean of sampled buckets bit for bit."""
    import paper_2308_09187_b200 as qgx
    K, d, bucket, sub, nlev = 8, 1 << 24, 8192, 64, 17
    ctx = qgx.qgx_create(0)
    try:
        c2 = gen.c2_gaussian(K=K, d=d, device="cuda")
        cfg = qgx.make_quant_cfg(np.linspace(0, 1, nlev), bucket, qgx.qgx_build_codebook_fixed(nlev, sub), c2.seed,
                                 code_type=qgx.QGX_CODE_HUFFMAN, nbins=1024)
        hist = qgx.qgx_update_levels(ctx, c2.v, cfg, qgx.QGX_REFIT_FIRST)
        # every coordinate adds its bucket's squared norm to one bin: the mass is bucket x the squared norm of everything
        total_sq = float((c2.v.double() ** 2).sum())
        assert abs(float(np.sum(hist)) - bucket * total_sq) <= 1e-6 * bucket * total_sq
        lev = np.array(cfg.level_list(), dtype=np.float32)
        cbo = o.codebook_from(cfg.cb.lengths(), cfg.cb.codes(), subblock=sub)
        mean, total = qgx.qgx_exchange(ctx, c2.v, cfg, 6, slot=0)
        qgx.qgx_sync_status(ctx)
        nb = d // bucket
        stream, bbits, tot = qgx.exchange_stream_tensors(ctx, 0, K, nb)
        words = (bbits.to(torch.int64) + 31) // 32
        offs = torch.cumsum(words, dim=1) - words
        assert torch.equal(tot, bbits.to(torch.int64).sum(dim=1)) and torch.equal(tot, total)
        for b in (0, 1, nb // 3, nb - 1):
            lo = b * bucket
            V = c2.v[:, lo:lo + bucket].cpu().numpy()
            first = [int(offs[k, b]) for k in range(K)]
            n_gpu = np.array([stream[k, first[k]].item() for k in range(K)], dtype=np.int32).view(np.float32).reshape(K, 1)
            assert np.all(np.abs(n_gpu - o.bucket_norms(V, bucket)) <= np.spacing(n_gpu))
            sym = o.quantize(V, bucket, lev, n_gpu, c2.seed, 6, coord_base=lo)
            st_ref, bb_ref, _ = o.encode(n_gpu, sym, bucket, cbo)
            for k in range(K):
                nw = int(words[k, b])
                assert int(bbits[k, b]) == int(bb_ref[k, 0])
                assert np.array_equal(stream[k, first[k]:first[k] + nw].cpu().numpy().view(np.uint32), st_ref[k, :nw])
            assert np.array_equal(mean[lo:lo + bucket].cpu().numpy(), o.average(n_gpu, sym, bucket, lev))
    finally:
        qgx.qgx_destroy(ctx)


@pytest.mark.parametrize("staged", [False, True], ids=["bucket in registers", "staged encode"])
def test_layerwise_config_on_sampled_buckets(staged):
    """The 16 layer-shaped tensors at their full sizes (each size twice), K = 16, bucket 4096, per-tensor tables and
    codes: first, last (the smallest tensors are one partial bucket) and one inner bucket of every tensor.  The
    tensors' exchanges run side by side on helper streams, so no encode kernel has the device to itself: every
    wait of the offset scan must still end (a wait that ran out would latch QGX_ERR_TIMEOUT)."""
    import paper_2308_09187_b200 as qgx
    ctx = qgx.qgx_create(0)
    try:
        if staged:
            qgx.qgx_set_encode_path(ctx, qgx.QGX_ENCODE_STAGED)
        lw = gen.c3_layerwise(K=16, device="cuda")
        K, d = lw.v.shape
        assert len(lw.sizes) == 16 and d == 2 * sum(gen.C3_TENSOR_SIZES)
        cfgs, at = [], 0
        for n in lw.sizes:
            cfg = qgx.make_quant_cfg(np.linspace(0, 1, lw.nlev), lw.bucket, qgx.qgx_build_codebook_fixed(lw.nlev, 128), lw.seed,
                                     code_type=qgx.QGX_CODE_HUFFMAN)
            qgx.qgx_update_levels(ctx, lw.v[:, at:at + n].contiguous(), cfg, qgx.QGX_REFIT_FIRST)
            cfgs.append(cfg)
            at += n
        mean, total = qgx.qgx_exchange_segments(ctx, lw.v, lw.sizes, cfgs, 9)
        qgx.qgx_sync_status(ctx)
        at, differing, checked = 0, 0, 0
        for n, cfg in zip(lw.sizes, cfgs):
            lev = np.array(cfg.level_list(), dtype=np.float32)
            nb = o.nbuckets(n, lw.bucket)
            for b in sorted({0, nb // 2, nb - 1}):
                lo = b * lw.bucket
                ln = min(lw.bucket, n - lo)
                V = lw.v[:, at + lo:at + lo + ln].cpu().numpy()
                norms = o.bucket_norms(V, lw.bucket)
                sym = o.quantize(V, lw.bucket, lev, norms, lw.seed, 9, coord_base=at + lo)
                ref = o.average(norms, sym, lw.bucket, lev)
                got = mean[at + lo:at + lo + ln].cpu().numpy()
                assert np.max(np.abs(got - ref)) <= 1e-5 * float(norms.max())
                differing += int(np.count_nonzero(got != ref))
                checked += K * ln
            at += n
        assert differing <= max(1, int(1e-6 * checked)) * K        # a flipped level changes one mean coordinate
        tb = total.cpu().numpy().astype(np.int64)
        assert np.all(tb > 2 * d) and np.all(tb < 13 * d)
    finally:
        qgx.qgx_destroy(ctx)


def test_affine_config_first_iterations():
    """V(x) = M x + b with n = 8192, K = 8, sigma = 1, bucket 4096, 17 adaptive levels: the first iterations at
    full size, teacher forced against the oracle (the library's fitted table handed to the oracle)."""
    import paper_2308_09187_b200 as qgx
    ctx = qgx.qgx_create(0)
    try:
        vi = gen.c4_affine(device="cuda")
        n = vi.M.shape[0]
        assert n == 8192 and vi.K == 8 and vi.bucket == 4096
        M, b = vi.M.cpu().numpy(), vi.b.cpu().numpy()
        lev = gen.uniform_levels(17).numpy().copy()
        cfg = qgx.make_quant_cfg(lev, vi.bucket, qgx.qgx_build_codebook_fixed(17, 128), vi.seed, code_type=qgx.QGX_CODE_HUFFMAN)
        cbo = o.codebook_fixed(17, 128)
        op, opo = qgx.make_operator(qgx.QGX_OP_DENSE_AFFINE, vi.M, vi.b), o.Op(o.OP_DENSE_AFFINE, M, b)
        st, st_o = qgx.EgState(vi.x0, vi.K), o.EgState(vi.x0.cpu().numpy(), vi.K)
        qgx.qgx_eg_init(ctx, st)
        for t in range(1, 4):
            nz = vi.noise(t)
            refit = 2 if t == 1 else 0
            st.X.copy_(torch.from_numpy(st_o.X)); st.Y.copy_(torch.from_numpy(st_o.Y)); st.Xbar.copy_(torch.from_numpy(st_o.Xbar))
            st.scalars.copy_(torch.tensor([st_o.sum_sq, float(st_o.gamma)], dtype=torch.float64))
            st.c.t = st_o.t
            qgx.qgx_eg_step(ctx, st, op, nz[0], nz[1], cfg, refit=refit)
            qgx.qgx_sync_status(ctx)
            if refit:
                lev = np.array(cfg.level_list(), dtype=np.float32)
                cbo = o.codebook_from(cfg.cb.lengths(), cfg.cb.codes(), subblock=128)
            nzh = nz.cpu().numpy()
            o.eg_step(st_o, opo, nzh[0], nzh[1], vi.bucket, lev, cbo, vi.seed)
            s, g = st.read_scalars()
            rel = lambda a, r: float(np.max(np.abs(a.astype(np.float64) - r)) / max(float(np.max(np.abs(r))), 1e-30))
            assert rel(st.Xhalf.cpu().numpy(), st_o.Xhalf) <= 1e-5 and rel(st.Y.cpu().numpy(), st_o.Y) <= 1e-5
            assert rel(st.X.cpu().numpy(), st_o.X) <= 1e-5
            assert abs(s - st_o.sum_sq) <= 1e-5 * st_o.sum_sq and abs(g - st_o.gamma) <= 1e-5 * st_o.gamma
    finally:
        qgx.qgx_destroy(ctx)

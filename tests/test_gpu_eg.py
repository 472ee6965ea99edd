"""Parity of qgx_eg_step and the operator kernels with the oracle: teacher-forced per step (the
library starts every step from the oracle's state) and free-running over whole trajectories."""
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


def _rel(a, b):
    b = np.asarray(b, dtype=np.float64)
    return float(np.max(np.abs(np.asarray(a, dtype=np.float64) - b)) / max(np.max(np.abs(b)), 1e-30))


def test_operators(q):
    qgx, ctx = q
    n = 1000
    M = gen.gaussian((n, n), 1, "cuda")
    b = gen.gaussian((n,), 2, "cuda")
    x = gen.gaussian((n,), 3, "cuda")
    out = qgx.qgx_apply_operator(ctx, qgx.make_operator(qgx.QGX_OP_DENSE_AFFINE, M, b), x)
    ref = o.apply_operator(o.Op(o.OP_DENSE_AFFINE, M.cpu().numpy(), b.cpu().numpy()), x.cpu().numpy())
    assert _rel(out.cpu().numpy(), ref) <= 1e-6
    A = gen.gaussian((513, 513), 4, "cuda")
    z = gen.gaussian((1026,), 5, "cuda")
    out = qgx.qgx_apply_operator(ctx, qgx.make_operator(qgx.QGX_OP_BILINEAR, A), z)
    ref = o.apply_operator(o.Op(o.OP_BILINEAR, A.cpu().numpy()), z.cpu().numpy())
    assert _rel(out.cpu().numpy(), ref) <= 1e-6
    D = gen.uniform((5000,), 6, "cuda", 0.01, 1.0)
    xx = gen.gaussian((5000,), 7, "cuda")
    out = qgx.qgx_apply_operator(ctx, qgx.make_operator(qgx.QGX_OP_DIAGONAL, D), xx)
    assert np.array_equal(out.cpu().numpy(), o.apply_operator(o.Op(o.OP_DIAGONAL, D.cpu().numpy()), xx.cpu().numpy()))
    qgx.qgx_sync_status(ctx)


def _load_state(qgx, st_gpu, st_or):
    st_gpu.X.copy_(torch.from_numpy(st_or.X))
    st_gpu.Y.copy_(torch.from_numpy(st_or.Y))
    st_gpu.Xbar.copy_(torch.from_numpy(st_or.Xbar))
    st_gpu.scalars.copy_(torch.tensor([st_or.sum_sq, float(st_or.gamma)], dtype=torch.float64))
    st_gpu.c.t = st_or.t


def _compare(st_gpu, st_or, tol=1e-5):
    s, g = st_gpu.read_scalars()
    assert _rel(st_gpu.Xhalf.cpu().numpy(), st_or.Xhalf) <= tol
    assert _rel(st_gpu.Y.cpu().numpy(), st_or.Y) <= tol
    assert _rel(st_gpu.X.cpu().numpy(), st_or.X) <= tol
    assert _rel(st_gpu.Xbar.cpu().numpy(), st_or.Xbar) <= tol
    assert abs(s - st_or.sum_sq) <= tol * max(st_or.sum_sq, 1e-30)
    assert abs(g - st_or.gamma) <= tol * st_or.gamma
    assert st_gpu.t == st_or.t


def test_bilinear_game_teacher_forced_and_free_running(q):
    """c1: n = 1024 (d = 2048), K = 4, bucket 512, 9 uniform levels, fixed-length code, 100 iterations."""
    qgx, ctx = q
    T = 100
    g = gen.c1_bilinear(T=T, device="cuda")
    A, z0, noise = g.A.cpu().numpy(), g.z0.cpu().numpy(), g.noise.cpu().numpy()
    lev = gen.uniform_levels(9).numpy()
    cb = qgx.qgx_build_codebook_fixed(9, 128)
    cbo = o.codebook_from(cb.lengths(), cb.codes(), subblock=128)
    cfg = qgx.make_quant_cfg(lev, g.bucket, cb, g.seed)
    op = qgx.make_operator(qgx.QGX_OP_BILINEAR, g.A)
    opo = o.Op(o.OP_BILINEAR, A)
    st_f = qgx.EgState(g.z0, g.K)          # free running
    st_t = qgx.EgState(g.z0, g.K)          # teacher forced
    qgx.qgx_eg_init(ctx, st_f)
    qgx.qgx_eg_init(ctx, st_t)
    st_o = o.EgState(z0, g.K)
    bits = torch.zeros((2, g.K), dtype=torch.int64, device="cuda")
    for t in range(T):
        _load_state(qgx, st_t, st_o)
        bits_o = o.eg_step(st_o, opo, noise[t, 0], noise[t, 1], g.bucket, lev, cbo, g.seed)
        qgx.qgx_eg_step(ctx, st_t, op, g.noise[t, 0], g.noise[t, 1], cfg, bits=bits)
        qgx.qgx_eg_step(ctx, st_f, op, g.noise[t, 0], g.noise[t, 1], cfg)
        if t % 10 == 0 or t == T - 1:
            qgx.qgx_sync_status(ctx)
            _compare(st_t, st_o)
            assert int(bits.sum().item()) == bits_o
    qgx.qgx_sync_status(ctx)
    _compare(st_f, st_o, tol=1e-4)          # free running: the same trajectory up to rare level flips
    s, gam = st_f.read_scalars()
    assert abs(1.0 / gam ** 2 - (1.0 + s) / g.K ** 2) <= 1e-6 * (1.0 + s) / g.K ** 2     # step-size identity
    assert float(st_f.Xbar.norm()) < float(g.z0.norm())                                   # towards z* = 0


def test_affine_vi_with_refits_teacher_forced(q):
    """c4 at reduced size: V(x) = M x + b, K = 8, noise sigma = 1, 17 adaptive levels refitted every 10 steps."""
    qgx, ctx = q
    n, T = 512, 40
    vi = gen.c4_affine(n=n, K=8, device="cuda", bucket=128)
    M, b = vi.M.cpu().numpy(), vi.b.cpu().numpy()
    xstar = np.linalg.solve(M.astype(np.float64), -b.astype(np.float64))
    assert np.linalg.norm(M.astype(np.float64) @ xstar + b) <= 1e-12 * np.linalg.norm(b)
    lev_o = gen.uniform_levels(17).numpy().copy()
    cb = qgx.qgx_build_codebook_fixed(17, 32)
    cbo = o.codebook_fixed(17, 32)
    cfg = qgx.make_quant_cfg(lev_o, vi.bucket, cb, vi.seed, code_type=qgx.QGX_CODE_HUFFMAN, nbins=256)
    op = qgx.make_operator(qgx.QGX_OP_DENSE_AFFINE, vi.M, vi.b)
    opo = o.Op(o.OP_DENSE_AFFINE, M, b)
    st_t = qgx.EgState(vi.x0, vi.K)
    qgx.qgx_eg_init(ctx, st_t)
    st_o = o.EgState(vi.x0.cpu().numpy(), vi.K)
    for t in range(1, T + 1):
        nz = vi.noise(t)
        nzh = nz.cpu().numpy()
        refit = 2 if t == 1 else (1 if (t - 1) % 10 == 0 else 0)
        _load_state(qgx, st_t, st_o)
        # both sides quantize with the same table and code: the library's refit result is handed to the oracle
        qgx.qgx_eg_step(ctx, st_t, op, nz[0], nz[1], cfg, refit=refit)
        if refit:
            lev_ref = lev_o.copy()
            a = o.apply_operator(opo, st_o.X)
            V = o.form_dual_vectors(a, nzh[0], vi.K)
            lev_ref, _ = o.refit(V, vi.bucket, 256, lev_ref, cbo, refit == 2, o.CODE_HUFFMAN)
            got = np.array(cfg.level_list(), dtype=np.float32)
            assert np.max(np.abs(got - lev_ref)) <= 1e-6
            lev_o = got.copy()
            cbo = o.codebook_from(cfg.cb.lengths(), cfg.cb.codes(), subblock=32)
        o.eg_step(st_o, opo, nzh[0], nzh[1], vi.bucket, lev_o, cbo, vi.seed)
        qgx.qgx_sync_status(ctx)
        _compare(st_t, st_o)
    err = np.linalg.norm(st_t.Xbar.cpu().numpy() - xstar) / np.linalg.norm(xstar)
    assert err < 1.0


def test_iteration_against_the_oracle_with_its_own_refits(q):
    """As above, but the oracle fits its own level tables and builds its own codes (first fit at t = 1, a continuing
    refit at t = 6): a wrong fit in the library would show in the iterates."""
    qgx, ctx = q
    n, T = 512, 10
    vi = gen.c4_affine(n=n, K=8, device="cuda", bucket=128)
    M, b = vi.M.cpu().numpy(), vi.b.cpu().numpy()
    lev_o = gen.uniform_levels(17).numpy().copy()
    cbo = o.codebook_fixed(17, 32)
    cfg = qgx.make_quant_cfg(lev_o, vi.bucket, qgx.qgx_build_codebook_fixed(17, 32), vi.seed, code_type=qgx.QGX_CODE_HUFFMAN, nbins=256)
    op = qgx.make_operator(qgx.QGX_OP_DENSE_AFFINE, vi.M, vi.b)
    opo = o.Op(o.OP_DENSE_AFFINE, M, b)
    st_t = qgx.EgState(vi.x0, vi.K)
    qgx.qgx_eg_init(ctx, st_t)
    st_o = o.EgState(vi.x0.cpu().numpy(), vi.K)
    for t in range(1, T + 1):
        nz = vi.noise(t)
        nzh = nz.cpu().numpy()
        refit = 2 if t == 1 else (1 if t == 6 else 0)
        _load_state(qgx, st_t, st_o)
        qgx.qgx_eg_step(ctx, st_t, op, nz[0], nz[1], cfg, refit=refit)
        o.eg_step(st_o, opo, nzh[0], nzh[1], vi.bucket, lev_o, cbo, vi.seed, refit=refit, code_type=o.CODE_HUFFMAN, nbins=256)
        qgx.qgx_sync_status(ctx)
        if refit:
            assert np.max(np.abs(np.array(cfg.level_list(), dtype=np.float32) - lev_o)) <= 1e-6
        _compare(st_t, st_o)


def test_diagonal_operator_scale_shape(q):
    """c5 at reduced size: diagonal operator, mixture noise reused every iteration, bucket 16384."""
    qgx, ctx = q
    K, d = 4, 3 * 16384 + 4000
    c5 = gen.c5_diagonal(K=K, d=d, device="cuda")
    D, x0, noise = c5.D.cpu().numpy(), c5.x0.cpu().numpy(), c5.noise.cpu().numpy()
    lev = gen.uniform_levels(17).numpy().copy()
    cb = qgx.qgx_build_codebook_fixed(17, 128)
    cfg = qgx.make_quant_cfg(lev, c5.bucket, cb, c5.seed, code_type=qgx.QGX_CODE_HUFFMAN)
    op = qgx.make_operator(qgx.QGX_OP_DIAGONAL, c5.D)
    opo = o.Op(o.OP_DIAGONAL, D)
    st = qgx.EgState(c5.x0, K)
    qgx.qgx_eg_init(ctx, st)
    st_o = o.EgState(x0, K)
    cbo = o.codebook_fixed(17, 128)
    for t in range(1, 4):
        refit = 2 if t == 1 else 0
        _load_state(qgx, st, st_o)
        qgx.qgx_eg_step(ctx, st, op, c5.noise[0], c5.noise[1], cfg, refit=refit)
        if refit:
            lev = np.array(cfg.level_list(), dtype=np.float32)
            cbo = o.codebook_from(cfg.cb.lengths(), cfg.cb.codes(), subblock=128)
        o.eg_step(st_o, opo, noise[0], noise[1], c5.bucket, lev, cbo, c5.seed)
        qgx.qgx_sync_status(ctx)
        _compare(st, st_o)


@pytest.mark.parametrize("method", ["da", "optda"])
def test_dual_averaging_and_optimistic_variant(q, method):
    """The one-exchange members of the family (Eq. Quantized DA, Eq. Quantized OptDA) against the oracle, teacher
    forced, with refits in between (the optimistic variant then compares vectors quantized with two different
    level tables).  Diagonal operator: the dual vectors are bit-identical on both sides."""
    qgx, ctx = q
    K, d, bucket, sub = 4, 3 * 2048 + 100, 2048, 64
    c5 = gen.c5_diagonal(K=K, d=d, device="cuda", bucket=bucket, seed=77)
    D, x0, noise = c5.D.cpu().numpy(), c5.x0.cpu().numpy(), c5.noise.cpu().numpy()
    m_gpu = qgx.QGX_METHOD_DA if method == "da" else qgx.QGX_METHOD_OPTDA
    m_or = o.METHOD_DA if method == "da" else o.METHOD_OPTDA
    lev = gen.uniform_levels(17).numpy().copy()
    cfg = qgx.make_quant_cfg(lev, bucket, qgx.qgx_build_codebook_fixed(17, sub), c5.seed, code_type=qgx.QGX_CODE_HUFFMAN)
    op, opo = qgx.make_operator(qgx.QGX_OP_DIAGONAL, c5.D), o.Op(o.OP_DIAGONAL, D)
    st = qgx.EgState(c5.x0, K)
    qgx.qgx_eg_init(ctx, st)
    st_o = o.EgState(x0, K)
    cbo = o.codebook_fixed(17, sub)
    mean_prev = torch.zeros(d, dtype=torch.float32, device="cuda")
    gp, mp = np.zeros((K, d), np.float32), np.zeros(d, np.float32)
    bits = torch.zeros(K, dtype=torch.int64, device="cuda")
    for t in range(1, 8):
        refit = 2 if t == 1 else (1 if t % 3 == 0 else 0)
        nz_t = (t % 2)                                   # alternate the two noise sets
        _load_state(qgx, st, st_o)
        mean_prev.copy_(torch.from_numpy(mp))
        qgx.qgx_family_step(ctx, st, m_gpu, op, c5.noise[nz_t], cfg, refit=refit, mean_prev=mean_prev, bits=bits)
        qgx.qgx_sync_status(ctx)
        if refit:
            lev = np.array(cfg.level_list(), dtype=np.float32)
            cbo = o.codebook_from(cfg.cb.lengths(), cfg.cb.codes(), subblock=sub)
        sent = o.family_step(st_o, m_or, opo, noise[nz_t], bucket, lev, cbo, c5.seed, gp, mp)
        _compare(st, st_o, tol=1e-6)
        assert int(bits.sum().item()) == sent
        if method == "optda":
            assert np.array_equal(mean_prev.cpu().numpy(), mp)
    assert st_o.sum_sq > 0


def test_optimistic_dual_averaging_free_running_on_the_affine_problem(q):
    """c4 at reduced size, free running (no teacher forcing): the library's own iterates approach the solution."""
    qgx, ctx = q
    n, T = 512, 120
    vi = gen.c4_affine(n=n, K=8, device="cuda", bucket=128)
    M, b = vi.M.cpu().numpy(), vi.b.cpu().numpy()
    xstar = np.linalg.solve(M.astype(np.float64), -b.astype(np.float64))
    cfg = qgx.make_quant_cfg(gen.uniform_levels(17).numpy(), vi.bucket, qgx.qgx_build_codebook_fixed(17, 32), vi.seed,
                             code_type=qgx.QGX_CODE_HUFFMAN, nbins=256)
    op = qgx.make_operator(qgx.QGX_OP_DENSE_AFFINE, vi.M, vi.b)
    st = qgx.EgState(vi.x0, vi.K)
    qgx.qgx_eg_init(ctx, st)
    mean_prev = torch.zeros(n, dtype=torch.float32, device="cuda")
    errs = {}
    for t in range(1, T + 1):
        refit = 2 if t == 1 else (1 if (t - 1) % 10 == 0 else 0)
        qgx.qgx_family_step(ctx, st, qgx.QGX_METHOD_OPTDA, op, vi.noise(t)[1], cfg, refit=refit, mean_prev=mean_prev)
        if t in (15, T):
            qgx.qgx_sync_status(ctx)
            errs[t] = float(np.linalg.norm(st.Xbar.cpu().numpy() - xstar) / np.linalg.norm(xstar))
    assert errs[T] < errs[15] < 1.0


def test_relative_noise_iteration(q):
    """Assumption 3: V_k = A(x) .* S_k with random player-update scales, fused into the quantizer's load; teacher
    forced against the oracle for the two-exchange iteration and the optimistic variant, then the fixed point."""
    qgx, ctx = q
    K, d, bucket, sub = 4, 2 * 4096 + 300, 4096, 64
    D = gen.uniform((d,), 21, "cuda", 0.2, 1.0)
    x0 = gen.gaussian((d,), 22, "cuda")
    op = qgx.make_operator(qgx.QGX_OP_DIAGONAL, D, noise_model=qgx.QGX_NOISE_RELATIVE)
    opo = o.Op(o.OP_DIAGONAL, D.cpu().numpy(), noise_model=o.NOISE_RELATIVE)
    lev = gen.uniform_levels(17).numpy().copy()
    cfg = qgx.make_quant_cfg(lev, bucket, qgx.qgx_build_codebook_fixed(17, sub), 5, code_type=qgx.QGX_CODE_HUFFMAN)
    cbo = o.codebook_fixed(17, sub)
    st, st_o = qgx.EgState(x0, K), o.EgState(x0.cpu().numpy(), K)
    qgx.qgx_eg_init(ctx, st)
    for t in range(1, 5):
        S = gen.player_scales((2, K, d), 128, 0.5, 900 + t, device="cuda")
        refit = 2 if t == 1 else 0
        _load_state(qgx, st, st_o)
        qgx.qgx_eg_step(ctx, st, op, S[0], S[1], cfg, refit=refit)
        qgx.qgx_sync_status(ctx)
        if refit:
            lev = np.array(cfg.level_list(), dtype=np.float32)
            cbo = o.codebook_from(cfg.cb.lengths(), cfg.cb.codes(), subblock=sub)
        Sh = S.cpu().numpy()
        o.eg_step(st_o, opo, Sh[0], Sh[1], bucket, lev, cbo, 5)
        _compare(st, st_o, tol=1e-6)
    # optimistic variant under the same oracle
    st2, st2_o = qgx.EgState(x0, K), o.EgState(x0.cpu().numpy(), K)
    qgx.qgx_eg_init(ctx, st2)
    mean_prev = torch.zeros(d, dtype=torch.float32, device="cuda")
    gp, mp = np.zeros((K, d), np.float32), np.zeros(d, np.float32)
    for t in range(1, 4):
        S = gen.player_scales((K, d), 128, 0.5, 950 + t, device="cuda")
        _load_state(qgx, st2, st2_o)
        mean_prev.copy_(torch.from_numpy(mp))
        qgx.qgx_family_step(ctx, st2, qgx.QGX_METHOD_OPTDA, op, S, cfg, mean_prev=mean_prev)
        qgx.qgx_sync_status(ctx)
        o.family_step(st2_o, o.METHOD_OPTDA, opo, S.cpu().numpy(), bucket, lev, cbo, 5, gp, mp)
        _compare(st2, st2_o, tol=1e-6)
    # at the solution nothing moves, whatever is drawn
    z = torch.zeros(d, dtype=torch.float32, device="cuda")
    st3 = qgx.EgState(z, K)
    qgx.qgx_eg_init(ctx, st3)
    S = gen.player_scales((2, K, d), 128, 0.5, 999, device="cuda")
    qgx.qgx_eg_step(ctx, st3, op, S[0], S[1], cfg)
    qgx.qgx_sync_status(ctx)
    s, g = st3.read_scalars()
    assert not st3.X.any().item() and s == 0.0 and g == K


def test_two_level_tables(q):
    """A level table and a code of its own for each exchange (footnote of Sec. 3.3): teacher forced against the
    oracle with refits, the second exchange on heavier-tailed vectors than the first."""
    qgx, ctx = q
    K, d, bucket, sub = 4, 2 * 2048 + 500, 2048, 64
    D = gen.uniform((d,), 31, "cuda", 0.05, 1.0)
    x0 = gen.gaussian((d,), 32, "cuda")
    n_t = gen.gaussian((K, d), 33, "cuda", std=0.2)
    n_h = gen.student_t3((K, d), 34, "cuda") * 0.3
    op, opo = qgx.make_operator(qgx.QGX_OP_DIAGONAL, D), o.Op(o.OP_DIAGONAL, D.cpu().numpy())
    lev0 = gen.uniform_levels(17).numpy()
    cfg_t = qgx.make_quant_cfg(lev0, bucket, qgx.qgx_build_codebook_fixed(17, sub), 8, code_type=qgx.QGX_CODE_HUFFMAN, nbins=512)
    cfg_h = qgx.make_quant_cfg(lev0, bucket, qgx.qgx_build_codebook_fixed(17, sub), 8, code_type=qgx.QGX_CODE_HUFFMAN, nbins=512)
    st, st_o = qgx.EgState(x0, K), o.EgState(x0.cpu().numpy(), K)
    qgx.qgx_eg_init(ctx, st)
    lt, lh = lev0.copy(), lev0.copy()
    ct, ch = o.codebook_fixed(17, sub), o.codebook_fixed(17, sub)
    nth, nhh = n_t.cpu().numpy(), n_h.cpu().numpy()
    for t in range(1, 6):
        refit = 2 if t == 1 else (1 if t == 4 else 0)
        _load_state(qgx, st, st_o)
        qgx.qgx_eg_step_two_tables(ctx, st, op, n_t, n_h, cfg_t, cfg_h, refit=refit)
        qgx.qgx_sync_status(ctx)
        if refit:
            # both sides quantize with the library's tables and codes (the fits themselves are compared below)
            got_t, got_h = np.array(cfg_t.level_list(), np.float32), np.array(cfg_h.level_list(), np.float32)
            lt_o, lh_o = lt.copy(), lh.copy()
            probe = o.EgState(st_o.X.copy(), K)
            probe.load(st_o.X, st_o.Y, st_o.Xbar, st_o.sum_sq, st_o.gamma, st_o.t)
            o.eg_step_two_tables(probe, opo, nth, nhh, bucket, lt_o, o.codebook_fixed(17, sub), lh_o, o.codebook_fixed(17, sub),
                                 8, refit=refit, code_type=o.CODE_HUFFMAN, nbins=512)
            # first fits and fits that continue from the fitted tables alike
            assert np.max(np.abs(got_t - lt_o)) <= 1e-6 and np.max(np.abs(got_h - lh_o)) <= 1e-6
            assert not np.array_equal(got_t, got_h)
            lt, lh = got_t.copy(), got_h.copy()
            ct = o.codebook_from(cfg_t.cb.lengths(), cfg_t.cb.codes(), subblock=sub)
            ch = o.codebook_from(cfg_h.cb.lengths(), cfg_h.cb.codes(), subblock=sub)
        o.eg_step_two_tables(st_o, opo, nth, nhh, bucket, lt, ct, lh, ch, 8)
        _compare(st, st_o, tol=1e-6)


def test_argument_errors_of_the_iteration_calls(q):
    """Wrong arguments come back as error codes; nothing is launched and the context stays usable."""
    qgx, ctx = q
    K, d, bucket = 2, 1024, 256
    D = gen.uniform((d,), 1, "cuda", 0.1, 1.0)
    x0 = gen.gaussian((d,), 2, "cuda")
    nz = gen.gaussian((K, d), 3, "cuda")
    op = qgx.make_operator(qgx.QGX_OP_DIAGONAL, D)
    cfg = qgx.make_quant_cfg(gen.uniform_levels(9).numpy(), bucket, qgx.qgx_build_codebook_fixed(9, 32), 1)
    st = qgx.EgState(x0, K)
    qgx.qgx_eg_init(ctx, st)
    mean_prev = torch.zeros(d, dtype=torch.float32, device="cuda")
    with pytest.raises(qgx.QgxError) as e:
        qgx.qgx_family_step(ctx, st, 7, op, nz, cfg, mean_prev=mean_prev)              # no such method
    assert e.value.status == qgx.QGX_ERR_INVALID_ARG
    with pytest.raises(qgx.QgxError) as e:
        qgx.qgx_family_step(ctx, st, qgx.QGX_METHOD_OPTDA, op, nz, cfg)                # needs mean_prev
    assert e.value.status == qgx.QGX_ERR_INVALID_ARG
    with pytest.raises(qgx.QgxError) as e:
        qgx.qgx_eg_step_two_tables(ctx, st, op, nz, nz, cfg, cfg)                      # one table given twice
    assert e.value.status == qgx.QGX_ERR_INVALID_ARG
    other = qgx.make_quant_cfg(gen.uniform_levels(9).numpy(), bucket, qgx.qgx_build_codebook_fixed(9, 64), 1)
    with pytest.raises(qgx.QgxError) as e:
        qgx.qgx_eg_step_two_tables(ctx, st, op, nz, nz, cfg, other)                    # different sub-block sizes
    assert e.value.status == qgx.QGX_ERR_INVALID_ARG
    # an optimistic step that is not the first needs the vectors kept by the step before it
    st.c.t = 5
    ctx2 = qgx.qgx_create(0)
    try:
        with pytest.raises(qgx.QgxError) as e:
            qgx.qgx_family_step(ctx2, st, qgx.QGX_METHOD_OPTDA, op, nz, cfg, mean_prev=mean_prev)
        assert e.value.status == qgx.QGX_ERR_INVALID_ARG
    finally:
        qgx.qgx_destroy(ctx2)
    st.c.t = 1
    assert st.t == 1
    qgx.qgx_family_step(ctx, st, qgx.QGX_METHOD_OPTDA, op, nz, cfg, mean_prev=mean_prev)   # and the context still works
    qgx.qgx_sync_status(ctx)
    assert st.t == 2

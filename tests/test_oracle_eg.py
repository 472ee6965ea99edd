"""Pins of the oracle's iteration (Algorithm 1, Eq. Q-GenX, adaptive step of Theorem 3).  CPU only."""
import math

import numpy as np

import qgx_inputs as gen
from oracle import qgx_oracle as o


def test_operators_against_fp64_matmul():
    rng = np.random.default_rng(1)
    n = 96
    M = rng.standard_normal((n, n)).astype(np.float32)
    b = rng.standard_normal(n).astype(np.float32)
    x = rng.standard_normal(n).astype(np.float32)
    ref = M.astype(np.float64) @ x.astype(np.float64) + b
    got = o.apply_operator(o.Op(o.OP_DENSE_AFFINE, M, b), x)
    assert np.max(np.abs(got - ref)) <= 1e-6 * np.max(np.abs(ref))
    A = rng.standard_normal((n, n)).astype(np.float32)
    z = rng.standard_normal(2 * n).astype(np.float32)
    ref2 = np.r_[A.astype(np.float64) @ z[n:], -(A.astype(np.float64).T @ z[:n])]
    got2 = o.apply_operator(o.Op(o.OP_BILINEAR, A), z)
    assert np.max(np.abs(got2 - ref2)) <= 1e-6 * np.max(np.abs(ref2))
    D = rng.uniform(0.01, 1, n).astype(np.float32)
    assert np.array_equal(o.apply_operator(o.Op(o.OP_DIAGONAL, D), x), D * x)


def test_two_dimensional_dual_extrapolation_by_hand():
    """K = 1, no noise, quantizer bypassed: the recursion of Eq. (Q-GenX) on V(x, y) = (y, -x)
    from z1 = (1, 0), worked by hand:
      gamma_1 = 1; V(z1) = (0, -1); z_{3/2} = (1, 1); V(z_{3/2}) = (1, -1); Y_2 = (-1, 1);
      sum = ||(0,-1) - (1,-1)||^2 = 1; gamma_2 = 1/sqrt(2); z_2 = (1 - 1/sqrt 2, 1/sqrt 2)."""
    op = o.Op(o.OP_BILINEAR, np.array([[1.0]], dtype=np.float32))
    st = o.EgState(np.array([1.0, 0.0], dtype=np.float32), K=1)
    lev = np.array([0.0, 1.0], dtype=np.float32)
    cb = o.codebook_fixed(2)
    assert st.gamma == 1.0 and st.t == 1
    o.eg_step(st, op, None, None, 2, lev, cb, seed=0, quantizer_off=True)
    r = 1.0 / math.sqrt(2.0)
    assert st.Xhalf.tolist() == [1.0, 1.0]
    assert st.Y.tolist() == [-1.0, 1.0]
    assert st.sum_sq == 1.0 and abs(st.gamma - r) < 1e-7
    assert np.allclose(st.X, [1.0 - r, r], atol=1e-7)
    assert st.Xbar.tolist() == [1.0, 1.0] and st.t == 2
    # second step, by the same rules in fp64
    x = np.array([1.0 - r, r])
    v1 = np.array([x[1], -x[0]])
    xh = x - r * v1
    v2 = np.array([xh[1], -xh[0]])
    Y = np.array([-1.0, 1.0]) - v2
    s = 1.0 + np.sum((v1 - v2) ** 2)
    g3 = 1.0 / math.sqrt(1.0 + s)
    o.eg_step(st, op, None, None, 2, lev, cb, seed=0, quantizer_off=True)
    assert np.allclose(st.Xhalf, xh, atol=1e-6) and np.allclose(st.Y, Y, atol=1e-6)
    assert abs(st.sum_sq - s) < 1e-6 and abs(st.gamma - g3) < 1e-6
    assert np.allclose(st.X, np.array([1.0, 0.0]) + g3 * Y, atol=1e-6)
    assert np.allclose(st.Xbar, (np.array([1.0, 1.0]) + xh) / 2, atol=1e-6)


def test_step_size_identity_and_bits():
    # 1/gamma_{T+1}^2 = (1 + sum_t sum_k ||Vhat_{k,t} - Vhat_{k,t+1/2}||^2) / K^2, checked every step
    g = gen.c1_bilinear(n=64, K=4, T=12, bucket=32)
    op = o.Op(o.OP_BILINEAR, g.A.numpy())
    st = o.EgState(g.z0.numpy(), K=4)
    lev = gen.uniform_levels(9).numpy()
    cb = o.codebook_fixed(9, 16)
    prev = 0.0
    for t in range(12):
        bits = o.eg_step(st, op, g.noise[t, 0].numpy(), g.noise[t, 1].numpy(), 32, lev, cb, seed=g.seed)
        assert bits > 0 and st.sum_sq > prev
        prev = st.sum_sq
        assert abs(1.0 / float(st.gamma) ** 2 - (1.0 + st.sum_sq) / 16.0) <= 1e-6 * (1.0 + st.sum_sq) / 16.0
    assert st.t == 13


def _run_c1(T, n=256, K=4, seed=1001):
    g = gen.c1_bilinear(n=n, K=K, T=T, seed=seed, bucket=128)
    op = o.Op(o.OP_BILINEAR, g.A.numpy())
    st = o.EgState(g.z0.numpy(), K=K)
    lev = gen.uniform_levels(9).numpy()
    cb = o.codebook_fixed(9, 32)
    for t in range(T):
        o.eg_step(st, op, g.noise[t, 0].numpy(), g.noise[t, 1].numpy(), g.bucket, lev, cb, seed=seed)
    return float(np.linalg.norm(st.Xbar)), float(np.linalg.norm(g.z0.numpy()))


def test_bilinear_game_ergodic_average_approaches_the_solution():
    # z* = 0 for min_x max_y x^T A y; the error of the ergodic average falls with T (Theorem 3: trend only)
    e25, z0 = _run_c1(25)
    e100, _ = _run_c1(100)
    assert e100 < e25 < z0


def _run_c4(T, K, n=128, seed=1004, refit_every=10):
    vi = gen.c4_affine(n=n, K=K, seed=seed, bucket=64, noise_std=1.0)
    M, b = vi.M.numpy(), vi.b.numpy()
    xstar = np.linalg.solve(M.astype(np.float64), -b.astype(np.float64))     # the zero of V(x) = M x + b
    assert np.linalg.norm(M.astype(np.float64) @ xstar + b) <= 1e-12 * np.linalg.norm(b)
    op = o.Op(o.OP_DENSE_AFFINE, M, b)
    st = o.EgState(vi.x0.numpy(), K=K)
    lev = gen.uniform_levels(17).numpy().copy()
    cb = o.codebook_fixed(17, 32)
    for t in range(1, T + 1):
        nz = vi.noise(t).numpy()
        refit = 2 if t == 1 else (1 if (t - 1) % refit_every == 0 else 0)
        o.eg_step(st, op, nz[0], nz[1], vi.bucket, lev, cb, seed=seed, refit=refit, code_type=o.CODE_HUFFMAN,
                  nbins=256)
    return float(np.linalg.norm(st.Xbar - xstar) / np.linalg.norm(xstar)), lev, cb


def test_affine_vi_error_falls_with_iterations_and_workers():
    e_short, _, _ = _run_c4(40, K=8)
    e_long, lev, cb = _run_c4(160, K=8)
    assert e_long < e_short
    errs1 = [_run_c4(160, K=1, seed=s)[0] for s in (1004, 2004)]
    errs8 = [_run_c4(160, K=8, seed=s)[0] for s in (1004, 2004)]
    assert np.mean(errs8) < np.mean(errs1)             # more workers, smaller error at equal T
    assert o.check_levels(lev) == o.OK and lev[1] < 1.0 / 16.0    # the table was refitted towards small u
    assert 1 <= min(cb.lengths()) <= cb.maxlen <= 12


def test_exchange_matches_its_parts():
    rng = np.random.default_rng(12)
    v = rng.standard_normal((3, 1000)).astype(np.float32)
    lev = gen.uniform_levels(9).numpy()
    cb = o.codebook_fixed(9, 128)
    mean, total, vhat = o.exchange(v, 256, lev, cb, seed=77, xid=5, return_vhat=True)
    norms = o.bucket_norms(v, 256)
    sym = o.quantize(v, 256, lev, norms, seed=77, xid=5)
    assert np.array_equal(vhat, o.dequantize(norms, sym, 256, lev))
    assert np.array_equal(mean, o.average(norms, sym, 256, lev))
    _, _, tb = o.encode(norms, sym, 256, cb)
    assert np.array_equal(total, tb)
    V = o.form_dual_vectors(v[0], v, 3)
    assert np.array_equal(V, v[0][None, :] + v)


# ---- the other two members of the family (Sec. 3.1: quantized dual averaging, optimistic dual averaging) ----

def _tiny(method):
    op = o.Op(o.OP_BILINEAR, np.array([[1.0]], dtype=np.float32))           # V(x, y) = (y, -x)
    st = o.EgState(np.array([1.0, 0.0], dtype=np.float32), K=1)
    lev = np.array([0.0, 1.0], dtype=np.float32)
    gp, mp = np.zeros((1, 2), np.float32), np.zeros(2, np.float32)
    step = lambda: o.family_step(st, method, op, None, 2, lev, o.codebook_fixed(2), 0, gp, mp, quantizer_off=True)
    return st, step, gp, mp


def test_dual_averaging_by_hand():
    """Eq. (Quantized DA) on V(x, y) = (y, -x) from z1 = (1, 0), K = 1, no noise, quantizer bypassed:
      g_1 = (0, -1); Y_2 = (0, 1); sum = ||g_1||^2 = 1; gamma_2 = 1/sqrt 2; z_2 = (1, 1/sqrt 2);
      g_2 = (1/sqrt 2, -1); Y_3 = (-1/sqrt 2, 2); sum = 2.5; gamma_3 = 1/sqrt 3.5; z_3 = z_1 + gamma_3 Y_3."""
    st, step, _, _ = _tiny(o.METHOD_DA)
    r = 1.0 / math.sqrt(2.0)
    step()
    assert st.Xhalf.tolist() == [1.0, 0.0] and st.Y.tolist() == [0.0, 1.0]       # X_{t+1/2} = X_t
    assert st.sum_sq == 1.0 and abs(st.gamma - r) < 1e-7 and st.t == 2
    assert np.allclose(st.X, [1.0, r], atol=1e-7) and st.Xbar.tolist() == [1.0, 0.0]
    step()
    g3 = 1.0 / math.sqrt(3.5)
    assert np.allclose(st.Y, [-r, 2.0], atol=1e-6) and abs(st.sum_sq - 2.5) < 1e-6 and abs(st.gamma - g3) < 1e-6
    assert np.allclose(st.X, [1.0 - g3 * r, 2.0 * g3], atol=1e-6)
    assert np.allclose(st.Xbar, [1.0, r / 2], atol=1e-6)


def test_optimistic_dual_averaging_by_hand():
    """Eq. (Quantized OptDA), same problem; the first iteration has no earlier feedback (taken as zero):
      z_{3/2} = z_1; g_{3/2} = (0, -1); Y_2 = (0, 1); sum = 1; gamma_2 = 1/sqrt 2; z_2 = (1, 1/sqrt 2);
      z_{5/2} = z_2 - gamma_2 g_{3/2} = (1, sqrt 2); g_{5/2} = (sqrt 2, -1); Y_3 = (-sqrt 2, 2);
      sum = 1 + ||g_{3/2} - g_{5/2}||^2 = 3; gamma_3 = 1/2; z_3 = (1 - sqrt 2 / 2, 1)."""
    st, step, gp, mp = _tiny(o.METHOD_OPTDA)
    r, s2 = 1.0 / math.sqrt(2.0), math.sqrt(2.0)
    step()
    assert st.Xhalf.tolist() == [1.0, 0.0] and st.Y.tolist() == [0.0, 1.0] and st.sum_sq == 1.0
    assert gp.tolist() == [[0.0, -1.0]] and mp.tolist() == [0.0, -1.0]
    assert np.allclose(st.X, [1.0, r], atol=1e-7)
    step()
    assert np.allclose(st.Xhalf, [1.0, s2], atol=1e-6) and np.allclose(gp, [[s2, -1.0]], atol=1e-6)
    assert np.allclose(st.Y, [-s2, 2.0], atol=1e-6) and abs(st.sum_sq - 3.0) < 1e-6 and abs(st.gamma - 0.5) < 1e-6
    assert np.allclose(st.X, [1.0 - s2 / 2, 1.0], atol=1e-6)
    assert np.allclose(st.Xbar, [1.0, s2 / 2], atol=1e-6) and st.t == 3


def test_family_closed_forms_for_a_constant_operator():
    """A(x) = b for all x (M = 0), K workers, no noise, quantizer bypassed.
    DA: sum after t steps = t K ||b||^2, so X_{T+1} = X_1 - T b K / sqrt(1 + T K ||b||^2).
    OptDA: only the first iteration adds to the sum (K ||b||^2), so X_{T+1} = X_1 - T b K / sqrt(1 + K ||b||^2)."""
    n, K, T = 6, 3, 7
    b = np.array([0.5, -1.0, 0.25, 2.0, 0.0, -0.125], dtype=np.float32)
    x1 = np.arange(n, dtype=np.float32)
    op = o.Op(o.OP_DENSE_AFFINE, np.zeros((n, n), np.float32), b)
    nb2 = float(np.dot(b.astype(np.float64), b.astype(np.float64)))
    lev = np.array([0.0, 1.0], dtype=np.float32)
    for method, total in ((o.METHOD_DA, T * K * nb2), (o.METHOD_OPTDA, K * nb2)):
        st = o.EgState(x1, K=K)
        gp, mp = np.zeros((K, n), np.float32), np.zeros(n, np.float32)
        for _ in range(T):
            o.family_step(st, method, op, None, 2, lev, o.codebook_fixed(2), 0, gp, mp, quantizer_off=True)
        assert abs(st.sum_sq - total) <= 1e-12 * total
        gam = K / math.sqrt(1.0 + total)
        assert abs(st.gamma - gam) <= 1e-6 * gam
        assert np.allclose(st.Y, -T * b.astype(np.float64), rtol=1e-6, atol=1e-6)
        assert np.allclose(st.X, x1 - gam * T * b.astype(np.float64), rtol=1e-5, atol=1e-5)


def test_family_step_is_the_pinned_exchange_plus_the_update_rules():
    """Quantizer on: the step's feedback is exactly what the (separately pinned) exchange returns for the dual
    vectors at X_{t+1/2} with exchange id 2t + 1, and the step-size sum grows by the squared differences."""
    vi = gen.c4_affine(n=96, K=4, seed=7, bucket=32, noise_std=0.5)
    M, b = vi.M.numpy(), vi.b.numpy()
    op = o.Op(o.OP_DENSE_AFFINE, M, b)
    lev = gen.uniform_levels(9).numpy().copy()
    cb = o.codebook_fixed(9, 16)
    for method in (o.METHOD_DA, o.METHOD_OPTDA):
        st = o.EgState(vi.x0.numpy(), K=4)
        gp, mp = np.zeros((4, 96), np.float32), np.zeros(96, np.float32)
        for t in range(1, 6):
            nz = vi.noise(t).numpy()[1]
            x_before, y_before, s_before, g_before = st.X.copy(), st.Y.copy(), st.sum_sq, gp.copy()
            gamma_t = np.float32(st.gamma)
            xh = (x_before - gamma_t * mp).astype(np.float32) if method == o.METHOD_OPTDA else x_before
            V = o.form_dual_vectors(o.apply_operator(op, xh), nz, 4)
            mean, tot, vhat = o.exchange(V, vi.bucket, lev, cb, vi.seed, 2 * t + 1, return_vhat=True)
            bits = o.family_step(st, method, op, nz, vi.bucket, lev, cb, vi.seed, gp, mp)
            assert np.array_equal(st.Xhalf, xh) and bits == int(tot.sum())
            assert np.array_equal(st.Y, y_before - mean)
            before = g_before if method == o.METHOD_OPTDA else np.zeros_like(vhat)
            inc = np.sum((before - vhat).astype(np.float64) ** 2)
            assert abs((st.sum_sq - s_before) - inc) <= 1e-12 * max(inc, 1.0)
            assert abs(st.gamma - 4.0 / math.sqrt(1.0 + st.sum_sq)) <= 1e-6 * st.gamma
            if method == o.METHOD_OPTDA:
                assert np.array_equal(gp, vhat) and np.array_equal(mp, mean)


def test_optimistic_dual_averaging_solves_the_bilinear_game_where_dual_averaging_does_not():
    """On min_x max_y x^T A y plain dual averaging is known to cycle or drift, the optimistic variant converges
    (the reason the family carries an extrapolation step): trend only."""
    def run(method, T):
        g = gen.c1_bilinear(n=64, K=4, T=T, seed=11, noise_std=0.05, bucket=64)
        op = o.Op(o.OP_BILINEAR, g.A.numpy())
        st = o.EgState(g.z0.numpy(), K=4)
        lev = gen.uniform_levels(9).numpy().copy()
        cb = o.codebook_fixed(9, 32)
        gp, mp = np.zeros((4, 128), np.float32), np.zeros(128, np.float32)
        noise = g.noise.numpy()
        for t in range(1, T + 1):
            o.family_step(st, method, op, noise[t - 1, 1], g.bucket, lev, cb, g.seed, gp, mp)
        return float(np.linalg.norm(st.Xbar)), float(np.linalg.norm(g.z0.numpy()))
    e_opt_short, z0 = run(o.METHOD_OPTDA, 40)
    e_opt_long, _ = run(o.METHOD_OPTDA, 240)
    e_da_long, _ = run(o.METHOD_DA, 240)
    assert e_opt_long < e_opt_short < z0
    assert e_opt_long < e_da_long


# ---- relative noise (Assumption 3; random player updating of the appendix on examples) ----

def test_relative_noise_oracle_is_a_product_with_mean_one_scales():
    a = np.array([2.0, -3.0, 0.0, 0.5], dtype=np.float32)
    S = np.array([[2.0, 0.0, 2.0, 0.0], [0.0, 2.0, 2.0, 2.0]], dtype=np.float32)
    assert o.form_dual_vectors_relative(a, S, 2).tolist() == [[4.0, -0.0, 0.0, 0.0], [0.0, -6.0, 0.0, 1.0]]
    assert o.form_dual_vectors_relative(a, None, 3).tolist() == [a.tolist()] * 3
    # where the operator vanishes the dual vectors vanish, whatever was drawn: the noise is relative
    assert not o.form_dual_vectors_relative(np.zeros(4, np.float32), S, 2).any()
    # the seeded scales: blocks of equal values in {0, 1/p}, mean one, relative variance 1/p - 1
    s = gen.player_scales((4, 1 << 16), 64, 0.25, seed=3).numpy()
    assert set(np.unique(s).tolist()) == {0.0, 4.0}
    assert np.all(s.reshape(4, -1, 64) == s.reshape(4, -1, 64)[:, :, :1])
    assert abs(s.mean() - 1.0) < 0.05 and abs(s.var() - 3.0) < 0.3
    assert np.array_equal(s, gen.player_scales((4, 1 << 16), 64, 0.25, seed=3).numpy())


def _relative_run(model, T, K=4, d=256, seed=5):
    D = gen.uniform((d,), seed, "cpu", 0.2, 1.0).numpy()
    x0 = gen.gaussian((d,), seed + 1, "cpu").numpy()
    op = o.Op(o.OP_DIAGONAL, D, noise_model=model)                 # gradient of a convex quadratic: co-coercive
    st = o.EgState(x0, K)
    lev = gen.uniform_levels(17).numpy().copy()
    cb = o.codebook_fixed(17, 32)
    sigma = float(np.linalg.norm(D * x0) / math.sqrt(d))          # absolute noise as large as the relative one at x0
    marks = {}
    for t in range(1, T + 1):
        if model == o.NOISE_RELATIVE:
            nz = gen.player_scales((2, K, d), 64, 0.5, seed * 1000 + t).numpy()
        else:
            nz = gen.gaussian((2, K, d), seed * 1000 + t, "cpu", std=sigma).numpy()
        refit = 2 if t == 1 else (1 if t % 20 == 1 else 0)
        o.eg_step(st, op, nz[0], nz[1], 512, lev, cb, seed, refit=refit, code_type=o.CODE_HUFFMAN, nbins=256)
        if t in (T // 4, T):
            nx = float(np.linalg.norm(x0))
            marks[t] = (float(np.linalg.norm(st.Xbar)) / nx, float(np.linalg.norm(st.X)) / nx, st.gamma)
    return marks


def test_relative_noise_gives_the_fast_regime():
    """Theorem 4 against Theorem 3, as trends: with relative noise and a co-coercive operator the squared differences
    are summable, so the adaptive step stops shrinking, the iterates themselves converge and the ergodic average
    gains about 1/T; with absolute noise of the same initial size the step keeps shrinking like 1/sqrt t and the
    average gains about 1/sqrt T."""
    T = 800
    rel, ab = _relative_run(o.NOISE_RELATIVE, T), _relative_run(o.NOISE_ADDITIVE, T)
    assert rel[T][2] > 0.95 * rel[T // 4][2]                       # step size settled
    assert ab[T][2] < 0.65 * ab[T // 4][2]                         # step size still falling
    assert rel[T // 4][0] / rel[T][0] > 2.5                        # four times the iterations: close to 4x
    assert ab[T // 4][0] / ab[T][0] < 2.0                          # close to 2x
    assert rel[T][1] < 0.02 < ab[T][1]                             # the last iterate itself


def test_relative_noise_special_cases():
    d, K = 96, 3
    D = gen.uniform((d,), 1, "cpu", 0.2, 1.0).numpy()
    lev = gen.uniform_levels(9).numpy().copy()
    cb = o.codebook_fixed(9, 32)
    # the solution is a fixed point whatever is drawn (under additive noise it is not)
    st = o.EgState(np.zeros(d, np.float32), K)
    S = gen.player_scales((2, K, d), 8, 0.5, seed=2).numpy()
    for _ in range(3):
        o.eg_step(st, o.Op(o.OP_DIAGONAL, D, noise_model=o.NOISE_RELATIVE), S[0], S[1], 32, lev, cb, 9)
    assert not st.X.any() and not st.Y.any() and st.sum_sq == 0.0 and st.gamma == K
    # scales of one are no noise at all
    x0 = gen.gaussian((d,), 4, "cpu").numpy()
    a, b = o.EgState(x0, K), o.EgState(x0, K)
    ones = np.ones((K, d), np.float32)
    for _ in range(3):
        o.eg_step(a, o.Op(o.OP_DIAGONAL, D, noise_model=o.NOISE_RELATIVE), ones, ones, 32, lev, cb, 9)
        o.eg_step(b, o.Op(o.OP_DIAGONAL, D), None, None, 32, lev, cb, 9)
    assert np.array_equal(a.X, b.X) and a.sum_sq == b.sum_sq


# ---- a level table of its own for each exchange (footnote of Sec. 3.3) ----

def test_two_level_tables():
    d, K, bucket = 1536, 4, 256
    D = gen.uniform((d,), 31, "cpu", 0.05, 1.0).numpy()
    x0 = gen.gaussian((d,), 32, "cpu").numpy()
    op = o.Op(o.OP_DIAGONAL, D)
    n_t = gen.gaussian((K, d), 33, "cpu", std=0.2).numpy()
    n_h = gen.student_t3((K, d), 34, "cpu").numpy() * np.float32(0.3)          # heavier tails at the half step
    lev0 = gen.uniform_levels(17).numpy()
    # equal tables, no refit: the single-table iteration, bit for bit
    a, b = o.EgState(x0, K), o.EgState(x0, K)
    la, lb, lc = lev0.copy(), lev0.copy(), lev0.copy()
    ca, cb_, cc = o.codebook_fixed(17, 32), o.codebook_fixed(17, 32), o.codebook_fixed(17, 32)
    for _ in range(2):
        bits_a = o.eg_step(a, op, n_t, n_h, bucket, la, ca, 3)
        bits_b = o.eg_step_two_tables(b, op, n_t, n_h, bucket, lb, cb_, lc, cc, 3)
        assert bits_a == bits_b and np.array_equal(a.X, b.X) and a.sum_sq == b.sum_sq and np.array_equal(a.Xbar, b.Xbar)
    # a refit fits each table to its own dual vectors: the pinned refit applied to V_t and to V_{t+1/2}
    st = o.EgState(x0, K)
    lt, lh = lev0.copy(), lev0.copy()
    ct, ch = o.codebook_fixed(17, 32), o.codebook_fixed(17, 32)
    V_t = o.form_dual_vectors(o.apply_operator(op, st.X), n_t, K)
    lt_ref, hist_t = o.refit(V_t, bucket, 256, lev0.copy(), o.codebook_fixed(17, 32), True, o.CODE_HUFFMAN)
    o.eg_step_two_tables(st, op, n_t, n_h, bucket, lt, ct, lh, ch, 3, refit=2, code_type=o.CODE_HUFFMAN, nbins=256)
    assert np.array_equal(lt, lt_ref)
    V_h = o.form_dual_vectors(o.apply_operator(op, st.Xhalf), n_h, K)
    lh_ref, hist_h = o.refit(V_h, bucket, 256, lev0.copy(), o.codebook_fixed(17, 32), True, o.CODE_HUFFMAN)
    assert np.array_equal(lh, lh_ref) and not np.array_equal(lt, lh)
    # what the second table is for: on the half-step vectors it has the smaller quantization variance (QAda objective)
    assert o.objective(hist_h, lh) < o.objective(hist_h, lt)
    assert o.objective(hist_t, lt) < o.objective(hist_t, lh)
    # and the realised error of the second exchange is smaller with its own table (same draws)
    def err(levels, cbk):
        _, _, vhat = o.exchange(V_h, bucket, levels, cbk, 3, 3, return_vhat=True)
        return float(np.sum((vhat.astype(np.float64) - V_h) ** 2))
    assert err(lh, ch) < err(lt, ct)

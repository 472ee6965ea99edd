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

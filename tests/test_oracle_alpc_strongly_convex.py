"""Pins for the oracle's strongly convex ALPC-SVRG step (Algorithm 2 with h = lambda_l1*||.||_1 + (sigma/2)*||.||^2):
the two updates against brute-force minimisation of the printed argmins, sigma = 0 against the general convex step
bit for bit, the weighted snapshot against fp64, and a full-precision run against an independently written fp64
loop of Algorithm 2 (CPU only)."""
import numpy as np
import pytest

import oracle as orc
from paper_1901_08924_b200 import synth


def _problem(n=64, d=24, loss="least_squares", seed=0, **kw):
    X, y, _ = synth.linear_problem(n, d, loss=loss, sparsity=0.3, noise=0.1, seed=seed)
    code = orc.LOGISTIC if loss == "logistic" else orc.LEAST_SQUARES
    args = dict(loss=code, lambda_l1=1e-3, N=4, B=2, b=4, clip_mode=orc.CLIP_STD, clip_value=2.5, seed=7)
    args.update(kw)
    return orc.Problem(X.numpy(), y.numpy(), **args)


@pytest.mark.parametrize("sigma", [0.05, 0.7, 3.0])
def test_updates_are_the_argmins_with_an_elastic_net(sigma):
    # steps 12-13 of Algorithm 2 by brute-force scalar minimisation (d = 1 problem)
    X = np.array([[1.0], [2.0], [-1.5], [0.5]], np.float32)
    y = np.array([1.0, -1.0, 1.0, 1.0], np.float32)
    lam, L = 0.3, 2.0
    P = orc.Problem(X, y, orc.LOGISTIC, lam, N=2, B=1, b=32, clip_mode=orc.CLIP_NONE, clip_value=1.0, seed=3)
    xs = np.array([0.4], np.float32)
    mu, _, _ = orc.full_grad(X, y, P.loss, xs)
    yk, zk = np.array([0.9], np.float32), np.array([-0.6], np.float32)
    tau1, tau2, alpha, w = 0.4, 0.5, 0.35, 1.75
    yn, zn, sn, t = orc.alpc_step(P, 2, tau1, tau2, alpha, 1 / (4 * L), xs, mu, yk, zk, np.array([0.25], np.float32),
                                  taps=True, sigma=sigma, weight=w)
    xk = t["x"][0]
    grid = np.linspace(-3, 3, 600001)
    h = lam * np.abs(grid) + 0.5 * sigma * grid ** 2
    oy = 2 * L * (grid - xk) ** 2 + t["v"][0] * grid + h
    oz = (grid - zk[0]) ** 2 / (2 * alpha) + t["vhat"][0] * grid + h
    assert abs(yn[0] - grid[oy.argmin()]) < 2e-5
    assert abs(zn[0] - grid[oz.argmin()]) < 2e-5
    assert sn[0] == pytest.approx(0.25 + w * yn[0], rel=1e-6)


def test_sigma_zero_and_unit_weight_reproduce_the_general_convex_step():
    P = _problem(n=60, d=21, N=3, B=2)
    rng = np.random.default_rng(1)
    xs, yk, zk, s0 = (rng.standard_normal(P.d).astype(np.float32) for _ in range(4))
    mu, _, _ = orc.full_grad(P.X, P.y, P.loss, xs)
    a = orc.alpc_step(P, 5, 0.5, 0.25, 0.2, 0.1, xs, mu, yk, zk, s0)
    c = orc.alpc_step(P, 5, 0.5, 0.25, 0.2, 0.1, xs, mu, yk, zk, s0, sigma=0.0, weight=1.0)
    for u, v in zip(a, c):
        assert (u.view(np.uint32) == v.view(np.uint32)).all()
    # sigma > 0 shrinks both iterates towards zero, by exactly the two factors
    e = orc.alpc_step(P, 5, 0.5, 0.25, 0.2, 0.1, xs, mu, yk, zk, s0, sigma=0.8, weight=1.0)
    assert np.allclose(e[0], a[0] / (1 + 0.8 * 0.1), rtol=1e-6, atol=1e-9)
    assert np.allclose(e[1], a[1] / (1 + 0.2 * 0.8), rtol=1e-6, atol=1e-9)


def test_weighted_snapshot_against_float64():
    rng = np.random.default_rng(2)
    m, d, alpha, sigma = 37, 50, 0.3, 0.2
    ys = rng.standard_normal((m, d)).astype(np.float32)
    theta = np.float32(1.0) + np.float32(alpha) * np.float32(sigma)
    w, wsum, ysum = np.float32(1.0), np.float32(0.0), np.zeros(d, np.float32)
    for t in range(m):  # the accumulation the step performs
        ysum = ysum + w * ys[t]
        wsum = np.float32(wsum + w)
        w = np.float32(w * theta)
    got = orc.weighted_snapshot(ysum, wsum)
    w64 = (1.0 + alpha * sigma) ** np.arange(m)
    exact = (w64[:, None] * ys.astype(np.float64)).sum(axis=0) / w64.sum()
    assert np.abs(got - exact).max() < 1e-5 * np.abs(exact).max() + 1e-6
    # equal weights: the plain mean of Algorithm 3
    assert np.allclose(orc.weighted_snapshot(ys.sum(axis=0, dtype=np.float32), np.float32(m)), ys.mean(axis=0), atol=1e-6)
    assert orc.ridge_term(np.array([3.0, -4.0], np.float32), 0.5) == pytest.approx(0.25 * 25.0)


def test_full_precision_run_follows_an_independent_loop_of_algorithm2():
    """b = 32, no clipping: the quantizer is the identity, so the epoch is Katyusha-style SVRG with double sampling;
    an fp64 loop written here from Algorithm 2 must give the same snapshot, and the objective must fall."""
    P = _problem(n=48, d=12, N=3, B=2, b=32, clip_mode=orc.CLIP_NONE, clip_value=1.0, lambda_l1=1e-3)
    X64, y64 = P.X.astype(np.float64), P.y.astype(np.float64)
    L = float((X64 ** 2).sum(axis=1).max())
    sigma, m = 0.05 * L, 20
    tau1, tau2 = float(np.sqrt(m * sigma / (6 * L))), 0.5
    alpha = 1.0 / (6 * tau1 * L)
    theta = np.float32(1.0) + np.float32(alpha) * np.float32(sigma)
    soft = lambda w, kap: np.sign(w) * np.maximum(np.abs(w) - kap, 0.0)
    grad_rows = lambda rows, x: (X64[rows].T * (X64[rows] @ x - y64[rows])).mean(axis=1)
    obj = lambda x: 0.5 * np.mean((X64 @ x - y64) ** 2) + P.lambda_l1 * np.abs(x).sum() + 0.5 * sigma * (x ** 2).sum()
    xs = np.zeros(P.d, np.float32)
    y = z = xs.copy()
    xs64 = xs.astype(np.float64)
    y64i, z64i = xs64.copy(), xs64.copy()
    n_i = P.n // P.N
    p0 = obj(xs64)
    for s in range(3):
        mu, _, _ = orc.full_grad(P.X, P.y, P.loss, xs)
        mu64 = grad_rows(np.arange(P.n), xs64)
        ysum, w, wsum = np.zeros(P.d, np.float32), np.float32(1.0), np.float32(0.0)
        acc64, w64, wsum64 = np.zeros(P.d), 1.0, 0.0
        for t in range(m):
            k = s * m + t
            y, z, ysum = orc.alpc_step(P, k, tau1, tau2, alpha, 1 / (4 * L), xs, mu, y, z, ysum, sigma=sigma, weight=w)
            wsum, w = np.float32(wsum + w), np.float32(w * theta)
            # the same step in fp64, from the algorithm box
            x = tau1 * z64i + tau2 * xs64 + (1 - tau1 - tau2) * y64i
            u = np.mean([grad_rows(orc.sample_batch(P.seed, orc.TAG_BATCH, i, k, P.B, i * n_i, n_i), x)
                         - grad_rows(orc.sample_batch(P.seed, orc.TAG_BATCH, i, k, P.B, i * n_i, n_i), xs64)
                         for i in range(P.N)], axis=0)
            J = orc.sample_batch(P.seed, orc.TAG_BATCH_J, 0, k, P.B, 0, P.n)
            v, vhat = u + mu64, grad_rows(J, x) - grad_rows(J, xs64) + mu64
            y64i = soft(x - v / (4 * L), P.lambda_l1 / (4 * L)) / (1 + sigma / (4 * L))
            z64i = soft(z64i - alpha * vhat, alpha * P.lambda_l1) / (1 + alpha * sigma)
            acc64, wsum64, w64 = acc64 + w64 * y64i, wsum64 + w64, w64 * (1 + alpha * sigma)
        xs = orc.weighted_snapshot(ysum, wsum)
        xs64 = acc64 / wsum64
        assert np.abs(xs - xs64).max() < 2e-4 * max(1.0, np.abs(xs64).max())
    assert obj(xs64) < 0.7 * p0
    assert orc.objective(P.X, P.y, P.loss, xs, P.lambda_l1) + orc.ridge_term(xs, sigma) == pytest.approx(obj(xs.astype(np.float64)), rel=1e-5)

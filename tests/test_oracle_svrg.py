"""Pins for the oracle's linear-model path: losses, full gradient, sampling, the SVRG estimator,
Algorithm 1's step and Algorithm 2's step (CPU only)."""
import math

import numpy as np
import pytest

import oracle as orc
from paper_1901_08924_b200 import synth


def _problem(n=64, d=24, loss="logistic", seed=0, **kw):
    X, y, _ = synth.linear_problem(n, d, loss=loss, sparsity=0.3, noise=0.1, seed=seed)
    code = orc.LOGISTIC if loss == "logistic" else orc.LEAST_SQUARES
    args = dict(loss=code, lambda_l1=1e-3, N=4, B=2, b=4, clip_mode=orc.CLIP_STD, clip_value=2.5, seed=7)
    args.update(kw)
    return orc.Problem(X.numpy(), y.numpy(), **args)


def _f64_loss(loss, m, y):
    return 0.5 * (m - y) ** 2 if loss == orc.LEAST_SQUARES else np.log1p(np.exp(-y * m))


@pytest.mark.parametrize("loss", [orc.LOGISTIC, orc.LEAST_SQUARES])
def test_loss_derivative_is_derivative_of_loss(loss):
    for m, y in [(0.25, 1.0), (-1.25, 1.0), (2.0, -1.0), (0.0, -1.0), (5.5, 0.25)]:  # dyadic: exact in fp32
        h = 2.0 ** -7
        num = (orc.loss_value(loss, m + h, y) - orc.loss_value(loss, m - h, y)) / (2 * h)
        assert abs(float(orc.loss_deriv(loss, m, y)) - num) < 1e-5
        assert abs(orc.loss_value(loss, m, y) - _f64_loss(loss, m, y)) < 1e-6
    if loss == orc.LOGISTIC:  # no overflow at large margins
        assert orc.loss_deriv(loss, 1000.0, 1.0) == 0 and orc.loss_deriv(loss, -1000.0, 1.0) == -1
        assert abs(orc.loss_value(loss, -1000.0, 1.0) - 1000.0) < 1e-9


@pytest.mark.parametrize("loss", ["logistic", "least_squares"])
def test_full_gradient_against_float64_and_finite_differences(loss):
    P = _problem(n=50, d=17, loss=loss)
    rng = np.random.default_rng(1)
    x = rng.standard_normal(P.d).astype(np.float32) * 0.5
    mu, margins, f = orc.full_grad(P.X, P.y, P.loss, x)
    X64, y64, x64 = P.X.astype(np.float64), P.y.astype(np.float64), x.astype(np.float64)
    m64 = X64 @ x64
    assert np.abs(margins - m64).max() < 1e-6
    g = (m64 - y64) if P.loss == orc.LEAST_SQUARES else (-y64 / (1 + np.exp(y64 * m64)))
    assert np.abs(mu - X64.T @ g / P.n).max() < 1e-6  # Algorithm 1 step 4: (1/n) sum of per-sample gradients
    assert abs(f - _f64_loss(P.loss, m64, y64).mean()) < 1e-6
    # gradient of f by central differences of the objective (lambda = 0)
    h = 1e-3
    for j in (0, 5, 16):
        e = np.zeros(P.d, np.float32)
        e[j] = h
        num = (orc.objective(P.X, P.y, P.loss, x + e, 0.0) - orc.objective(P.X, P.y, P.loss, x - e, 0.0)) / (2 * h)
        assert abs(num - mu[j]) < 2e-4
    assert abs(orc.objective(P.X, P.y, P.loss, x, 0.25) - (f + 0.25 * np.abs(x64).sum())) < 1e-9


def test_sampling_range_uniformity_and_streams():
    n_i, B = 37, 4
    counts = np.zeros(n_i)
    for k in range(3000):
        idx = orc.sample_batch(5, orc.TAG_BATCH, 2, k, B, 2 * n_i, n_i)
        assert ((idx >= 2 * n_i) & (idx < 3 * n_i)).all()
        np.add.at(counts, idx - 2 * n_i, 1)
    expect = 3000 * B / n_i
    assert ((counts - expect) ** 2 / expect).sum() < 80  # 36 dof, p ~ 3e-5
    a = orc.sample_batch(5, orc.TAG_BATCH, 0, 9, 8, 0, 1000)
    assert (a != orc.sample_batch(5, orc.TAG_BATCH, 1, 9, 8, 0, 1000)).any()      # workers independent
    assert (a != orc.sample_batch(5, orc.TAG_BATCH_J, 0, 9, 8, 0, 1000)).any()    # J independent of i_B
    assert (a != orc.sample_batch(5, orc.TAG_BATCH, 0, 10, 8, 0, 1000)).any()     # iterations independent
    assert (a != orc.sample_batch(6, orc.TAG_BATCH, 0, 9, 8, 0, 1000)).any()


@pytest.mark.parametrize("loss", ["logistic", "least_squares"])
def test_estimator_equals_full_gradient_at_snapshot(loss):
    # at x = x~ the difference u vanishes, so v = grad f(x~) exactly and all codes are the zero code
    P = _problem(loss=loss)
    rng = np.random.default_rng(2)
    xs = rng.standard_normal(P.d).astype(np.float32)
    mu, _, _ = orc.full_grad(P.X, P.y, P.loss, xs)
    xn, t = orc.lpc_inner_step(P, k=3, eta=0.1, x=xs, xs=xs, mu=mu, taps=True)
    assert (t["coef"] == 0).all() and (t["u"] == 0).all() and (t["delta"] == 0).all()
    assert (t["v"] == mu).all()
    for i in range(P.N):
        assert (orc.unpack(t["words"][i], P.d, P.b) == 2 ** (P.b - 1)).all()
    w = xs.astype(np.float64) - 0.1 * mu
    expect = np.sign(w) * np.maximum(np.abs(w) - 0.1 * P.lambda_l1, 0)
    assert np.abs(xn - expect).max() < 1e-6


@pytest.mark.parametrize("loss", ["logistic", "least_squares"])
def test_estimator_is_unbiased_over_batches(loss):
    # B = 1: averaging c_a X_a over every row a, plus mu, is grad f(x) (Assumption 1)
    P = _problem(n=8, d=6, loss=loss, B=1, N=1)
    rng = np.random.default_rng(3)
    x = rng.standard_normal(P.d).astype(np.float32)
    xs = rng.standard_normal(P.d).astype(np.float32)
    mu, _, _ = orc.full_grad(P.X, P.y, P.loss, xs)
    gx, _, _ = orc.full_grad(P.X, P.y, P.loss, x)
    acc = np.zeros(P.d)
    for a in range(P.n):
        c = orc.svrg_coef(P.X, P.y, P.loss, [a], x, xs)
        acc += orc.svrg_diff_from_coef(P.X, [a], c)
    assert np.abs(acc / P.n + mu - gx).max() < 1e-6


def test_svrg_difference_against_float64():
    P = _problem(n=40, d=33, loss="logistic", B=4)
    rng = np.random.default_rng(4)
    x, xs = (rng.standard_normal(P.d).astype(np.float32) for _ in range(2))
    idx = np.array([3, 17, 3, 39])
    c = orc.svrg_coef(P.X, P.y, P.loss, idx, x, xs)
    u = orc.svrg_diff_from_coef(P.X, idx, c)
    X64, y64 = P.X.astype(np.float64), P.y.astype(np.float64)
    g = lambda v: -y64[idx] / (1 + np.exp(y64[idx] * (X64[idx] @ v.astype(np.float64))))
    c64 = g(x) - g(xs)
    assert np.abs(c - c64).max() < 1e-6
    assert np.abs(u - (c64[:, None] * X64[idx]).mean(axis=0)).max() < 1e-6  # (1/B) sum over the batch


def _prox_svrg_reference(P, x0, S, m, eta):
    """Independently written minibatch prox-SVRG in float64 (no quantization), using the oracle only
    for the batch indices so that both runs see the same samples."""
    X, y = P.X.astype(np.float64), P.y.astype(np.float64)
    grad = (lambda rows, v: X[rows].T * ((X[rows] @ v) - y[rows])) if P.loss == orc.LEAST_SQUARES else \
        (lambda rows, v: X[rows].T * (-y[rows] / (1 + np.exp(y[rows] * (X[rows] @ v)))))
    snap = x0.astype(np.float64)
    x = snap.copy()
    n_i = P.n // P.N
    for s in range(S):
        full = grad(np.arange(P.n), snap).mean(axis=1)
        x = snap.copy()
        for t in range(m):
            k = s * m + t
            u = np.zeros(P.d)
            for i in range(P.N):
                rows = orc.sample_batch(P.seed, orc.TAG_BATCH, i, k, P.B, i * n_i, n_i)
                u += (grad(rows, x) - grad(rows, snap)).mean(axis=1)
            w = x - eta * (u / P.N + full)
            x = np.sign(w) * np.maximum(np.abs(w) - eta * P.lambda_l1, 0)
        snap = x.copy()
    return snap


@pytest.mark.parametrize("loss", ["logistic", "least_squares"])
def test_full_precision_bypass_is_prox_svrg(loss):
    # Section 3: with u~ = (1/N) sum u^i Algorithm 1 is minibatch prox-SVRG
    P = _problem(n=48, d=12, loss=loss, b=32, clip_mode=orc.CLIP_NONE)
    rng = np.random.default_rng(6)
    x0 = rng.standard_normal(P.d).astype(np.float32) * 0.3
    S, m, eta = 2, 15, 0.2
    snap = x0.copy()
    for s in range(S):
        mu, _, _ = orc.full_grad(P.X, P.y, P.loss, snap)
        x = snap.copy()
        for t in range(m):
            x = orc.lpc_inner_step(P, s * m + t, eta, x, snap, mu)
        snap = x
    ref = _prox_svrg_reference(P, x0, S, m, eta)
    assert np.abs(snap - ref).max() < 2e-5
    p0 = orc.objective(P.X, P.y, P.loss, x0, P.lambda_l1)
    assert orc.objective(P.X, P.y, P.loss, snap, P.lambda_l1) < p0


def test_quantized_step_stays_close_to_full_precision_step():
    # scheme (a): the only precision loss is Q itself, bounded per coordinate by delta_i (Lemma 1's
    # support), so |x+_quantized - x+_fp| <= eta * mean_i delta_i
    P = _problem(n=64, d=40, loss="least_squares", b=4, clip_mode=orc.CLIP_NONE)
    P32 = _problem(n=64, d=40, loss="least_squares", b=32, clip_mode=orc.CLIP_NONE)
    rng = np.random.default_rng(8)
    x, xs = (rng.standard_normal(P.d).astype(np.float32) for _ in range(2))
    mu, _, _ = orc.full_grad(P.X, P.y, P.loss, xs)
    xq, t = orc.lpc_inner_step(P, 5, 0.1, x, xs, mu, taps=True)
    xf = orc.lpc_inner_step(P32, 5, 0.1, x, xs, mu)
    assert (t["delta"] > 0).all()
    assert np.abs(xq - xf).max() <= 0.1 * float(t["delta"].mean()) * (1 + 1e-5) + 1e-7
    # and the packed messages decode to the taps
    for i in range(P.N):
        w, dlt, _ = orc.quantize_pack(t["u"][i], P.b, P.clip_mode, P.clip_value, P.seed, i, 5)
        assert (w == t["words"][i]).all() and dlt == t["delta"][i]


def test_alpc_updates_are_the_argmins_of_algorithm2():
    # steps 12-13 of Algorithm 2 by brute-force scalar minimisation (d = 1 problem)
    X = np.array([[1.0], [2.0], [-1.5], [0.5]], np.float32)
    y = np.array([1.0, -1.0, 1.0, 1.0], np.float32)
    lam, L = 0.3, 2.0
    P = orc.Problem(X, y, orc.LOGISTIC, lam, N=2, B=1, b=32, clip_mode=orc.CLIP_NONE, clip_value=1.0, seed=3)
    xs = np.array([0.4], np.float32)
    mu, _, _ = orc.full_grad(X, y, P.loss, xs)
    yk, zk = np.array([0.9], np.float32), np.array([-0.6], np.float32)
    tau1, tau2, alpha = 0.4, 0.5, 0.35
    yn, zn, sn, t = orc.alpc_step(P, 2, tau1, tau2, alpha, 1 / (4 * L), xs, mu, yk, zk, np.zeros(1, np.float32), taps=True)
    xk = tau1 * zk[0] + tau2 * xs[0] + (1 - tau1 - tau2) * yk[0]
    assert abs(t["x"][0] - xk) < 1e-6
    grid = np.linspace(-3, 3, 600001)
    oy = 2 * L * (grid - xk) ** 2 + t["v"][0] * grid + lam * np.abs(grid)
    oz = (grid - zk[0]) ** 2 / (2 * alpha) + t["vhat"][0] * grid + lam * np.abs(grid)
    assert abs(yn[0] - grid[oy.argmin()]) < 2e-5
    assert abs(zn[0] - grid[oz.argmin()]) < 2e-5
    assert sn[0] == yn[0]


def test_alpc_estimators_against_float64():
    P = _problem(n=60, d=21, loss="least_squares", b=32, clip_mode=orc.CLIP_NONE, N=3, B=2, lambda_l1=0.0)
    rng = np.random.default_rng(12)
    xs, yk, zk = (rng.standard_normal(P.d).astype(np.float32) for _ in range(3))
    mu, _, _ = orc.full_grad(P.X, P.y, P.loss, xs)
    tau1, tau2, alpha, L = 0.5, 0.25, 0.2, 1.5
    k = 11
    yn, zn, sn, t = orc.alpc_step(P, k, tau1, tau2, alpha, 1 / (4 * L), xs, mu, yk, zk, yk, taps=True)
    X64, y64 = P.X.astype(np.float64), P.y.astype(np.float64)
    x = tau1 * zk + tau2 * xs + (1 - tau1 - tau2) * yk
    diff = lambda rows: (X64[rows].T * ((X64[rows] @ x) - (X64[rows] @ xs.astype(np.float64)))).mean(axis=1)
    n_i = P.n // P.N
    u = np.mean([diff(orc.sample_batch(P.seed, orc.TAG_BATCH, i, k, P.B, i * n_i, n_i)) for i in range(P.N)], axis=0)
    J = orc.sample_batch(P.seed, orc.TAG_BATCH_J, 0, k, P.B, 0, P.n)  # one shared batch from all rows
    assert np.abs(t["v"] - (u + mu)).max() < 1e-5
    assert np.abs(t["vhat"] - (diff(J) + mu)).max() < 1e-5
    assert np.abs(yn - (x - t["v"] / (4 * L))).max() < 1e-6      # lambda = 0: plain gradient steps
    assert np.abs(zn - (zk - alpha * t["vhat"])).max() < 1e-6
    assert np.abs(sn - (yk + yn)).max() < 1e-6


def test_alpc_with_one_bit_budget_still_uses_full_precision_for_z():
    # double sampling: z moves with the unquantized v^ whatever b is
    Pq = _problem(n=60, d=21, loss="least_squares", b=2, N=3, B=2)
    Pf = _problem(n=60, d=21, loss="least_squares", b=32, clip_mode=orc.CLIP_NONE, N=3, B=2)
    rng = np.random.default_rng(13)
    xs, yk, zk = (rng.standard_normal(Pq.d).astype(np.float32) for _ in range(3))
    mu, _, _ = orc.full_grad(Pq.X, Pq.y, Pq.loss, xs)
    a = orc.alpc_step(Pq, 4, 0.5, 0.25, 0.2, 0.1, xs, mu, yk, zk, yk, taps=True)
    c = orc.alpc_step(Pf, 4, 0.5, 0.25, 0.2, 0.1, xs, mu, yk, zk, yk, taps=True)
    assert (a[1] == c[1]).all() and (a[3]["vhat"] == c[3]["vhat"]).all()
    assert (a[0] != c[0]).any()

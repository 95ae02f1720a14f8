"""Pins for the oracle's outer rule of Algorithm 3 (ALPC-SVRG, general convex case): the per-epoch parameters against
the printed formulas, the snapshot against the plain mean, and whole epochs in full precision (b = 32, no clipping)
against an fp64 loop written here from the algorithm box (CPU only)."""
import numpy as np
import pytest

import oracle as orc
from paper_1901_08924_b200 import synth


def test_epoch_parameters_follow_step_3():
    L = 3.7
    for s in (0, 1, 2, 10, 1000):
        tau1, alpha = orc.alpc3_epoch_params(s, L)
        assert tau1 == np.float32(2.0 / (s + 4))
        assert alpha == np.float32((s + 4) / (12.0 * L))  # 1/(6 L tau1) with tau1 = 2/(s+4)
    # tau1 falls from 1/2 and alpha grows linearly in s
    t0, a0 = orc.alpc3_epoch_params(0, L)
    t4, a4 = orc.alpc3_epoch_params(4, L)
    assert t0 == np.float32(0.5) and t4 == np.float32(0.25) and a4 == pytest.approx(2 * a0, rel=1e-6)


def test_snapshot_is_the_plain_mean_of_the_epochs_iterates():
    rng = np.random.default_rng(0)
    m, d = 29, 40
    ys = rng.standard_normal((m, d)).astype(np.float32)
    ysum = np.zeros(d, np.float32)
    for t in range(m):
        ysum = ysum + ys[t]
    got = orc.alpc3_mean_snapshot(ysum, m)
    assert np.abs(got - ys.astype(np.float64).mean(axis=0)).max() < 1e-6
    assert (orc.alpc3_mean_snapshot(np.full(3, 8.0, np.float32), 4) == 2.0).all()


def test_full_precision_epochs_follow_an_independent_loop_of_algorithm3():
    X, y, _ = synth.linear_problem(60, 10, loss="least_squares", sparsity=0.4, noise=0.05, seed=4)
    P = orc.Problem(X.numpy(), y.numpy(), orc.LEAST_SQUARES, 2e-3, N=3, B=2, b=32, clip_mode=orc.CLIP_NONE,
                    clip_value=1.0, seed=11)
    X64, y64 = P.X.astype(np.float64), P.y.astype(np.float64)
    L = float((X64 ** 2).sum(axis=1).max())
    m, tau2 = 25, 0.5
    soft = lambda w, kap: np.sign(w) * np.maximum(np.abs(w) - kap, 0.0)
    grad_rows = lambda rows, x: (X64[rows].T * (X64[rows] @ x - y64[rows])).mean(axis=1)
    obj = lambda x: 0.5 * np.mean((X64 @ x - y64) ** 2) + P.lambda_l1 * np.abs(x).sum()
    n_i = P.n // P.N
    xs = np.zeros(P.d, np.float32)
    yv = zv = xs.copy()
    xs64 = np.zeros(P.d)
    y64i, z64i = xs64.copy(), xs64.copy()
    p0 = obj(xs64)
    for s in range(4):
        mu, _, _ = orc.full_grad(P.X, P.y, P.loss, xs)
        yv, zv, xs = orc.alpc3_epoch(P, s, m, L, tau2, xs, mu, yv, zv)
        # the same epoch in fp64, from the two algorithm boxes
        tau1 = 2.0 / (s + 4)
        alpha = 1.0 / (6.0 * L * tau1)
        mu64 = grad_rows(np.arange(P.n), xs64)
        acc = np.zeros(P.d)
        for t in range(m):
            k = s * m + t
            x = tau1 * z64i + tau2 * xs64 + (1 - tau1 - tau2) * y64i
            u = np.mean([grad_rows(orc.sample_batch(P.seed, orc.TAG_BATCH, i, k, P.B, i * n_i, n_i), x)
                         - grad_rows(orc.sample_batch(P.seed, orc.TAG_BATCH, i, k, P.B, i * n_i, n_i), xs64)
                         for i in range(P.N)], axis=0)
            J = orc.sample_batch(P.seed, orc.TAG_BATCH_J, 0, k, P.B, 0, P.n)
            v, vhat = u + mu64, grad_rows(J, x) - grad_rows(J, xs64) + mu64
            y64i = soft(x - v / (4 * L), P.lambda_l1 / (4 * L))
            z64i = soft(z64i - alpha * vhat, alpha * P.lambda_l1)
            acc += y64i
        xs64 = acc / m
        assert np.abs(xs - xs64).max() < 2e-4 * max(1.0, np.abs(xs64).max()), s
        assert np.abs(yv - y64i).max() < 2e-4 * max(1.0, np.abs(y64i).max())  # y and z carry over
        assert np.abs(zv - z64i).max() < 2e-4 * max(1.0, np.abs(z64i).max())
    assert obj(xs64) < 0.7 * p0

"""GPU parity for the strongly convex case of ALPC-SVRG (Algorithm 2 with an elastic-net h): single steps and whole
epochs with Theorem 3's parameters against the oracle, bit for bit on least squares, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_1901_08924_b200 import lpc, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _bits(a):
    a = a.detach().cpu().numpy() if isinstance(a, torch.Tensor) else np.asarray(a)
    return a.view(np.uint32) if a.dtype == np.float32 else a


def _same(a, b):
    return (_bits(a) == _bits(b)).all()


def _setup(n, d, loss, N, B, b, clip=(orc.CLIP_STD, 2.5), lam=1e-3, seed=7):
    X, y, _ = synth.linear_problem(n, d, loss=loss, sparsity=0.2, noise=0.1, seed=0)
    code = orc.LOGISTIC if loss == "logistic" else orc.LEAST_SQUARES
    P = orc.Problem(X.numpy(), y.numpy(), code, lam, N, B, b, clip[0], clip[1], seed)
    ctx = lpc.Context(X.to(DEV), y.to(DEV), code, lam, N, B, b, clip[0], clip[1], seed)
    return P, ctx


@pytest.mark.parametrize("loss", ["least_squares", "logistic"])
@pytest.mark.parametrize("n,d,N,B,b", [(96, 64, 4, 2, 4), (256, 1000, 4, 4, 2), (64, 4096, 2, 8, 8)])
def test_single_steps_with_weights(loss, n, d, N, B, b):
    P, ctx = _setup(n, d, loss, N, B, b)
    rng = np.random.default_rng(3)
    xs, y, z = ((rng.standard_normal(P.d) * 0.2).astype(np.float32) for _ in range(3))
    mu, margins, _ = orc.full_grad(P.X, P.y, P.loss, xs)
    for w, t in ((lpc.BUF_XTILDE, xs), (lpc.BUF_MU, mu), (lpc.BUF_MARGINS, margins), (lpc.BUF_Y, y), (lpc.BUF_Z, z)):
        ctx.set_buffer(w, torch.from_numpy(t).to(DEV))
    ctx.set_buffer(lpc.BUF_YSUM, torch.zeros(P.d, device=DEV))
    sigma, tau1, tau2, alpha, inv4L = 0.6, 0.4, 0.5, 0.35, 0.125
    ctx.set_strong_convexity(sigma)
    theta = np.float32(np.float32(1.0) + np.float32(alpha) * np.float32(sigma))
    ysum, w = np.zeros(P.d, np.float32), np.float32(1.0)
    for k in (5, 6, 7):  # consecutive steps of one epoch: weights 1, theta, theta*theta
        ctx.alpc_double_sample_step(tau1, tau2, alpha, inv4L, k)
        ctx.sync_status()
        y, z, ysum = orc.alpc_step(P, k, tau1, tau2, alpha, inv4L, xs, mu, y, z, ysum, sigma=sigma, weight=w)
        w = np.float32(w * theta)
        if P.loss == orc.LEAST_SQUARES:
            assert _same(ctx.get_buffer(lpc.BUF_Y), y) and _same(ctx.get_buffer(lpc.BUF_Z), z)
            assert _same(ctx.get_buffer(lpc.BUF_YSUM), ysum)
        else:
            for buf, ref in ((lpc.BUF_Y, y), (lpc.BUF_Z, z), (lpc.BUF_YSUM, ysum)):
                got = ctx.get_buffer(buf).cpu().numpy()
                assert np.linalg.norm(got - ref) <= 1e-5 * np.linalg.norm(ref) + 1e-7
            # carry the library's state so that later steps are compared from the same bits
            y, z, ysum = (ctx.get_buffer(bf).cpu().numpy() for bf in (lpc.BUF_Y, lpc.BUF_Z, lpc.BUF_YSUM))
    ctx.close()


def test_epochs_follow_algorithm2_with_the_theorem_parameters():
    P, ctx = _setup(1024, 512, "least_squares", N=4, B=4, b=4, clip=(orc.CLIP_STD, 2.0), lam=1e-4, seed=21)
    m, S = 40, 3
    L = float((P.X.astype(np.float64) ** 2).sum(axis=1).max())
    sigma = np.float32(0.02 * L)
    tau1 = np.float32(np.sqrt(m * float(sigma) / (6 * L)))
    alpha = np.float32(1.0 / (6.0 * float(tau1) * L))
    inv4L = np.float32(1.0 / (4.0 * L))
    theta = np.float32(np.float32(1.0) + alpha * sigma)
    x0 = np.zeros(P.d, np.float32)
    ctx.set_iterate(torch.from_numpy(x0).to(DEV))
    ctx.set_strong_convexity(float(sigma))
    ctx.alpc_begin()
    snap, y, z = x0.copy(), x0.copy(), x0.copy()
    p0 = ctx.objective()
    assert p0 == pytest.approx(orc.objective(P.X, P.y, P.loss, x0, P.lambda_l1), rel=1e-9)
    for s in range(S):
        ctx.snapshot_full_grad()
        mu = ctx.get_buffer(lpc.BUF_MU).cpu().numpy()
        ctx.alpc_double_sample_steps(float(tau1), 0.5, float(alpha), float(inv4L), s * m, m)
        assert ctx.query(lpc.INFO_LOOP_LAUNCHES) == s + 1  # the weighted steps of an epoch run as one launch
        ctx.alpc_end_epoch(m)
        ysum, w, wsum = np.zeros(P.d, np.float32), np.float32(1.0), np.float32(0.0)
        for t in range(m):
            y, z, ysum = orc.alpc_step(P, s * m + t, tau1, 0.5, alpha, inv4L, snap, mu, y, z, ysum, sigma=sigma, weight=w)
            wsum, w = np.float32(wsum + w), np.float32(w * theta)
        snap = orc.weighted_snapshot(ysum, wsum)
        assert _same(ctx.get_iterate(), snap)
        assert _same(ctx.get_buffer(lpc.BUF_Y), y) and _same(ctx.get_buffer(lpc.BUF_Z), z)
    ctx.sync_status()
    pe = ctx.objective()
    assert pe < p0
    ref = orc.objective(P.X, P.y, P.loss, snap, P.lambda_l1) + orc.ridge_term(snap, sigma)
    assert pe == pytest.approx(ref, rel=1e-9)
    ctx.close()


@pytest.mark.parametrize("loss", ["least_squares", "logistic"])
def test_one_launch_loop_equals_single_steps_with_weights(loss):
    P, ctx = _setup(512, 1024, loss, N=4, B=4, b=4)
    ref = lpc.Context(ctx.X, ctx.y, P.loss, P.lambda_l1, P.N, P.B, P.b, P.clip_mode, P.clip_value, P.seed)
    x0 = (np.random.default_rng(5).standard_normal(P.d) * 0.1).astype(np.float32)
    tau1, tau2, alpha, inv4L, count = 0.4, 0.5, 0.3, 0.2, 11
    for cx in (ctx, ref):
        cx.set_strong_convexity(0.35)
        cx.set_iterate(torch.from_numpy(x0).to(DEV))
        cx.alpc_begin()
        cx.snapshot_full_grad()
        cx.alpc_double_sample_step(tau1, tau2, alpha, inv4L, 0)  # the loop then starts from the second weight
    ctx.alpc_double_sample_steps(tau1, tau2, alpha, inv4L, 1, count)
    for k in range(1, 1 + count):
        ref.alpc_double_sample_step(tau1, tau2, alpha, inv4L, k)
    for cx in (ctx, ref):
        cx.sync_status()
    assert ctx.query(lpc.INFO_LOOP_LAUNCHES) == 1 and ref.query(lpc.INFO_LOOP_LAUNCHES) == 0
    for w in (lpc.BUF_X, lpc.BUF_Y, lpc.BUF_Z, lpc.BUF_YSUM):
        assert _same(ctx.get_buffer(w), ref.get_buffer(w)), w
    for cx in (ctx, ref):
        cx.alpc_end_epoch(count + 1)
        cx.sync_status()
    assert _same(ctx.get_iterate(), ref.get_iterate())  # same sum of weights on both paths
    ctx.close()
    ref.close()


def test_sigma_zero_is_the_general_convex_path_and_bad_values_are_rejected():
    P, ctx = _setup(256, 128, "least_squares", N=4, B=2, b=4)
    ref = lpc.Context(ctx.X, ctx.y, P.loss, P.lambda_l1, P.N, P.B, P.b, P.clip_mode, P.clip_value, P.seed)
    ctx.set_strong_convexity(0.5)
    ctx.set_strong_convexity(0.0)  # back to h = lambda_l1*||.||_1
    x0 = (np.random.default_rng(5).standard_normal(P.d) * 0.1).astype(np.float32)
    for cx in (ctx, ref):
        cx.set_iterate(torch.from_numpy(x0).to(DEV))
        cx.alpc_begin()
        cx.snapshot_full_grad()
        cx.alpc_double_sample_steps(0.4, 0.5, 0.3, 0.2, 0, 7)
        cx.alpc_end_epoch(7)
        cx.sync_status()
    for w in (lpc.BUF_X, lpc.BUF_Y, lpc.BUF_Z):
        assert _same(ctx.get_buffer(w), ref.get_buffer(w))
    for bad in (-1.0, float("nan"), float("inf")):
        with pytest.raises(lpc.LpcError):
            ctx.set_strong_convexity(bad)
    ctx.close()
    ref.close()

"""GPU parity of the linear-model path (snapshot full gradient, fused inner step, ALPC step,
objective, trajectories) against the CPU oracle, through the C ABI.

Chain of custody for one step: from identical state (x, snapshot, mu, cached margins) the sampled
rows, the coefficients, u, the scales, the packed codes and the new iterate must all match bit for
bit for least squares.  For the logistic loss the coefficient goes through exp(), which is not
bit-portable between libraries, so the coefficients are compared to one ulp and everything
downstream is compared bitwise after the oracle is handed the GPU's coefficients when they differ.
"""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_1901_08924_b200 import lpc, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _bits(a):
    a = a.detach().cpu().numpy() if isinstance(a, torch.Tensor) else np.asarray(a)
    return a.view(np.uint32) if a.dtype == np.float32 else a


def _same(a, b):
    return (_bits(a) == _bits(b)).all()


def _setup(n, d, loss, N, B, b, clip=(orc.CLIP_STD, 2.5), lam=1e-3, seed=7, data_seed=0, col_scale=None):
    X, y, _ = synth.linear_problem(n, d, loss=loss, sparsity=0.2, noise=0.1, seed=data_seed, col_scale_range=col_scale)
    code = orc.LOGISTIC if loss == "logistic" else orc.LEAST_SQUARES
    P = orc.Problem(X.numpy(), y.numpy(), code, lam, N, B, b, clip[0], clip[1], seed)
    ctx = lpc.Context(X.to(DEV), y.to(DEV), code, lam, N, B, b, clip[0], clip[1], seed)
    return P, ctx


def _inject_snapshot(ctx, P, xs):
    """Oracle snapshot state copied into the context, so that both sides start from the same bits."""
    mu, margins, f = orc.full_grad(P.X, P.y, P.loss, xs)
    ctx.set_buffer(lpc.BUF_XTILDE, torch.from_numpy(xs).to(DEV))
    ctx.set_buffer(lpc.BUF_MU, torch.from_numpy(mu).to(DEV))
    ctx.set_buffer(lpc.BUF_MARGINS, torch.from_numpy(margins).to(DEV))
    return mu


@pytest.mark.parametrize("loss", ["least_squares", "logistic"])
# the last three: many tiles per CTA (the ring of stages wraps, both row warps get tiles), a ragged last tile on a deep
# ring, and a row wider than 8,192 columns (one row per tile, 16 values per compute thread)
@pytest.mark.parametrize("n,d", [(64, 8), (96, 64), (200, 1000), (120, 1500), (64, 3072), (1000, 4096), (48, 8192),
                                 (20000, 1024), (5004, 2048), (36, 12288)])
def test_snapshot_full_gradient(loss, n, d):
    P, ctx = _setup(n, d, loss, N=4, B=2, b=4)
    rng = np.random.default_rng(d)
    x = (rng.standard_normal(d) * 0.5).astype(np.float32)
    ctx.set_iterate(torch.from_numpy(x).to(DEV))
    mu_out = torch.empty(d, device=DEV)
    f = ctx.snapshot_full_grad(mu_out, want_f=True)
    ctx.sync_status()
    mu, margins, fr = orc.full_grad(P.X, P.y, P.loss, x)
    assert _same(ctx.get_buffer(lpc.BUF_MARGINS), margins)          # balanced-tree margins: bit-exact
    assert _same(ctx.get_buffer(lpc.BUF_XTILDE), x)
    g = mu_out.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(g - mu) <= 2e-6 * np.linalg.norm(mu) + 1e-12  # fp32 column sums vs fp64
    assert _same(ctx.get_buffer(lpc.BUF_MU), mu_out)
    assert abs(f - fr) <= 1e-12 + 1e-10 * abs(fr)
    Pv = ctx.objective()
    assert abs(Pv - orc.objective(P.X, P.y, P.loss, x, P.lambda_l1)) <= 1e-10 * max(1.0, abs(Pv))
    x2 = (rng.standard_normal(d)).astype(np.float32)
    assert abs(ctx.objective(torch.from_numpy(x2).to(DEV)) - orc.objective(P.X, P.y, P.loss, x2, P.lambda_l1)) <= 1e-9
    ctx.close()


def _check_step(P, ctx, k, eta, x, xs, mu):
    xn, t = orc.lpc_inner_step(P, k, eta, x, xs, mu, taps=True)
    ctx.set_iterate(torch.from_numpy(x).to(DEV))
    ctx.inner_step(eta, k)
    ctx.sync_status()
    idx = ctx.get_buffer(lpc.BUF_BATCH_IDX).cpu().numpy()[: P.N]
    coef = ctx.get_buffer(lpc.BUF_COEF).cpu().numpy()[: P.N]
    assert (idx == t["idx"]).all()
    if P.loss == orc.LEAST_SQUARES:
        assert _same(coef, t["coef"])
    else:
        assert np.abs(coef - t["coef"]).max() <= 1.2e-7 * max(1.0, np.abs(t["coef"]).max())
    if not _same(coef, t["coef"]):  # hand the GPU's coefficients to the oracle and redo the rest of the step
        W = max(P.W, 1)
        words = np.zeros((P.N, W), np.uint32)
        for i in range(P.N):
            t["u"][i] = orc.svrg_diff_from_coef(P.X, idx[i], coef[i])
            w, t["delta"][i], t["clipped"][i] = orc.quantize_pack(t["u"][i], P.b, P.clip_mode, P.clip_value, P.seed, i, k)
            words[i, : w.size] = w
        t["words"] = words[:, : P.W]
        xn, t["v"] = orc.unpack_average_prox(words, t["delta"], P.d, P.b, mu, x, eta, P.lambda_l1, want_v=True)
    assert _same(ctx.get_buffer(lpc.BUF_U), t["u"])
    assert _same(ctx.get_buffer(lpc.BUF_DELTA), t["delta"])
    codes = ctx.get_buffer(lpc.BUF_CODES).cpu().numpy().view(np.uint32)
    assert (codes[:, : P.W] == t["words"]).all() and (codes[:, P.W:] == 0).all()
    assert (ctx.get_buffer(lpc.BUF_CLIPPED).cpu().numpy().view(np.uint32) == t["clipped"]).all()
    assert _same(ctx.get_buffer(lpc.BUF_V), t["v"])
    assert _same(ctx.get_iterate(), xn)
    return xn


@pytest.mark.parametrize("loss", ["least_squares", "logistic"])
@pytest.mark.parametrize("cfg", [
    dict(n=64, d=8, N=4, B=1, b=2), dict(n=96, d=100, N=3, B=2, b=4), dict(n=256, d=1000, N=4, B=1, b=2),
    dict(n=256, d=1000, N=4, B=3, b=3), dict(n=128, d=2048, N=2, B=8, b=8), dict(n=128, d=4096, N=16, B=8, b=4),
    dict(n=64, d=8192, N=4, B=16, b=2), dict(n=64, d=5000, N=2, B=4, b=1), dict(n=64, d=3000, N=2, B=4, b=32),
    dict(n=64, d=12288, N=2, B=2, b=5), dict(n=32, d=16384, N=2, B=2, b=4),
    # minibatches larger than shared memory holds: the rows stream through the ring in batch order
    dict(n=2048, d=1000, N=2, B=101, b=4), dict(n=1024, d=4096, N=4, B=256, b=4), dict(n=512, d=8192, N=2, B=65, b=2),
    dict(n=4096, d=256, N=2, B=1024, b=8), dict(n=256, d=16384, N=2, B=70, b=3),
])
def test_inner_step_chain_of_custody(loss, cfg):
    c = dict(cfg)
    P, ctx = _setup(c.pop("n"), c.pop("d"), loss, **c)
    ctx.set_option(lpc.OPT_TAP_U, 1)
    rng = np.random.default_rng(1)
    xs = (rng.standard_normal(P.d) * 0.3).astype(np.float32)
    x = (xs + rng.standard_normal(P.d).astype(np.float32) * 0.05).astype(np.float32)
    mu = _inject_snapshot(ctx, P, xs)
    for k in (0, 1, 1000003):
        x = _check_step(P, ctx, k, 0.05, x, xs, mu)
    ctx.close()


@pytest.mark.parametrize("cs", [1, 2, 4, 8])
@pytest.mark.parametrize("clip", [(orc.CLIP_NONE, 1.0), (orc.CLIP_LAMBDA, 0.9), (orc.CLIP_STD, 2.0)])
def test_inner_step_cluster_sizes_and_clip_rules(cs, clip):
    P, ctx = _setup(128, 4096, "least_squares", N=4, B=4, b=4, clip=clip)
    ctx.set_option(lpc.OPT_TAP_U, 1)
    ctx.set_option(lpc.OPT_CLUSTER_SIZE, cs)
    rng = np.random.default_rng(cs)
    xs = (rng.standard_normal(P.d) * 0.3).astype(np.float32)
    x = (xs + rng.standard_normal(P.d).astype(np.float32) * 0.05).astype(np.float32)
    mu = _inject_snapshot(ctx, P, xs)
    _check_step(P, ctx, 5, 0.05, x, xs, mu)
    ctx.close()


def test_global_sampling_option():
    P, ctx = _setup(128, 256, "least_squares", N=4, B=4, b=4)
    P.partition_local = False
    ctx.set_option(lpc.OPT_SAMPLE_GLOBAL, 1)
    ctx.set_option(lpc.OPT_TAP_U, 1)
    rng = np.random.default_rng(2)
    xs = rng.standard_normal(P.d).astype(np.float32)
    x = (xs + 0.1 * rng.standard_normal(P.d)).astype(np.float32)
    mu = _inject_snapshot(ctx, P, xs)
    _check_step(P, ctx, 3, 0.1, x, xs, mu)
    ctx.close()


@pytest.mark.parametrize("loss", ["least_squares", "logistic"])
def test_first_step_of_epoch_sends_zeros(loss):
    # x = snapshot: u = 0 exactly (cached margins are bit-identical to recomputed ones), v = mu
    P, ctx = _setup(200, 1000, loss, N=4, B=2, b=2)
    ctx.set_option(lpc.OPT_TAP_U, 1)
    x = (np.random.default_rng(3).standard_normal(P.d) * 0.2).astype(np.float32)
    ctx.set_iterate(torch.from_numpy(x).to(DEV))
    ctx.snapshot_full_grad()
    ctx.inner_step(0.1, 0)
    ctx.sync_status()
    assert (ctx.get_buffer(lpc.BUF_U) == 0).all() and (ctx.get_buffer(lpc.BUF_DELTA) == 0).all()
    assert _same(ctx.get_buffer(lpc.BUF_V), ctx.get_buffer(lpc.BUF_MU))
    codes = ctx.get_buffer(lpc.BUF_CODES).cpu().numpy().view(np.uint32)
    for i in range(P.N):
        assert (orc.unpack(codes[i], P.d, P.b) == 2).all()
    ctx.close()


def _oracle_epochs(P, x0, S, m, eta, mu_of=None):
    snap = x0.copy()
    traj = []
    for s in range(S):
        mu = mu_of(s, snap) if mu_of else orc.full_grad(P.X, P.y, P.loss, snap)[0]
        x = snap.copy()
        for t in range(m):
            x = orc.lpc_inner_step(P, s * m + t, eta, x, snap, mu)
        snap = x
        traj.append(orc.objective(P.X, P.y, P.loss, snap, P.lambda_l1))
    return snap, traj


def test_trajectory_tiny_config_full():
    # the smallest workload in full: logistic + L1, 4000 x 1000, 4 workers, B=1, b=2, clip 2.5 std, eta 0.1,
    # one epoch of 1000 steps
    P, ctx = _setup(4000, 1000, "logistic", N=4, B=1, b=2, clip=(orc.CLIP_STD, 2.5), lam=1e-4, seed=0)
    x0 = np.zeros(P.d, np.float32)
    ctx.set_iterate(torch.from_numpy(x0).to(DEV))
    p_start = ctx.objective()
    ctx.snapshot_full_grad()
    ctx.inner_steps(0.1, 0, 1000)
    ctx.sync_status()
    p_gpu = ctx.objective()
    snap, traj = _oracle_epochs(P, x0, 1, 1000, 0.1)
    assert abs(p_gpu - traj[-1]) <= 1e-4 * abs(traj[-1])
    assert p_gpu < p_start
    xg = ctx.get_iterate().cpu().numpy()
    assert np.linalg.norm(xg - snap) <= 1e-4 * np.linalg.norm(snap)
    s1, s2 = ctx.comm_bits()
    assert s1 == 32 * 1000 * 4 * 3 and s2 == 1000 * orc.broadcast_bits(1000, 2, 4)
    ctx.close()


def test_trajectory_least_squares_bitwise_within_epochs():
    # least squares has no transcendental on the path: with the snapshot gradient shared, whole epochs
    # (graph replay included) reproduce the oracle bit for bit
    P, ctx = _setup(1024, 512, "least_squares", N=4, B=2, b=4, clip=(orc.CLIP_STD, 3.0), lam=1e-4, seed=11)
    m, S, eta = 160, 2, 0.05
    x0 = np.zeros(P.d, np.float32)
    ctx.set_iterate(torch.from_numpy(x0).to(DEV))
    mus = []

    def mu_of(s, snap):
        return mus[s]

    snap_gpu = []
    for s in range(S):
        ctx.snapshot_full_grad()
        mus.append(ctx.get_buffer(lpc.BUF_MU).cpu().numpy())
        ctx.inner_steps(eta, s * m, m)
        snap_gpu.append(ctx.get_iterate().cpu().numpy())
    ctx.sync_status()
    snap, traj = _oracle_epochs(P, x0, S, m, eta, mu_of)
    assert _same(snap_gpu[-1], snap)
    assert abs(ctx.objective() - traj[-1]) <= 1e-10 * abs(traj[-1])
    assert traj[-1] < orc.objective(P.X, P.y, P.loss, x0, P.lambda_l1)
    ctx.close()


def test_graph_replay_equals_plain_launches_and_resume():
    P, ctx = _setup(512, 1024, "logistic", N=4, B=2, b=4, seed=5)
    x0 = (np.random.default_rng(0).standard_normal(P.d) * 0.1).astype(np.float32)
    ctx.set_iterate(torch.from_numpy(x0).to(DEV))
    ctx.snapshot_full_grad()
    ctx.inner_step(0.1, 0)  # move away from the snapshot
    state = [ctx.get_buffer(w) for w in (lpc.BUF_X, lpc.BUF_XTILDE, lpc.BUF_MU, lpc.BUF_MARGINS)]
    ctx.inner_steps(0.1, 1, 300)  # two graph replays + 44 plain steps
    a = ctx.get_iterate()
    ctx.sync_status()
    # a fresh context resumed from the saved state, stepping one launch at a time
    ctx2 = lpc.Context(ctx.X, ctx.y, P.loss, P.lambda_l1, P.N, P.B, P.b, P.clip_mode, P.clip_value, P.seed)
    for w, t in zip((lpc.BUF_X, lpc.BUF_XTILDE, lpc.BUF_MU, lpc.BUF_MARGINS), state):
        ctx2.set_buffer(w, t)
    ctx2.set_option(lpc.OPT_USE_GRAPH, 0)
    ctx2.inner_steps(0.1, 1, 150)
    for k in range(151, 301):
        ctx2.inner_step(0.1, k)
    ctx2.sync_status()
    assert _same(a, ctx2.get_iterate())
    assert ctx.comm_bits()[1] == 301 * orc.broadcast_bits(P.d, P.b, P.N)
    ctx.close()
    ctx2.close()


@pytest.mark.parametrize("cfg", [
    dict(n=64, d=8, N=4, B=1, b=2), dict(n=256, d=1000, N=4, B=1, b=2), dict(n=256, d=1000, N=4, B=3, b=3),
    dict(n=128, d=4096, N=16, B=8, b=4), dict(n=64, d=8192, N=4, B=16, b=8), dict(n=64, d=5000, N=2, B=4, b=1),
    dict(n=64, d=3000, N=2, B=4, b=32), dict(n=64, d=12288, N=2, B=2, b=5), dict(n=256, d=2048, N=32, B=2, b=4),
])
@pytest.mark.parametrize("mode", ["persistent", "graph"])
def test_multi_step_paths_equal_single_launches(cfg, mode):
    # the one-launch persistent loop and the graph replay must give the bits of one-step-at-a-time launches
    c = dict(cfg)
    P, ctx = _setup(c.pop("n"), c.pop("d"), "logistic", **c)
    ref = lpc.Context(ctx.X, ctx.y, P.loss, P.lambda_l1, P.N, P.B, P.b, P.clip_mode, P.clip_value, P.seed)
    x0 = (np.random.default_rng(9).standard_normal(P.d) * 0.1).astype(np.float32)
    count = 131 if mode == "graph" else 7
    for cx in (ctx, ref):
        cx.set_option(lpc.OPT_TAP_U, 1)
        cx.set_iterate(torch.from_numpy(x0).to(DEV))
        cx.snapshot_full_grad()
        cx.inner_step(0.05, 0)
    if mode == "graph":
        ctx.set_option(lpc.OPT_PERSISTENT, 0)
    ctx.inner_steps(0.05, 1, count)
    for k in range(1, 1 + count):
        ref.inner_step(0.05, k)
    ctx.sync_status()
    ref.sync_status()
    for w in (lpc.BUF_X, lpc.BUF_CODES, lpc.BUF_DELTA, lpc.BUF_CLIPPED, lpc.BUF_BATCH_IDX, lpc.BUF_COEF, lpc.BUF_U, lpc.BUF_V):
        got, want = ctx.get_buffer(w), ref.get_buffer(w)
        if w in (lpc.BUF_BATCH_IDX, lpc.BUF_COEF):
            got, want = got[: P.N], want[: P.N]
        assert _same(got, want), w
    assert ctx.comm_bits() == ref.comm_bits()
    assert ctx.query(lpc.INFO_LOOP_LAUNCHES) == (1 if mode == "persistent" else 0)  # the intended path really ran
    assert ref.query(lpc.INFO_LOOP_LAUNCHES) == 0
    ctx.close()
    ref.close()


@pytest.mark.parametrize("loss", ["least_squares", "logistic"])
@pytest.mark.parametrize("cfg", [dict(n=128, d=1000, N=4, B=2, b=2), dict(n=128, d=8192, N=4, B=16, b=8),
                                 dict(n=64, d=4096, N=2, B=4, b=4), dict(n=1024, d=2048, N=2, B=130, b=4)])
def test_alpc_step_chain_of_custody(loss, cfg):
    c = dict(cfg)
    P, ctx = _setup(c.pop("n"), c.pop("d"), loss, lam=1e-3, **c)
    ctx.set_option(lpc.OPT_TAP_U, 1)
    rng = np.random.default_rng(4)
    xs, y, z = ((rng.standard_normal(P.d) * 0.2).astype(np.float32) for _ in range(3))
    ysum = np.abs(rng.standard_normal(P.d)).astype(np.float32)
    mu = _inject_snapshot(ctx, P, xs)
    tau1, tau2, alpha, inv4L = 0.4, 0.5, 0.35, 0.125
    for k in (2, 9):
        for w, t in ((lpc.BUF_Y, y), (lpc.BUF_Z, z), (lpc.BUF_YSUM, ysum)):
            ctx.set_buffer(w, torch.from_numpy(t).to(DEV))
        ctx.alpc_double_sample_step(tau1, tau2, alpha, inv4L, k)
        ctx.sync_status()
        yn, zn, sn, t = orc.alpc_step(P, k, tau1, tau2, alpha, inv4L, xs, mu, y, z, ysum, taps=True)
        assert _same(ctx.get_buffer(lpc.BUF_X), t["x"])  # the coupled point
        idx = ctx.get_buffer(lpc.BUF_BATCH_IDX).cpu().numpy()
        assert (idx[P.N] == orc.sample_batch(P.seed, orc.TAG_BATCH_J, 0, k, P.B, 0, P.n)).all()  # one shared batch J
        if P.loss == orc.LEAST_SQUARES:
            assert _same(ctx.get_buffer(lpc.BUF_VHAT), t["vhat"])
            assert _same(ctx.get_buffer(lpc.BUF_V), t["v"])
            assert _same(ctx.get_buffer(lpc.BUF_Y), yn) and _same(ctx.get_buffer(lpc.BUF_Z), zn)
            assert _same(ctx.get_buffer(lpc.BUF_YSUM), sn)
        else:
            for w, ref in ((lpc.BUF_VHAT, t["vhat"]), (lpc.BUF_Y, yn), (lpc.BUF_Z, zn), (lpc.BUF_YSUM, sn)):
                got = ctx.get_buffer(w).cpu().numpy()
                assert np.linalg.norm(got - ref) <= 1e-5 * np.linalg.norm(ref) + 1e-7
        y, z, ysum = yn, zn, sn
    ctx.close()


def test_alpc_epochs_follow_algorithm3():
    # tau_1 = 2/(s+4), alpha = 1/(6 L tau_1), tau_2 = 1/2, snapshot = mean of the epoch's y iterates
    P, ctx = _setup(1024, 512, "least_squares", N=4, B=4, b=4, clip=(orc.CLIP_STD, 2.0), lam=1e-4, seed=21)
    m, S = 130, 3
    L = float((P.X.astype(np.float64) ** 2).sum(axis=1).max())
    x0 = np.zeros(P.d, np.float32)
    ctx.set_iterate(torch.from_numpy(x0).to(DEV))
    ctx.alpc_begin()
    snap, y, z = x0.copy(), x0.copy(), x0.copy()
    p0 = ctx.objective()
    for s in range(S):
        tau1, alpha = orc.alpc3_epoch_params(s, L)  # the oracle's outer rule (Algorithm 3 step 3)
        inv4L = np.float32(1.0 / (4.0 * L))
        ctx.snapshot_full_grad()
        mu = ctx.get_buffer(lpc.BUF_MU).cpu().numpy()
        ctx.alpc_double_sample_steps(float(tau1), 0.5, float(alpha), float(inv4L), s * m, m)
        ctx.alpc_end_epoch(m)
        y, z, snap = orc.alpc3_epoch(P, s, m, L, 0.5, snap, mu, y, z)
        assert _same(ctx.get_iterate(), snap)
        assert _same(ctx.get_buffer(lpc.BUF_Y), y) and _same(ctx.get_buffer(lpc.BUF_Z), z)
    ctx.sync_status()
    assert ctx.objective() < p0
    ctx.close()


def test_host_buffer_job_matches_context_path():
    P, ctx = _setup(512, 256, "least_squares", N=4, B=2, b=4, seed=3)
    S, m, eta = 2, 140, 0.05
    x0 = torch.zeros(P.d)
    xh, Ph, bits = lpc.svrg_run_host(torch.from_numpy(P.X), torch.from_numpy(P.y), P.loss, P.lambda_l1, P.N, P.B, P.b,
                                     P.clip_mode, P.clip_value, P.seed, S, m, eta, x0)
    ctx.set_iterate(x0.to(DEV))
    for s in range(S):
        ctx.snapshot_full_grad()
        ctx.inner_steps(eta, s * m, m)
    ctx.sync_status()
    assert _same(ctx.get_iterate(), xh)
    assert abs(ctx.objective() - Ph) <= 1e-12 * abs(Ph)
    assert bits == ctx.comm_bits()[1]
    ctx.close()


def test_unsupported_and_invalid_calls_are_refused():
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, 2, 1, 4, lpc.CLIP_NONE, 1.0, 0)
    assert lpc.lib().lpc_inner_step(q._h, 0.1, 0) == lpc.ERR_UNSUPPORTED
    assert lpc.lib().lpc_snapshot_full_grad(q._h, None, None) == lpc.ERR_UNSUPPORTED
    assert lpc.lib().lpc_quantize_pack(q._h, None, None, 10, 10, None, 1, 0, None, None, None) == lpc.ERR_INVALID_ARG
    q.close()


@pytest.mark.parametrize("cfg", [
    dict(n=256, d=1000, N=4, B=2, b=2), dict(n=128, d=4096, N=16, B=8, b=4), dict(n=64, d=8192, N=4, B=16, b=8),
    dict(n=64, d=5000, N=2, B=4, b=1), dict(n=64, d=3000, N=2, B=4, b=32), dict(n=96, d=12288, N=3, B=2, b=5),
    dict(n=128, d=8192, N=32, B=16, b=2),
])
@pytest.mark.parametrize("loss", ["least_squares", "logistic"])
def test_alpc_one_launch_loop_equals_single_steps(cfg, loss):
    # Algorithm 2's steps run as one persistent launch must give the bits of one-step-at-a-time launches
    c = dict(cfg)
    P, ctx = _setup(c.pop("n"), c.pop("d"), loss, **c)
    ref = lpc.Context(ctx.X, ctx.y, P.loss, P.lambda_l1, P.N, P.B, P.b, P.clip_mode, P.clip_value, P.seed)
    x0 = (np.random.default_rng(5).standard_normal(P.d) * 0.1).astype(np.float32)
    tau1, tau2, alpha, inv4L, count = 0.4, 0.5, 0.3, 0.2, 9
    for cx in (ctx, ref):
        cx.set_option(lpc.OPT_TAP_U, 1)
        cx.set_iterate(torch.from_numpy(x0).to(DEV))
        cx.alpc_begin()
        cx.snapshot_full_grad()
        cx.alpc_double_sample_step(tau1, tau2, alpha, inv4L, 0)
    ctx.alpc_double_sample_steps(tau1, tau2, alpha, inv4L, 1, count)
    for k in range(1, 1 + count):
        ref.alpc_double_sample_step(tau1, tau2, alpha, inv4L, k)
    ctx.sync_status()
    ref.sync_status()
    assert ctx.query(lpc.INFO_LOOP_LAUNCHES) == 1 and ref.query(lpc.INFO_LOOP_LAUNCHES) == 0
    for w in (lpc.BUF_X, lpc.BUF_Y, lpc.BUF_Z, lpc.BUF_YSUM, lpc.BUF_VHAT, lpc.BUF_V, lpc.BUF_CODES, lpc.BUF_DELTA,
              lpc.BUF_CLIPPED, lpc.BUF_BATCH_IDX, lpc.BUF_COEF, lpc.BUF_U):
        assert _same(ctx.get_buffer(w), ref.get_buffer(w)), w
    assert ctx.comm_bits() == ref.comm_bits()
    ctx.close()
    ref.close()


def test_average_divisor_option_leaves_the_training_loops_alone():
    # LPC_OPT_AVERAGE_DIVISOR belongs to lpc_unpack_average_prox; single steps, graph replay and the one-launch loop all
    # keep averaging over the N workers (Eq. 3) and agree bit for bit
    P, ctx = _setup(512, 256, "least_squares", N=4, B=2, b=4, seed=9)
    count, eta = 130, 0.05
    results = []
    for mode in ("single", "graph", "loop"):
        c = lpc.Context(ctx.X, ctx.y, P.loss, P.lambda_l1, P.N, P.B, P.b, P.clip_mode, P.clip_value, P.seed)
        c.set_option(lpc.OPT_AVERAGE_DIVISOR, 3)
        c.snapshot_full_grad()
        if mode == "single":
            for k in range(count):
                c.inner_step(eta, k)
        else:
            c.set_option(lpc.OPT_PERSISTENT, 1 if mode == "loop" else 0)
            c.inner_steps(eta, 0, count)
        c.sync_status()
        assert c.query(lpc.INFO_LOOP_LAUNCHES) == (1 if mode == "loop" else 0)
        results.append(c.get_iterate().cpu().numpy())
        c.close()
    assert _same(results[0], results[1]) and _same(results[0], results[2])
    # and they are the oracle's iterates (which know no such option)
    ctx.snapshot_full_grad()
    mu = ctx.get_buffer(lpc.BUF_MU).cpu().numpy()
    x0 = np.zeros(P.d, np.float32)
    xr = x0
    for k in range(count):
        xr = orc.lpc_inner_step(P, k, eta, xr, x0, mu)
    assert _same(results[0], xr)
    ctx.close()


def test_loop_without_the_cooperative_attribute_gives_the_same_bits():
    # the profiling configuration of the one-launch loop: a plain cluster launch of the same grid
    P, ctx = _setup(512, 1000, "least_squares", N=4, B=2, b=4, seed=13)
    ref = lpc.Context(ctx.X, ctx.y, P.loss, P.lambda_l1, P.N, P.B, P.b, P.clip_mode, P.clip_value, P.seed)
    ctx.set_option(lpc.OPT_LOOP_COOPERATIVE, 0)
    for c in (ctx, ref):
        c.snapshot_full_grad()
        c.inner_steps(0.05, 0, 40)
        c.sync_status()
        assert c.query(lpc.INFO_LOOP_LAUNCHES) == 1
    assert _same(ctx.get_iterate(), ref.get_iterate())
    assert _same(ctx.get_buffer(lpc.BUF_CODES), ref.get_buffer(lpc.BUF_CODES))
    ctx.close()
    ref.close()

"""Parity at the full sizes of the workloads, in the launch configuration the benchmark times.

Where the oracle can do the whole job in seconds it does (least-squares epoch, layer-wise DNN
aggregation); elsewhere it checks what it can compute one by one: scales from full passes, codes and
updated coordinates in sampled windows, sampled margins.
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


def test_least_squares_workload_full_epoch_bitwise():
    # 131,072 x 4,096, N = 16, B = 8, b = 4, clip 3 std, m = 1,024: one whole epoch through the one-launch loop
    n, d, N, B, b, m = 131072, 4096, 16, 8, 4, 1024
    X, y, _ = synth.linear_problem(n, d, loss="least_squares", sparsity=0.05, noise=0.01, seed=0, device=DEV)
    eta = 1.0 / (6.0 * float((X.double() ** 2).sum(dim=1).max().item()))
    ctx = lpc.Context(X, y, lpc.LEAST_SQUARES, 1e-4, N, B, b, lpc.CLIP_STD, 3.0, 0)
    Xh, yh = X.cpu().numpy(), y.cpu().numpy()
    P = orc.Problem(Xh, yh, orc.LEAST_SQUARES, 1e-4, N, B, b, orc.CLIP_STD, 3.0, 0)
    x0 = (np.random.default_rng(0).standard_normal(d) * 0.01).astype(np.float32)
    ctx.set_iterate(torch.from_numpy(x0).to(DEV))
    f = ctx.snapshot_full_grad(want_f=True)
    mu_g = ctx.get_buffer(lpc.BUF_MU).cpu().numpy()
    mu, margins, fr = orc.full_grad(Xh, yh, P.loss, x0)
    assert (_bits(ctx.get_buffer(lpc.BUF_MARGINS)) == _bits(margins)).all()
    assert np.linalg.norm(mu_g - mu) <= 2e-6 * np.linalg.norm(mu)
    assert abs(f - fr) <= 1e-10 * abs(fr)
    ctx.inner_steps(eta, 0, m)
    ctx.sync_status()
    assert ctx.query(lpc.INFO_LOOP_LAUNCHES) == 1
    x = x0.copy()
    for k in range(m):
        x = orc.lpc_inner_step(P, k, eta, x, x0, mu_g)
    xg = ctx.get_iterate().cpu().numpy()
    assert (_bits(xg) == _bits(x)).all()
    pg = ctx.objective()
    assert abs(pg - orc.objective(Xh, yh, P.loss, x, P.lambda_l1)) <= 1e-10 * abs(pg)
    assert ctx.comm_bits() == (32 * d * N * (N - 1), m * orc.broadcast_bits(d, b, N))
    ctx.close()


@pytest.mark.parametrize("b", [2, 8])
def test_alpc_workload_full_size_steps(b):
    # 262,144 x 8,192 logistic with ill-conditioned columns, N = 32, B = 16, clip 2 std (ALPC, double sampling)
    n, d, N, B = 262144, 8192, 32, 16
    X, y, _ = synth.linear_problem(n, d, loss="logistic", sparsity=0.02, noise=0.1, seed=1, col_scale_range=(0.1, 10.0),
                                   device=DEV)
    ctx = lpc.Context(X, y, lpc.LOGISTIC, 1e-5, N, B, b, lpc.CLIP_STD, 2.0, 5)
    Xh, yh = X.cpu().numpy(), y.cpu().numpy()
    P = orc.Problem(Xh, yh, orc.LOGISTIC, 1e-5, N, B, b, orc.CLIP_STD, 2.0, 5)
    L = 0.25 * float((X * X).sum(dim=1).max().item())
    x0 = np.zeros(d, np.float32)
    ctx.set_iterate(torch.from_numpy(x0).to(DEV))
    ctx.alpc_begin()
    ctx.snapshot_full_grad()
    ctx.sync_status()
    rows = np.random.default_rng(2).integers(0, n, 64)
    mg = ctx.get_buffer(lpc.BUF_MARGINS).cpu().numpy()
    for a in rows:  # sampled margins, bit for bit
        assert _bits(mg[a:a + 1])[0] == _bits(np.array([orc.margin(Xh[a], x0)], np.float32))[0]
    mu = ctx.get_buffer(lpc.BUF_MU).cpu().numpy()
    tau1, alpha, inv4L = np.float32(0.5), np.float32(1.0 / (6.0 * L * 0.5)), np.float32(1.0 / (4.0 * L))
    yv, zv, ys = x0.copy(), x0.copy(), x0.copy()
    steps = 6
    for k in range(steps):
        ctx.alpc_double_sample_step(float(tau1), 0.5, float(alpha), float(inv4L), k)
        yv, zv, ys, t = orc.alpc_step(P, k, tau1, 0.5, alpha, inv4L, x0, mu, yv, zv, ys, taps=True)
        ctx.sync_status()
        idx = ctx.get_buffer(lpc.BUF_BATCH_IDX).cpu().numpy()
        assert (idx[N] == orc.sample_batch(P.seed, orc.TAG_BATCH_J, 0, k, B, 0, n)).all()
        for w, ref in ((lpc.BUF_Y, yv), (lpc.BUF_Z, zv), (lpc.BUF_YSUM, ys), (lpc.BUF_VHAT, t["vhat"])):
            got = ctx.get_buffer(w).cpu().numpy()
            assert np.linalg.norm(got - ref) <= 1e-5 * np.linalg.norm(ref) + 1e-9, (k, w)
        # continue from the GPU's state so that one-ulp differences in exp() do not accumulate in the comparison
        yv, zv, ys = (ctx.get_buffer(w).cpu().numpy() for w in (lpc.BUF_Y, lpc.BUF_Z, lpc.BUF_YSUM))
    ctx.close()


def test_sweep_full_length_sampled_windows():
    # 8 worker vectors of 2^26 heavy-tailed values, b = 4, clip 2 std: scales from full passes, codes and updated
    # coordinates in sampled windows
    N, length, b, seed, k = 8, 1 << 26, 4, 11, 3
    U = synth.gradient_vectors(N, length, "student_t3", seed=4, device=DEV)
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, N, 1, b, lpc.CLIP_STD, 2.0, seed)
    codes, delta, clipped = q.quantize_pack(U, k)
    x = torch.zeros(length, device=DEV)
    q.unpack_average_prox(codes, delta, length, x, 1.0, 1e-3)
    q.sync_status()
    Uh = U.cpu().numpy()
    sc = [orc.scale(Uh[i], b, orc.CLIP_STD, 2.0) for i in range(N)]
    dl = delta.cpu().numpy()[:, 0]
    assert (_bits(dl) == _bits(np.array([s["delta"] for s in sc], np.float32))).all()
    lower = [-(np.float32(s["T"]) + np.float32(s["delta"])) for s in sc]
    want_clip = [int(((Uh[i] > sc[i]["T"]) | (Uh[i] < lower[i])).sum()) for i in range(N)]
    assert clipped.cpu().numpy()[:, 0].tolist() == want_clip
    W = 2048
    starts = [0, 8192 * 1000 + 8, (1 << 25) - 1024, length - W]
    ch = codes.cpu().numpy().view(np.uint32)
    xh = x.cpu().numpy()
    for s0 in starts:
        words = np.zeros((N, W * b // 32), np.uint32)
        for i in range(N):
            c = np.array([orc.quantize_coord(Uh[i, j], sc[i]["rdelta"], b, orc.rounding_bits(seed, i, k, 0, j)) + 8
                          for j in range(s0, s0 + W)], np.uint32)
            words[i] = orc.pack(c, b)
        assert (ch[:, s0 * b // 32:(s0 + W) * b // 32] == words).all(), s0
        ref = orc.unpack_average_prox(words, dl, W, b, None, np.zeros(W, np.float32), 1.0, 1e-3)
        assert (_bits(xh[s0:s0 + W]) == _bits(ref)).all(), s0
    q.close()


def test_dnn_shaped_aggregation_full_bitwise():
    # 62 tensors, 11,689,512 parameters, N = 16, b = 4, per-tensor clip 2.5 std; u = current - snapshot gradient
    N, b, seed, k = 16, 4, 2, 9
    cur, snap, mu, offs = synth.dnn_gradients(N, seed=3, device=DEV)
    total, nseg = offs[-1], len(offs) - 1
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, N, 1, b, lpc.CLIP_STD, 2.5, seed)
    codes, delta, clipped = q.quantize_pack(cur, k, U_sub=snap, seg_offsets=offs)
    x = torch.zeros(total, device=DEV)
    q.unpack_average_prox(codes, delta, total, x, -1.0, 0.0, mu=mu, seg_offsets=offs)  # x = v
    q.sync_status()
    u = (cur - snap).cpu().numpy()
    woff, stride = lpc.packed_layout(total, b, offs)
    ch, dh, clh, xh, muh = codes.cpu().numpy().view(np.uint32), delta.cpu().numpy(), clipped.cpu().numpy(), x.cpu().numpy(), mu.cpu().numpy()
    base = 0
    for s in range(nseg):
        ln = offs[s + 1] - offs[s]
        W = orc.packed_words(ln, b)
        words = np.zeros((N, W), np.uint32)
        for i in range(N):
            words[i], dli, cli = orc.quantize_pack(u[i, offs[s]:offs[s + 1]], b, orc.CLIP_STD, 2.5, seed, i, k, base)
            assert _bits(np.array([dli], np.float32))[0] == _bits(dh[i, s:s + 1])[0] and cli == clh[i, s]
        assert (ch[:, woff[s]:woff[s] + W] == words).all(), s
        ref = orc.unpack_average_prox(words, dh[:, s], ln, b, muh[offs[s]:offs[s + 1]], np.zeros(ln, np.float32), -1.0, 0.0)
        assert (_bits(xh[offs[s]:offs[s + 1]]) == _bits(ref)).all(), s
        base += (ln + 7) // 8
    q.close()


def test_server_schemes_and_entropy_count_full_length():
    # 8 worker vectors of 2^26 Gaussian values of different magnitudes, b = 4, clip 2 std, in the launch shapes the
    # benchmark times: unified scale from full passes, codes / server streams / updated coordinates in sampled windows;
    # worker 0's own message (own scale) and its histogram in full
    N, length, b, seed, k = 8, 1 << 26, 4, 13, 5
    U = synth.gradient_vectors(N, length, "gauss", seed=6, device=DEV)
    U *= torch.linspace(0.5, 1.5, N, device=DEV).unsqueeze(1)
    Uh = U.cpu().numpy()
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, N, 1, b, lpc.CLIP_STD, 2.0, seed)
    # -- own scales: worker 0 in full against the oracle, then its histogram and the two counts
    codes, delta, _ = q.quantize_pack(U, k)
    hist, ent, huf = q.message_entropy(codes, length)
    q.sync_status()
    w0, d0, _ = orc.quantize_pack(Uh[0], b, orc.CLIP_STD, 2.0, seed=seed, worker=0, k=k)
    ch = codes.cpu().numpy().view(np.uint32)
    assert (ch[0, : w0.size] == w0).all() and _bits(delta.cpu().numpy()[0, :1])[0] == _bits(np.array([d0], np.float32))[0]
    h0 = orc.code_histogram(w0, length, b)
    hg = hist.cpu().numpy()
    assert (hg[0, 0].astype(np.uint64) == h0).all()
    assert (hg.sum(axis=2) == length).all()
    assert huf[0, 0] == orc.huffman_bits(h0) and ent[0, 0] == pytest.approx(orc.entropy_bits(h0), rel=1e-12)
    # -- unified scale
    q.set_option(lpc.OPT_SHARED_SCALE, 1)
    codes, delta, clipped = q.quantize_pack(U, k)
    srv_b, bo = q.server_reduce(codes, length, lpc.SCHEME_SERVER_SUM, k)
    srv_c, _ = q.server_reduce(codes, length, lpc.SCHEME_SERVER_REQUANTIZE, k)
    xb, xc = torch.zeros(length, device=DEV), torch.zeros(length, device=DEV)
    wb = lpc.Context(None, None, lpc.LOGISTIC, 0.0, 1, 1, bo, lpc.CLIP_NONE, 1.0, seed)
    wb.set_option(lpc.OPT_AVERAGE_DIVISOR, N)
    wc = lpc.Context(None, None, lpc.LOGISTIC, 0.0, 1, 1, b, lpc.CLIP_NONE, 1.0, seed)
    d1 = delta[:1].contiguous()
    wb.unpack_average_prox(srv_b, d1, length, xb, 1.0, 1e-3)
    wc.unpack_average_prox(srv_c, d1, length, xc, 1.0, 1e-3)
    for c in (q, wb, wc):
        c.sync_status()
    sc = [orc.scale(Uh[i], b, orc.CLIP_STD, 2.0) for i in range(N)]
    best = max(sc, key=lambda s: s["T"])
    dl = delta.cpu().numpy()
    assert (_bits(dl) == _bits(np.float32(best["delta"]))).all()
    lower = -(np.float32(best["T"]) + np.float32(best["delta"]))
    want_clip = [int(((Uh[i] > best["T"]) | (Uh[i] < lower)).sum()) for i in range(N)]
    assert clipped.cpu().numpy()[:, 0].tolist() == want_clip
    W = 2048
    ch = codes.cpu().numpy().view(np.uint32)
    sb, sc_ = srv_b.cpu().numpy().view(np.uint32).ravel(), srv_c.cpu().numpy().view(np.uint32).ravel()
    xbh, xch = xb.cpu().numpy(), xc.cpu().numpy()
    for s0 in [0, 8192 * 1000 + 32, (1 << 25) - 1024, length - W]:
        words = np.zeros((N, W * b // 32), np.uint32)
        for i in range(N):
            c = np.array([orc.quantize_coord(Uh[i, j], best["rdelta"], b, orc.rounding_bits(seed, i, k, 0, j)) + 8
                          for j in range(s0, s0 + W)], np.uint32)
            words[i] = orc.pack(c, b)
        assert (ch[:, s0 * b // 32:(s0 + W) * b // 32] == words).all(), s0
        ref_b = orc.server_reduce(words, W, b, False)
        ref_c = orc.server_reduce(words, W, b, True, seed=seed, k=k, block_base=s0 // 8)
        assert (sb[s0 * bo // 32:(s0 + W) * bo // 32] == ref_b).all(), s0
        assert (sc_[s0 * b // 32:(s0 + W) * b // 32] == ref_c).all(), s0
        zero = np.zeros(W, np.float32)
        assert (_bits(xbh[s0:s0 + W]) == _bits(orc.unpack_scaled_prox(ref_b, best["delta"], W, bo, N, None, zero, 1.0, 1e-3))).all()
        assert (_bits(xch[s0:s0 + W]) == _bits(orc.unpack_scaled_prox(ref_c, best["delta"], W, b, 1, None, zero, 1.0, 1e-3))).all()
    for c in (q, wb, wc):
        c.close()


@pytest.mark.parametrize("B,b", [(256, 2), (256, 8), (1024, 2)])
def test_fused_worker_kernel_large_minibatches_bench_shape(B, b):
    # The streaming worker kernel in the launch shape the benchmark times on it: d = 8,192, N = 32 workers, logistic
    # loss on ill-conditioned columns, clip 2 std, clusters of 4 CTAs, a ring of 6 (B = 256) or 5 (B = 1,024) stages.
    # The matrix has fewer rows than the benchmark's (the launch shape does not depend on n; the oracle pays per row).
    n, d, N = 8192, 8192, 32
    X, y, _ = synth.linear_problem(n, d, loss="logistic", sparsity=0.02, noise=0.1, seed=1, col_scale_range=(0.1, 10.0))
    Xh, yh = X.numpy(), y.numpy()
    P = orc.Problem(Xh, yh, orc.LOGISTIC, 1e-5, N, B, b, orc.CLIP_STD, 2.0, 3)
    ctx = lpc.Context(X.to(DEV), y.to(DEV), lpc.LOGISTIC, 1e-5, N, B, b, lpc.CLIP_STD, 2.0, 3)
    assert ctx.query(lpc.INFO_STEP_CLUSTER_SIZE) == 4
    assert ctx.query(lpc.INFO_STEP_RING_STAGES) == (6 if B == 256 else 5)
    ctx.set_option(lpc.OPT_TAP_U, 1)
    rng = np.random.default_rng(B + b)
    xs = (rng.standard_normal(d) * 0.02).astype(np.float32)
    x = (xs + rng.standard_normal(d).astype(np.float32) * 0.005).astype(np.float32)
    mu, margins, _ = orc.full_grad(Xh, yh, P.loss, xs)
    ctx.set_buffer(lpc.BUF_XTILDE, torch.from_numpy(xs).to(DEV))
    ctx.set_buffer(lpc.BUF_MU, torch.from_numpy(mu).to(DEV))
    ctx.set_buffer(lpc.BUF_MARGINS, torch.from_numpy(margins).to(DEV))
    k, eta = 7, 0.01
    ctx.set_iterate(torch.from_numpy(x).to(DEV))
    ctx.inner_step(eta, k)
    ctx.sync_status()
    _, t = orc.lpc_inner_step(P, k, eta, x, xs, mu, taps=True)
    idx = ctx.get_buffer(lpc.BUF_BATCH_IDX).cpu().numpy()[:N]
    coef = ctx.get_buffer(lpc.BUF_COEF).cpu().numpy()[:N]
    assert (idx == t["idx"]).all()
    # the logistic derivative goes through exp on both sides: coefficients within an ulp of their largest, and everything
    # after them bit for bit once the oracle is handed the coefficients the kernel used
    assert np.abs(coef - t["coef"]).max() <= 1.2e-7 * max(1.0, np.abs(t["coef"]).max())
    words = np.zeros((N, P.W), np.uint32)
    delta = np.zeros(N, np.float32)
    clipped = np.zeros(N, np.uint32)
    u = np.zeros((N, d), np.float32)
    for i in range(N):
        u[i] = orc.svrg_diff_from_coef(Xh, idx[i], coef[i])
        w, delta[i], clipped[i] = orc.quantize_pack(u[i], b, orc.CLIP_STD, 2.0, 3, i, k)
        words[i] = w[: P.W]
    xn, v = orc.unpack_average_prox(words, delta, d, b, mu, x, eta, P.lambda_l1, want_v=True)
    assert (_bits(ctx.get_buffer(lpc.BUF_U)) == _bits(u)).all()
    assert (_bits(ctx.get_buffer(lpc.BUF_DELTA)) == _bits(delta)).all()
    codes = ctx.get_buffer(lpc.BUF_CODES).cpu().numpy().view(np.uint32)
    assert (codes[:, : P.W] == words).all() and (codes[:, P.W:] == 0).all()
    assert (ctx.get_buffer(lpc.BUF_CLIPPED).cpu().numpy().view(np.uint32) == clipped).all()
    assert (_bits(ctx.get_buffer(lpc.BUF_V)) == _bits(v)).all()
    assert (_bits(ctx.get_iterate()) == _bits(xn)).all()
    ctx.close()

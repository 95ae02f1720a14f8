"""The error path of the bounded device-side waits, without hanging or faulting anything: a tiny kernel waits on an
mbarrier phase that nothing completes and polls a tagged word that nobody writes, through the same wait routines
as the training kernels; both give up after a millisecond or two, the status reaches the host as LPC_ERR_TIMEOUT,
and the context goes on working."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_1901_08924_b200 import lpc, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_timeout_is_reported_once_and_the_loop_still_matches_the_oracle():
    n, d, N, B, b, seed = 256, 512, 4, 2, 4, 1
    X, y, _ = synth.linear_problem(n, d, loss="least_squares", sparsity=0.1, noise=0.01, seed=2)
    ctx = lpc.Context(X.to(DEV), y.to(DEV), lpc.LEAST_SQUARES, 1e-4, N, B, b, lpc.CLIP_STD, 3.0, seed)
    ctx.snapshot_full_grad()
    ctx.inner_steps(0.05, 0, 4)
    assert ctx.status() == lpc.OK
    ctx.debug_wait_timeout(2_000_000)
    assert ctx.status() == lpc.ERR_TIMEOUT
    assert ctx.status() == lpc.OK  # reported once
    # the one-launch loop after the raised abort flag: four more steps, eight in all, against the oracle
    ctx.inner_steps(0.05, 4, 4)
    ctx.sync_status()
    P = orc.Problem(X.numpy(), y.numpy(), orc.LEAST_SQUARES, 1e-4, N, B, b, orc.CLIP_STD, 3.0, seed)
    x0 = np.zeros(d, np.float32)
    mu = ctx.get_buffer(lpc.BUF_MU).cpu().numpy()
    xr = x0
    for k in range(8):
        xr = orc.lpc_inner_step(P, k, 0.05, xr, x0, mu)
    assert (ctx.get_iterate().cpu().numpy().view(np.uint32) == xr.view(np.uint32)).all()
    with pytest.raises(lpc.LpcError):
        ctx.debug_wait_timeout(10)  # below the smallest limit
    ctx.close()


def test_timeout_on_a_quantizer_only_context():
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, 2, 1, 4, lpc.CLIP_NONE, 1.0, 0)
    q.debug_wait_timeout(1_000_000)
    assert q.status() == lpc.ERR_TIMEOUT
    U = torch.randn((2, 1000), device=DEV)
    codes, delta, _ = q.quantize_pack(U, 0)
    assert q.status() == lpc.OK
    w, dl, _ = orc.quantize_pack(U[1].cpu().numpy(), 4, orc.CLIP_NONE, 1.0, 0, 1, 0)
    assert (codes[1].cpu().numpy().view(np.uint32)[: w.size] == w).all()
    q.close()

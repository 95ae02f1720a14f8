"""GPU parity of the stand-alone quantize+pack and unpack+average+prox entry points against the
CPU oracle, through the C ABI.  Codes, scales, clipped counts and the updated iterate must match
bit for bit (the random streams and the fp32 operation order are part of the definition)."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_1901_08924_b200 import lpc, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _u32(t):
    return t.detach().cpu().numpy().view(np.uint32)


def _oracle_quantize(U, b, clip_mode, clip_value, seed, k, seg_offsets=None, U_sub=None):
    """Reference packed buffer in the library's layout: returns (codes (N, stride), delta (N, nseg), clipped)."""
    N, length = U.shape
    offs = [0, length] if seg_offsets is None else list(seg_offsets)
    nseg = len(offs) - 1
    woff, stride = lpc.packed_layout(length, b, None if seg_offsets is None else offs)
    codes = np.zeros((N, stride), np.uint32)
    delta = np.zeros((N, nseg), np.float32)
    clipped = np.zeros((N, nseg), np.uint32)
    V = U if U_sub is None else (U - U_sub).astype(np.float32)
    base = 0
    for s in range(nseg):
        ln = offs[s + 1] - offs[s]
        for i in range(N):
            w, dl, cl = orc.quantize_pack(V[i, offs[s]:offs[s + 1]], b, clip_mode, clip_value, seed, i, k, base)
            codes[i, woff[s]:woff[s] + w.size] = w
            delta[i, s], clipped[i, s] = dl, cl
        base += (ln + 7) // 8
    return codes, delta, clipped


def _ctx(N, b, clip_mode, clip_value, seed):
    return lpc.Context(None, None, lpc.LOGISTIC, 0.0, N, 1, b, clip_mode, clip_value, seed)


def test_philox_streams_match_oracle_bitwise():
    for (seed, tag, worker, k, block0) in [(0, 0, 0, 0, 0), (0x123456789ABCDEF0, 1, 77, (3 << 32) + 5, 1000),
                                           (42, 2, 0xABCDEF, 2 ** 40, 0xFFFFFF00)]:
        got = _u32(lpc.debug_stream_blocks(seed, tag, worker, k, block0, 300))
        for i in (0, 1, 2, 17, 255, 299):
            want = orc.stream_block(seed, tag, worker, k, (block0 + i) & 0xFFFFFFFF)
            assert (got[i] == want).all()


@pytest.mark.parametrize("b", [1, 2, 3, 4, 5, 7, 8, 12, 16, 32])
@pytest.mark.parametrize("clip", [(orc.CLIP_NONE, 1.0), (orc.CLIP_LAMBDA, 0.85), (orc.CLIP_STD, 2.5)])
@pytest.mark.parametrize("one_launch", [1, 0])
def test_quantize_pack_bit_exact(b, clip, one_launch):
    # one_launch = 1: the single cooperative launch that short vectors take (b = 32 always takes three launches)
    N, seed, k = 3, 1234, 7
    rng = np.random.default_rng(b * 10 + clip[0])
    for length in (1, 7, 8, 9, 31, 33, 257, 2047, 8191, 8192, 8193, 3 * 8192 + 1001):
        U = rng.standard_normal((N, length)).astype(np.float32)
        U[0] *= 1e-3
        ctx = _ctx(N, b, clip[0], clip[1], seed)
        ctx.set_option(lpc.OPT_ONE_LAUNCH_QUANTIZE, one_launch)
        codes, delta, clipped = ctx.quantize_pack(torch.from_numpy(U).to(DEV), k)
        ctx.sync_status()
        assert ctx.query(lpc.INFO_QUANT_ONE_LAUNCH) == (1 if one_launch and b != 32 else 0)
        rc, rd, rcl = _oracle_quantize(U, b, clip[0], clip[1], seed, k)
        assert (delta.cpu().numpy() == rd).all(), (length, delta, rd)
        assert (_u32(codes) == rc).all(), length
        assert (_u32(clipped) == rcl).all(), length
        ctx.close()


@pytest.mark.parametrize("b", [2, 4, 6])
def test_quantize_segments_difference_and_strided_rows(b):
    # per-tensor scales, u = cur - snap formed on the fly, rows with a stride larger than len
    N, seed, k = 4, 99, 3
    offs = [0, 4, 4, 1000, 1064, 9400, 9400 + 8192 * 2, 9400 + 8192 * 2 + 12]
    length = offs[-1]
    rng = np.random.default_rng(5)
    scale = np.repeat(10.0 ** rng.uniform(-4, -1, len(offs) - 1), np.diff(offs)).astype(np.float32)
    cur = (rng.standard_normal((N, length)) * scale).astype(np.float32)
    snap = (rng.standard_normal((N, length)) * scale).astype(np.float32)
    ld = length + 20
    cur_d = torch.zeros((N, ld), device=DEV)
    snap_d = torch.zeros((N, ld), device=DEV)
    cur_d[:, :length] = torch.from_numpy(cur).to(DEV)
    snap_d[:, :length] = torch.from_numpy(snap).to(DEV)
    ctx = _ctx(N, b, orc.CLIP_STD, 2.5, seed)
    codes, delta, clipped = ctx.quantize_pack(cur_d[:, :length], k, U_sub=snap_d[:, :length], seg_offsets=offs)
    ctx.sync_status()
    rc, rd, rcl = _oracle_quantize(cur, b, orc.CLIP_STD, 2.5, seed, k, offs, U_sub=snap)
    assert (delta.cpu().numpy() == rd).all()
    assert (_u32(codes) == rc).all()
    assert (_u32(clipped) == rcl).all()
    # segments with offsets that are not multiples of 4 take the scalar-load path
    offs2 = [0, 3, 1001, 1001 + 8195]
    U = rng.standard_normal((N, offs2[-1])).astype(np.float32)
    codes, delta, clipped = ctx.quantize_pack(torch.from_numpy(U).to(DEV), k, seg_offsets=offs2)
    ctx.sync_status()
    rc, rd, rcl = _oracle_quantize(U, b, orc.CLIP_STD, 2.5, seed, k, offs2)
    assert (delta.cpu().numpy() == rd).all() and (_u32(codes) == rc).all() and (_u32(clipped) == rcl).all()
    ctx.close()


def test_degenerate_and_nonfinite_inputs():
    N, b = 2, 4
    ctx = _ctx(N, b, orc.CLIP_STD, 2.5, 0)
    U = torch.zeros((N, 100), device=DEV)
    U[1, 50] = 3.0  # worker 1: a single outlier -> std clip far below the max
    codes, delta, clipped = ctx.quantize_pack(U, 0)
    ctx.sync_status()
    rc, rd, rcl = _oracle_quantize(U.cpu().numpy(), b, orc.CLIP_STD, 2.5, 0, 0)
    assert (delta.cpu().numpy() == rd).all() and delta[0, 0] == 0
    assert (_u32(codes) == rc).all() and (_u32(clipped) == rcl).all() and clipped[1, 0] == 1
    assert (orc.unpack(_u32(codes)[0], 100, b) == 8).all()  # zero vector -> all codes are the zero code
    U[0, 3] = float("nan")
    ctx.quantize_pack(U, 1)
    assert ctx.status() == lpc.ERR_NONFINITE
    U[0, 3] = float("inf")
    ctx.quantize_pack(U, 2)
    assert ctx.status() == lpc.ERR_NONFINITE
    assert ctx.status() == lpc.OK  # the flag is cleared once reported
    # empty vector: nothing to do, no error
    E = torch.zeros((N, 0), device=DEV)
    codes, delta, clipped = ctx.quantize_pack(E, 0)
    ctx.sync_status()
    assert codes.shape == (N, 0)
    ctx.close()


@pytest.mark.parametrize("b", [1, 2, 3, 4, 8, 11, 16, 32])
@pytest.mark.parametrize("N", [1, 5, 8])
def test_unpack_average_prox_bit_exact(b, N):
    seed, k = 5, 11
    rng = np.random.default_rng(b + N)
    for length in (1, 8, 9, 100, 8191, 8200, 2 * 8192 + 77):
        U = rng.standard_normal((N, length)).astype(np.float32)
        mu = rng.standard_normal(length).astype(np.float32)
        x0 = rng.standard_normal(length).astype(np.float32)
        rc, rd, _ = _oracle_quantize(U, b, orc.CLIP_STD, 2.0, seed, k)
        ctx = _ctx(N, b, orc.CLIP_STD, 2.0, seed)
        x = torch.from_numpy(x0).to(DEV)
        v = torch.empty(length, device=DEV)
        ctx.unpack_average_prox(torch.from_numpy(rc.view(np.int32)).to(DEV), torch.from_numpy(rd).to(DEV), length, x,
                                0.3, 1e-3 * 50, mu=torch.from_numpy(mu).to(DEV), v_out=v)
        ctx.sync_status()
        W = orc.packed_words(length, b)
        xr, vr = orc.unpack_average_prox(rc[:, :max(W, 1)], rd[:, 0], length, b, mu, x0, 0.3, 1e-3 * 50, want_v=True)
        assert (x.cpu().numpy().view(np.uint32) == xr.view(np.uint32)).all(), length
        assert (v.cpu().numpy().view(np.uint32) == vr.view(np.uint32)).all(), length
        # mu = None means no snapshot term
        x2 = torch.from_numpy(x0).to(DEV)
        ctx.unpack_average_prox(torch.from_numpy(rc.view(np.int32)).to(DEV), torch.from_numpy(rd).to(DEV), length, x2,
                                1.0, 1e-3)
        xr2 = orc.unpack_average_prox(rc[:, :max(W, 1)], rd[:, 0], length, b, None, x0, 1.0, 1e-3)
        assert (x2.cpu().numpy().view(np.uint32) == xr2.view(np.uint32)).all()
        ctx.close()


def test_round_trip_segmented_dnn_shapes_small():
    # quantize -> aggregate on a scaled-down layer list (same code path as the 62-tensor workload)
    shapes = [(16, 3, 3, 3), (16,), (16,), (32, 16, 3, 3), (32,), (32,), (10, 32), (10,)]
    N, b, seed, k = 4, 4, 3, 2
    cur, snap, mu, offs = synth.dnn_gradients(N, shapes, seed=1)
    ctx = _ctx(N, b, orc.CLIP_STD, 2.5, seed)
    codes, delta, clipped = ctx.quantize_pack(cur.to(DEV), k, U_sub=snap.to(DEV), seg_offsets=offs)
    x = torch.zeros(offs[-1], device=DEV)
    ctx.unpack_average_prox(codes, delta, offs[-1], x, -1.0, 0.0, mu=mu.to(DEV), seg_offsets=offs)  # x = v
    ctx.sync_status()
    rc, rd, _ = _oracle_quantize(cur.numpy(), b, orc.CLIP_STD, 2.5, seed, k, offs, U_sub=snap.numpy())
    assert (_u32(codes) == rc).all() and (delta.cpu().numpy() == rd).all()
    woff, stride = lpc.packed_layout(offs[-1], b, offs)
    want = np.zeros(offs[-1], np.float32)
    for s in range(len(shapes)):
        ln = offs[s + 1] - offs[s]
        W = orc.packed_words(ln, b)
        want[offs[s]:offs[s + 1]] = orc.unpack_average_prox(rc[:, woff[s]:woff[s] + W], rd[:, s], ln, b,
                                                            mu.numpy()[offs[s]:offs[s + 1]], np.zeros(ln, np.float32),
                                                            -1.0, 0.0)
    assert (x.cpu().numpy().view(np.uint32) == want.view(np.uint32)).all()
    # aggregated gradient against the unquantized mean: per coordinate within the mean over workers of
    # (one grid step + the part of |u| beyond the clip threshold T = 7*delta)
    u = cur - snap
    err = (x.cpu() - (u.mean(dim=0) + mu)).abs()
    dl = delta.cpu()
    for s in range(len(shapes)):
        us = u[:, offs[s]:offs[s + 1]]
        bound = (dl[:, s:s + 1] * 1.0001 + (us.abs() - 7 * dl[:, s:s + 1]).clamp(min=0)).mean(dim=0)
        assert (err[offs[s]:offs[s + 1]] <= bound + 1e-9).all()
    ctx.close()


def test_bit_counters_follow_table1():
    N, b, length = 4, 2, 1000
    ctx = _ctx(N, b, orc.CLIP_NONE, 1.0, 0)
    ctx.quantize_pack(torch.randn((N, length), device=DEV), 0)
    ctx.quantize_pack(torch.randn((N, length), device=DEV), 1)
    s1, s2 = ctx.comm_bits()
    assert s1 == 0 and s2 == 2 * orc.broadcast_bits(length, b, N) == 2 * 24384
    ctx.close()

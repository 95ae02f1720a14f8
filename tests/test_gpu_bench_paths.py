"""Parity on every launch shape the benchmark's quantizer/aggregator legs time.

The second pass of lpc_quantize_pack has a software-pipelined loop that only runs of several whole tiles
enter, and lpc_unpack_average_prox spreads a tile over 4, 2 or 1 CTAs depending on the tile count.  The
tests here drive each of those shapes for every fixed code width, compare with the oracle element by
element where it finishes in seconds and in sampled windows (plus scales and clipped counts from full
oracle passes) at the full lengths, and assert through lpc_query that the intended shape really ran.
"""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_1901_08924_b200 import lpc, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"
TILE = 8192
RUN = 8  # tiles per CTA of the quantizer's second pass


def _u32(t):
    return t.detach().cpu().numpy().view(np.uint32)


def _bits(a):
    a = np.asarray(a)
    return a.view(np.uint32) if a.dtype == np.float32 else a


def _ctx(N, b, clip_mode, clip_value, seed):
    return lpc.Context(None, None, lpc.LOGISTIC, 0.0, N, 1, b, clip_mode, clip_value, seed)


def _offset(b):
    return 0 if b == 1 else 1 << (b - 1)


def _rows_aligned(U):
    """U on the device with a row stride that is a multiple of 4 floats, so that every worker's vector starts on a
    16-byte boundary (the pipelined loop needs that)."""
    N, length = U.shape
    buf = torch.zeros((N, (length + 3) // 4 * 4), device=DEV)
    buf[:, :length] = torch.from_numpy(U).to(DEV)
    return buf[:, :length]


@pytest.mark.parametrize("b", [1, 2, 3, 4, 8])
def test_quantize_runs_of_whole_tiles_bit_exact(b):
    # runs of 2, 5, 8 whole tiles, a full run plus one tile and a ragged tail, two full runs plus a tail
    N, seed, k = 3, 77, 5
    rng = np.random.default_rng(100 + b)
    for length, want_runs in ((2 * TILE, 1), (5 * TILE + 3, 0), (8 * TILE, 1), (9 * TILE + 17, 1), (16 * TILE + 5, 2),
                              (13 * TILE, 2)):
        U = rng.standard_normal((N, length)).astype(np.float32)
        U[1] *= 37.0
        ctx = _ctx(N, b, orc.CLIP_STD, 2.0, seed)
        ctx.set_option(lpc.OPT_ONE_LAUNCH_QUANTIZE, 0)  # the three-launch path that long vectors take
        codes, delta, clipped = ctx.quantize_pack(_rows_aligned(U), k)
        ctx.sync_status()
        assert ctx.query(lpc.INFO_QUANT_PIPELINED_RUNS) == want_runs, length
        assert ctx.query(lpc.INFO_QUANT_ONE_LAUNCH) == 0
        W = orc.packed_words(length, b)
        for i in range(N):
            w, dl, cl = orc.quantize_pack(U[i], b, orc.CLIP_STD, 2.0, seed, i, k)
            assert _bits(np.float32(dl).reshape(1))[0] == _u32(delta)[i, 0], (length, i)
            assert (_u32(codes)[i, :W] == w).all(), (length, i)
            assert (_u32(codes)[i, W:] == 0).all()
            assert int(_u32(clipped)[i, 0]) == cl
        ctx.close()


@pytest.mark.parametrize("b", [2, 3, 8])
def test_quantize_runs_with_subtrahend_bit_exact(b):
    # u = cur - snap formed on the fly inside the pipelined loop (one sweep per step instead of two)
    N, seed, k = 2, 9, 1
    rng = np.random.default_rng(b)
    length = 10 * TILE + 100
    cur = rng.standard_normal((N, length)).astype(np.float32)
    snap = rng.standard_normal((N, length)).astype(np.float32)
    ctx = _ctx(N, b, orc.CLIP_STD, 2.5, seed)
    ctx.set_option(lpc.OPT_ONE_LAUNCH_QUANTIZE, 0)
    codes, delta, clipped = ctx.quantize_pack(torch.from_numpy(cur).to(DEV), k, U_sub=torch.from_numpy(snap).to(DEV))
    ctx.sync_status()
    assert ctx.query(lpc.INFO_QUANT_PIPELINED_RUNS) == 1
    u = (cur - snap).astype(np.float32)
    W = orc.packed_words(length, b)
    for i in range(N):
        w, dl, cl = orc.quantize_pack(u[i], b, orc.CLIP_STD, 2.5, seed, i, k)
        assert (_u32(codes)[i, :W] == w).all() and int(_u32(clipped)[i, 0]) == cl
        assert _bits(np.float32(dl).reshape(1))[0] == _u32(delta)[i, 0]
    ctx.close()


def _window_check(Uh, sc, ch, xh, dl, b, seed, k, starts, W):
    """Codes and updated coordinates of the windows [s0, s0 + W) against the oracle, coordinate by coordinate."""
    N = Uh.shape[0]
    for s0 in starts:
        words = np.zeros((N, W * b // 32), np.uint32)
        for i in range(N):
            c = np.array([orc.quantize_coord(Uh[i, j], sc[i]["rdelta"], b, orc.rounding_bits(seed, i, k, 0, j)) + _offset(b)
                          for j in range(s0, s0 + W)], np.uint32)
            words[i] = orc.pack(c, b)
        assert (ch[:, s0 * b // 32:(s0 + W) * b // 32] == words).all(), s0
        ref = orc.unpack_average_prox(words, dl, W, b, None, np.zeros(W, np.float32), 1.0, 1e-3)
        assert (_bits(xh[s0:s0 + W]) == _bits(ref)).all(), s0


def _full_length_case(N, log2_len, b, dist, clip, seed, k, want_split):
    length = 1 << log2_len
    U = synth.gradient_vectors(N, length, dist, seed=seed + 1, device=DEV)
    q = _ctx(N, b, orc.CLIP_STD, clip, seed)
    codes, delta, clipped = q.quantize_pack(U, k)
    assert q.query(lpc.INFO_QUANT_ONE_LAUNCH) == 0  # longer than L2 holds: statistics, scale and codes as three launches
    assert q.query(lpc.INFO_QUANT_PIPELINED_RUNS) == length // (TILE * RUN)
    x = torch.zeros(length, device=DEV)
    q.unpack_average_prox(codes, delta, length, x, 1.0, 1e-3)
    q.sync_status()
    assert q.query(lpc.INFO_AGGREGATE_SPLIT) == want_split
    Uh = U.cpu().numpy()
    del U
    sc = [orc.scale(Uh[i], b, orc.CLIP_STD, clip) for i in range(N)]
    dl = delta.cpu().numpy()[:, 0]
    assert (_bits(dl) == _bits(np.array([s["delta"] for s in sc], np.float32))).all()
    lower = [-np.float32(s["T"]) if b == 1 else -(np.float32(s["T"]) + np.float32(s["delta"])) for s in sc]
    want_clip = [int(((Uh[i] > sc[i]["T"]) | (Uh[i] < lower[i])).sum()) for i in range(N)]
    assert clipped.cpu().numpy()[:, 0].tolist() == want_clip
    W = 1024
    starts = [0, TILE * 37 + 32, length // 2 - 512, length - W]
    _window_check(Uh, sc, codes.cpu().numpy().view(np.uint32), x.cpu().numpy(), dl, b, seed, k, starts, W)
    q.close()


@pytest.mark.parametrize("b", [1, 2, 8])
def test_sweep_2p26_other_widths_sampled_windows(b):
    # the sweep's longest timed length at the widths that the b = 4 full-length test does not cover; one CTA per
    # aggregator tile (8,192 tiles)
    _full_length_case(8, 26, b, "gauss", 2.0, seed=20 + b, k=2, want_split=1)


@pytest.mark.parametrize("b", [1, 2, 4, 8])
def test_aggregator_two_ctas_per_tile_2p23(b):
    # 2^23 coordinates = 1,024 tiles: between one and two waves of resident CTAs, two CTAs share a tile
    _full_length_case(8, 23, b, "student_t3", 2.0, seed=30 + b, k=4, want_split=2)


@pytest.mark.parametrize("clip", [1.0, 4.0])
def test_sweep_2p24_other_clip_values(clip):
    # clip 1 std (a third of the coordinates outside the hull) and 4 std (almost none) on heavy-tailed values
    _full_length_case(8, 24, 4, "student_t3", clip, seed=41, k=6, want_split=1)


def test_sweep_2p28_sampled_windows():
    # the longest vectors of the sweep: 8 x 2^28 heavy-tailed values (8.6 GB), b = 4, clip 2 std
    _full_length_case(8, 28, 4, "student_t3", 2.0, seed=51, k=7, want_split=1)


@pytest.mark.parametrize("b", [3])
def test_three_level_codes_full_length_windows(b):
    # the paper's own setting (three positive levels, b = 3): 24 bits per thread, three words per four lanes
    N, length, seed, k = 8, 1 << 22, 61, 8
    U = synth.gradient_vectors(N, length, "gauss", seed=seed, device=DEV)
    q = _ctx(N, b, orc.CLIP_STD, 2.0, seed)
    codes, delta, clipped = q.quantize_pack(U, k)
    x = torch.zeros(length, device=DEV)
    q.unpack_average_prox(codes, delta, length, x, 1.0, 1e-3)
    q.sync_status()
    assert q.query(lpc.INFO_QUANT_PIPELINED_RUNS) == length // (TILE * RUN) and q.query(lpc.INFO_AGGREGATE_SPLIT) == 4
    assert q.query(lpc.INFO_QUANT_ONE_LAUNCH) == 0  # 8 x 2^22 values = 134 MB
    Uh = U.cpu().numpy()
    W = orc.packed_words(length, b)
    ch = codes.cpu().numpy().view(np.uint32)
    words = np.zeros((N, W), np.uint32)
    dl = np.zeros(N, np.float32)
    for i in range(N):
        words[i], dl[i], cl = orc.quantize_pack(Uh[i], b, orc.CLIP_STD, 2.0, seed, i, k)
        assert cl == int(clipped.cpu().numpy()[i, 0])
    assert (ch[:, :W] == words).all()
    assert (_bits(delta.cpu().numpy()[:, 0]) == _bits(dl)).all()
    ref = orc.unpack_average_prox(words, dl, length, b, None, np.zeros(length, np.float32), 1.0, 1e-3)
    assert (_bits(x.cpu().numpy()) == _bits(ref)).all()
    q.close()


@pytest.mark.parametrize("b", [1, 2, 3, 4, 8, 16])
@pytest.mark.parametrize("log2_len", [16, 20])
def test_one_launch_quantizer_short_vectors_bit_exact(b, log2_len):
    # the sweep's short vectors (8 x 2^16, 8 x 2^20) stay in L2 between the statistics and the codes: one cooperative
    # launch; at 2^20 the 1,024 tiles exceed the resident CTAs, so a CTA takes several tiles of different workers.
    # Twice in a row: the arrival counters carry over from call to call.
    N, seed = 8, 71
    length = 1 << log2_len
    U = synth.gradient_vectors(N, length, "student_t3", seed=b + log2_len)
    q = _ctx(N, b, orc.CLIP_STD, 2.0, seed)
    Ud = U.to(DEV)
    for k in (3, 4):
        codes, delta, clipped = q.quantize_pack(Ud, k)
        q.sync_status()
        assert q.query(lpc.INFO_QUANT_ONE_LAUNCH) == 1
        W = orc.packed_words(length, b)
        for i in range(N):
            w, dl, cl = orc.quantize_pack(U[i].numpy(), b, orc.CLIP_STD, 2.0, seed, i, k)
            assert (_u32(codes)[i, :W] == w).all(), (k, i)
            assert _bits(np.float32(dl).reshape(1))[0] == _u32(delta)[i, 0] and int(_u32(clipped)[i, 0]) == cl
    # the three-launch path on the same input gives the same bits
    q.set_option(lpc.OPT_ONE_LAUNCH_QUANTIZE, 0)
    c2, d2, cl2 = q.quantize_pack(Ud, 4)
    q.sync_status()
    assert q.query(lpc.INFO_QUANT_ONE_LAUNCH) == 0
    assert torch.equal(c2, codes) and torch.equal(d2.view(torch.int32), delta.view(torch.int32)) and torch.equal(cl2, clipped)
    q.close()

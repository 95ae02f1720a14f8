"""Pins for the oracle's parameter-server schemes (b) and (c) of Section 3.2 (CPU only).

Checked against what the paper and arithmetic fix: the unified scale is the largest worker scale; adding
grid indices loses nothing (scheme (b) equals the average of the decoded vectors); the sums fit the
ceil(log N) extra bits in the worst case; the second quantization of scheme (c) is unbiased and leaves grid
points alone (exhaustive over all 65,536 rounding values); Table 1's bit counts.
"""
import math
import os

import numpy as np
import pytest

import oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _vectors(N, d, seed, spread=True):
    rng = np.random.default_rng(seed)
    U = rng.standard_normal((N, d)).astype(np.float32)
    if spread:
        U *= rng.uniform(0.2, 3.0, size=(N, 1)).astype(np.float32)  # workers with different magnitudes
    return U


def test_table1_parameter_server_rows():
    rows = [l.split()[1:] for l in open(os.path.join(GOLDEN, "table1_bits.txt")) if l.startswith("ps")]
    assert len(rows) == 5
    for d, b, N, bits_b, bits_c in (map(int, r) for r in rows):
        assert orc.scheme_bits(orc.SCHEME_B, d, b, N) == bits_b
        assert orc.scheme_bits(orc.SCHEME_C, d, b, N) == bits_c
        assert orc.scheme_bits(orc.SCHEME_A, d, b, N) == orc.broadcast_bits(d, b, N)
        assert orc.sum_bits_per_coordinate(b, N) == b + math.ceil(math.log2(N))
        # (c) sends b bits each way, (b) widens only the way back
        assert bits_b - bits_c == N * d * math.ceil(math.log2(N))


@pytest.mark.parametrize("b", [2, 3, 4, 8])
@pytest.mark.parametrize("clip", [(orc.CLIP_NONE, 1.0), (orc.CLIP_LAMBDA, 0.5), (orc.CLIP_STD, 2.0)])
def test_unified_scale_is_the_largest_worker_scale(b, clip):
    U = _vectors(5, 333, 7)
    own = [orc.scale(U[i], b, *clip) for i in range(5)]
    words, delta, clipped = orc.quantize_pack_shared(U, b, *clip, seed=3, k=11)
    assert delta == max(o["delta"] for o in own)
    i_star = int(np.argmax([o["T"] for o in own]))
    # the worker that owns the scale sends exactly what it would send on its own
    w_own, d_own, c_own = orc.quantize_pack(U[i_star], b, *clip, seed=3, worker=i_star, k=11)
    assert d_own == delta and (w_own == words[i_star]).all() and c_own == clipped[i_star]
    # the others are quantized on the same grid: every decoded value is an index times the shared delta,
    # inside the shared hull, and within one grid step of the (clipped) input
    T = own[i_star]["T"]
    for i in range(5):
        idx = orc.unpack(words[i], 333, b).astype(np.int64) - 2 ** (b - 1)
        assert idx.min() >= -(2 ** (b - 1)) and idx.max() <= 2 ** (b - 1) - 1
        clippedu = np.clip(U[i].astype(np.float64), -(np.float64(T) + np.float64(delta)), np.float64(T))
        assert np.abs(idx * np.float64(delta) - clippedu).max() <= np.float64(delta) * (1 + 1e-5)
        outside = int(((U[i] > T) | (U[i] < -(np.float32(T) + np.float32(delta)))).sum())
        assert clipped[i] == outside


def test_all_zero_workers_and_all_zero_input():
    U = _vectors(3, 50, 1)
    U[1] = 0
    words, delta, _ = orc.quantize_pack_shared(U, 4, seed=1)
    assert delta > 0 and (orc.unpack(words[1], 50, 4) == 8).all()  # zeros on the shared grid
    words, delta, clipped = orc.quantize_pack_shared(np.zeros((3, 50), np.float32), 4, seed=1)
    assert delta == 0 and (clipped == 0).all()
    for i in range(3):
        assert (orc.unpack(words[i], 50, 4) == 8).all()


@pytest.mark.parametrize("N", [2, 3, 4, 7, 16])
@pytest.mark.parametrize("b", [2, 4, 8])
def test_scheme_b_sum_is_lossless(N, b):
    d = 211
    U = _vectors(N, d, 100 + N + b)
    words, delta, _ = orc.quantize_pack_shared(U, b, orc.CLIP_STD, 2.5, seed=5, k=2)
    sums = orc.server_reduce(words, d, b, requantize=False)
    bo = orc.sum_bits_per_coordinate(b, N)
    assert sums.size == orc.packed_words(d, bo)
    K = orc.unpack(sums, d, bo).astype(np.int64) - 2 ** (bo - 1)
    idx = np.stack([orc.unpack(words[i], d, b).astype(np.int64) - 2 ** (b - 1) for i in range(N)])
    assert (K == idx.sum(axis=0)).all()
    # worker side: (delta*K)/N equals the mean of the decoded vectors (Eq. 3) up to two fp32 roundings
    x0 = np.zeros(d, np.float32)
    _, ut = orc.unpack_scaled_prox(sums, delta, d, bo, N, None, x0, 1.0, 0.0, want_utilde=True)
    exact = np.float64(delta) * idx.sum(axis=0) / N
    assert np.abs(ut - exact).max() <= 2.0 ** -22 * np.abs(exact).max()
    # and the broadcast scheme (a) on the same messages gives the same average within fp32 summation error
    xa, uta = orc.unpack_average_prox(words, np.full(N, delta, np.float32), d, b, None, x0, 1.0, 0.0, want_utilde=True)
    assert np.abs(uta - exact).max() <= N * 2.0 ** -23 * np.abs(exact).max()


def test_sum_fits_the_extra_bits_in_the_worst_case():
    for b in (2, 3, 5, 8):
        for N in (2, 3, 5, 8, 64):
            if b + math.ceil(math.log2(N)) > 16:
                continue
            bo = orc.sum_bits_per_coordinate(b, N)
            lo = np.tile(orc.pack(np.zeros(9, np.uint32), b), (N, 1))                      # every index -2^(b-1)
            hi = np.tile(orc.pack(np.full(9, 2 ** b - 1, np.uint32), b), (N, 1))           # every index 2^(b-1)-1
            klo = orc.unpack(orc.server_reduce(lo, 9, b, False), 9, bo).astype(np.int64) - 2 ** (bo - 1)
            khi = orc.unpack(orc.server_reduce(hi, 9, b, False), 9, bo).astype(np.int64) - 2 ** (bo - 1)
            assert (klo == -N * 2 ** (b - 1)).all() and (khi == N * (2 ** (b - 1) - 1)).all()


def _requant_all_r16(K, N, b):
    """Index chosen by the oracle's rule for the average K/N, for every 16-bit rounding value."""
    s = np.float32(np.float32(K) / np.float32(N))
    return np.array([orc.quantize_coord(s, 1.0, b, r) for r in range(0, 65536)], dtype=np.int64)


@pytest.mark.parametrize("N,K", [(3, 1), (3, -4), (4, 7), (5, -11), (7, 20), (16, -57)])
def test_requantization_is_unbiased_exhaustively(N, K):
    b = 4
    k = _requant_all_r16(K, N, b)
    lo = math.floor(K / N)
    assert set(np.unique(k)) <= {lo, lo + 1}                      # rule (1): one of the two neighbours
    assert abs(k.mean() - K / N) <= 2.0 ** -16                    # E Q(s) = s on the 2^-16 grid of the rounding variable
    var = k.var()
    f = K / N - lo
    assert abs(var - f * (1 - f)) <= 2.0 ** -14 and var <= 0.25 + 1e-12  # (x-z)(z+delta-x) <= delta^2/4


def test_requantization_keeps_grid_points():
    for N in (2, 4, 5):
        for q in (-8, -3, 0, 2, 7):
            k = _requant_all_r16(q * N, N, 4)
            assert (k == q).all()


def test_scheme_c_stream_and_mean():
    N, d, b = 6, 4096, 4
    U = _vectors(N, d, 77)
    words, delta, _ = orc.quantize_pack_shared(U, b, orc.CLIP_STD, 2.0, seed=9, k=4)
    idx = np.stack([orc.unpack(words[i], d, b).astype(np.int64) - 8 for i in range(N)])
    avg = idx.sum(axis=0) / N
    out = orc.server_reduce(words, d, b, requantize=True, seed=9, k=4)
    assert out.size == orc.packed_words(d, b)
    kq = orc.unpack(out, d, b).astype(np.int64) - 8
    assert (np.abs(kq - avg) < 1).all() and (kq[avg == np.round(avg)] == avg[avg == np.round(avg)]).all()
    # the rounding variables are the server's own stream: block j/8, lane j%8 of tag 4, independent of the workers'
    blk = orc.stream_block(9, 4, 0, 4, 5)
    r16 = [(int(blk[l >> 1]) >> (16 * (l & 1))) & 0xFFFF for l in range(8)]
    for l in range(8):
        j = 40 + l
        s = np.float32(np.float32(idx[:, j].sum()) / np.float32(N))
        assert kq[j] == orc.quantize_coord(s, 1.0, b, r16[l])
    # different iterations draw different variables; the error of the second quantization averages out
    errs = []
    for k in range(40):
        o = orc.server_reduce(words, d, b, True, seed=9, k=k)
        errs.append((orc.unpack(o, d, b).astype(np.int64) - 8 - avg).mean())
    assert abs(np.mean(errs)) < 4 * 0.5 / math.sqrt(40 * d)
    # worker side of scheme (c): u~ = delta * index
    _, ut = orc.unpack_scaled_prox(out, delta, d, b, 1, None, np.zeros(d, np.float32), 1.0, 0.0, want_utilde=True)
    assert (ut == (np.float32(delta) * kq.astype(np.float32))).all()


def test_unsupported_widths_are_rejected():
    U = _vectors(2, 16, 1)
    for b in (1, 32):
        with pytest.raises(orc.OracleError):
            orc.quantize_pack_shared(U, b)
    words, _, _ = orc.quantize_pack_shared(_vectors(64, 16, 1), 12)
    with pytest.raises(orc.OracleError):
        orc.server_reduce(words, 16, 12, requantize=False)  # 12 + 6 bits > 16

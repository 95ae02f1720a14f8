"""Pins for the oracle's RNG, quantizer, packing and aggregation (CPU only).

Each test checks the oracle against something fixed by the paper or by mathematics, not against
a retyped copy of the oracle's own formula.
"""
import math
import os

import numpy as np
import pytest

import oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---- Philox ----------------------------------------------------------------------------------

def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if l[0] != "#"]
    assert len(rows) == 3
    for r in rows:
        v = [int(t, 16) for t in r]
        out = orc.philox4x32_10(v[0:4], v[4:6])
        assert [int(o) for o in out] == v[6:10]


def test_stream_counter_layout():
    # the stream helper is the raw generator at counter (block, k_lo, worker|tag<<24, k_hi), key = seed
    seed, tag, worker, k, block = 0x1234567811223344, 2, 77, (5 << 32) | 9, 1234
    a = orc.stream_block(seed, tag, worker, k, block)
    b = orc.philox4x32_10([block, 9, 77 | (2 << 24), 5], [0x11223344, 0x12345678])
    assert (a == b).all()


def test_rounding_bits_lanes_and_uniformity():
    seed, worker, k = 42, 3, 17
    blk = orc.stream_block(seed, orc.TAG_ROUND, worker, k, 5)
    halves = []
    for w in blk:
        halves += [int(w) & 0xFFFF, int(w) >> 16]
    got = [orc.rounding_bits(seed, worker, k, 0, 40 + l) for l in range(8)]
    assert got == halves
    assert orc.rounding_bits(seed, worker, k, 5, 3) == halves[3]  # block_base shifts the stream
    r = np.array([orc.rounding_bits(7, 0, 0, 0, j) for j in range(40000)], dtype=np.float64)
    assert abs(r.mean() - 32767.5) < 4 * 65536 / math.sqrt(12 * r.size)
    hist = np.bincount((r // 4096).astype(int), minlength=16)
    chi2 = ((hist - r.size / 16) ** 2 / (r.size / 16)).sum()
    assert chi2 < 45  # 15 dof, p ~ 1e-4


# ---- pairwise sums ---------------------------------------------------------------------------

def _pairwise_numpy(v):
    v = np.asarray(v, dtype=np.float32)
    p = 1
    while p < v.size:
        p *= 2
    w = np.zeros(p, dtype=np.float32)
    w[: v.size] = v
    while w.size > 1:
        w = (w[0::2] + w[1::2]).astype(np.float32)
    return w[0]


@pytest.mark.parametrize("n", [1, 2, 3, 7, 8, 9, 100, 1000, 1024, 4097, 70001])
def test_tree_sum_is_pairwise_and_accurate(n):
    rng = np.random.default_rng(n)
    v = rng.standard_normal(n).astype(np.float32)
    s = orc.tree_sum(v)
    assert s == _pairwise_numpy(v)  # level-by-level evaluation of the same tree, bit for bit
    exact = v.astype(np.float64).sum()
    bound = (math.log2(max(n, 2)) + 1) * 2.0 ** -24 * np.abs(v).astype(np.float64).sum()
    assert abs(float(s) - exact) <= bound
    assert orc.tree_sumsq(v) == _pairwise_numpy((v * v).astype(np.float32))
    w = rng.standard_normal(n).astype(np.float32)
    assert orc.tree_dot(v, w) == _pairwise_numpy((v * w).astype(np.float32))


def test_tree_sum_invariant_under_aligned_blocks():
    rng = np.random.default_rng(5)
    v = rng.standard_normal(5000).astype(np.float32)
    full = orc.tree_sum(v)
    for blk in (8, 256, 1024):
        parts = [orc.tree_sum(np.pad(v[i:i + blk], (0, blk - len(v[i:i + blk])))) for i in range(0, v.size, blk)]
        assert orc.tree_sum(np.array(parts, dtype=np.float32)) == full


# ---- quantizer: rule (1), Lemma 1 -------------------------------------------------------------

def _enumerate(u, rdelta, b):
    return np.array([orc.quantize_coord(u, rdelta, b, r) for r in range(65536)], dtype=np.int64)


@pytest.mark.parametrize("b", [2, 3, 4, 8])
def test_unbiased_and_variance_by_exhaustive_enumeration(b):
    # delta = 0.25 exactly (rdelta = 4): x inside the hull must satisfy E[Q(x)] = x (Section 2.2,
    # rule 1) and E(Q(x)-x)^2 = (x-z)(z+delta-x) <= delta^2/4 (Lemma 1).  The rounding variable
    # has 16 bits, so the mean is exact up to delta * 2^-17.
    delta, rdelta = np.float32(0.25), np.float32(4.0)
    Lv = 2 ** (b - 1) - 1
    rng = np.random.default_rng(b)
    xs = rng.uniform(-(Lv + 1) * 0.25, Lv * 0.25, size=6).astype(np.float32)
    for x in xs:
        kq = _enumerate(x, rdelta, b)
        z = math.floor(float(x) / 0.25) * 0.25
        assert set(np.unique(kq)) <= {round(z / 0.25), round(z / 0.25) + 1}
        q = kq * 0.25
        assert abs(q.mean() - float(x)) <= 0.25 * 2.0 ** -17 + 1e-12
        var = ((q - float(x)) ** 2).mean()
        expect = (float(x) - z) * (z + 0.25 - float(x))
        assert abs(var - expect) <= 0.25 ** 2 * 2.0 ** -15
        assert var <= 0.25 ** 2 / 4 + 1e-12
        assert (np.diff(kq) <= 0).all()  # the decision is a threshold on the rounding variable


@pytest.mark.parametrize("b", [2, 3, 4, 5, 8, 12, 16])
def test_codebook_points_are_fixed_points(b):
    # every point of dom(delta,b), including both extremes, maps to itself for every draw
    rdelta = np.float32(4.0)
    for k in range(-2 ** (b - 1), 2 ** (b - 1)) if b <= 8 else (-2 ** (b - 1), -1, 0, 1, 2 ** (b - 1) - 1):
        x = np.float32(k * 0.25)
        for r in (0, 1, 32767, 65535):
            assert orc.quantize_coord(x, rdelta, b, r) == k


@pytest.mark.parametrize("b", [2, 4, 8])
def test_projection_outside_hull(b):
    # rule (2): outside the hull -> smallest / largest codebook value, deterministically
    rdelta = np.float32(4.0)
    lo, hi = -2 ** (b - 1), 2 ** (b - 1) - 1
    for r in (0, 40000, 65535):
        assert orc.quantize_coord(np.float32(hi * 0.25 + 0.01), rdelta, b, r) == hi
        assert orc.quantize_coord(np.float32(1e30), rdelta, b, r) == hi
        assert orc.quantize_coord(np.float32(lo * 0.25 - 0.01), rdelta, b, r) == lo
        assert orc.quantize_coord(np.float32(-1e30), rdelta, b, r) == lo


def test_one_bit_extension_is_unbiased_on_its_interval():
    # b=1 (not defined by Eq. 2): two code points -T,+T; unbiased for |x| <= T
    T = np.float32(2.0)
    for x in (-2.0, -1.3, 0.0, 0.7, 2.0):
        bits = np.array([orc.quantize_coord(np.float32(x), np.float32(0.5), 1, r) for r in range(65536)])
        q = (2 * bits - 1) * float(T)
        assert abs(q.mean() - x) <= 2 * float(T) * 2.0 ** -17 + 1e-12
    assert orc.quantize_coord(np.float32(9.0), np.float32(0.5), 1, 65535) == 1
    assert orc.quantize_coord(np.float32(-9.0), np.float32(0.5), 1, 0) == 0


# ---- scale: Eq. 2 -----------------------------------------------------------------------------

def test_scale_follows_eq2():
    rng = np.random.default_rng(0)
    u = rng.standard_normal(1000).astype(np.float32)
    M = np.abs(u).max()
    for b in (2, 3, 4, 8):
        Lv = 2 ** (b - 1) - 1
        s = orc.scale(u, b, orc.CLIP_NONE)
        assert s["M"] == M and s["T"] == M
        assert s["delta"] == np.float32(M) / np.float32(Lv)
        lam = np.float32(0.85)
        s = orc.scale(u, b, orc.CLIP_LAMBDA, lam)
        assert s["T"] == lam * M and s["delta"] == (lam * M) / np.float32(Lv)
    # c*std reading: T = min(c*std, M) with the population standard deviation
    s = orc.scale(u, 4, orc.CLIP_STD, 2.5)
    assert abs(float(s["T"]) - 2.5 * u.astype(np.float64).std()) < 1e-5
    s = orc.scale(u, 4, orc.CLIP_STD, 100.0)
    assert s["T"] == M
    # degenerate scale: u = 0 gives delta = 0
    s = orc.scale(np.zeros(10, np.float32), 4, orc.CLIP_STD, 2.5)
    assert s["degenerate"] and s["delta"] == 0
    with pytest.raises(orc.OracleError) as e:
        orc.scale(np.array([1.0, np.inf], np.float32), 4)
    assert e.value.code == orc.ERR_NONFINITE
    with pytest.raises(orc.OracleError):
        orc.scale(np.array([np.nan, 1.0], np.float32), 4)


def test_lambda_one_keeps_every_coordinate_in_hull():
    # Section 3.1 "Unbiased quantization": lambda = 1 -> no coordinate is clipped
    rng = np.random.default_rng(1)
    for b in (2, 3, 4, 8):
        for trial in range(20):
            u = (rng.standard_normal(257) * 10.0 ** rng.uniform(-6, 6)).astype(np.float32)
            words, delta, clipped, idx = orc.quantize_pack(u, b, orc.CLIP_NONE, seed=trial, want_index=True)
            assert clipped == 0
            assert idx.min() >= -2 ** (b - 1) and idx.max() <= 2 ** (b - 1) - 1
            assert np.abs(idx * float(delta) - u).max() <= float(delta) * (1 + 1e-6)


def test_clipped_count_and_projection_in_vector_quantizer():
    u = np.array([1.0, -1.0, 0.2, -0.2, 0.5, 0.74, -0.76, 0.0], dtype=np.float32)
    b, lam = 3, np.float32(0.5)  # T = 0.5, delta = 0.5/3, hull = [-(T+delta), T]
    words, delta, clipped, idx = orc.quantize_pack(u, b, orc.CLIP_LAMBDA, lam, want_index=True)
    assert delta == np.float32(0.5) / np.float32(3)
    assert clipped == 4  # 1.0, -1.0, 0.74 and -0.76 lie outside [-0.6667, 0.5]
    assert idx[0] == 3 and idx[1] == -4 and idx[5] == 3 and idx[6] == -4 and idx[7] == 0


def test_monte_carlo_mean_of_vector_quantizer():
    # Section 3.1: with the clip disabled E[Q(u)] = u; tiny vector, many seeds
    u = np.array([0.9, -0.33, 0.05, -1.0, 0.41], dtype=np.float32)
    for b in (2, 4):
        acc = np.zeros(u.size)
        S = 4000
        for seed in range(S):
            _, delta, _, idx = orc.quantize_pack(u, b, orc.CLIP_NONE, seed=seed, want_index=True)
            acc += idx * float(delta)
        err = np.abs(acc / S - u)
        assert (err <= 4 * float(delta) / 2 / math.sqrt(S) + 1e-6).all()


@pytest.mark.parametrize("dist", ["gauss", "student"])
def test_vector_error_bound(dist):
    # supplement, Lemma 3: E||Q(w)-w||^2 <= (d-d_l) delta^2/4 + d_l (1-lambda)^2 ||w||^2
    rng = np.random.default_rng(3)
    d, b, lam = 400, 4, np.float32(0.6)
    w = (rng.standard_normal(d) if dist == "gauss" else rng.standard_t(3, d)).astype(np.float32)
    errs = []
    for seed in range(200):
        _, delta, clipped, idx = orc.quantize_pack(w, b, orc.CLIP_LAMBDA, lam, seed=seed, want_index=True)
        errs.append(((idx * float(delta) - w.astype(np.float64)) ** 2).sum())
    rhs = (d - clipped) * float(delta) ** 2 / 4 + clipped * (1 - float(lam)) ** 2 * (w.astype(np.float64) ** 2).sum()
    assert clipped > 0
    assert np.mean(errs) <= rhs


# ---- b = 32 ------------------------------------------------------------------------------------

def test_b32_is_identity():
    rng = np.random.default_rng(9)
    u = rng.standard_normal(100).astype(np.float32)
    words, delta, clipped = orc.quantize_pack(u, 32, orc.CLIP_NONE)
    assert (words.view(np.float32) == u).all() and delta == 1.0 and clipped == 0
    x = orc.unpack_average_prox(words[None, :], [delta], u.size, 32, None, np.zeros_like(u), -1.0, 0.0)
    assert (x == u).all()  # x+ = 0 - (-1)*u


# ---- packing and bit counts --------------------------------------------------------------------

@pytest.mark.parametrize("b", list(range(1, 17)))
def test_pack_layout_and_round_trip(b):
    rng = np.random.default_rng(b)
    for n in list(range(1, 70)) + [127, 128, 129, 255, 256, 257]:
        codes = rng.integers(0, 2 ** b, size=n, dtype=np.uint32)
        words = orc.pack(codes, b)
        assert words.size == (n * b + 31) // 32 == orc.packed_words(n, b)
        big = sum(int(c) << (j * b) for j, c in enumerate(codes))  # the stream as one integer
        expect = [(big >> (32 * w)) & 0xFFFFFFFF for w in range(words.size)]
        assert [int(w) for w in words] == expect
        assert (orc.unpack(words, n, b) == codes).all()


def test_bit_counts_match_table1():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "table1_bits.txt")) if l[0] != "#" and not l.startswith("ps")]
    for d, b, N, msg, bc in (map(int, r) for r in rows):
        assert orc.message_bits(d, b) == msg
        assert orc.broadcast_bits(d, b, N) == bc
        if N > 1:
            assert math.isclose(32 * d * N * (N - 1) / bc, 32 / (32 / d + b), rel_tol=1e-12)


def test_offset_binary_codes_in_stream():
    # grid index k is stored as k + 2^(b-1); zero vector -> every code is 2^(b-1)
    for b in (2, 3, 4, 8):
        words, delta, clipped, idx = orc.quantize_pack(np.zeros(37, np.float32), b, want_index=True)
        assert delta == 0 and clipped == 0 and (idx == 0).all()
        assert (orc.unpack(words, 37, b) == 2 ** (b - 1)).all()
    u = np.array([3.0, -3.0, 1.0, -4.0], np.float32)  # T=4?  no: CLIP_LAMBDA below fixes delta = 1
    words, delta, _, idx = orc.quantize_pack(u, 3, orc.CLIP_LAMBDA, np.float32(0.75), want_index=True)
    assert delta == 1.0 and list(idx) == [3, -3, 1, -4]
    assert list(orc.unpack(words, 4, 3)) == [7, 1, 5, 0]


# ---- aggregation (Eq. 3) and the proximal step -------------------------------------------------

def test_prox_is_the_argmin_of_its_definition():
    # prox_{eta h}(w) = argmin_y lambda|y| + (y-w)^2/(2 eta), brute force on a fine grid
    grid = np.linspace(-3, 3, 600001)
    for w, eta, lam in [(1.3, 0.5, 1.0), (-0.7, 0.3, 2.0), (0.2, 1.0, 0.5), (-2.0, 0.1, 0.0), (0.0, 1.0, 1.0)]:
        obj = lam * np.abs(grid) + (grid - w) ** 2 / (2 * eta)
        brute = grid[obj.argmin()]
        assert abs(float(orc.soft_threshold(w, eta * lam)) - brute) <= 2e-5


def test_average_and_step_against_float64():
    rng = np.random.default_rng(11)
    N, d, b = 5, 203, 4
    U = rng.standard_normal((N, d)).astype(np.float32)
    mu = rng.standard_normal(d).astype(np.float32)
    x = rng.standard_normal(d).astype(np.float32)
    W = orc.packed_words(d, b)
    words = np.zeros((N, W), np.uint32)
    delta = np.zeros(N, np.float32)
    deq = np.zeros((N, d))
    for i in range(N):
        words[i], delta[i], _, idx = orc.quantize_pack(U[i], b, orc.CLIP_STD, 2.5, seed=1, worker=i, k=4, want_index=True)
        deq[i] = idx.astype(np.float64) * float(delta[i])
    eta, lam = 0.3, 0.05
    xn, v, ut = orc.unpack_average_prox(words, delta, d, b, mu, x, eta, lam, want_v=True, want_utilde=True)
    ut64 = deq.mean(axis=0)  # Eq. 3
    v64 = ut64 + mu
    w64 = x - eta * v64
    x64 = np.sign(w64) * np.maximum(np.abs(w64) - eta * lam, 0)
    assert np.abs(ut - ut64).max() < 1e-6 and np.abs(v - v64).max() < 1e-6 and np.abs(xn - x64).max() < 1e-6
    # workers draw different rounding streams
    w0, _, _ = orc.quantize_pack(U[0], b, seed=1, worker=0, k=4)
    w1, _, _ = orc.quantize_pack(U[0], b, seed=1, worker=1, k=4)
    w2, _, _ = orc.quantize_pack(U[0], b, seed=1, worker=0, k=5)
    assert (w0 != w1).any() and (w0 != w2).any()

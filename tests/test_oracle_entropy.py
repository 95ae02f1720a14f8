"""Pins for the oracle's entropy-coding count (Section 5.1 passes the codes through Huffman's code): histogram,
empirical entropy and Huffman length against textbook cases, closed forms, Shannon's bounds and a brute-force
search over all prefix-code length assignments on tiny alphabets."""
import itertools
import math

import numpy as np
import pytest

import oracle as orc


def test_histogram_counts_every_code_once():
    rng = np.random.default_rng(0)
    for b in (1, 2, 3, 4, 8, 11):
        n = 1000 + b
        codes = rng.integers(0, 2 ** b, size=n, dtype=np.uint32)
        h = orc.code_histogram(orc.pack(codes, b), n, b)
        assert h.sum() == n and (h == np.bincount(codes, minlength=2 ** b)).all()
    assert orc.code_histogram(np.zeros(1, np.uint32), 0, 4).sum() == 0


def test_uniform_and_dyadic_histograms_have_closed_forms():
    for b in (1, 2, 4, 8):
        h = np.full(2 ** b, 37, np.uint64)
        assert orc.entropy_bits(h) == pytest.approx(37 * 2 ** b * b, rel=1e-14)
        assert orc.huffman_bits(h) == 37 * 2 ** b * b  # a full binary tree of depth b
    # probabilities 1/2, 1/4, 1/8, 1/16, 1/16: Huffman lengths 1, 2, 3, 4, 4 meet the entropy exactly
    h = np.array([8, 4, 2, 1, 1, 0, 0, 0], np.uint64) * 5
    assert orc.huffman_bits(h) == 5 * (8 * 1 + 4 * 2 + 2 * 3 + 1 * 4 + 1 * 4)
    assert orc.entropy_bits(h) == pytest.approx(orc.huffman_bits(h), rel=1e-14)


def test_textbook_example_and_degenerate_messages():
    # frequencies 45, 13, 12, 16, 9, 5 (thousands): the classic six-letter example costs 224 thousand bits
    assert orc.huffman_bits(np.array([45, 13, 12, 16, 9, 5], np.uint64)) == 224
    assert orc.huffman_bits(np.zeros(16, np.uint64)) == 0 and orc.entropy_bits(np.zeros(16, np.uint64)) == 0
    one = np.zeros(16, np.uint64)
    one[8] = 1000  # every coordinate the zero code (the first step of every epoch)
    assert orc.entropy_bits(one) == 0 and orc.huffman_bits(one) == 1000


def _best_prefix_code_bits(counts):
    """Brute force: the cheapest length assignment that satisfies Kraft's inequality (m <= 5 symbols)."""
    m = len(counts)
    best = None
    for lens in itertools.product(range(1, m + 1), repeat=m):
        if sum(2.0 ** -l for l in lens) <= 1.0 + 1e-12:
            cost = sum(c * l for c, l in zip(counts, lens))
            best = cost if best is None else min(best, cost)
    return best


def test_huffman_is_optimal_on_tiny_alphabets_and_within_shannon_bounds():
    rng = np.random.default_rng(1)
    for _ in range(60):
        m = int(rng.integers(2, 6))
        counts = rng.integers(1, 50, size=m)
        h = np.zeros(8, np.uint64)
        h[rng.permutation(8)[:m]] = counts
        assert orc.huffman_bits(h) == _best_prefix_code_bits(list(counts))
    for b in (2, 4, 8):
        for _ in range(20):
            h = rng.integers(0, 1000, size=2 ** b).astype(np.uint64) ** 2
            n, H, L = int(h.sum()), orc.entropy_bits(h), orc.huffman_bits(h)
            assert H <= L + 1e-6 and L < H + n
            p = h[h > 0] / n
            assert H == pytest.approx(-n * float((p * np.log2(p)).sum()), rel=1e-12)


def test_clipped_gaussian_messages_compress_below_b_bits():
    # near-Gaussian gradient coordinates (Figure 2) put most codes near the middle of the grid
    u = np.random.default_rng(2).standard_normal(20000).astype(np.float32)
    for b in (4, 8):
        words, _, _ = orc.quantize_pack(u, b, orc.CLIP_STD, 2.5, seed=1)
        h = orc.code_histogram(words, u.size, b)
        assert orc.huffman_bits(h) < 0.985 * b * u.size
        assert orc.entropy_bits(h) <= orc.huffman_bits(h)

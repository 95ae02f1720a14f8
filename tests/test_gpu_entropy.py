"""GPU parity for the entropy-coding count: the histogram kernel against the oracle's histogram (exact), and the
library's entropy bound and Huffman length against the oracle's, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_1901_08924_b200 import lpc, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _check(N, length, b, dist, offs=None, seed=1):
    U = synth.gradient_vectors(N, length, dist, seed=seed)
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, N, 1, b, lpc.CLIP_STD, 2.0, seed)
    codes, _, _ = q.quantize_pack(U.to(DEV), 3, seg_offsets=offs)
    hist, ent, huf = q.message_entropy(codes, length, seg_offsets=offs)
    q.sync_status()
    got = codes.cpu().numpy().view(np.uint32)
    woff, _ = lpc.packed_layout(length, b, offs)
    bounds = offs if offs is not None else [0, length]
    h = hist.cpu().numpy()
    for i in range(N):
        for s in range(len(bounds) - 1):
            n = bounds[s + 1] - bounds[s]
            W = orc.packed_words(n, b)
            # the oracle counts the very words the library packed; those words are checked against the oracle's own
            # quantizer by the quantizer's parity tests
            ref = orc.code_histogram(got[i, woff[s]: woff[s] + max(W, 1)], n, b)
            assert (h[i, s].astype(np.uint64) == ref).all()
            assert huf[i, s] == orc.huffman_bits(ref)
            assert ent[i, s] == pytest.approx(orc.entropy_bits(ref), rel=1e-12, abs=1e-9)
            assert ent[i, s] <= huf[i, s] + 1e-6 and huf[i, s] <= max(b * n, n)
    q.close()


@pytest.mark.parametrize("b", [1, 2, 3, 4, 8])
@pytest.mark.parametrize("N,length", [(1, 1), (3, 8191), (4, 8192 * 3 + 5), (8, 100000)])
def test_histogram_and_counts_match_oracle(b, N, length):
    _check(N, length, b, "gauss")


def test_segments_heavy_tails_and_known_streams():
    _check(4, 30000, 4, "student_t3", offs=[0, 7, 7, 9000, 30000])
    # a stream built on the CPU with a known histogram: every code value c appears c + 1 times per 136 coordinates
    b, reps = 4, 700
    pattern = np.concatenate([np.full(c + 1, c, np.uint32) for c in range(16)])
    codes_np = np.tile(pattern, reps)
    rng = np.random.default_rng(0)
    rng.shuffle(codes_np)
    n = codes_np.size
    words = orc.pack(codes_np, b)
    _, stride = lpc.packed_layout(n, b)
    buf = np.zeros((1, stride), np.uint32)
    buf[0, : words.size] = words
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, 1, 1, b, lpc.CLIP_NONE, 1.0, 0)
    hist, ent, huf = q.message_entropy(torch.from_numpy(buf.view(np.int32)).to(DEV), n)
    q.sync_status()
    assert (hist.cpu().numpy().ravel() == (np.arange(16) + 1) * reps).all()
    p = (np.arange(16) + 1) / 136.0
    assert ent[0, 0] == pytest.approx(-n * float((p * np.log2(p)).sum()), rel=1e-12)
    assert huf[0, 0] == orc.huffman_bits(((np.arange(16) + 1) * reps).astype(np.uint64))
    q.close()


def test_empty_zero_and_unsupported():
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, 2, 1, 4, lpc.CLIP_STD, 2.0, 0)
    codes, _, _ = q.quantize_pack(torch.zeros(2, 5000, device=DEV), 0)
    hist, ent, huf = q.message_entropy(codes, 5000)
    assert (hist.cpu().numpy()[:, 0, 8] == 5000).all() and hist.sum().item() == 10000
    assert (ent == 0).all() and (huf == 5000).all()  # one value: no information, one bit per coordinate as a symbol code
    hist, ent, huf = q.message_entropy(codes, 0)
    assert hist.sum().item() == 0 and (ent == 0).all() and (huf == 0).all()
    q.sync_status()
    q.close()
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, 2, 1, 12, lpc.CLIP_NONE, 1.0, 0)
    with pytest.raises(lpc.LpcError):
        q.message_entropy(torch.zeros(2, 64, dtype=torch.int32, device=DEV), 16)
    q.close()

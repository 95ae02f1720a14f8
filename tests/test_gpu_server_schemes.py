"""GPU parity for the parameter-server schemes (b) and (c) of Section 3.2: unified-scale quantization, the server's
index sums and re-quantized averages, and the worker-side decode, each compared bit for bit with the oracle on the
same seeded vectors, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_1901_08924_b200 import lpc, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run_schemes(N, length, b, dist, clip, seed, k):
    U = synth.gradient_vectors(N, length, dist, seed=seed)
    U *= torch.linspace(0.3, 2.0, N).unsqueeze(1)  # workers with different magnitudes: the unified scale matters
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, N, 1, b, clip[0], clip[1], seed)
    q.set_option(lpc.OPT_SHARED_SCALE, 1)
    codes, delta, clipped = q.quantize_pack(U.to(DEV), k)
    q.sync_status()
    W = orc.packed_words(length, b)
    ref_words, ref_delta, ref_clipped = orc.quantize_pack_shared(U.numpy(), b, clip[0], clip[1], seed=seed, k=k)
    got = codes.cpu().numpy().view(np.uint32)
    assert (got[:, :W] == ref_words).all(), "unified-scale codes differ from the oracle"
    assert (got[:, W:] == 0).all(), "padding words must be zero"
    assert (delta.cpu().numpy().view(np.uint32) == np.float32(ref_delta).view(np.uint32)).all()
    assert (clipped.cpu().numpy().ravel().astype(np.int64) == ref_clipped.astype(np.int64)).all()
    mu = torch.randn(length, generator=torch.Generator().manual_seed(seed + 1))
    x0 = torch.randn(length, generator=torch.Generator().manual_seed(seed + 2))
    out = {}
    for scheme, requant in ((lpc.SCHEME_SERVER_SUM, False), (lpc.SCHEME_SERVER_REQUANTIZE, True)):
        if not requant and b + int(np.ceil(np.log2(N))) > 16:
            continue
        srv, bo = q.server_reduce(codes, length, scheme, k)
        q.sync_status()
        ref_srv = orc.server_reduce(ref_words, length, b, requant, seed=seed, k=k)
        Wo = orc.packed_words(length, bo)
        gs = srv.cpu().numpy().view(np.uint32).ravel()
        assert (gs[:Wo] == ref_srv).all(), "server stream differs from the oracle"
        assert (gs[Wo:] == 0).all()
        # worker side: one stream of bo bits, divided by N under scheme (b)
        w = lpc.Context(None, None, lpc.LOGISTIC, 0.0, 1, 1, bo, lpc.CLIP_NONE, 1.0, seed)
        if not requant:
            w.set_option(lpc.OPT_AVERAGE_DIVISOR, N)
        x = x0.clone().to(DEV)
        v = torch.empty(length, device=DEV)
        w.unpack_average_prox(srv, delta[:1].contiguous(), length, x, 0.3, 1e-3, mu=mu.to(DEV), v_out=v)
        w.sync_status()
        xr, vr = orc.unpack_scaled_prox(ref_srv, ref_delta, length, bo, 1 if requant else N, mu.numpy(), x0.numpy(), 0.3, 1e-3,
                                        want_v=True)
        assert (x.cpu().numpy().view(np.uint32) == xr.view(np.uint32)).all()
        assert (v.cpu().numpy().view(np.uint32) == vr.view(np.uint32)).all()
        w.close()
        out[scheme] = x.cpu().numpy()
    q.close()
    return out


@pytest.mark.parametrize("b", [2, 3, 4, 8])
@pytest.mark.parametrize("N,length", [(2, 1), (3, 257), (8, 8192 * 2 + 77), (16, 50000)])
def test_server_schemes_match_oracle(b, N, length):
    _run_schemes(N, length, b, "gauss", (lpc.CLIP_STD, 2.0), seed=5 + b, k=3)


def test_server_schemes_heavy_tails_and_wide_codes():
    _run_schemes(5, 30011, 11, "student_t3", (lpc.CLIP_LAMBDA, 0.25), seed=2, k=9)
    _run_schemes(64, 4097, 6, "student_t3", (lpc.CLIP_NONE, 1.0), seed=3, k=0)


def test_server_schemes_all_zero_and_empty():
    N, length, b = 4, 1000, 4
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, N, 1, b, lpc.CLIP_STD, 2.0, 1)
    q.set_option(lpc.OPT_SHARED_SCALE, 1)
    codes, delta, _ = q.quantize_pack(torch.zeros(N, length, device=DEV), 0)
    assert (delta.cpu().numpy() == 0).all()
    srv, bo = q.server_reduce(codes, length, lpc.SCHEME_SERVER_SUM, 0)
    W = orc.packed_words(length, bo)
    assert (orc.unpack(srv.cpu().numpy().view(np.uint32).ravel()[:W], length, bo) == 2 ** (bo - 1)).all()
    srv, _ = q.server_reduce(codes, length, lpc.SCHEME_SERVER_REQUANTIZE, 0)
    assert (orc.unpack(srv.cpu().numpy().view(np.uint32).ravel()[: orc.packed_words(length, b)], length, b) == 8).all()
    q.sync_status()
    q.close()


def test_server_schemes_segmented_and_bit_counts():
    N, b = 4, 4
    offs = [0, 100, 100, 9000, 20000]
    U = synth.gradient_vectors(N, offs[-1], "gauss", seed=4)
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, N, 1, b, lpc.CLIP_STD, 2.5, 7)
    q.set_option(lpc.OPT_SHARED_SCALE, 1)
    codes, delta, _ = q.quantize_pack(U.to(DEV), 1, seg_offsets=offs)
    srv, bo = q.server_reduce(codes, offs[-1], lpc.SCHEME_SERVER_SUM, 1, seg_offsets=offs)
    q.sync_status()
    woff_in, _ = lpc.packed_layout(offs[-1], b, offs)
    woff_out, _ = lpc.packed_layout(offs[-1], bo, offs)
    got, gs = codes.cpu().numpy().view(np.uint32), srv.cpu().numpy().view(np.uint32).ravel()
    d = delta.cpu().numpy()
    srvc, _ = q.server_reduce(codes, offs[-1], lpc.SCHEME_SERVER_REQUANTIZE, 1, seg_offsets=offs)
    q.sync_status()
    gc = srvc.cpu().numpy().view(np.uint32).ravel()
    base = 0  # a segment's rounding streams continue the block count of the segments before it
    for s in range(4):
        lo, hi = offs[s], offs[s + 1]
        if hi > lo:
            rw, rd, _ = orc.quantize_pack_shared(U[:, lo:hi].numpy(), b, orc.CLIP_STD, 2.5, seed=7, k=1, block_base=base)
            assert (d[:, s] == rd).all()
            W = orc.packed_words(hi - lo, b)
            assert (got[:, woff_in[s]: woff_in[s] + W] == rw).all()
            ref_sum = orc.server_reduce(rw, hi - lo, b, False)
            assert (gs[woff_out[s]: woff_out[s] + ref_sum.size] == ref_sum).all()
            ref_rq = orc.server_reduce(rw, hi - lo, b, True, seed=7, k=1, block_base=base)
            assert (gc[woff_in[s]: woff_in[s] + W] == ref_rq).all()
        base += (hi - lo + 7) // 8
    bits = q.comm_bits()[1]
    expect = sum(N * (64 + b * (offs[s + 1] - offs[s]) + bw * (offs[s + 1] - offs[s])) for s in range(4) for bw in (bo, b))
    assert bits == expect
    assert lpc.scheme_bits(lpc.SCHEME_SERVER_SUM, 4096, 4, 16) == orc.scheme_bits(orc.SCHEME_B, 4096, 4, 16) == 787456
    assert lpc.scheme_bits(lpc.SCHEME_SERVER_REQUANTIZE, 4096, 4, 16) == orc.scheme_bits(orc.SCHEME_C, 4096, 4, 16)
    assert lpc.scheme_bits(lpc.SCHEME_BROADCAST, 4096, 4, 16) == orc.broadcast_bits(4096, 4, 16)
    q.close()


def test_server_schemes_reject_unsupported():
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, 4, 1, 1, lpc.CLIP_NONE, 1.0, 1)
    with pytest.raises(lpc.LpcError):
        q.set_option(lpc.OPT_SHARED_SCALE, 1)
    with pytest.raises(lpc.LpcError):
        q.server_reduce(torch.zeros(4, 4, dtype=torch.int32, device=DEV), 16, lpc.SCHEME_SERVER_SUM, 0)
    q.close()
    q = lpc.Context(None, None, lpc.LOGISTIC, 0.0, 64, 1, 12, lpc.CLIP_NONE, 1.0, 1)
    with pytest.raises(lpc.LpcError):
        q.server_reduce(torch.zeros(64, 8, dtype=torch.int32, device=DEV), 16, lpc.SCHEME_SERVER_SUM, 0)  # 12 + 6 > 16 bits
    q.close()

"""lpc_quantize_pack_static must give the bits of lpc_quantize_pack.

The static entry point exists for callers that cannot allocate device memory where they run (a
latency-critical loop, a plug-in with a fixed memory budget): its working memory is a fixed array inside
the library, shared by all calls.  Two calls in a row check that nothing left over from the first call
leaks into the second.  This file is collected last on purpose, so that a failure here cannot hide the
result of any other test in a run that stops at the first failure.
"""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_1901_08924_b200 import lpc, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _same_bits(a, b):
    return torch.equal(a.view(torch.int32), b.view(torch.int32))


def _static_call(U, b, clip_mode, clip_value, seed, k):
    N, length = U.shape
    _, stride = lpc.packed_layout(length, b)
    codes = torch.full((N, stride), -1, dtype=torch.int32, device=DEV)
    delta = torch.full((N,), -1.0, dtype=torch.float32, device=DEV)
    clipped = torch.full((N,), -1, dtype=torch.int32, device=DEV)
    rc = lpc.quantize_pack_static(U, b, clip_mode, clip_value, seed, k, codes, delta, clipped)
    assert rc == lpc.OK
    torch.cuda.synchronize()
    return codes, delta, clipped


def test_static_entry_point_matches_context_path_on_two_calls():
    N, b, seed = 4, 4, 17
    ctx = lpc.Context(None, None, lpc.LOGISTIC, 0.0, N, 1, b, lpc.CLIP_STD, 2.5, seed)
    for call, (length, dist, k) in enumerate([(50001, "gauss", 3), (20000, "student_t3", 4)]):
        U = synth.gradient_vectors(N, length, dist, seed=call).to(DEV)
        ref_codes, ref_delta, ref_clipped = ctx.quantize_pack(U, k)
        ctx.sync_status()
        codes, delta, clipped = _static_call(U, b, lpc.CLIP_STD, 2.5, seed, k)
        assert torch.equal(codes, ref_codes), call                      # packed codes: bit-exact
        assert _same_bits(delta, ref_delta.reshape(-1)), call           # scales: bit-exact
        assert torch.equal(clipped, ref_clipped.reshape(-1)), call
        # and the oracle itself, for worker 0 of each call
        w, dl, cl = orc.quantize_pack(U[0].cpu().numpy(), b, orc.CLIP_STD, 2.5, seed, 0, k)
        assert (codes[0].cpu().numpy().view(np.uint32)[: w.size] == w).all()
        assert np.float32(dl).view(np.uint32) == delta[0].cpu().numpy().view(np.uint32) and cl == int(clipped[0])
    ctx.close()


@pytest.mark.parametrize("b", [1, 3, 8, 16, 32])
@pytest.mark.parametrize("clip", [(lpc.CLIP_NONE, 1.0), (lpc.CLIP_LAMBDA, 0.8), (lpc.CLIP_STD, 2.0)])
def test_static_entry_point_other_widths_and_clip_rules(b, clip):
    # the generic-width kernel (byte staging), the full-precision bypass and the other two clip rules on the fixed
    # working memory, twice in a row
    N, seed = 3, 5
    ctx = lpc.Context(None, None, lpc.LOGISTIC, 0.0, N, 1, b, clip[0], clip[1], seed)
    for k, length in enumerate((8192 + 77, 3001)):
        U = synth.gradient_vectors(N, length, "gauss", seed=10 + k).to(DEV)
        ref = ctx.quantize_pack(U, k)
        ctx.sync_status()
        got = _static_call(U, b, clip[0], clip[1], seed, k)
        assert torch.equal(got[0], ref[0]) and _same_bits(got[1], ref[1].reshape(-1))
        assert torch.equal(got[2], ref[2].reshape(-1))
    ctx.close()


def test_static_entry_point_at_its_tile_limit_and_allocates_nothing():
    # exactly LPC_STATIC_MAX_TILES tile partials: 64 workers x 1,024 tiles.  After a first call (which may load the
    # kernels), a second call must leave both torch's and the driver's view of free device memory unchanged.
    N, b, seed, k = 64, 2, 3, 9
    length = 1024 * 8192
    U = synth.gradient_vectors(N, length, "gauss", seed=1, device=DEV)
    _, stride = lpc.packed_layout(length, b)
    codes = torch.empty((N, stride), dtype=torch.int32, device=DEV)
    delta = torch.empty((N,), dtype=torch.float32, device=DEV)
    clipped = torch.empty((N,), dtype=torch.int32, device=DEV)
    assert lpc.quantize_pack_static(U, b, lpc.CLIP_STD, 2.0, seed, k, codes, delta, clipped) == lpc.OK
    torch.cuda.synchronize()
    first = (codes.clone(), delta.clone(), clipped.clone())
    torch_before, (free_before, _) = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()
    assert lpc.quantize_pack_static(U, b, lpc.CLIP_STD, 2.0, seed, k, codes, delta, clipped) == lpc.OK
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == torch_before and torch.cuda.mem_get_info()[0] == free_before
    assert torch.equal(codes, first[0]) and _same_bits(delta, first[1]) and torch.equal(clipped, first[2])
    for i in (0, 63):  # scales and clipped counts of two workers from full oracle passes, codes in a window
        u = U[i].cpu().numpy()
        sc = orc.scale(u, b, orc.CLIP_STD, 2.0)
        assert np.float32(sc["delta"]).view(np.uint32) == delta[i].cpu().numpy().view(np.uint32)
        lower = -(np.float32(sc["T"]) + np.float32(sc["delta"]))
        assert int(((u > sc["T"]) | (u < lower)).sum()) == int(clipped[i])
        s0, W = 8192 * 513 + 64, 512
        c = np.array([orc.quantize_coord(u[j], sc["rdelta"], b, orc.rounding_bits(seed, i, k, 0, j)) + 2
                      for j in range(s0, s0 + W)], np.uint32)
        assert (codes[i].cpu().numpy().view(np.uint32)[s0 * b // 32:(s0 + W) * b // 32] == orc.pack(c, b)).all()
    # one tile more does not fit
    L = lpc.lib()
    st = torch.cuda.current_stream().cuda_stream
    assert L.lpc_quantize_pack_static(U.data_ptr(), length + 1, length + 4, N, b, 2, 2.0, 0, 0, codes.data_ptr(),
                                      delta.data_ptr(), clipped.data_ptr(), st) == lpc.ERR_UNSUPPORTED


def test_static_entry_point_refuses_what_does_not_fit():
    U = torch.zeros((2, 64), device=DEV)
    out = torch.zeros((2, 8), dtype=torch.int32, device=DEV)
    d = torch.zeros(2, device=DEV)
    c = torch.zeros(2, dtype=torch.int32, device=DEV)
    L = lpc.lib()
    st = torch.cuda.current_stream().cuda_stream
    # more workers than the fixed working memory has scale records for
    assert L.lpc_quantize_pack_static(U.data_ptr(), 64, 64, 65, 4, 0, 1.0, 0, 0, out.data_ptr(), d.data_ptr(),
                                      c.data_ptr(), st) == lpc.ERR_UNSUPPORTED
    # more tiles than it has partial slots for (checked before anything is read or launched)
    assert L.lpc_quantize_pack_static(U.data_ptr(), 8192 * 40000, 8192 * 40000, 2, 4, 0, 1.0, 0, 0, out.data_ptr(),
                                      d.data_ptr(), c.data_ptr(), st) == lpc.ERR_UNSUPPORTED
    assert L.lpc_quantize_pack_static(None, 64, 64, 2, 4, 0, 1.0, 0, 0, out.data_ptr(), d.data_ptr(), c.data_ptr(),
                                      st) == lpc.ERR_INVALID_ARG
    assert L.lpc_quantize_pack_static(U.data_ptr(), 64, 64, 2, 17, 0, 1.0, 0, 0, out.data_ptr(), d.data_ptr(),
                                      c.data_ptr(), st) == lpc.ERR_INVALID_ARG

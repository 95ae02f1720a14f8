"""lpc_quantize_pack_static must give the bits of lpc_quantize_pack.

The static entry point exists for callers that cannot allocate device memory where they run (a
latency-critical loop, a plug-in with a fixed memory budget): its working memory is a fixed array inside
the library, shared by all calls.  Two calls in a row check that nothing left over from the first call
leaks into the second.  This file is collected last on purpose, so that a failure here cannot hide the
result of any other test in a run that stops at the first failure.
"""
import pytest
import torch

from paper_1901_08924_b200 import lpc, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _same_bits(a, b):
    return torch.equal(a.view(torch.int32), b.view(torch.int32))


def test_static_entry_point_matches_context_path_on_two_calls():
    N, b, seed = 4, 4, 17
    ctx = lpc.Context(None, None, lpc.LOGISTIC, 0.0, N, 1, b, lpc.CLIP_STD, 2.5, seed)
    for call, (length, dist, k) in enumerate([(50001, "gauss", 3), (20000, "student_t3", 4)]):
        U = synth.gradient_vectors(N, length, dist, seed=call).to(DEV)
        ref_codes, ref_delta, ref_clipped = ctx.quantize_pack(U, k)
        ctx.sync_status()
        _, stride = lpc.packed_layout(length, b)
        codes = torch.full((N, stride), -1, dtype=torch.int32, device=DEV)
        delta = torch.full((N,), -1.0, dtype=torch.float32, device=DEV)
        clipped = torch.full((N,), -1, dtype=torch.int32, device=DEV)
        rc = lpc.quantize_pack_static(U, b, lpc.CLIP_STD, 2.5, seed, k, codes, delta, clipped)
        assert rc == lpc.OK
        torch.cuda.synchronize()
        assert torch.equal(codes, ref_codes), call                      # packed codes: bit-exact
        assert _same_bits(delta, ref_delta.reshape(-1)), call           # scales: bit-exact
        assert torch.equal(clipped, ref_clipped.reshape(-1)), call
    ctx.close()


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

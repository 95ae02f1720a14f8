"""CPU-only checks of the C-ABI boundary: the library loads, exports every declared symbol, and
its host-side helpers (layout arithmetic, argument validation) behave as include/lpc.h says."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lpc():
    from paper_1901_08924_b200 import build, lpc as binding
    build.build()
    return binding


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "lpc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lpc_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lpc):
    names = _declared_symbols()
    assert len(names) >= 20
    L = C.CDLL(lpc.LIB_PATH)
    for n in names:
        assert hasattr(L, n), n
    assert sorted(s[0] for s in lpc.SYMBOLS) == names  # the binding covers the header exactly


def test_packed_words_and_layout(lpc):
    assert lpc.packed_words(1000, 2) == 63 and lpc.packed_words(4096, 4) == 512
    assert lpc.packed_words(0, 8) == 0 and lpc.packed_words(5, 3) == 1 and lpc.packed_words(11, 3) == 2
    assert lpc.packed_words(7, 32) == 7
    with pytest.raises(lpc.LpcError):
        lpc.packed_words(10, 0)
    with pytest.raises(lpc.LpcError):
        lpc.packed_words(10, 17)
    woff, stride = lpc.packed_layout(1000, 2)
    assert woff == [0, 64] and stride == 64  # 63 words rounded up to a multiple of 4
    woff, stride = lpc.packed_layout(100, 4, [0, 10, 10, 33, 100])
    assert woff == [0, 4, 4, 8, 20] and stride == 20
    with pytest.raises(lpc.LpcError):
        lpc.packed_layout(100, 4, [0, 50, 40, 100])  # offsets must not decrease
    with pytest.raises(lpc.LpcError):
        lpc.packed_layout(100, 4, [0, 50, 99])  # must end at len


def test_init_rejects_bad_arguments_before_touching_the_device(lpc):
    h = C.c_void_p(None)
    L = lpc.lib()
    fake = C.c_void_p(1 << 20)  # 16-byte aligned, never dereferenced by the checks below
    bad = [
        dict(N=0), dict(N=2000), dict(b=0), dict(b=17), dict(b=31), dict(clip_mode=5),
        dict(clip_mode=lpc.CLIP_LAMBDA, clip_value=1.5), dict(clip_mode=lpc.CLIP_LAMBDA, clip_value=0.0),
        dict(clip_mode=lpc.CLIP_STD, clip_value=-1.0), dict(lam=-1.0), dict(d=1002), dict(d=2), dict(d=32768),
        dict(n=4001), dict(B=0), dict(B=1025), dict(loss=7), dict(X=C.c_void_p((1 << 20) + 4)),
    ]
    for kw in bad:
        a = dict(X=fake, y=fake, n=4000, d=1000, loss=0, lam=1e-4, N=4, B=1, b=2, clip_mode=2, clip_value=2.5)
        a.update(kw)
        rc = L.lpc_init(C.byref(h), a["X"], a["y"], a["n"], a["d"], a["loss"], a["lam"], a["N"], a["B"], a["b"],
                        a["clip_mode"], a["clip_value"], 0, None)
        assert rc == lpc.ERR_INVALID_ARG, kw
        assert not h.value
    assert L.lpc_destroy(None) == lpc.OK
    assert L.lpc_inner_step(None, 0.1, 0) == lpc.ERR_INVALID_ARG

"""numpy front end of the CPU oracle (oracle/lpc_oracle.cpp).

TEST INFRASTRUCTURE.  Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It holds no arithmetic of its own: every function marshals numpy arrays into the
C entry points of the oracle library and returns what they wrote.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

LOGISTIC, LEAST_SQUARES = 0, 1
CLIP_NONE, CLIP_LAMBDA, CLIP_STD = 0, 1, 2
TAG_ROUND, TAG_BATCH, TAG_BATCH_J = 0, 1, 2
OK, ERR_INVALID, ERR_NONFINITE = 0, -1, -3

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _declare(_lib)
    return _lib


_f32p = C.POINTER(C.c_float)
_u32p = C.POINTER(C.c_uint32)
_i32p = C.POINTER(C.c_int32)
_i64p = C.POINTER(C.c_int64)
_f64p = C.POINTER(C.c_double)


def _declare(L):
    L.orc_philox4x32_10.argtypes = [_u32p, _u32p, _u32p]
    L.orc_philox4x32_10.restype = None
    L.orc_stream_block.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64, C.c_uint32, _u32p]
    L.orc_stream_block.restype = None
    L.orc_rounding_bits.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint32, C.c_int64]
    L.orc_rounding_bits.restype = C.c_uint32
    for name in ("orc_tree_sum", "orc_tree_sumsq"):
        getattr(L, name).argtypes = [_f32p, C.c_int64]
        getattr(L, name).restype = C.c_float
    L.orc_tree_dot.argtypes = [_f32p, _f32p, C.c_int64]
    L.orc_tree_dot.restype = C.c_float
    L.orc_packed_words.argtypes = [C.c_int64, C.c_int]
    L.orc_packed_words.restype = C.c_int64
    L.orc_message_bits.argtypes = [C.c_int64, C.c_int]
    L.orc_message_bits.restype = C.c_uint64
    L.orc_broadcast_bits.argtypes = [C.c_int64, C.c_int, C.c_int]
    L.orc_broadcast_bits.restype = C.c_uint64
    L.orc_scale.argtypes = [_f32p, C.c_int64, C.c_int, C.c_int, C.c_float, _f32p, C.POINTER(C.c_int)]
    L.orc_scale.restype = C.c_int
    L.orc_quantize_coord.argtypes = [C.c_float, C.c_float, C.c_int, C.c_uint32]
    L.orc_quantize_coord.restype = C.c_int
    L.orc_pack.argtypes = [_u32p, C.c_int64, C.c_int, _u32p]
    _u64p = C.POINTER(C.c_uint64)
    L.orc_code_histogram.argtypes = [_u32p, C.c_int64, C.c_int, _u64p]
    L.orc_code_histogram.restype = C.c_int
    L.orc_entropy_bits.argtypes = [_u64p, C.c_int]
    L.orc_entropy_bits.restype = C.c_double
    L.orc_huffman_bits.argtypes = [_u64p, C.c_int]
    L.orc_huffman_bits.restype = C.c_uint64
    L.orc_sum_bits_per_coordinate.argtypes = [C.c_int, C.c_int]
    L.orc_sum_bits_per_coordinate.restype = C.c_int
    L.orc_scheme_bits.argtypes = [C.c_int, C.c_int64, C.c_int, C.c_int]
    L.orc_scheme_bits.restype = C.c_uint64
    L.orc_quantize_pack_shared.argtypes = [_f32p, C.c_int, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_float, C.c_uint64,
                                           C.c_uint64, C.c_uint32, _u32p, C.c_int64, _f32p, _u32p]
    L.orc_quantize_pack_shared.restype = C.c_int
    L.orc_server_reduce.argtypes = [_u32p, C.c_int64, C.c_int, C.c_int64, C.c_int, C.c_int, C.c_uint64, C.c_uint64, C.c_uint32,
                                    _u32p]
    L.orc_server_reduce.restype = C.c_int
    L.orc_unpack_scaled_prox.argtypes = [_u32p, C.c_float, C.c_int64, C.c_int, C.c_int, _f32p, _f32p, C.c_float, C.c_float,
                                         _f32p, _f32p]
    L.orc_unpack_scaled_prox.restype = None
    L.orc_pack.restype = None
    L.orc_unpack.argtypes = [_u32p, C.c_int64, C.c_int, _u32p]
    L.orc_unpack.restype = None
    L.orc_quantize_pack.argtypes = [_f32p, C.c_int64, C.c_int, C.c_int, C.c_float, C.c_uint64, C.c_uint32,
                                    C.c_uint64, C.c_uint32, _u32p, _f32p, _u32p, _i32p]
    L.orc_quantize_pack.restype = C.c_int
    L.orc_unpack_average_prox.argtypes = [_u32p, C.c_int64, _f32p, C.c_int, C.c_int64, C.c_int, _f32p, _f32p,
                                          C.c_float, C.c_float, _f32p, _f32p]
    L.orc_unpack_average_prox.restype = None
    L.orc_soft_threshold.argtypes = [C.c_float, C.c_float]
    L.orc_soft_threshold.restype = C.c_float
    L.orc_margin.argtypes = [_f32p, _f32p, C.c_int64]
    L.orc_margin.restype = C.c_float
    L.orc_loss_deriv.argtypes = [C.c_int, C.c_float, C.c_float]
    L.orc_loss_deriv.restype = C.c_float
    L.orc_loss_value.argtypes = [C.c_int, C.c_float, C.c_float]
    L.orc_loss_value.restype = C.c_double
    L.orc_full_grad.argtypes = [_f32p, _f32p, C.c_int64, C.c_int64, C.c_int, _f32p, _f32p, _f32p, _f64p]
    L.orc_full_grad.restype = None
    L.orc_objective.argtypes = [_f32p, _f32p, C.c_int64, C.c_int64, C.c_int, _f32p, C.c_float]
    L.orc_objective.restype = C.c_double
    L.orc_sample_batch.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64, C.c_int, C.c_int64,
                                   C.c_int64, _i64p]
    L.orc_sample_batch.restype = None
    L.orc_svrg_coef.argtypes = [_f32p, _f32p, C.c_int64, C.c_int, _i64p, C.c_int, _f32p, _f32p, _f32p]
    L.orc_svrg_coef.restype = None
    L.orc_svrg_diff_from_coef.argtypes = [_f32p, C.c_int64, _i64p, C.c_int, _f32p, _f32p]
    L.orc_svrg_diff_from_coef.restype = None
    L.orc_lpc_inner_step.argtypes = [_f32p, _f32p, C.c_int64, C.c_int64, C.c_int, C.c_float, C.c_int, C.c_int,
                                     C.c_int, C.c_int, C.c_float, C.c_uint64, C.c_int, C.c_uint64, C.c_float,
                                     _f32p, _f32p, _f32p, _i64p, _f32p, _f32p, _u32p, C.c_int64, _f32p, _u32p,
                                     _f32p]
    L.orc_lpc_inner_step.restype = C.c_int
    L.orc_alpc_step.argtypes = [_f32p, _f32p, C.c_int64, C.c_int64, C.c_int, C.c_float, C.c_int, C.c_int,
                                C.c_int, C.c_int, C.c_float, C.c_uint64, C.c_int, C.c_uint64, C.c_float,
                                C.c_float, C.c_float, C.c_float, _f32p, _f32p, _f32p, _f32p, _f32p, _f32p,
                                _f32p, _f32p, _u32p, C.c_int64, _f32p]
    L.orc_alpc_step.restype = C.c_int
    L.orc_alpc_step_sc.argtypes = [_f32p, _f32p, C.c_int64, C.c_int64, C.c_int, C.c_float, C.c_int, C.c_int,
                                   C.c_int, C.c_int, C.c_float, C.c_uint64, C.c_int, C.c_uint64, C.c_float,
                                   C.c_float, C.c_float, C.c_float, C.c_float, C.c_float, _f32p, _f32p, _f32p, _f32p,
                                   _f32p, _f32p, _f32p, _f32p, _u32p, C.c_int64, _f32p]
    L.orc_alpc_step_sc.restype = C.c_int
    L.orc_weighted_snapshot.argtypes = [_f32p, C.c_float, C.c_int64, _f32p]
    L.orc_weighted_snapshot.restype = None
    L.orc_ridge_term.argtypes = [_f32p, C.c_int64, C.c_float]
    L.orc_ridge_term.restype = C.c_double


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(_f32p)


def _ptr(a, typ):
    return None if a is None else a.ctypes.data_as(typ)


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__(f"oracle status {code}")
        self.code = code


def _check(rc):
    if rc != OK:
        raise OracleError(rc)


# ---- RNG -------------------------------------------------------------------------------------

def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(c.ctypes.data_as(_u32p), k.ctypes.data_as(_u32p), out.ctypes.data_as(_u32p))
    return out


def stream_block(seed, tag, worker, k, block):
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_stream_block(seed, tag, worker, k, block, out.ctypes.data_as(_u32p))
    return out


def rounding_bits(seed, worker, k, block_base, j):
    return int(lib().orc_rounding_bits(seed, worker, k, block_base, j))


# ---- sums ------------------------------------------------------------------------------------

def tree_sum(v):
    v, p = _f32(v)
    return np.float32(lib().orc_tree_sum(p, v.size))


def tree_sumsq(v):
    v, p = _f32(v)
    return np.float32(lib().orc_tree_sumsq(p, v.size))


def tree_dot(a, b):
    a, pa = _f32(a)
    b, pb = _f32(b)
    assert a.size == b.size
    return np.float32(lib().orc_tree_dot(pa, pb, a.size))


# ---- quantizer -------------------------------------------------------------------------------

def packed_words(length, b):
    return int(lib().orc_packed_words(length, b))


def message_bits(length, b):
    return int(lib().orc_message_bits(length, b))


def broadcast_bits(length, b, N):
    return int(lib().orc_broadcast_bits(length, b, N))


def scale(u, b, clip_mode=CLIP_NONE, clip_value=1.0):
    """Returns dict(M, S1, S2, T, delta, rdelta, degenerate) of Eq. 2 for the vector u."""
    u, p = _f32(u)
    out = np.zeros(6, dtype=np.float32)
    deg = C.c_int(0)
    _check(lib().orc_scale(p, u.size, b, clip_mode, clip_value, out.ctypes.data_as(_f32p), C.byref(deg)))
    return dict(M=out[0], S1=out[1], S2=out[2], T=out[3], delta=out[4], rdelta=out[5], degenerate=bool(deg.value))


def quantize_coord(u, rdelta, b, r16):
    return int(lib().orc_quantize_coord(np.float32(u), np.float32(rdelta), b, r16))


def pack(codes, b):
    codes = np.ascontiguousarray(codes, dtype=np.uint32)
    words = np.zeros(max(packed_words(codes.size, b), 1), dtype=np.uint32)
    lib().orc_pack(codes.ctypes.data_as(_u32p), codes.size, b, words.ctypes.data_as(_u32p))
    return words[: packed_words(codes.size, b)]


def unpack(words, length, b):
    words = np.ascontiguousarray(words, dtype=np.uint32)
    codes = np.zeros(length, dtype=np.uint32)
    lib().orc_unpack(words.ctypes.data_as(_u32p), length, b, codes.ctypes.data_as(_u32p))
    return codes


def quantize_pack(u, b, clip_mode=CLIP_NONE, clip_value=1.0, seed=0, worker=0, k=0, block_base=0,
                  want_index=False):
    """One worker vector (or one tensor segment).  Returns (words, delta, clipped[, index])."""
    u, p = _f32(u)
    W = packed_words(u.size, b)
    words = np.zeros(max(W, 1), dtype=np.uint32)
    delta = C.c_float(0)
    clipped = C.c_uint32(0)
    index = np.zeros(max(u.size, 1), dtype=np.int32) if want_index else None
    rc = lib().orc_quantize_pack(p, u.size, b, clip_mode, clip_value, seed, worker, k, block_base,
                                 words.ctypes.data_as(_u32p), C.byref(delta),
                                 C.cast(C.byref(clipped), _u32p), _ptr(index, _i32p))
    _check(rc)
    res = (words[:W], np.float32(delta.value), int(clipped.value))
    return res + (index[: u.size],) if want_index else res


def unpack_average_prox(words, delta, length, b, mu, x, eta, lambda_l1, want_v=False, want_utilde=False):
    """words: (N, stride) uint32; delta: (N,).  Returns x_new (and v, u~ when asked)."""
    words = np.ascontiguousarray(words, dtype=np.uint32)
    assert words.ndim == 2
    N, stride = words.shape
    delta, pd = _f32(delta)
    assert delta.size == N
    xn = np.array(x, dtype=np.float32, copy=True)
    mu_a = None if mu is None else np.ascontiguousarray(mu, dtype=np.float32)
    v = np.zeros(length, dtype=np.float32) if want_v else None
    ut = np.zeros(length, dtype=np.float32) if want_utilde else None
    lib().orc_unpack_average_prox(words.ctypes.data_as(_u32p), stride, pd, N, length, b, _ptr(mu_a, _f32p),
                                  xn.ctypes.data_as(_f32p), eta, lambda_l1, _ptr(v, _f32p), _ptr(ut, _f32p))
    out = (xn,)
    if want_v:
        out += (v,)
    if want_utilde:
        out += (ut,)
    return out if len(out) > 1 else xn


def code_histogram(words, length, b):
    """Counts of the 2^b code values in a packed message."""
    words = np.ascontiguousarray(words, dtype=np.uint32)
    hist = np.zeros(1 << b, dtype=np.uint64)
    _check(lib().orc_code_histogram(words.ctypes.data_as(_u32p), length, b, hist.ctypes.data_as(C.POINTER(C.c_uint64))))
    return hist


def entropy_bits(hist):
    """n * H: the empirical-entropy bound on the message's payload, in bits."""
    hist = np.ascontiguousarray(hist, dtype=np.uint64)
    return float(lib().orc_entropy_bits(hist.ctypes.data_as(C.POINTER(C.c_uint64)), hist.size))


def huffman_bits(hist):
    """Payload length in bits under a Huffman code built for this histogram."""
    hist = np.ascontiguousarray(hist, dtype=np.uint64)
    return int(lib().orc_huffman_bits(hist.ctypes.data_as(C.POINTER(C.c_uint64)), hist.size))


SCHEME_A, SCHEME_B, SCHEME_C = 0, 1, 2


def sum_bits_per_coordinate(b, N):
    """Width of the server's sum stream under scheme (b): b + ceil(log2 N)."""
    return int(lib().orc_sum_bits_per_coordinate(b, N))


def scheme_bits(scheme, d, b, N):
    """Bits of one communication step 2 under scheme (a), (b) or (c) (Table 1)."""
    return int(lib().orc_scheme_bits(scheme, d, b, N))


def quantize_pack_shared(U, b, clip_mode=CLIP_NONE, clip_value=1.0, seed=0, k=0, block_base=0):
    """All N worker vectors (rows of U) with the unified scale of schemes (b)/(c).
    Returns (words (N, W), delta, clipped (N,))."""
    U = np.ascontiguousarray(U, dtype=np.float32)
    N, length = U.shape
    W = max(packed_words(length, b), 1)
    words = np.zeros((N, W), dtype=np.uint32)
    delta = np.zeros(1, dtype=np.float32)
    clipped = np.zeros(N, dtype=np.uint32)
    _check(lib().orc_quantize_pack_shared(U.ctypes.data_as(_f32p), N, length, length, b, clip_mode, clip_value, seed, k,
                                          block_base, words.ctypes.data_as(_u32p), W, delta.ctypes.data_as(_f32p),
                                          clipped.ctypes.data_as(_u32p)))
    return words[:, : packed_words(length, b)], np.float32(delta[0]), clipped


def server_reduce(words, length, b, requantize, seed=0, k=0, block_base=0):
    """The server of scheme (b) (requantize False: index sums, b + ceil(log2 N) bits) or (c) (True: b bits)."""
    words = np.ascontiguousarray(words, dtype=np.uint32)
    N, stride = words.shape
    bo = b if requantize else sum_bits_per_coordinate(b, N)
    out = np.zeros(max(packed_words(length, bo), 1), dtype=np.uint32)
    _check(lib().orc_server_reduce(words.ctypes.data_as(_u32p), stride, N, length, b, 1 if requantize else 0, seed, k,
                                   block_base, out.ctypes.data_as(_u32p)))
    return out[: packed_words(length, bo)]


def unpack_scaled_prox(words, delta, length, bits, divisor, mu, x, eta, lambda_l1, want_v=False, want_utilde=False):
    """A worker after the server's message: u~ = (delta * index) / divisor, then the proximal step."""
    words = np.ascontiguousarray(words, dtype=np.uint32)
    xn = np.array(x, dtype=np.float32, copy=True)
    mu_a = None if mu is None else np.ascontiguousarray(mu, dtype=np.float32)
    v = np.zeros(length, dtype=np.float32) if want_v else None
    ut = np.zeros(length, dtype=np.float32) if want_utilde else None
    lib().orc_unpack_scaled_prox(words.ctypes.data_as(_u32p), np.float32(delta), length, bits, divisor, _ptr(mu_a, _f32p),
                                 xn.ctypes.data_as(_f32p), eta, lambda_l1, _ptr(v, _f32p), _ptr(ut, _f32p))
    out = (xn,)
    if want_v:
        out += (v,)
    if want_utilde:
        out += (ut,)
    return out if len(out) > 1 else xn


def soft_threshold(w, kappa):
    return np.float32(lib().orc_soft_threshold(np.float32(w), np.float32(kappa)))


# ---- linear model ----------------------------------------------------------------------------

def margin(Xa, x):
    return tree_dot(Xa, x)


def loss_deriv(loss, m, y):
    return np.float32(lib().orc_loss_deriv(loss, np.float32(m), np.float32(y)))


def loss_value(loss, m, y):
    return float(lib().orc_loss_value(loss, np.float32(m), np.float32(y)))


def full_grad(X, y, loss, x):
    """Returns (mu, margins, f)."""
    X, pX = _f32(X)
    y, py = _f32(y)
    x, px = _f32(x)
    n, d = X.shape
    mu = np.zeros(d, dtype=np.float32)
    margins = np.zeros(n, dtype=np.float32)
    f = C.c_double(0)
    lib().orc_full_grad(pX, py, n, d, loss, px, mu.ctypes.data_as(_f32p), margins.ctypes.data_as(_f32p),
                        C.byref(f))
    return mu, margins, f.value


def objective(X, y, loss, x, lambda_l1):
    X, pX = _f32(X)
    y, py = _f32(y)
    x, px = _f32(x)
    n, d = X.shape
    return float(lib().orc_objective(pX, py, n, d, loss, px, lambda_l1))


def sample_batch(seed, tag, worker, k, B, lo, span):
    idx = np.zeros(B, dtype=np.int64)
    lib().orc_sample_batch(seed, tag, worker, k, B, lo, span, idx.ctypes.data_as(_i64p))
    return idx


def svrg_coef(X, y, loss, idx, x, xs):
    X, pX = _f32(X)
    y, py = _f32(y)
    x, px = _f32(x)
    xs, pxs = _f32(xs)
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    coef = np.zeros(idx.size, dtype=np.float32)
    lib().orc_svrg_coef(pX, py, X.shape[1], loss, idx.ctypes.data_as(_i64p), idx.size, px, pxs,
                        coef.ctypes.data_as(_f32p))
    return coef


def svrg_diff_from_coef(X, idx, coef):
    X, pX = _f32(X)
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    coef, pc = _f32(coef)
    u = np.zeros(X.shape[1], dtype=np.float32)
    lib().orc_svrg_diff_from_coef(pX, X.shape[1], idx.ctypes.data_as(_i64p), idx.size, pc,
                                  u.ctypes.data_as(_f32p))
    return u


class Problem:
    """The finite-sum problem of Eq. 1 with the quantizer settings: plain data holder."""

    def __init__(self, X, y, loss, lambda_l1, N, B, b, clip_mode, clip_value, seed, partition_local=True):
        self.X = np.ascontiguousarray(X, dtype=np.float32)
        self.y = np.ascontiguousarray(y, dtype=np.float32)
        self.n, self.d = self.X.shape
        self.loss, self.lambda_l1 = loss, float(lambda_l1)
        self.N, self.B, self.b = N, B, b
        self.clip_mode, self.clip_value = clip_mode, float(clip_value)
        self.seed, self.partition_local = seed, bool(partition_local)
        self.W = packed_words(self.d, b)


def lpc_inner_step(P, k, eta, x, xs, mu, taps=False):
    """Algorithm 1 steps 6-10 for all workers.  Returns x_new, or (x_new, taps dict)."""
    xn = np.array(x, dtype=np.float32, copy=True)
    xs, pxs = _f32(xs)
    mu, pmu = _f32(mu)
    t = None
    if taps:
        t = dict(idx=np.zeros((P.N, P.B), dtype=np.int64), coef=np.zeros((P.N, P.B), dtype=np.float32),
                 u=np.zeros((P.N, P.d), dtype=np.float32), words=np.zeros((P.N, max(P.W, 1)), dtype=np.uint32),
                 delta=np.zeros(P.N, dtype=np.float32), clipped=np.zeros(P.N, dtype=np.uint32),
                 v=np.zeros(P.d, dtype=np.float32))
    g = (lambda name, typ: _ptr(t[name], typ)) if taps else (lambda name, typ: None)
    rc = lib().orc_lpc_inner_step(P.X.ctypes.data_as(_f32p), P.y.ctypes.data_as(_f32p), P.n, P.d, P.loss,
                                  P.lambda_l1, P.N, P.B, P.b, P.clip_mode, P.clip_value, P.seed,
                                  int(P.partition_local), k, eta, pxs, pmu, xn.ctypes.data_as(_f32p),
                                  g("idx", _i64p), g("coef", _f32p), g("u", _f32p), g("words", _u32p),
                                  max(P.W, 1), g("delta", _f32p), g("clipped", _u32p), g("v", _f32p))
    _check(rc)
    if taps:
        t["words"] = t["words"][:, : P.W]
        return xn, t
    return xn


def weighted_snapshot(ysum, wsum):
    """Algorithm 2's snapshot from the weighted sum of the epoch's y iterates and the sum of the weights."""
    ysum, p = _f32(ysum)
    out = np.zeros_like(ysum)
    lib().orc_weighted_snapshot(p, np.float32(wsum), ysum.size, out.ctypes.data_as(_f32p))
    return out


def ridge_term(x, sigma):
    x, p = _f32(x)
    return float(lib().orc_ridge_term(p, x.size, np.float32(sigma)))


def alpc_step(P, k, tau1, tau2, alpha, inv4L, xs, mu, y, z, ysum, taps=False, sigma=None, weight=1.0):
    """Algorithm 2 steps 5-13.  Returns (y_new, z_new, ysum_new[, taps]).  sigma (with weight): the strongly convex
    case with h = lambda_l1*||.||_1 + (sigma/2)*||.||^2 and the snapshot weight of this step."""
    xs, pxs = _f32(xs)
    mu, pmu = _f32(mu)
    yn = np.array(y, dtype=np.float32, copy=True)
    zn = np.array(z, dtype=np.float32, copy=True)
    sn = np.array(ysum, dtype=np.float32, copy=True)
    t = None
    if taps:
        t = dict(x=np.zeros(P.d, dtype=np.float32), v=np.zeros(P.d, dtype=np.float32),
                 vhat=np.zeros(P.d, dtype=np.float32), words=np.zeros((P.N, max(P.W, 1)), dtype=np.uint32),
                 delta=np.zeros(P.N, dtype=np.float32))
    g = (lambda name, typ: _ptr(t[name], typ)) if taps else (lambda name, typ: None)
    head = (P.X.ctypes.data_as(_f32p), P.y.ctypes.data_as(_f32p), P.n, P.d, P.loss, P.lambda_l1, P.N, P.B, P.b,
            P.clip_mode, P.clip_value, P.seed, int(P.partition_local), k, tau1, tau2, alpha, inv4L)
    tail = (pxs, pmu, yn.ctypes.data_as(_f32p), zn.ctypes.data_as(_f32p), sn.ctypes.data_as(_f32p),
            g("x", _f32p), g("v", _f32p), g("vhat", _f32p), g("words", _u32p), max(P.W, 1), g("delta", _f32p))
    if sigma is None:
        rc = lib().orc_alpc_step(*head, *tail)
    else:
        rc = lib().orc_alpc_step_sc(*head, np.float32(sigma), np.float32(weight), *tail)
    _check(rc)
    if taps:
        t["words"] = t["words"][:, : P.W]
        return yn, zn, sn, t
    return yn, zn, sn


def alpc3_epoch_params(s, L):
    """Algorithm 3 step 3: (tau_1, alpha) of epoch s for smoothness L, as fp32 values."""
    t, a = C.c_float(0), C.c_float(0)
    lib().orc_alpc3_epoch_params(C.c_int64(s), C.c_double(L), C.byref(t), C.byref(a))
    return np.float32(t.value), np.float32(a.value)


def alpc3_mean_snapshot(ysum, m):
    """Algorithm 3 step 5 from the running sum of the epoch's y iterates."""
    ysum, p = _f32(ysum)
    out = np.zeros_like(ysum)
    lib().orc_alpc3_mean_snapshot(p, C.c_int64(m), ysum.size, out.ctypes.data_as(_f32p))
    return out


def alpc3_epoch(P, s, m, L, tau2, xs, mu, y, z):
    """One epoch of Algorithm 3 after its full-gradient step.  Returns (y, z, next snapshot)."""
    xs, pxs = _f32(xs)
    mu, pmu = _f32(mu)
    yn = np.array(y, dtype=np.float32, copy=True)
    zn = np.array(z, dtype=np.float32, copy=True)
    nxt = np.zeros(P.d, dtype=np.float32)
    rc = lib().orc_alpc3_epoch(P.X.ctypes.data_as(_f32p), P.y.ctypes.data_as(_f32p), C.c_int64(P.n), C.c_int64(P.d),
                               P.loss, C.c_float(P.lambda_l1), P.N, P.B, P.b, P.clip_mode, C.c_float(P.clip_value),
                               C.c_uint64(P.seed), int(P.partition_local), C.c_int64(s), C.c_int64(m), C.c_double(L),
                               C.c_float(tau2), pxs, pmu, yn.ctypes.data_as(_f32p), zn.ctypes.data_as(_f32p),
                               nxt.ctypes.data_as(_f32p))
    _check(rc)
    return yn, zn, nxt

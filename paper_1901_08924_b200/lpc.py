"""Thin Python binding of the C-ABI library (include/lpc.h): argument marshalling only.

Torch is used for device memory and streams; every step of the method runs inside
liblpcsvrg.so.  There is no CPU fallback: if the library is missing or cannot be loaded the
import of a symbol fails loudly.
"""
import ctypes as C
import os

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
# LPC_LIBRARY selects another build of the same library (the phase-stamping build of paper_1901_08924_b200.trace)
LIB_PATH = os.environ.get("LPC_LIBRARY") or os.path.join(HERE, "liblpcsvrg.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_NONFINITE, ERR_CUDA, ERR_TIMEOUT = 0, -1, -2, -3, -4, -5
LOGISTIC, LEAST_SQUARES = 0, 1
CLIP_NONE, CLIP_LAMBDA, CLIP_STD = 0, 1, 2
(BUF_X, BUF_XTILDE, BUF_MU, BUF_MARGINS, BUF_Y, BUF_Z, BUF_YSUM, BUF_CODES, BUF_DELTA, BUF_CLIPPED, BUF_BATCH_IDX,
 BUF_COEF, BUF_U, BUF_V, BUF_VHAT) = range(15)
OPT_SAMPLE_GLOBAL, OPT_TAP_U, OPT_CLUSTER_SIZE, OPT_USE_GRAPH, OPT_PROFILE, OPT_PERSISTENT = 0, 1, 2, 3, 4, 5
OPT_SHARED_SCALE, OPT_AVERAGE_DIVISOR, OPT_ONE_LAUNCH_QUANTIZE, OPT_LOOP_COOPERATIVE = 6, 7, 8, 9
SCHEME_BROADCAST, SCHEME_SERVER_SUM, SCHEME_SERVER_REQUANTIZE = 0, 1, 2
(INFO_STEP_CLUSTER_SIZE, INFO_LOOP_CLUSTER_SIZE, INFO_LOOP_LAUNCHES, INFO_SNAPSHOT_ROWS_PER_TILE, INFO_SNAPSHOT_STAGES,
 INFO_ALPC_LOOP_CLUSTER_SIZE, INFO_LOOP_ROW_SLOTS, INFO_ALPC_LOOP_ROW_SLOTS, INFO_STEP_RING_STAGES,
 INFO_AGGREGATE_SPLIT, INFO_QUANT_PIPELINED_RUNS, INFO_LOOP_COORDS_PER_THREAD, INFO_ALPC_LOOP_COORDS_PER_THREAD,
 INFO_QUANT_ONE_LAUNCH) = range(14)
KERNEL_NAMES = ["snapshot", "worker", "aggregate", "quant_stats", "quant_pack", "other", "inner_loop", "quant_fused"]

# every symbol that include/lpc.h declares: (name, restype, argtypes)
_vp, _i64, _i32, _u64, _f32, _int = C.c_void_p, C.c_int64, C.c_int32, C.c_uint64, C.c_float, C.c_int
_i64p, _u64p, _f64p = C.POINTER(C.c_int64), C.POINTER(C.c_uint64), C.POINTER(C.c_double)
SYMBOLS = [
    ("lpc_init", _int, [C.POINTER(_vp), _vp, _vp, _i64, _i32, _int, _f32, _i32, _i32, _i32, _int, _f32, _u64, _vp]),
    ("lpc_destroy", _int, [_vp]),
    ("lpc_set_option", _int, [_vp, _int, _i64]),
    ("lpc_last_error", C.c_char_p, [_vp]),
    ("lpc_sync_status", _int, [_vp]),
    ("lpc_get_buffer", _int, [_vp, _int, _vp, C.c_size_t]),
    ("lpc_set_buffer", _int, [_vp, _int, _vp, C.c_size_t]),
    ("lpc_set_iterate", _int, [_vp, _vp]),
    ("lpc_get_iterate", _int, [_vp, _vp]),
    ("lpc_snapshot_full_grad", _int, [_vp, _vp, _f64p]),
    ("lpc_inner_step", _int, [_vp, _f32, _u64]),
    ("lpc_inner_steps", _int, [_vp, _f32, _u64, _i64]),
    ("lpc_packed_layout", _int, [_i64, _i32, _i64p, _i32, _i64p, _i64p]),
    ("lpc_packed_words", _int, [_i64, _i32, _i64p]),
    ("lpc_quantize_pack", _int, [_vp, _vp, _vp, _i64, _i64, _i64p, _i32, _u64, _vp, _vp, _vp]),
    ("lpc_unpack_average_prox", _int, [_vp, _vp, _vp, _i64, _i64p, _i32, _vp, _vp, _f32, _f32, _vp]),
    ("lpc_message_entropy", _int, [_vp, _vp, _i64, _i64p, _i32, _vp, _f64p, _u64p]),
    ("lpc_server_reduce", _int, [_vp, _vp, _i64, _i64p, _i32, _int, _u64, _vp]),
    ("lpc_sum_bits", _int, [_i32, _i32, C.POINTER(C.c_int32)]),
    ("lpc_scheme_bits", _int, [_int, _i64, _i32, _i32, _u64p]),
    ("lpc_alpc_begin", _int, [_vp]),
    ("lpc_set_strong_convexity", _int, [_vp, _f32]),
    ("lpc_alpc_double_sample_step", _int, [_vp, _f32, _f32, _f32, _f32, _u64]),
    ("lpc_alpc_double_sample_steps", _int, [_vp, _f32, _f32, _f32, _f32, _u64, _i64]),
    ("lpc_alpc_end_epoch", _int, [_vp, _i64]),
    ("lpc_objective", _int, [_vp, _vp, _f64p]),
    ("lpc_comm_bits", _int, [_vp, _u64p, _u64p]),
    ("lpc_get_profile", _int, [_vp, _f64p, _i64p, _i32]),
    ("lpc_query", _int, [_vp, _int, _i64p]),
    ("lpc_svrg_run_host", _int, [_vp, _vp, _i64, _i32, _int, _f32, _i32, _i32, _i32, _int, _f32, _u64, _i32, _i64,
                                 _f32, _vp, _f64p, _u64p]),
    ("lpc_quantize_pack_static", _int, [_vp, _i64, _i64, _i32, _i32, _int, _f32, _u64, _u64, _vp, _vp, _vp, _vp]),
    ("lpc_debug_wait_timeout", _int, [_vp, _u64]),
    ("lpc_debug_stream_blocks", _int, [_u64, C.c_uint32, C.c_uint32, _u64, C.c_uint32, _i64, _vp, _vp]),
]

_lib = None


def lib():
    """Loads liblpcsvrg.so (built in-tree by paper_1901_08924_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_1901_08924_b200.build` "
                               "(there is no fallback implementation)")
        L = C.CDLL(LIB_PATH)
        for name, res, args in SYMBOLS:
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


class LpcError(RuntimeError):
    def __init__(self, code, text=""):
        super().__init__(f"lpc status {code}: {text}")
        self.code = code


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _seg(seg_offsets):
    if seg_offsets is None:
        return None, 1
    arr = (C.c_int64 * len(seg_offsets))(*[int(v) for v in seg_offsets])
    return arr, len(seg_offsets) - 1


def packed_words(length, b):
    out = C.c_int64(0)
    rc = lib().lpc_packed_words(length, b, C.byref(out))
    if rc != OK:
        raise LpcError(rc)
    return out.value


def sum_bits(b, N):
    out = C.c_int32(0)
    rc = lib().lpc_sum_bits(b, N, C.byref(out))
    if rc != OK:
        raise LpcError(rc, "lpc_sum_bits")
    return out.value


def scheme_bits(scheme, d, b, N):
    out = C.c_uint64(0)
    rc = lib().lpc_scheme_bits(scheme, d, b, N, C.byref(out))
    if rc != OK:
        raise LpcError(rc, "lpc_scheme_bits")
    return out.value


def packed_layout(length, b, seg_offsets=None):
    """Returns (word_offsets list of nseg+1, stride_words)."""
    arr, nseg = _seg(seg_offsets)
    woff = (C.c_int64 * (nseg + 1))()
    stride = C.c_int64(0)
    rc = lib().lpc_packed_layout(length, b, arr, nseg, woff, C.byref(stride))
    if rc != OK:
        raise LpcError(rc)
    return list(woff), stride.value


class Context:
    """Owns one lpc_ctx.  X and y are CUDA fp32 tensors kept alive by this object (or None for a
    quantizer-only context)."""

    def __init__(self, X, y, loss, lambda_l1, N, B, b, clip_mode, clip_value, seed, stream=None):
        self._h = C.c_void_p(None)
        self.X, self.y = X, y
        if X is not None:
            assert X.is_cuda and X.dtype == torch.float32 and X.is_contiguous() and X.dim() == 2
            assert y.is_cuda and y.dtype == torch.float32 and y.is_contiguous() and y.numel() == X.shape[0]
            n, d = X.shape
            self.device = X.device
        else:
            n, d = 0, 0
            self.device = torch.device("cuda", torch.cuda.current_device())
        self.n, self.d, self.N, self.B, self.b = n, d, N, B, b
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        rc = lib().lpc_init(C.byref(self._h), _ptr(X), _ptr(y), n, d, loss, lambda_l1, N, B, b, clip_mode, clip_value,
                            seed, C.c_void_p(self.stream.cuda_stream))
        if rc != OK:
            self._h = C.c_void_p(None)
            raise LpcError(rc, "lpc_init")
        if X is not None:
            _, self.stride_words = packed_layout(d, b)

    def _ck(self, rc):
        if rc != OK:
            raise LpcError(rc, lib().lpc_last_error(self._h).decode())

    def close(self):
        if self._h:
            lib().lpc_destroy(self._h)
            self._h = C.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_option(self, option, value):
        self._ck(lib().lpc_set_option(self._h, option, value))

    def sync_status(self):
        """Waits for the stream; raises LpcError for a recorded device-side error."""
        self._ck(lib().lpc_sync_status(self._h))

    def status(self):
        return lib().lpc_sync_status(self._h)

    _BUF_DTYPE = {BUF_CODES: torch.int32, BUF_CLIPPED: torch.int32, BUF_BATCH_IDX: torch.int64}

    def _buf_shape(self, which):
        N, B, d = self.N, self.B, self.d
        return {BUF_MARGINS: (self.n,), BUF_CODES: (N, self.stride_words), BUF_DELTA: (N,), BUF_CLIPPED: (N,),
                BUF_BATCH_IDX: (N + 1, B), BUF_COEF: (N + 1, B), BUF_U: (N, d)}.get(which, (d,))

    def get_buffer(self, which):
        t = torch.empty(self._buf_shape(which), dtype=self._BUF_DTYPE.get(which, torch.float32), device=self.device)
        self._ck(lib().lpc_get_buffer(self._h, which, _ptr(t), t.numel() * t.element_size()))
        return t

    def set_buffer(self, which, t):
        assert t.is_cuda and t.is_contiguous()
        self._ck(lib().lpc_set_buffer(self._h, which, _ptr(t), t.numel() * t.element_size()))

    def set_iterate(self, x):
        assert x.is_cuda and x.dtype == torch.float32 and x.numel() == self.d
        self._ck(lib().lpc_set_iterate(self._h, _ptr(x)))

    def get_iterate(self):
        x = torch.empty(self.d, dtype=torch.float32, device=self.device)
        self._ck(lib().lpc_get_iterate(self._h, _ptr(x)))
        return x

    def snapshot_full_grad(self, mu_out=None, want_f=False):
        f = C.c_double(0)
        self._ck(lib().lpc_snapshot_full_grad(self._h, _ptr(mu_out), C.byref(f) if want_f else None))
        return f.value if want_f else None

    def inner_step(self, eta, k):
        self._ck(lib().lpc_inner_step(self._h, eta, k))

    def inner_steps(self, eta, k0, count):
        self._ck(lib().lpc_inner_steps(self._h, eta, k0, count))

    def quantize_pack(self, U, k, U_sub=None, seg_offsets=None, codes_out=None, delta_out=None, clipped_out=None):
        """U: (N, len) fp32 CUDA tensor (row stride = U.stride(0)).  Returns (codes, delta, clipped)."""
        assert U.is_cuda and U.dtype == torch.float32 and U.dim() == 2 and U.shape[0] == self.N and U.stride(1) == 1
        length, ld = U.shape[1], (U.stride(0) if U.shape[0] > 1 else max(U.shape[1], 1))
        if U_sub is not None:
            assert U_sub.shape == U.shape and U_sub.stride() == U.stride() and U_sub.dtype == torch.float32
        arr, nseg = _seg(seg_offsets)
        _, stride = packed_layout(length, self.b, seg_offsets)
        if codes_out is None:
            codes_out = torch.empty((self.N, stride), dtype=torch.int32, device=U.device)
        if delta_out is None:
            delta_out = torch.empty((self.N, nseg), dtype=torch.float32, device=U.device)
        if clipped_out is None:
            clipped_out = torch.empty((self.N, nseg), dtype=torch.int32, device=U.device)
        self._ck(lib().lpc_quantize_pack(self._h, _ptr(U), _ptr(U_sub), length, ld, arr, nseg, k, _ptr(codes_out),
                                         _ptr(delta_out), _ptr(clipped_out)))
        return codes_out, delta_out, clipped_out

    def unpack_average_prox(self, codes, delta, length, x, eta, lambda_l1, mu=None, seg_offsets=None, v_out=None):
        arr, nseg = _seg(seg_offsets)
        self._ck(lib().lpc_unpack_average_prox(self._h, _ptr(codes), _ptr(delta), length, arr, nseg, _ptr(mu), _ptr(x),
                                               eta, lambda_l1, _ptr(v_out)))
        return x

    def message_entropy(self, codes, length, seg_offsets=None, hist_out=None, host_counts=True):
        """Histogram of every (worker, segment) message and, on the host, its entropy bound and Huffman length in bits.
        Returns (hist (N, nseg, 2^b) int64 CUDA tensor, entropy (N, nseg) or None, huffman (N, nseg) or None)."""
        arr, nseg = _seg(seg_offsets)
        if hist_out is None:
            hist_out = torch.empty((self.N, nseg, 1 << self.b), dtype=torch.int64, device=codes.device)
        ent = (C.c_double * (self.N * nseg))() if host_counts else None
        huf = (C.c_uint64 * (self.N * nseg))() if host_counts else None
        self._ck(lib().lpc_message_entropy(self._h, _ptr(codes), length, arr, nseg, _ptr(hist_out), ent, huf))
        if not host_counts:
            return hist_out, None, None
        import numpy as np
        return (hist_out, np.array(ent[:], dtype=np.float64).reshape(self.N, nseg),
                np.array(huf[:], dtype=np.uint64).reshape(self.N, nseg))

    def server_reduce(self, codes, length, scheme, k, seg_offsets=None, codes_out=None):
        """The server of scheme (b) or (c): N streams of b bits in, one stream out.  Returns (codes_out, bits_out)."""
        arr, nseg = _seg(seg_offsets)
        bo = sum_bits(self.b, self.N) if scheme == SCHEME_SERVER_SUM else self.b
        _, stride = packed_layout(length, bo, seg_offsets)
        if codes_out is None:
            codes_out = torch.empty((1, stride), dtype=torch.int32, device=codes.device)
        self._ck(lib().lpc_server_reduce(self._h, _ptr(codes), length, arr, nseg, scheme, k, _ptr(codes_out)))
        return codes_out, bo

    def set_strong_convexity(self, sigma):
        self._ck(lib().lpc_set_strong_convexity(self._h, sigma))

    def alpc_begin(self):
        self._ck(lib().lpc_alpc_begin(self._h))

    def alpc_double_sample_step(self, tau1, tau2, alpha, inv4L, k):
        self._ck(lib().lpc_alpc_double_sample_step(self._h, tau1, tau2, alpha, inv4L, k))

    def alpc_double_sample_steps(self, tau1, tau2, alpha, inv4L, k0, count):
        self._ck(lib().lpc_alpc_double_sample_steps(self._h, tau1, tau2, alpha, inv4L, k0, count))

    def alpc_end_epoch(self, m):
        self._ck(lib().lpc_alpc_end_epoch(self._h, m))

    def objective(self, x=None):
        P = C.c_double(0)
        self._ck(lib().lpc_objective(self._h, _ptr(x), C.byref(P)))
        return P.value

    def query(self, what):
        out = C.c_int64(0)
        self._ck(lib().lpc_query(self._h, what, C.byref(out)))
        return out.value

    def get_profile(self, reset=True):
        """Returns {kernel name: (total ms, launches)} measured since profiling was switched on / last reset."""
        n = len(KERNEL_NAMES)
        ms, cnt = (C.c_double * n)(), (C.c_int64 * n)()
        self._ck(lib().lpc_get_profile(self._h, ms, cnt, 1 if reset else 0))
        return {KERNEL_NAMES[i]: (ms[i], cnt[i]) for i in range(n)}

    def debug_wait_timeout(self, limit_ns):
        """Enqueues a kernel whose bounded waits run out after limit_ns (see lpc_debug_wait_timeout)."""
        self._ck(lib().lpc_debug_wait_timeout(self._h, limit_ns))

    def comm_bits(self):
        a, b = C.c_uint64(0), C.c_uint64(0)
        self._ck(lib().lpc_comm_bits(self._h, C.byref(a), C.byref(b)))
        return a.value, b.value


def svrg_run_host(X, y, loss, lambda_l1, N, B, b, clip_mode, clip_value, seed, S, m, eta, x0):
    """Whole LPC-SVRG job from HOST tensors (pinned recommended).  Returns (x, objective, step2_bits)."""
    assert not X.is_cuda and X.dtype == torch.float32 and X.is_contiguous()
    assert not y.is_cuda and not x0.is_cuda
    n, d = X.shape
    x = x0.clone().contiguous()
    P, bits = C.c_double(0), C.c_uint64(0)
    rc = lib().lpc_svrg_run_host(_ptr(X), _ptr(y), n, d, loss, lambda_l1, N, B, b, clip_mode, clip_value, seed, S, m, eta,
                                 _ptr(x), C.byref(P), C.byref(bits))
    if rc != OK:
        raise LpcError(rc, "lpc_svrg_run_host")
    return x, P.value, bits.value


def debug_stream_blocks(seed, tag, worker, k, block0, count, device=None):
    out = torch.empty((count, 4), dtype=torch.int32, device=device or torch.device("cuda", torch.cuda.current_device()))
    st = torch.cuda.current_stream(out.device)
    rc = lib().lpc_debug_stream_blocks(seed, tag, worker, k, block0, count, _ptr(out), C.c_void_p(st.cuda_stream))
    if rc != OK:
        raise LpcError(rc, "lpc_debug_stream_blocks")
    return out


def quantize_pack_static(U, b, clip_mode, clip_value, seed, k, codes_out, delta_out, clipped_out):
    """Quantize + pack without any device allocation inside the library (see lpc_quantize_pack_static).

    The caller supplies every buffer: U (N, len) fp32, codes_out (N, stride_words) int32 with stride_words from
    packed_layout(len, b), delta_out (N,) fp32, clipped_out (N,) int32.  Returns the status code.
    """
    assert U.is_cuda and U.dtype == torch.float32 and U.dim() == 2 and U.stride(1) == 1
    N, length = U.shape
    ld = U.stride(0) if N > 1 else max(length, 1)
    st = torch.cuda.current_stream(U.device)
    with torch.cuda.device(U.device):  # the library looks its working memory up on the current device
        return lib().lpc_quantize_pack_static(_ptr(U), length, ld, N, b, clip_mode, clip_value, seed, k, _ptr(codes_out),
                                              _ptr(delta_out), _ptr(clipped_out), C.c_void_p(st.cuda_stream))

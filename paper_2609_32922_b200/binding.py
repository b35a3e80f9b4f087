"""Thin ctypes binding of ``libscgemm.so`` (the C ABI declared in ``include/sc_gemm.h``).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.  PyTorch is used
for device memory and streams.  A missing library, or a CUDA device that is absent, is an error: there
is no CPU path here.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libscgemm.so")

SC_OK, SC_ERR_ARG, SC_ERR_SHAPE, SC_ERR_LENGTH, SC_ERR_NONFINITE = 0, 1, 2, 3, 4
SC_ERR_BUDGET, SC_ERR_WORKSPACE, SC_ERR_CUDA, SC_ERR_TIMEOUT = 5, 6, 7, 8
SC_BIPOLAR_XNOR, SC_UNIPOLAR_AND = 0, 1
SC_SCALE_NONE, SC_SCALE_PER_ROW, SC_SCALE_PER_TENSOR = 0, 1, 2
SC_CORE_AUTO, SC_CORE_POPC, SC_CORE_CSA, SC_CORE_SIMPLE, SC_CORE_UMMA, SC_CORE_UMMA_PAIR = 0, 1, 2, 3, 4, 5
SC_QUANT_DIRECT257, SC_QUANT_INT8_THEN_257 = 0, 1
SC_L_CAP = 1024

EXPORTS = (
    "sc_create", "sc_destroy", "sc_status_string", "sc_device_status", "sc_row_stats", "sc_assign_lengths",
    "sc_ladder_lengths", "sc_stream_bytes", "sc_encode", "sc_debug_unpack", "sc_workspace_bytes", "sc_matmul",
    "sc_selftest_comparator", "sc_selftest_expansion", "sc_selftest_bounded_wait", "sc_microbench", "sc_profile_enable", "sc_profile_read", "sc_launch_count", "sc_last_core_selected",
    "sc_assign_lengths_static", "sc_weights_bytes", "sc_weights_prepare", "sc_weights_release",
    "sc_workspace_bytes_prepared", "sc_matmul_prepared", "sc_surrogate_noise",
    "sc_workspace_bytes_batched", "sc_matmul_batched", "sc_workspace_bytes_cbsg", "sc_matmul_cbsg", "sc_cbsg_scc",
)


class sc_params(ctypes.Structure):
    _fields_ = [("mode", ctypes.c_int32), ("scale_a", ctypes.c_int32), ("scale_w", ctypes.c_int32),
                ("group", ctypes.c_int32), ("seed", ctypes.c_uint64), ("stream_id", ctypes.c_uint32),
                ("core", ctypes.c_uint32), ("quant", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class ScError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__("%s: %s (code %d)" % (where, status_string(code), code))
        self.code = code


_lib = None


def load():
    """Opens the shared library (built by ``paper_2609_32922_b200.build``); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError("%s not found: build it with `python -m paper_2609_32922_b200.build`" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    c = ctypes
    vp, i32, i64, f64, sz = c.c_void_p, c.c_int32, c.c_int64, c.c_double, c.c_size_t
    pp = c.POINTER(sc_params)
    lib.sc_create.argtypes = [c.POINTER(vp), c.c_int]
    lib.sc_destroy.argtypes = [vp]
    lib.sc_status_string.argtypes = [c.c_int]
    lib.sc_status_string.restype = c.c_char_p
    lib.sc_device_status.argtypes = [vp, c.POINTER(i32)]
    lib.sc_row_stats.argtypes = [vp, vp, i64, i64, vp, vp]
    lib.sc_assign_lengths.argtypes = [vp, vp, i64, i32, f64, i32, i32, vp, c.POINTER(f64), vp]
    lib.sc_ladder_lengths.argtypes = [vp, vp, i64, i32, c.POINTER(i32), c.POINTER(c.c_float), i32, vp, vp]
    lib.sc_stream_bytes.argtypes = [i64, i64, i32, i32]
    lib.sc_stream_bytes.restype = sz
    lib.sc_encode.argtypes = [vp, vp, i64, i64, i32, vp, i32, pp, vp, vp, vp]
    lib.sc_debug_unpack.argtypes = [vp, vp, i64, i64, i32, i32, vp, vp, vp]
    lib.sc_workspace_bytes.argtypes = [i64, i64, i64, i32, pp]
    lib.sc_workspace_bytes.restype = sz
    lib.sc_matmul.argtypes = [vp, vp, vp, i64, i64, i64, vp, i32, pp, vp, vp, vp, sz, vp]
    lib.sc_weights_bytes.argtypes = [i64, i64, i32, pp]
    lib.sc_weights_bytes.restype = sz
    lib.sc_weights_prepare.argtypes = [vp, vp, i64, i64, i32, pp, vp, sz, vp, c.POINTER(vp)]
    lib.sc_weights_release.argtypes = [vp]
    lib.sc_workspace_bytes_prepared.argtypes = [i64, i64, i64, i32, pp]
    lib.sc_workspace_bytes_prepared.restype = sz
    lib.sc_matmul_prepared.argtypes = [vp, vp, vp, i64, vp, i32, pp, vp, vp, vp, sz, vp]
    lib.sc_workspace_bytes_batched.argtypes = [i64, i64, i64, i64, i32, pp]
    lib.sc_workspace_bytes_batched.restype = sz
    lib.sc_matmul_batched.argtypes = [vp, vp, vp, i64, i64, i64, i64, i32, vp, i32, pp, vp, vp, vp, sz, vp]
    lib.sc_matmul_batched.restype = c.c_int
    lib.sc_workspace_bytes_cbsg.argtypes = [i64, i64, i64, i32, pp]
    lib.sc_workspace_bytes_cbsg.restype = sz
    lib.sc_matmul_cbsg.argtypes = [vp, vp, vp, i64, i64, i64, vp, i32, pp, vp, vp, vp, sz, vp]
    lib.sc_matmul_cbsg.restype = c.c_int
    lib.sc_cbsg_scc.argtypes = [vp, vp, vp, i64, i32, c.c_uint64, c.c_uint32, vp, vp, vp, sz, vp]
    lib.sc_cbsg_scc.restype = c.c_int
    lib.sc_surrogate_noise.argtypes = [vp, vp, i64, i64, vp, i32, f64, c.c_uint64, c.c_uint32, vp, vp]
    lib.sc_surrogate_noise.restype = c.c_int
    lib.sc_selftest_comparator.argtypes = []
    lib.sc_selftest_comparator.restype = i32
    lib.sc_selftest_expansion.argtypes = []
    lib.sc_selftest_expansion.restype = i32
    lib.sc_microbench.argtypes = [vp, i32, i32, c.POINTER(c.c_float), c.POINTER(f64)]
    lib.sc_selftest_bounded_wait.argtypes = [vp, i64, c.POINTER(i32), c.POINTER(i64)]
    lib.sc_selftest_bounded_wait.restype = c.c_int
    lib.sc_profile_enable.argtypes = [vp, i32]
    lib.sc_profile_read.argtypes = [vp, c.POINTER(c.c_float)]
    lib.sc_launch_count.argtypes = [vp, c.POINTER(i64)]
    lib.sc_last_core_selected.argtypes = [vp, c.POINTER(i32)]
    lib.sc_last_core_selected.restype = c.c_int
    lib.sc_assign_lengths_static.argtypes = [vp, i64, i32, f64, i32, i32, vp, vp, vp, vp]
    lib.sc_assign_lengths_static.restype = c.c_int
    for name in ("sc_create", "sc_destroy", "sc_device_status", "sc_row_stats", "sc_assign_lengths",
                 "sc_ladder_lengths", "sc_encode", "sc_debug_unpack", "sc_matmul", "sc_microbench",
                 "sc_profile_enable", "sc_profile_read", "sc_launch_count", "sc_weights_prepare",
                 "sc_weights_release", "sc_matmul_prepared"):
        getattr(lib, name).restype = c.c_int
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load().sc_status_string(int(code)).decode()


def _check(code: int, where: str):
    if code != SC_OK:
        raise ScError(code, where)


def make_params(mode=SC_BIPOLAR_XNOR, scale_a=SC_SCALE_PER_ROW, scale_w=SC_SCALE_PER_TENSOR, group=1, seed=0,
                stream_id=0, core=SC_CORE_AUTO, quant=SC_QUANT_DIRECT257) -> sc_params:
    return sc_params(mode, scale_a, scale_w, group, seed, stream_id, core, quant, 0)


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream_handle(stream) -> Optional[int]:
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream or None


# ---- the C entry points, same names ---------------------------------------------------------------
def sc_create(device: int = 0) -> int:
    h = ctypes.c_void_p()
    _check(load().sc_create(ctypes.byref(h), device), "sc_create")
    return h.value


def sc_destroy(ctx: int):
    _check(load().sc_destroy(ctx), "sc_destroy")


def sc_device_status(ctx: int) -> int:
    code = ctypes.c_int32(0)
    _check(load().sc_device_status(ctx, ctypes.byref(code)), "sc_device_status")
    return int(code.value)


def sc_row_stats(ctx, A, g, stream=None):
    M, K = A.shape
    _check(load().sc_row_stats(ctx, _ptr(A), M, K, _ptr(g), _stream_handle(stream)), "sc_row_stats")


def sc_assign_lengths(ctx, g, group, avg_budget, Lmin, Lmax, L_out, want_realized=False, stream=None):
    avg = ctypes.c_double(0.0)
    _check(load().sc_assign_lengths(ctx, _ptr(g), g.numel(), group, float(avg_budget), Lmin, Lmax, _ptr(L_out),
                                    ctypes.byref(avg) if want_realized else None, _stream_handle(stream)),
           "sc_assign_lengths")
    return float(avg.value) if want_realized else None


def sc_ladder_lengths(ctx, g, group, ladder, tau, L_out, stream=None):
    n = len(ladder)
    lad = (ctypes.c_int32 * n)(*[int(x) for x in ladder])
    th = (ctypes.c_float * max(n - 1, 1))(*[float(x) for x in tau]) if n > 1 else None
    _check(load().sc_ladder_lengths(ctx, _ptr(g), g.numel(), group, lad, th, n, _ptr(L_out), _stream_handle(stream)),
           "sc_ladder_lengths")


def sc_stream_bytes(stream_rows, depth, Lmax, mode) -> int:
    return int(load().sc_stream_bytes(stream_rows, depth, Lmax, mode))


def sc_encode(ctx, X, tensor_id, L_or_none, Lmax, params, streams_out, scales_out, stream=None):
    rows, cols = X.shape
    _check(load().sc_encode(ctx, _ptr(X), rows, cols, tensor_id, _ptr(L_or_none), Lmax, ctypes.byref(params),
                            _ptr(streams_out), _ptr(scales_out), _stream_handle(stream)), "sc_encode")


def sc_debug_unpack(ctx, streams, stream_rows, depth, Lmax, mode, bits_out, neg_out=None, stream=None):
    _check(load().sc_debug_unpack(ctx, _ptr(streams), stream_rows, depth, Lmax, mode, _ptr(bits_out), _ptr(neg_out),
                                  _stream_handle(stream)), "sc_debug_unpack")


def sc_workspace_bytes(M, K, N, Lmax, params) -> int:
    return int(load().sc_workspace_bytes(M, K, N, Lmax, ctypes.byref(params)))


def sc_matmul(ctx, A, W, L, Lmax, params, P, C, ws, stream=None):
    M, K = A.shape
    K2, N = W.shape
    assert K == K2
    _check(load().sc_matmul(ctx, _ptr(A), _ptr(W), M, K, N, _ptr(L), Lmax, ctypes.byref(params), _ptr(P), _ptr(C),
                            _ptr(ws), ws.numel() * ws.element_size(), _stream_handle(stream)), "sc_matmul")


def sc_weights_bytes(K, N, Lmax, params) -> int:
    return int(load().sc_weights_bytes(K, N, Lmax, ctypes.byref(params)))


def sc_weights_prepare(ctx, W, Lmax, params, wbuf, stream=None) -> int:
    K, N = W.shape
    out = ctypes.c_void_p()
    _check(load().sc_weights_prepare(ctx, _ptr(W), K, N, Lmax, ctypes.byref(params), _ptr(wbuf),
                                     wbuf.numel() * wbuf.element_size(), _stream_handle(stream), ctypes.byref(out)),
           "sc_weights_prepare")
    return out.value


def sc_weights_release(weights: int):
    _check(load().sc_weights_release(weights), "sc_weights_release")


def sc_workspace_bytes_prepared(M, K, N, Lmax, params) -> int:
    return int(load().sc_workspace_bytes_prepared(M, K, N, Lmax, ctypes.byref(params)))


def sc_matmul_prepared(ctx, A, weights, L, Lmax, params, P, C, ws, stream=None):
    _check(load().sc_matmul_prepared(ctx, _ptr(A), weights, A.shape[0], _ptr(L), Lmax, ctypes.byref(params), _ptr(P),
                                     _ptr(C), _ptr(ws), ws.numel() * ws.element_size(), _stream_handle(stream)),
           "sc_matmul_prepared")


def sc_workspace_bytes_batched(B, M, K, N, Lmax, params) -> int:
    return int(load().sc_workspace_bytes_batched(B, M, K, N, Lmax, ctypes.byref(params)))


def sc_matmul_batched(ctx, A, W, w_transposed, L, Lmax, params, P, C, ws, stream=None):
    B, M, K = A.shape
    N = W.shape[1] if w_transposed else W.shape[2]
    assert W.shape[0] == B and (W.shape[2] if w_transposed else W.shape[1]) == K
    _check(load().sc_matmul_batched(ctx, _ptr(A), _ptr(W), B, M, K, N, 1 if w_transposed else 0, _ptr(L), Lmax,
                                    ctypes.byref(params), _ptr(P), _ptr(C), _ptr(ws), ws.numel() * ws.element_size(),
                                    _stream_handle(stream)), "sc_matmul_batched")


def sc_workspace_bytes_cbsg(M, K, N, Lmax, params) -> int:
    return int(load().sc_workspace_bytes_cbsg(M, K, N, Lmax, ctypes.byref(params)))


def sc_matmul_cbsg(ctx, A, W, L, Lmax, params, P, C, ws, stream=None):
    M, K = A.shape
    K2, N = W.shape
    assert K == K2
    _check(load().sc_matmul_cbsg(ctx, _ptr(A), _ptr(W), M, K, N, _ptr(L), Lmax, ctypes.byref(params), _ptr(P), _ptr(C),
                                 _ptr(ws), ws.numel() * ws.element_size(), _stream_handle(stream)), "sc_matmul_cbsg")


def sc_cbsg_scc(ctx, Ta, Tw, L, seed, stream_id, counts, scc, ws, stream=None):
    _check(load().sc_cbsg_scc(ctx, _ptr(Ta), _ptr(Tw), Ta.numel(), L, seed, stream_id, _ptr(counts), _ptr(scc), _ptr(ws),
                              ws.numel() * ws.element_size(), _stream_handle(stream)), "sc_cbsg_scc")


SC_SURROGATE_COEFF = 2.324


def sc_surrogate_noise(ctx, Y, L, group, coeff, seed, stream_id, out, stream=None):
    M, N = Y.shape
    _check(load().sc_surrogate_noise(ctx, _ptr(Y), M, N, _ptr(L), group, float(coeff), seed, stream_id, _ptr(out),
                                     _stream_handle(stream)), "sc_surrogate_noise")


def sc_selftest_comparator() -> int:
    return int(load().sc_selftest_comparator())


def sc_selftest_expansion() -> int:
    return int(load().sc_selftest_expansion())


def sc_selftest_bounded_wait(ctx, limit_cycles: int):
    """Returns (site word, counter a, counter b), (clocks waited by the timed-out warp, by the aborted warp)."""
    site, cyc = (ctypes.c_int32 * 3)(), (ctypes.c_int64 * 2)()
    _check(load().sc_selftest_bounded_wait(ctx, int(limit_cycles), site, cyc), "sc_selftest_bounded_wait")
    return tuple(int(x) for x in site), tuple(int(x) for x in cyc)


def sc_microbench(ctx, kind: int, iters: int):
    ms, words = ctypes.c_float(0), ctypes.c_double(0)
    _check(load().sc_microbench(ctx, kind, iters, ctypes.byref(ms), ctypes.byref(words)), "sc_microbench")
    return float(ms.value), float(words.value)


PROFILE_PHASES = ("scales", "plan", "encode_a", "encode_w", "core", "decode", "total", "reserved")


def sc_profile_enable(ctx, on: bool):
    _check(load().sc_profile_enable(ctx, 1 if on else 0), "sc_profile_enable")


def sc_profile_read(ctx) -> dict:
    ms = (ctypes.c_float * 8)()
    _check(load().sc_profile_read(ctx, ms), "sc_profile_read")
    return {name: float(ms[k]) for k, name in enumerate(PROFILE_PHASES) if name != "reserved"}


def sc_last_core_selected(ctx) -> int:
    v = ctypes.c_int32(0)
    _check(load().sc_last_core_selected(ctx, ctypes.byref(v)), "sc_last_core_selected")
    return int(v.value)


def sc_launch_count(ctx) -> int:
    n = ctypes.c_int64(0)
    _check(load().sc_launch_count(ctx, ctypes.byref(n)), "sc_launch_count")
    return int(n.value)


SC_STATIC_MAX_GROUPS = 262144


def sc_assign_lengths_static(g, group, avg_budget, Lmin, Lmax, L_out, status_out=None, total_out=None, stream=None):
    """Context-free, allocation-free length assignment: every buffer is the caller's, the scratch is a
    fixed array inside the library.  For callers that may not allocate device memory."""
    _check(load().sc_assign_lengths_static(_ptr(g), g.numel(), group, float(avg_budget), Lmin, Lmax, _ptr(L_out),
                                           _ptr(status_out), _ptr(total_out), _stream_handle(stream)),
           "sc_assign_lengths_static")


# ---- convenience: owns a context and the torch buffers of repeated calls -------------------------------
class ScGemm:
    """Holds a library context on one device plus a reusable workspace; methods only allocate and call."""

    def __init__(self, device: int = 0):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: the SC-GEMM library has no CPU path")
        self.torch = torch
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        self.ctx = sc_create(device)
        self._ws = None

    def close(self):
        if self.ctx:
            sc_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def workspace(self, nbytes: int):
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = None
            self._ws = self.torch.empty(nbytes, dtype=self.torch.uint8, device=self.device)
        return self._ws

    def row_stats(self, A):
        g = self.torch.empty(A.shape[0], dtype=self.torch.float32, device=self.device)
        sc_row_stats(self.ctx, A, g)
        return g

    def assign_lengths(self, g, group, avg_budget, Lmin, Lmax, want_realized=False):
        n = (g.numel() + group - 1) // group
        L = self.torch.empty(n, dtype=self.torch.int32, device=self.device)
        r = sc_assign_lengths(self.ctx, g, group, avg_budget, Lmin, Lmax, L, want_realized)
        return (L, r) if want_realized else L

    def ladder_lengths(self, g, group, ladder, tau):
        n = (g.numel() + group - 1) // group
        L = self.torch.empty(n, dtype=self.torch.int32, device=self.device)
        sc_ladder_lengths(self.ctx, g, group, ladder, tau, L)
        return L

    def matmul(self, A, W, L, Lmax, params, want_P=True, out_C=None, out_P=None):
        M, K = A.shape
        N = W.shape[1]
        t = self.torch
        C = out_C if out_C is not None else t.empty((M, N), dtype=t.float32, device=self.device)
        P = out_P if out_P is not None else (t.empty((M, N), dtype=t.int32, device=self.device) if want_P else None)
        ws = self.workspace(sc_workspace_bytes(M, K, N, Lmax, params))
        sc_matmul(self.ctx, A, W, L, Lmax, params, P, C, ws)
        return P, C

    def matmul_batched(self, A, W, w_transposed, L, Lmax, params, want_P=True):
        B, M, K = A.shape
        N = W.shape[1] if w_transposed else W.shape[2]
        t = self.torch
        C = t.empty((B, M, N), dtype=t.float32, device=self.device)
        P = t.empty((B, M, N), dtype=t.int32, device=self.device) if want_P else None
        ws = self.workspace(sc_workspace_bytes_batched(B, M, K, N, Lmax, params))
        sc_matmul_batched(self.ctx, A, W, w_transposed, L, Lmax, params, P, C, ws)
        return P, C

    def matmul_cbsg(self, A, W, L, Lmax, params, want_P=True):
        M, K = A.shape
        N = W.shape[1]
        t = self.torch
        C = t.empty((M, N), dtype=t.float32, device=self.device)
        P = t.empty((M, N), dtype=t.int32, device=self.device) if want_P else None
        ws = self.workspace(sc_workspace_bytes_cbsg(M, K, N, Lmax, params))
        sc_matmul_cbsg(self.ctx, A, W, L, Lmax, params, P, C, ws)
        return P, C

    def prepare_weights(self, W, Lmax, params):
        """Returns (record, buffer, (K, N)); keep the buffer alive while the record is in use."""
        K, N = W.shape
        wbuf = self.torch.empty(sc_weights_bytes(K, N, Lmax, params), dtype=self.torch.uint8, device=self.device)
        return sc_weights_prepare(self.ctx, W, Lmax, params, wbuf), wbuf, (K, N)

    def matmul_prepared(self, A, prepared, L, Lmax, params, want_P=True, out_C=None, out_P=None):
        record, _wbuf, (K, N) = prepared
        M = A.shape[0]
        t = self.torch
        C = out_C if out_C is not None else t.empty((M, N), dtype=t.float32, device=self.device)
        P = out_P if out_P is not None else (t.empty((M, N), dtype=t.int32, device=self.device) if want_P else None)
        ws = self.workspace(sc_workspace_bytes_prepared(M, K, N, Lmax, params))
        sc_matmul_prepared(self.ctx, A, record, L, Lmax, params, P, C, ws)
        return P, C

    def encode(self, X, tensor_id, L_or_none, Lmax, params):
        t = self.torch
        rows, cols = X.shape
        stream_rows, depth = (rows, cols) if tensor_id == 0 else (cols, rows)
        streams = t.empty(sc_stream_bytes(stream_rows, depth, Lmax, params.mode), dtype=t.uint8, device=self.device)
        scales = t.empty(stream_rows, dtype=t.float32, device=self.device)
        sc_encode(self.ctx, X, tensor_id, L_or_none, Lmax, params, streams, scales)
        return streams, scales

    def unpack(self, streams, stream_rows, depth, Lmax, mode):
        t = self.torch
        bits = t.empty((stream_rows, depth, Lmax), dtype=t.uint8, device=self.device)
        neg = t.empty((stream_rows, depth, Lmax), dtype=t.uint8, device=self.device) if mode == SC_UNIPOLAR_AND else None
        sc_debug_unpack(self.ctx, streams, stream_rows, depth, Lmax, mode, bits, neg)
        return bits, neg

    def device_status(self) -> int:
        return sc_device_status(self.ctx)

"""ctypes front end of the CPU oracle (``sc_oracle.c``).

TEST INFRASTRUCTURE ONLY: the test-suite, the smoke check and the benchmark's
cpu-baseline leg may import this module; the CUDA library and its Python binding
must not.  Nothing here computes: every function marshals numpy arrays into the C
oracle and chains its steps in the order of the paper (scales -> encode -> gate and
popcount -> decode, Sec. 3.1, Sec. 4.2 and Eq. (1); length assignment, Sec. 4.4).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sc_oracle.c")
_LIB = os.path.join(_HERE, "libsc_oracle.so")

BIPOLAR_XNOR = 0
UNIPOLAR_AND = 1
SCALE_NONE = 0
SCALE_PER_ROW = 1      # A: per row of A; W: per output column of W (a row of B in C = A B^T)
SCALE_PER_TENSOR = 2

OK, ERR_ARG, ERR_LENGTH, ERR_NONFINITE, ERR_BUDGET = 0, 1, 3, 4, 5

_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math, no FMA contraction); returns the .so path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".%d.tmp" % os.getpid()
            cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
                   "-fno-fast-math", "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    lib = ctypes.CDLL(_LIB)
    c = ctypes
    f32p, i32p, i64p, u8p, u32p = (c.POINTER(c.c_float), c.POINTER(c.c_int32), c.POINTER(c.c_int64),
                                   c.POINTER(c.c_uint8), c.POINTER(c.c_uint32))
    lib.sco_philox4x32_10.argtypes = [u32p, u32p, u32p]
    lib.sco_philox4x32_10.restype = None
    lib.sco_normalise.argtypes = [c.c_float, c.c_float]
    lib.sco_normalise.restype = c.c_float
    lib.sco_boundary_bipolar.argtypes = [c.c_float]
    lib.sco_boundary_bipolar.restype = c.c_int32
    lib.sco_boundary_unipolar.argtypes = [c.c_float, i32p]
    lib.sco_boundary_unipolar.restype = c.c_int32
    lib.sco_boundary_bipolar_int8.argtypes = [c.c_float]
    lib.sco_boundary_bipolar_int8.restype = c.c_int32
    lib.sco_boundary_unipolar_int8.argtypes = [c.c_float, i32p]
    lib.sco_boundary_unipolar_int8.restype = c.c_int32
    lib.sco_random_byte.argtypes = [c.c_uint64, c.c_uint32, c.c_int32, c.c_uint64, c.c_int32]
    lib.sco_random_byte.restype = c.c_uint32
    lib.sco_stream_bit.argtypes = [c.c_uint64, c.c_uint32, c.c_int32, c.c_uint64, c.c_int32, c.c_int32]
    lib.sco_stream_bit.restype = c.c_int32
    for name in ("sco_scales_rows", "sco_scales_cols"):
        getattr(lib, name).argtypes = [f32p, c.c_int64, c.c_int64, f32p]
        getattr(lib, name).restype = c.c_int32
    lib.sco_scale_tensor.argtypes = [f32p, c.c_int64, f32p]
    lib.sco_scale_tensor.restype = c.c_int32
    lib.sco_row_absmax.argtypes = [f32p, c.c_int64, c.c_int64, f32p]
    lib.sco_row_absmax.restype = None
    lib.sco_encode.argtypes = [f32p, c.c_int64, c.c_int64, i64p, c.c_int64, i64p, c.c_int64,
                               c.c_int32, c.c_int32, f32p, f32p, c.c_float,
                               c.c_uint64, c.c_uint32, c.c_int32, u8p, i32p, u8p]
    lib.sco_encode.restype = c.c_int32
    lib.sco_encode_quant.argtypes = [f32p, c.c_int64, c.c_int64, i64p, c.c_int64, i64p, c.c_int64,
                                     c.c_int32, c.c_int32, c.c_int32, f32p, f32p, c.c_float,
                                     c.c_uint64, c.c_uint32, c.c_int32, u8p, i32p, u8p]
    lib.sco_encode_quant.restype = c.c_int32
    lib.sco_gate_accumulate.argtypes = [c.c_int32, u8p, u8p, c.c_int32, u8p, u8p, c.c_int32,
                                        c.c_int64, c.c_int64, c.c_int64, i32p, i32p]
    lib.sco_gate_accumulate.restype = c.c_int32
    lib.sco_decode.argtypes = [c.c_int32, i32p, c.c_int64, c.c_int64, c.c_int64, i32p, f32p, f32p, f32p]
    lib.sco_decode.restype = None
    lib.sco_assign_lengths.argtypes = [f32p, c.c_int64, c.c_int32, c.c_double, c.c_int32, c.c_int32,
                                       i32p, c.POINTER(c.c_double)]
    lib.sco_assign_lengths.restype = c.c_int32
    lib.sco_ladder_lengths.argtypes = [f32p, c.c_int64, c.c_int32, i32p, f32p, c.c_int32, i32p]
    lib.sco_ladder_lengths.restype = c.c_int32
    lib.sco_sobol8.argtypes = [c.c_int32, c.c_uint32]
    lib.sco_sobol8.restype = c.c_uint32
    lib.sco_cbsg_scramble.argtypes = [c.c_uint64, c.c_uint32, u8p]
    lib.sco_cbsg_scramble.restype = None
    lib.sco_cbsg_pair.argtypes = [c.c_int32, c.c_int32, c.c_int32, u8p, i32p]
    lib.sco_cbsg_pair.restype = c.c_int32
    lib.sco_scc.argtypes = [c.c_int32] * 4
    lib.sco_scc.restype = c.c_double
    lib.sco_cbsg_gate_accumulate.argtypes = [i32p, i32p, c.c_int64, c.c_int64, c.c_int64, i32p, c.c_uint64, c.c_uint32, i32p]
    lib.sco_cbsg_gate_accumulate.restype = c.c_int32
    lib.sco_standard_normal.argtypes = [c.c_uint64, c.c_uint32, c.c_uint64]
    lib.sco_standard_normal.restype = c.c_double
    lib.sco_surrogate_noise.argtypes = [f32p, c.c_int64, c.c_int64, i32p, c.c_double, c.c_uint64, c.c_uint32, f32p]
    lib.sco_surrogate_noise.restype = c.c_int32
    _lib = lib
    return lib


class OracleError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__("oracle %s failed with code %d" % (where, code))
        self.code = code


def _ptr(a, ctype):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctype))


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def num_threads() -> int:
    """Threads the OpenMP loops of the oracle use (OMP_NUM_THREADS, else the cores this process may run on)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    return len(os.sched_getaffinity(0))


# --------------------------------------------------------------------------- scalar steps
def philox4x32_10(counter, key):
    ctr = np.asarray(counter, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    _load().sco_philox4x32_10(_ptr(ctr, ctypes.c_uint32), _ptr(k, ctypes.c_uint32), _ptr(out, ctypes.c_uint32))
    return out


def normalise(x: float, sigma: float) -> float:
    return float(_load().sco_normalise(float(x), float(sigma)))


def boundary_bipolar(v: float) -> int:
    return int(_load().sco_boundary_bipolar(float(v)))


def boundary_unipolar(v: float):
    s = ctypes.c_int32(0)
    t = int(_load().sco_boundary_unipolar(float(v), ctypes.byref(s)))
    return t, int(s.value)


QUANT_DIRECT257, QUANT_INT8_THEN_257 = 0, 1


def boundary_bipolar_int8(v: float) -> int:
    """Sec. 4.2 two-step variant: int8 grid (q_max = 127) first, then the nearest of the 257 boundaries."""
    return int(_load().sco_boundary_bipolar_int8(float(v)))


def boundary_unipolar_int8(v: float):
    s = ctypes.c_int32(0)
    t = int(_load().sco_boundary_unipolar_int8(float(v), ctypes.byref(s)))
    return t, int(s.value)


def random_byte(seed: int, stream_id: int, tensor_id: int, elem: int, l: int) -> int:
    return int(_load().sco_random_byte(seed, stream_id, tensor_id, elem, l))


def stream_bit(seed: int, stream_id: int, tensor_id: int, elem: int, l: int, T: int) -> int:
    return int(_load().sco_stream_bit(seed, stream_id, tensor_id, elem, l, T))


# --------------------------------------------------------------------------- tensor steps
def scales(X, kind: int, axis: str):
    """sigma for a tensor. ``axis`` = 'row' (A: one per row) or 'col' (W: one per output column)."""
    X = _f32(X)
    rows, cols = X.shape
    lib = _load()
    if kind == SCALE_NONE:
        s = ctypes.c_float(0)                      # only for the non-finite check; sigma stays 1
        code = lib.sco_scale_tensor(_ptr(X, ctypes.c_float), X.size, ctypes.byref(s))
        sig = np.ones(rows if axis == "row" else cols, dtype=np.float32)
    elif kind == SCALE_PER_TENSOR:
        s = ctypes.c_float(0)
        code = lib.sco_scale_tensor(_ptr(X, ctypes.c_float), X.size, ctypes.byref(s))
        sig = np.full(rows if axis == "row" else cols, s.value, dtype=np.float32)
    elif kind == SCALE_PER_ROW:
        sig = np.zeros(rows if axis == "row" else cols, dtype=np.float32)
        fn = lib.sco_scales_rows if axis == "row" else lib.sco_scales_cols
        code = fn(_ptr(X, ctypes.c_float), rows, cols, _ptr(sig, ctypes.c_float))
    else:
        raise ValueError("scale kind")
    if code != OK:
        raise OracleError(code, "scales")
    return sig


def row_absmax(X):
    X = _f32(X)
    g = np.zeros(X.shape[0], dtype=np.float32)
    _load().sco_row_absmax(_ptr(X, ctypes.c_float), X.shape[0], X.shape[1], _ptr(g, ctypes.c_float))
    return g


def encode(X, tensor_id: int, mode: int, L: int, seed: int, stream_id: int = 0,
           sigma_row=None, sigma_col=None, sigma_tensor: float = 1.0, row_sel=None, col_sel=None, quant: int = 0):
    """Streams of X[row_sel, col_sel]: returns (bits[nr, nc, L] uint8, T[nr, nc] int32, sign[nr, nc] uint8)."""
    X = _f32(X)
    rows, cols = X.shape
    rs = None if row_sel is None else np.ascontiguousarray(row_sel, dtype=np.int64)
    cs = None if col_sel is None else np.ascontiguousarray(col_sel, dtype=np.int64)
    nr = rows if rs is None else rs.size
    nc = cols if cs is None else cs.size
    bits = np.zeros((nr, nc, max(L, 0)), dtype=np.uint8)
    T = np.zeros((nr, nc), dtype=np.int32)
    sign = np.zeros((nr, nc), dtype=np.uint8)
    sr = None if sigma_row is None else _f32(sigma_row)
    sc = None if sigma_col is None else _f32(sigma_col)
    code = _load().sco_encode_quant(_ptr(X, ctypes.c_float), rows, cols, _ptr(rs, ctypes.c_int64), nr,
                              _ptr(cs, ctypes.c_int64), nc, tensor_id, mode, quant,
                              _ptr(sr, ctypes.c_float), _ptr(sc, ctypes.c_float), float(sigma_tensor),
                              seed, stream_id, L, _ptr(bits, ctypes.c_uint8), _ptr(T, ctypes.c_int32),
                              _ptr(sign, ctypes.c_uint8))
    if code != OK:
        raise OracleError(code, "encode")
    return bits, T, sign


def gate_accumulate(mode: int, abits, asign, wbits, wsign, L_rows):
    """abits[m, K, La], wbits[K, n, Lw] (uint8 0/1) -> int32 popcount accumulators [m, n] (Eq. (1))."""
    abits = np.ascontiguousarray(abits, dtype=np.uint8)
    wbits = np.ascontiguousarray(wbits, dtype=np.uint8)
    m, K, La = abits.shape
    K2, n, Lw = wbits.shape
    assert K == K2
    L_rows = np.ascontiguousarray(L_rows, dtype=np.int32)
    assert L_rows.shape == (m,)
    a_s = None if asign is None else np.ascontiguousarray(asign, dtype=np.uint8)
    w_s = None if wsign is None else np.ascontiguousarray(wsign, dtype=np.uint8)
    P = np.zeros((m, n), dtype=np.int32)
    code = _load().sco_gate_accumulate(mode, _ptr(abits, ctypes.c_uint8), _ptr(a_s, ctypes.c_uint8), La,
                                       _ptr(wbits, ctypes.c_uint8), _ptr(w_s, ctypes.c_uint8), Lw,
                                       m, K, n, _ptr(L_rows, ctypes.c_int32), _ptr(P, ctypes.c_int32))
    if code != OK:
        raise OracleError(code, "gate_accumulate")
    return P


def decode(mode: int, P, K: int, L_rows, sigma_a, sigma_w):
    P = np.ascontiguousarray(P, dtype=np.int32)
    m, n = P.shape
    L_rows = np.ascontiguousarray(L_rows, dtype=np.int32)
    sa, sw = _f32(sigma_a), _f32(sigma_w)
    assert sa.shape == (m,) and sw.shape == (n,) and L_rows.shape == (m,)
    C = np.zeros((m, n), dtype=np.float32)
    _load().sco_decode(mode, _ptr(P, ctypes.c_int32), m, n, K, _ptr(L_rows, ctypes.c_int32),
                       _ptr(sa, ctypes.c_float), _ptr(sw, ctypes.c_float), _ptr(C, ctypes.c_float))
    return C


def expand_lengths(L_groups, M: int, group: int):
    """Entry g of L_groups applies to rows [g*group, (g+1)*group)."""
    L_groups = np.asarray(L_groups, dtype=np.int32)
    return np.repeat(L_groups, group)[:M].copy()


def matmul(A, W, L_rows, mode: int, scale_a: int, scale_w: int, seed: int, stream_id: int = 0,
           row_sel=None, col_sel=None, quant: int = 0):
    """The whole path on the output entries (row_sel x col_sel): returns dict(P, C, sigma_a, sigma_w).

    ``L_rows`` has one entry per row of A (already expanded from groups).  Scales are always taken
    over the full tensors; streams are generated for the selected rows / columns only, with the
    element indices of the full tensors, so the entries equal those of a full evaluation.
    """
    A, W = _f32(A), _f32(W)
    M, K = A.shape
    K2, N = W.shape
    assert K == K2
    L_rows = np.ascontiguousarray(L_rows, dtype=np.int32)
    assert L_rows.shape == (M,)
    rs = np.arange(M, dtype=np.int64) if row_sel is None else np.ascontiguousarray(row_sel, dtype=np.int64)
    cs = np.arange(N, dtype=np.int64) if col_sel is None else np.ascontiguousarray(col_sel, dtype=np.int64)
    sig_a = scales(A, scale_a, "row")
    sig_w = scales(W, scale_w, "col")
    Lsel = L_rows[rs]
    Lmax = int(Lsel.max()) if Lsel.size else 0
    abits, _, asign = encode(A, 0, mode, Lmax, seed, stream_id, sigma_row=sig_a, row_sel=rs, quant=quant)
    wbits, _, wsign = encode(W, 1, mode, Lmax, seed, stream_id, sigma_col=sig_w, col_sel=cs, quant=quant)
    P = gate_accumulate(mode, abits, asign, wbits, wsign, Lsel)
    C = decode(mode, P, K, Lsel, sig_a[rs], sig_w[cs])
    return {"P": P, "C": C, "sigma_a": sig_a, "sigma_w": sig_w}


def assign_lengths(g, group: int, avg_budget: float, Lmin: int, Lmax: int):
    """Sec. 4.4 length assignment: returns (L per group, realised average over rows)."""
    g = _f32(g)
    M = g.size
    ngroups = (M + group - 1) // group
    L = np.zeros(ngroups, dtype=np.int32)
    avg = ctypes.c_double(0)
    code = _load().sco_assign_lengths(_ptr(g, ctypes.c_float), M, group, float(avg_budget), Lmin, Lmax,
                                      _ptr(L, ctypes.c_int32), ctypes.byref(avg))
    if code != OK:
        raise OracleError(code, "assign_lengths")
    return L, float(avg.value)


def ladder_lengths(g, group: int, ladder, tau):
    g = _f32(g)
    M = g.size
    ladder = np.ascontiguousarray(ladder, dtype=np.int32)
    tau = np.ascontiguousarray(tau, dtype=np.float32)
    assert tau.size == ladder.size - 1
    L = np.zeros((M + group - 1) // group, dtype=np.int32)
    code = _load().sco_ladder_lengths(_ptr(g, ctypes.c_float), M, group, _ptr(ladder, ctypes.c_int32),
                                      _ptr(tau if tau.size else None, ctypes.c_float), ladder.size,
                                      _ptr(L, ctypes.c_int32))
    if code != OK:
        raise OracleError(code, "ladder_lengths")
    return L


SURROGATE_COEFF = 2.324    # alpha(L) = 2.324 / L reproduces the printed alpha column of Sec. 3.2's table


def standard_normal(seed: int, stream_id: int, cell: int) -> float:
    return float(_load().sco_standard_normal(seed, stream_id, cell))


def surrogate_noise(Y, L_rows, coeff: float, seed: int, stream_id: int = 0):
    """Sec. 3.2: Y (1 + (coeff / L_i) Z) with Z standard normal per output cell; rows with L = 0 give 0."""
    Y = _f32(Y)
    M, N = Y.shape
    L_rows = np.ascontiguousarray(L_rows, dtype=np.int32)
    assert L_rows.size == M
    out = np.zeros((M, N), dtype=np.float32)
    code = _load().sco_surrogate_noise(_ptr(Y, ctypes.c_float), M, N, _ptr(L_rows, ctypes.c_int32), float(coeff), seed,
                                       stream_id, _ptr(out, ctypes.c_float))
    if code != OK:
        raise OracleError(code, "surrogate_noise")
    return out


def matmul_batched(A, W, L_rows, mode: int, scale_a: int, scale_w: int, seed: int, stream_id: int = 0,
                   w_transposed: bool = False, batches=None):
    """B independent products C_b = A_b W_b (attention per head: Q K^T with the keys given as rows,
    probabilities times V), as a composition of the single-product steps above.

    ``A`` is [B, M, K]; ``W`` is [B, K, N], or [B, N, K] with ``w_transposed`` (the weight operand is then
    stored with its output columns as rows).  ``L_rows`` has one entry per stacked row b*M + i.  The stream
    of an element is indexed by its position in the caller's tensor as stored (flat index); scales are
    per stacked row of A, per (product, output column) of W, or per whole tensor.  ``batches`` restricts
    the evaluation to some products (their entries are those of a full evaluation).
    Returns dict(P[B', M, N], C[B', M, N], sigma_a[B*M], sigma_w[B*N]).
    """
    A, W = np.ascontiguousarray(A, dtype=np.float32), np.ascontiguousarray(W, dtype=np.float32)
    B, M, K = A.shape
    if w_transposed:
        B2, N, K2 = W.shape
    else:
        B2, K2, N = W.shape
    assert B == B2 and K == K2
    L_rows = np.ascontiguousarray(L_rows, dtype=np.int32)
    assert L_rows.shape == (B * M,)
    A2 = A.reshape(B * M, K)                                   # stacked rows: element index (b M + i) K + d
    sig_a = scales(A2, scale_a, "row")
    if w_transposed:
        W2 = W.reshape(B * N, K)                               # element index (b N + j) K + d
        sig_w = scales(W2, scale_w, "row")                     # one per (product, output column)
    else:
        W2 = W.reshape(B * K, N)                               # element index (b K + d) N + j
        if scale_w == SCALE_PER_ROW:
            sig_w = np.concatenate([scales(W[b], scale_w, "col") for b in range(B)])
        else:
            sig_w = np.tile(scales(W2, scale_w, "col"), B)     # the whole-tensor scale (or 1), repeated
    which = range(B) if batches is None else list(batches)
    P_all, C_all = [], []
    for b in which:
        rows = b * M + np.arange(M, dtype=np.int64)
        Lb = L_rows[rows]
        Lmax = int(Lb.max()) if Lb.size else 0
        abits, _, asign = encode(A2, 0, mode, Lmax, seed, stream_id, sigma_row=sig_a, row_sel=rows)
        if w_transposed:
            wrows = b * N + np.arange(N, dtype=np.int64)
            wb, _, ws = encode(W2, 1, mode, Lmax, seed, stream_id, sigma_row=sig_w, row_sel=wrows)
            wbits, wsign = np.ascontiguousarray(wb.transpose(1, 0, 2)), np.ascontiguousarray(ws.T)
        else:
            wrows = b * K + np.arange(K, dtype=np.int64)
            wbits, _, wsign = encode(W2, 1, mode, Lmax, seed, stream_id, sigma_col=sig_w[b * N:(b + 1) * N],
                                     row_sel=wrows)
        P = gate_accumulate(mode, abits, asign, wbits, wsign, Lb)
        P_all.append(P)
        C_all.append(decode(mode, P, K, Lb, sig_a[rows], sig_w[b * N:(b + 1) * N]))
    return {"P": np.stack(P_all), "C": np.stack(C_all), "sigma_a": sig_a, "sigma_w": sig_w}


# ---- Sec. 4.2 / Appendix A.1: Sobol-8 streams with conditional bitstream generation ---------------------
def sobol8(dim: int, n: int) -> int:
    return int(_load().sco_sobol8(dim, n))


def cbsg_scramble(seed: int, stream_id: int = 0):
    out = np.zeros(3, dtype=np.uint8)
    _load().sco_cbsg_scramble(seed, stream_id, _ptr(out, ctypes.c_uint8))
    return out


def cbsg_pair(Ta: int, Tw: int, L: int, scr):
    """One multiplier run: (XNOR count, [n11, n10, n01, n00])."""
    scr = np.ascontiguousarray(scr, dtype=np.uint8)
    counts = np.zeros(4, dtype=np.int32)
    p = _load().sco_cbsg_pair(Ta, Tw, L, _ptr(scr, ctypes.c_uint8), _ptr(counts, ctypes.c_int32))
    return int(p), counts


def scc(a: int, b: int, c: int, d: int) -> float:
    return float(_load().sco_scc(a, b, c, d))


def matmul_cbsg(A, W, L_rows, scale_a: int, scale_w: int, seed: int, stream_id: int = 0, row_sel=None, col_sel=None,
                quant: int = 0):
    """Bipolar SC product with the Sobol-8 / conditional-generation streams: dict(P, C, sigma_a, sigma_w)."""
    A, W = _f32(A), _f32(W)
    M, K = A.shape
    K2, N = W.shape
    assert K == K2
    L_rows = np.ascontiguousarray(L_rows, dtype=np.int32)
    rs = np.arange(M, dtype=np.int64) if row_sel is None else np.ascontiguousarray(row_sel, dtype=np.int64)
    cs = np.arange(N, dtype=np.int64) if col_sel is None else np.ascontiguousarray(col_sel, dtype=np.int64)
    sig_a = scales(A, scale_a, "row")
    sig_w = scales(W, scale_w, "col")
    _, Ta, _ = encode(A, 0, BIPOLAR_XNOR, 0, seed, stream_id, sigma_row=sig_a, row_sel=rs, quant=quant)   # boundaries only
    _, Tw, _ = encode(W, 1, BIPOLAR_XNOR, 0, seed, stream_id, sigma_col=sig_w, col_sel=cs, quant=quant)
    Lsel = np.ascontiguousarray(L_rows[rs])
    P = np.zeros((rs.size, cs.size), dtype=np.int32)
    code = _load().sco_cbsg_gate_accumulate(_ptr(np.ascontiguousarray(Ta), ctypes.c_int32),
                                            _ptr(np.ascontiguousarray(Tw), ctypes.c_int32), rs.size, K, cs.size,
                                            _ptr(Lsel, ctypes.c_int32), seed, stream_id, _ptr(P, ctypes.c_int32))
    if code != OK:
        raise OracleError(code, "matmul_cbsg")
    C = decode(BIPOLAR_XNOR, P, K, Lsel, sig_a[rs], sig_w[cs])
    return {"P": P, "C": C, "sigma_a": sig_a, "sigma_w": sig_w}

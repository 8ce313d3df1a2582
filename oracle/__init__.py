"""ctypes front end of the CPU oracle (``tsid_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this module;
it is used by the tests, by the smoke check and by the bench's CPU-baseline leg.
The arithmetic lives in the C file; this module only builds it with gcc,
marshals numpy arrays and returns numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tsid_oracle.c")
_LIB = os.path.join(_HERE, "libtsid_oracle.so")

CLIP_NONE, CLIP_ASYM_STEP, CLIP_ASYM_GRAD, CLIP_ASYM_ENTRY = 0, 1, 2, 3
NORM_NONE, NORM_COUNT = 0, 1
# levels of the emulation switch (argument bf16_emulate; True means EMU_BF16)
EMU_NONE, EMU_BF16, EMU_TENSOR = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, no fast-math).  Returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_bf16_round.restype = C.c_float
        _lib.orc_bf16_round.argtypes = [C.c_float]
        _lib.orc_fp16_round.restype = C.c_float
        _lib.orc_fp16_round.argtypes = [C.c_float]
        _lib.orc_clip_nested.restype = C.c_double
        _lib.orc_clip_nested.argtypes = [C.c_double, C.c_double]
    return _lib


def _p(a, ct):
    return a.ctypes.data_as(C.POINTER(ct))


def _coo(rows, cols, vals):
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    cols = np.ascontiguousarray(cols, dtype=np.int32)
    vals = np.ascontiguousarray(vals, dtype=np.float32)
    assert rows.shape == cols.shape == vals.shape and rows.ndim == 1
    return rows, cols, vals


def _fac(X, nrow, k):
    X = np.ascontiguousarray(X, dtype=np.float32)
    assert X.shape == (nrow, k), (X.shape, nrow, k)
    return X


def bf16_round(x: float) -> float:
    return float(_L().orc_bf16_round(C.c_float(x)))


def fp16_round(x: float) -> float:
    return float(_L().orc_fp16_round(C.c_float(x)))


def clip_nested(g: float, xi: float) -> float:
    return float(_L().orc_clip_nested(g, xi))


def residuals(m, n, k, rows, cols, vals, P, Q, bf16_emulate=False):
    rows, cols, vals = _coo(rows, cols, vals)
    P, Q = _fac(P, m, k), _fac(Q, n, k)
    e = np.empty(rows.shape[0], dtype=np.float64)
    _L().orc_residuals(C.c_int32(m), C.c_int32(n), C.c_int32(k), C.c_int64(rows.shape[0]),
                       _p(rows, C.c_int32), _p(cols, C.c_int32), _p(vals, C.c_float),
                       _p(P, C.c_float), _p(Q, C.c_float), C.c_int(int(bf16_emulate)),
                       _p(e, C.c_double))
    return e


@dataclass
class Step:
    GP: np.ndarray  # raw sums E Q, float64 (m, k)
    GQ: np.ndarray  # raw sums E^T P, float64 (n, k)
    DP: np.ndarray  # clipped direction, float64
    DQ: np.ndarray
    P: np.ndarray   # updated factors, float32
    Q: np.ndarray


def grad_step(m, n, k, rows, cols, vals, P, Q, eta, lam, xi,
              clip=CLIP_NONE, norm_p=NORM_NONE, norm_q=NORM_NONE, bf16_emulate=False) -> Step:
    rows, cols, vals = _coo(rows, cols, vals)
    P, Q = _fac(P, m, k), _fac(Q, n, k)
    GP = np.empty((m, k)); GQ = np.empty((n, k)); DP = np.empty((m, k)); DQ = np.empty((n, k))
    Pn = np.empty((m, k), dtype=np.float32); Qn = np.empty((n, k), dtype=np.float32)
    _L().orc_grad_step(C.c_int32(m), C.c_int32(n), C.c_int32(k), C.c_int64(rows.shape[0]),
                       _p(rows, C.c_int32), _p(cols, C.c_int32), _p(vals, C.c_float),
                       _p(P, C.c_float), _p(Q, C.c_float),
                       C.c_double(eta), C.c_double(lam), C.c_double(xi),
                       C.c_int(clip), C.c_int(norm_p), C.c_int(norm_q), C.c_int(int(bf16_emulate)),
                       _p(GP, C.c_double), _p(GQ, C.c_double), _p(DP, C.c_double), _p(DQ, C.c_double),
                       _p(Pn, C.c_float), _p(Qn, C.c_float))
    return Step(GP, GQ, DP, DQ, Pn, Qn)


def loss(m, n, k, rows, cols, vals, P, Q, lam, bf16_emulate=False):
    """Returns (SSE, objective)."""
    rows, cols, vals = _coo(rows, cols, vals)
    P, Q = _fac(P, m, k), _fac(Q, n, k)
    sse = C.c_double(0.0); obj = C.c_double(0.0)
    _L().orc_loss(C.c_int32(m), C.c_int32(n), C.c_int32(k), C.c_int64(rows.shape[0]),
                  _p(rows, C.c_int32), _p(cols, C.c_int32), _p(vals, C.c_float),
                  _p(P, C.c_float), _p(Q, C.c_float), C.c_double(lam), C.c_int(int(bf16_emulate)),
                  C.byref(sse), C.byref(obj))
    return sse.value, obj.value


def fit(m, n, k, rows, cols, vals, P, Q, epochs, eta, lam, xi,
        clip=CLIP_NONE, norm_p=NORM_NONE, norm_q=NORM_NONE, bf16_emulate=False, history=True):
    """Runs `epochs` steps on copies of P, Q.  Returns (P, Q, sse_history or None)."""
    rows, cols, vals = _coo(rows, cols, vals)
    P = _fac(P, m, k).copy(); Q = _fac(Q, n, k).copy()
    hist = np.empty(epochs + 1, dtype=np.float64) if history else None
    _L().orc_fit(C.c_int32(m), C.c_int32(n), C.c_int32(k), C.c_int64(rows.shape[0]),
                 _p(rows, C.c_int32), _p(cols, C.c_int32), _p(vals, C.c_float),
                 _p(P, C.c_float), _p(Q, C.c_float), C.c_int32(epochs),
                 C.c_double(eta), C.c_double(lam), C.c_double(xi),
                 C.c_int(clip), C.c_int(norm_p), C.c_int(norm_q), C.c_int(int(bf16_emulate)),
                 _p(hist, C.c_double) if history else None)
    return P, Q, hist


@dataclass
class Layout:
    row_ptr: np.ndarray  # int64 (m+1)
    col_idx: np.ndarray  # int32 (nnz), CSR order
    val_csr: np.ndarray  # float32
    col_ptr: np.ndarray  # int64 (n+1)
    row_idx: np.ndarray  # int32 (nnz), CSC order
    val_csc: np.ndarray  # float32
    perm: np.ndarray     # uint32: CSR position of CSC entry t


def layout(m, n, rows, cols, vals) -> Layout:
    rows, cols, vals = _coo(rows, cols, vals)
    nnz = rows.shape[0]
    out = Layout(np.empty(m + 1, np.int64), np.empty(nnz, np.int32), np.empty(nnz, np.float32),
                 np.empty(n + 1, np.int64), np.empty(nnz, np.int32), np.empty(nnz, np.float32),
                 np.empty(nnz, np.uint32))
    _L().orc_layout(C.c_int32(m), C.c_int32(n), C.c_int64(nnz),
                    _p(rows, C.c_int32), _p(cols, C.c_int32), _p(vals, C.c_float),
                    _p(out.row_ptr, C.c_int64), _p(out.col_idx, C.c_int32), _p(out.val_csr, C.c_float),
                    _p(out.col_ptr, C.c_int64), _p(out.row_idx, C.c_int32), _p(out.val_csc, C.c_float),
                    _p(out.perm, C.c_uint32))
    return out


def splitmix64_at(seed: int, index1: int) -> int:
    f = _L().orc_splitmix64_at
    f.restype = C.c_uint64
    f.argtypes = [C.c_uint64, C.c_uint64]
    return int(f(seed, index1))


def sample_template(m, n, rows, cols, vals, alpha, seed):
    """Returns (colmap int32[n], rows', cols', vals', d)."""
    rows, cols, vals = _coo(rows, cols, vals)
    nnz = rows.shape[0]
    colmap = np.empty(n, np.int32)
    ro, co, vo = np.empty(nnz, np.int32), np.empty(nnz, np.int32), np.empty(nnz, np.float32)
    d = C.c_int32(0); kept = C.c_int64(0)
    _L().orc_sample_template(C.c_int32(m), C.c_int32(n), C.c_int64(nnz), C.c_double(alpha), C.c_uint64(seed),
                             _p(rows, C.c_int32), _p(cols, C.c_int32), _p(vals, C.c_float),
                             _p(colmap, C.c_int32), _p(ro, C.c_int32), _p(co, C.c_int32), _p(vo, C.c_float),
                             C.byref(d), C.byref(kept))
    k = kept.value
    return colmap, ro[:k].copy(), co[:k].copy(), vo[:k].copy(), d.value


def extend(m, d, k, col_ptr, row_idx, vals, P, Q, eta, lam, iters, C0=None, beta1=0.9, beta2=0.999, eps=1e-8):
    """Stage II (Eq. 10 + Adam).  Returns (C float64 [ncols, d], sse)."""
    col_ptr = np.ascontiguousarray(col_ptr, dtype=np.int64)
    row_idx = np.ascontiguousarray(row_idx, dtype=np.int32)
    vals = np.ascontiguousarray(vals, dtype=np.float32)
    ncols = col_ptr.shape[0] - 1
    P, Q = _fac(P, m, k), _fac(Q, d, k)
    Cm = np.zeros((ncols, d), dtype=np.float64) if C0 is None else np.ascontiguousarray(C0, dtype=np.float64).copy()
    sse = C.c_double(0.0)
    _L().orc_extend(C.c_int32(m), C.c_int32(d), C.c_int32(k), C.c_int32(ncols), _p(col_ptr, C.c_int64),
                    _p(row_idx, C.c_int32), _p(vals, C.c_float), _p(P, C.c_float), _p(Q, C.c_float),
                    C.c_double(eta), C.c_double(lam), C.c_double(beta1), C.c_double(beta2), C.c_double(eps),
                    C.c_int32(iters), _p(Cm, C.c_double), C.byref(sse))
    return Cm, sse.value


def extend_mixed(m, d, k, col_ptr, row_idx, vals, P, Q, eta, lam, iters, C0=None, beta1=0.9, beta2=0.999, eps=1e-8,
                 round_operands=True):
    """Stage II with the operands of its two products rounded to bfloat16 (the paper's mixed precision, Sec. 5.2).
    round_operands=False is the same iteration in full precision.  Returns (C float64 [ncols, d], sse)."""
    col_ptr = np.ascontiguousarray(col_ptr, dtype=np.int64)
    row_idx = np.ascontiguousarray(row_idx, dtype=np.int32)
    vals = np.ascontiguousarray(vals, dtype=np.float32)
    ncols = col_ptr.shape[0] - 1
    P, Q = _fac(P, m, k), _fac(Q, d, k)
    Cm = np.zeros((ncols, d), dtype=np.float64) if C0 is None else np.ascontiguousarray(C0, dtype=np.float64).copy()
    sse = C.c_double(0.0)
    _L().orc_extend_mixed(C.c_int32(m), C.c_int32(d), C.c_int32(k), C.c_int32(ncols), _p(col_ptr, C.c_int64),
                          _p(row_idx, C.c_int32), _p(vals, C.c_float), _p(P, C.c_float), _p(Q, C.c_float),
                          C.c_double(eta), C.c_double(lam), C.c_double(beta1), C.c_double(beta2), C.c_double(eps),
                          C.c_int32(iters), C.c_int(int(round_operands)), _p(Cm, C.c_double), C.byref(sse))
    return Cm, sse.value

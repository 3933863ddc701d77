"""ctypes front end of the CPU oracle (``slim_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline / reference
legs may import this package.  The GPU library and its Python binding never do.

The C source is compiled on first use with ``gcc -O2 -fopenmp`` into
``oracle/liboracle.so`` (rebuilt when the source is newer).  All arithmetic
lives in the C file; this module only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "slim_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None

OK, BAD_ARG, BAD_MASK, CODE_RANGE = 0, 1, 3, 4


class OracleError(RuntimeError):
    def __init__(self, code, row=-1, group=-1):
        super().__init__(f"oracle error {code} (row {row}, group {group})")
        self.code, self.row, self.group = code, row, group


def build(force: bool = False) -> str:
    """Compile the oracle shared library if missing or stale; return its path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared",
                               _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        P = ctypes.c_void_p
        lib.oracle_pack.argtypes = [P, P, ctypes.c_int, ctypes.c_int, P, P, P, P]
        lib.oracle_pack.restype = ctypes.c_int
        lib.oracle_unpack.argtypes = [P, P, ctypes.c_int, ctypes.c_int, P, P]
        lib.oracle_unpack.restype = ctypes.c_int
        lib.oracle_repack_tiled.argtypes = [P, P, ctypes.c_int, ctypes.c_int, P]
        lib.oracle_repack_tiled.restype = ctypes.c_int
        lib.oracle_linear_fwd.argtypes = [P, ctypes.c_int, P, P, ctypes.c_float, P, P, ctypes.c_int,
                                          ctypes.c_int, ctypes.c_int, P, ctypes.c_int, P]
        lib.oracle_linear_fwd.restype = ctypes.c_int
        lib.oracle_linear_fwd_dense.argtypes = [P, ctypes.c_int, P, P, ctypes.c_float, P, P,
                                                ctypes.c_int, ctypes.c_int, ctypes.c_int, P, P]
        lib.oracle_linear_fwd_dense.restype = ctypes.c_int
        lib.oracle_quant_adapter.argtypes = [P, ctypes.c_int, ctypes.c_int, P, P]
        lib.oracle_quant_adapter.restype = ctypes.c_int
        lib.oracle_dequant_adapter.argtypes = [P, P, ctypes.c_int, ctypes.c_int, P]
        lib.oracle_dequant_adapter.restype = ctypes.c_int
        lib.oracle_linear_fwd_q.argtypes = [P, ctypes.c_int, P, P, ctypes.c_float, P, P, P, P, ctypes.c_int,
                                            ctypes.c_int, ctypes.c_int, P, ctypes.c_int, P]
        lib.oracle_linear_fwd_q.restype = ctypes.c_int
        lib.oracle_slim_quant.argtypes = [P, ctypes.c_int, ctypes.c_int, P, P, P, P]
        lib.oracle_slim_quant.restype = ctypes.c_int
        lib.oracle_mask_top2.argtypes = [P, P, ctypes.c_int, ctypes.c_int, P]
        lib.oracle_mask_top2.restype = ctypes.c_int
        lib.oracle_flop_reduction.argtypes = [ctypes.c_double] * 5
        lib.oracle_flop_reduction.restype = ctypes.c_double
        lib.oracle_num_threads.argtypes = []
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a)
    if a.dtype != dtype:
        raise TypeError(f"expected {dtype}, got {a.dtype}")
    return a


def pack(codes: np.ndarray, mask: np.ndarray):
    """codes int8 [d_out, d_in], mask uint8 [d_out, d_in] -> (vals, meta) uint8."""
    codes, mask = _c(codes, np.int8), _c(mask, np.uint8)
    d_out, d_in = codes.shape
    vals = np.zeros((d_out, d_in // 4), np.uint8)
    meta = np.zeros((d_out, d_in // 8), np.uint8)
    br, bg = ctypes.c_int(-1), ctypes.c_int(-1)
    rc = _load().oracle_pack(_p(codes), _p(mask), d_out, d_in, _p(vals), _p(meta),
                             ctypes.addressof(br), ctypes.addressof(bg))
    if rc != OK:
        raise OracleError(rc, br.value, bg.value)
    return vals, meta


def unpack(vals: np.ndarray, meta: np.ndarray):
    """Inverse of :func:`pack` -> (codes int8, mask uint8), both [d_out, d_in]."""
    vals, meta = _c(vals, np.uint8), _c(meta, np.uint8)
    d_out, d_in = vals.shape[0], vals.shape[1] * 4
    codes = np.empty((d_out, d_in), np.int8)
    mask = np.empty((d_out, d_in), np.uint8)
    rc = _load().oracle_unpack(_p(vals), _p(meta), d_out, d_in, _p(codes), _p(mask))
    if rc != OK:
        raise OracleError(rc)
    return codes, mask


def repack_tiled(vals: np.ndarray, meta: np.ndarray) -> np.ndarray:
    """(vals, meta) -> the decode-tiled copy, uint8 [ceil(d_out / 64) * 64 * d_in * 3 / 8]."""
    vals, meta = _c(vals, np.uint8), _c(meta, np.uint8)
    d_out, d_in = vals.shape[0], vals.shape[1] * 4
    out = np.zeros((d_out + 63) // 64 * 64 * d_in * 3 // 8, np.uint8)
    rc = _load().oracle_repack_tiled(_p(vals), _p(meta), d_out, d_in, _p(out))
    if rc != OK:
        raise OracleError(rc)
    return out


def linear_fwd(X, vals, meta, s, L, R, rows=None) -> np.ndarray:
    """Factored fp64 forward.  X/L/R are uint16 bfloat16 bit patterns.
    ``rows`` optionally restricts the evaluated token rows."""
    X, vals, meta = _c(X, np.uint16), _c(vals, np.uint8), _c(meta, np.uint8)
    b, d_in = X.shape
    d_out = vals.shape[0]
    r = 0 if L is None else L.shape[1]
    if r:
        L, R = _c(L, np.uint16), _c(R, np.uint16)
        assert L.shape == (d_out, r) and R.shape == (r, d_in)
    rows_a = None if rows is None else _c(np.asarray(rows, np.int32), np.int32)
    nm = b if rows_a is None else len(rows_a)
    Y = np.empty((nm, d_out), np.float64)
    rc = _load().oracle_linear_fwd(_p(X), b, _p(vals), _p(meta), float(s),
                                   _p(L) if r else None, _p(R) if r else None, r, d_out, d_in,
                                   _p(rows_a), nm, _p(Y))
    if rc != OK:
        raise OracleError(rc)
    return Y


def quant_adapter(A: np.ndarray):
    """bf16 bit patterns A[rows][cols] -> (codes uint8 [rows][cols / 2], scales uint16 [rows][ceil(cols / 128)])."""
    A = _c(A, np.uint16)
    rows, cols = A.shape
    codes = np.zeros((rows, cols // 2), np.uint8)
    scales = np.zeros((rows, (cols + 127) // 128), np.uint16)
    rc = _load().oracle_quant_adapter(_p(A), rows, cols, _p(codes), _p(scales))
    if rc != OK:
        raise OracleError(rc)
    return codes, scales


def dequant_adapter(codes: np.ndarray, scales: np.ndarray) -> np.ndarray:
    """The fp64 values (code x scale) a quantized adapter stands for."""
    codes, scales = _c(codes, np.uint8), _c(scales, np.uint16)
    rows, cols = codes.shape[0], codes.shape[1] * 2
    assert scales.shape == (rows, (cols + 127) // 128)
    out = np.empty((rows, cols), np.float64)
    rc = _load().oracle_dequant_adapter(_p(codes), _p(scales), rows, cols, _p(out))
    if rc != OK:
        raise OracleError(rc)
    return out


def linear_fwd_q(X, vals, meta, s, Lq, Ls, Rq, Rs, rows=None) -> np.ndarray:
    """Factored fp64 forward with quantized adapters (codes and scales of L and of R)."""
    X, vals, meta = _c(X, np.uint16), _c(vals, np.uint8), _c(meta, np.uint8)
    Lq, Ls, Rq, Rs = _c(Lq, np.uint8), _c(Ls, np.uint16), _c(Rq, np.uint8), _c(Rs, np.uint16)
    b, d_in = X.shape
    d_out, r = vals.shape[0], Lq.shape[1] * 2
    assert Lq.shape == (d_out, r // 2) and Rq.shape == (r, d_in // 2)
    assert Ls.shape == (d_out, (r + 127) // 128) and Rs.shape == (r, (d_in + 127) // 128)
    rows_a = None if rows is None else _c(np.asarray(rows, np.int32), np.int32)
    nm = b if rows_a is None else len(rows_a)
    Y = np.empty((nm, d_out), np.float64)
    rc = _load().oracle_linear_fwd_q(_p(X), b, _p(vals), _p(meta), float(s), _p(Lq), _p(Ls), _p(Rq), _p(Rs), r,
                                     d_out, d_in, _p(rows_a), nm, _p(Y))
    if rc != OK:
        raise OracleError(rc)
    return Y


def slim_quant(W: np.ndarray):
    """SLiM-Quant scale search on a float32 matrix: (codes int8 like W, scale float32, alpha float64,
    table float64 [29][2] of the (alpha, E(alpha)) pairs tried: ten coarse, then nineteen fine)."""
    W = _c(W, np.float32)
    d_out, d_in = W.shape
    codes = np.empty((d_out, d_in), np.int8)
    scale = np.zeros(1, np.float32)
    alpha = np.zeros(1, np.float64)
    table = np.zeros((29, 2), np.float64)
    rc = _load().oracle_slim_quant(_p(W), d_out, d_in, _p(codes), _p(scale), _p(alpha), _p(table))
    if rc != OK:
        raise OracleError(rc)
    return codes, np.float32(scale[0]), float(alpha[0]), table


def mask_top2(codes: np.ndarray, xbar=None) -> np.ndarray:
    """2:4 mask of int8 codes: per group of four along d_in the two largest |code| * xbar[k] (xbar None: |code|)."""
    codes = _c(codes, np.int8)
    d_out, d_in = codes.shape
    xb = None if xbar is None else _c(xbar, np.float32)
    assert xb is None or xb.shape == (d_in,)
    mask = np.empty((d_out, d_in), np.uint8)
    rc = _load().oracle_mask_top2(_p(codes), _p(xb), d_out, d_in, _p(mask))
    if rc != OK:
        raise OracleError(rc)
    return mask


def linear_fwd_dense(X, vals, meta, s, L, R, return_weight=False):
    """Unfactored fp64 forward through the explicit W_eff = s*Q + L@R."""
    X, vals, meta = _c(X, np.uint16), _c(vals, np.uint8), _c(meta, np.uint8)
    b, d_in = X.shape
    d_out = vals.shape[0]
    r = 0 if L is None else L.shape[1]
    if r:
        L, R = _c(L, np.uint16), _c(R, np.uint16)
    Y = np.empty((b, d_out), np.float64)
    We = np.empty((d_out, d_in), np.float64) if return_weight else None
    rc = _load().oracle_linear_fwd_dense(_p(X), b, _p(vals), _p(meta), float(s),
                                         _p(L) if r else None, _p(R) if r else None, r,
                                         d_out, d_in, _p(Y), _p(We))
    if rc != OK:
        raise OracleError(rc)
    return (Y, We) if return_weight else Y


def flop_reduction(d, n, a, V, rr) -> float:
    return float(_load().oracle_flop_reduction(float(d), float(n), float(a), float(V), float(rr)))


def num_threads() -> int:
    return int(_load().oracle_num_threads())

"""Python face of the CPU oracle (test infrastructure, never a product path).

`contract()` and `points()` call the plain C loop nest in gett_oracle.c
(Listing 3 of the paper: free loops, contracted loops with an accumulator, then
the alpha/beta update).  `canonical_tables()` in oracle.tables gives the integer
offset tables by div/mod.  Only tests, the smoke check and the benchmark's
cpu-baseline leg import this package; it imports nothing of the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gett_oracle.c")
_LIB = os.path.join(_HERE, "libgett_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile gett_oracle.c with gcc into libgett_oracle.so (idempotent)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-pthread",
                               "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Tensor(ctypes.Structure):
    _fields_ = [("nmodes", ctypes.c_int32),
                ("extent", ctypes.POINTER(ctypes.c_int64)),
                ("stride", ctypes.POINTER(ctypes.c_int64)),
                ("label", ctypes.POINTER(ctypes.c_int32))]


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        tp = ctypes.POINTER(_Tensor)
        lib.gett_oracle_contract.restype = ctypes.c_int
        lib.gett_oracle_contract.argtypes = [tp, tp, tp, ctypes.c_int, ctypes.c_double,
                                             ctypes.c_void_p, ctypes.c_void_p, ctypes.c_double,
                                             ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                             ctypes.c_int]
        lib.gett_oracle_points.restype = ctypes.c_int
        lib.gett_oracle_points.argtypes = [tp, tp, tp, ctypes.c_int, ctypes.c_double,
                                           ctypes.c_void_p, ctypes.c_void_p, ctypes.c_double,
                                           ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
                                           ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int]
        _lib = lib
    return _lib


class OracleError(ValueError):
    CODES = {1: "invalid argument", 2: "bad labels", 3: "extent mismatch"}

    def __init__(self, code: int):
        super().__init__(f"oracle error {code}: {self.CODES.get(code, '?')}")
        self.code = code


def _mk(spec):
    """spec has .labels/.extents/.strides; returns (struct, keepalive)."""
    n = len(spec.labels)
    ext = (ctypes.c_int64 * max(n, 1))(*spec.extents)
    st = (ctypes.c_int64 * max(n, 1))(*spec.strides)
    lab = (ctypes.c_int32 * max(n, 1))(*spec.labels)
    return _Tensor(n, ext, st, lab), (ext, st, lab)


def _operand(x: np.ndarray, dtype: int) -> np.ndarray:
    want = np.float32 if dtype == 0 else np.float64 if dtype == 3 else np.uint16
    x = np.ascontiguousarray(x)
    if x.dtype != want:
        raise TypeError(f"operand dtype {x.dtype}, expected {want}")
    return x


def default_threads() -> int:
    return os.cpu_count() or 1


def contract(con, dtype: int, alpha: float, A: np.ndarray, B: np.ndarray, beta: float,
             C_old: Optional[np.ndarray], threads: int = 1,
             want_abs: bool = True) -> Tuple[np.ndarray, Optional[np.ndarray]]:
    """Whole contraction.  Returns (C_ref, absacc) as float64 arrays over C's
    storage span (entries C does not address stay 0).  absacc[o] = sum |a||b|."""
    lib = _load()
    ta, ka = _mk(con.A)
    tb, kb = _mk(con.B)
    tc, kc = _mk(con.C)
    A = _operand(A, dtype)
    B = _operand(B, dtype)
    if A.size < con.A.span or B.size < con.B.span:
        raise ValueError("operand smaller than its span")
    cref = np.zeros(con.C.span, dtype=np.float64)
    cabs = np.zeros(con.C.span, dtype=np.float64) if want_abs else None
    cold = None
    if beta != 0.0:
        cold = np.ascontiguousarray(C_old, dtype=np.float64 if dtype == 3 else np.float32)
        if cold.size < con.C.span:
            raise ValueError("C_old smaller than its span")
    rc = lib.gett_oracle_contract(ctypes.byref(ta), ctypes.byref(tb), ctypes.byref(tc), dtype,
                                  float(alpha), A.ctypes.data, B.ctypes.data, float(beta),
                                  cold.ctypes.data if cold is not None else None,
                                  cref.ctypes.data, cabs.ctypes.data if want_abs else None,
                                  int(threads))
    if rc:
        raise OracleError(rc)
    return cref, cabs


def points(con, dtype: int, alpha: float, A: np.ndarray, B: np.ndarray, beta: float,
           C_old: Optional[np.ndarray], pts: np.ndarray,
           threads: int = 1) -> Tuple[np.ndarray, np.ndarray]:
    """Chosen outputs only.  pts[p, i] is the index of C's i-th mode.
    Returns (values, absacc), one float64 per point."""
    lib = _load()
    ta, ka = _mk(con.A)
    tb, kb = _mk(con.B)
    tc, kc = _mk(con.C)
    A = _operand(A, dtype)
    B = _operand(B, dtype)
    pts = np.ascontiguousarray(pts, dtype=np.int64).reshape(-1, max(len(con.C.labels), 1))
    n = pts.shape[0] if len(con.C.labels) else int(pts.shape[0])
    out = np.zeros(n, dtype=np.float64)
    ab = np.zeros(n, dtype=np.float64)
    cold = None
    if beta != 0.0:
        cold = np.ascontiguousarray(C_old, dtype=np.float64 if dtype == 3 else np.float32)
    rc = lib.gett_oracle_points(ctypes.byref(ta), ctypes.byref(tb), ctypes.byref(tc), dtype,
                                float(alpha), A.ctypes.data, B.ctypes.data, float(beta),
                                cold.ctypes.data if cold is not None else None, n,
                                pts.ctypes.data, out.ctypes.data, ab.ctypes.data, int(threads))
    if rc:
        raise OracleError(rc)
    return out, ab


def c_offsets(con) -> np.ndarray:
    """Storage offsets of every element C addresses, first mode fastest."""
    off = np.zeros(1, dtype=np.int64)
    for e, s in zip(con.C.extents, con.C.strides):
        off = (np.arange(e, dtype=np.int64)[:, None] * s + off[None, :]).reshape(-1)
    return off


def tolerance_ratio(C_gpu: np.ndarray, C_ref: np.ndarray, absacc: np.ndarray,
                    alpha: float, beta: float, C_old: Optional[np.ndarray],
                    offsets: Optional[np.ndarray] = None) -> float:
    """max|C_gpu - C_ref| / max(|alpha| * sum|a||b| + |beta| |C_old|): numerator and
    denominator each maximised over all outputs (the acceptance figure)."""
    sel = slice(None) if offsets is None else offsets
    num = float(np.max(np.abs(C_gpu[sel].astype(np.float64) - C_ref[sel])))
    scale = abs(alpha) * absacc[sel]
    if beta != 0.0 and C_old is not None:
        scale = scale + abs(beta) * np.abs(C_old[sel].astype(np.float64))
    den = float(np.max(scale))
    return num / den if den > 0 else (0.0 if num == 0 else float("inf"))

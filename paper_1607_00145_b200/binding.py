"""ctypes binding with the same names as include/gett.h (argument marshalling only)."""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional, Sequence

import numpy as np

GETT_MAX_MODES = 12
GETT_F32, GETT_BF16_F32, GETT_F16_F32, GETT_F64 = 0, 1, 2, 3
GETT_PATH_AUTO, GETT_PATH_SIMT, GETT_PATH_FFMA, GETT_PATH_UMMA = 0, 1, 2, 3
GETT_LOAD_SCALAR, GETT_LOAD_VEC_FREE, GETT_LOAD_VEC_K = 0, 1, 2
GETT_LOAD_TMA_FREE, GETT_LOAD_TMA_K, GETT_LOAD_VEC_KT = 3, 4, 5
GETT_EPI_AUTO, GETT_EPI_DIRECT, GETT_EPI_STAGED = 0, 1, 2
GETT_OPT_NO_TMA, GETT_OPT_NO_PAIR, GETT_OPT_NO_EXCHANGE, GETT_OPT_NO_ATOMS = 1, 2, 4, 8
GETT_OPT_STREAMK, GETT_OPT_NO_STREAMK = 16, 32
TABLE_NAMES = ("A_M", "A_K", "B_N", "B_K", "C_M", "C_N")

_HERE = os.path.dirname(os.path.abspath(__file__))


def library_path() -> str:
    """The in-tree shared library; GETT_LIBRARY names another build of it."""
    return os.environ.get("GETT_LIBRARY") or os.path.join(_HERE, "libgett_b200.so")


class _Desc(ctypes.Structure):
    _fields_ = [("nmodes", ctypes.c_int32),
                ("extent", ctypes.POINTER(ctypes.c_int64)),
                ("stride", ctypes.POINTER(ctypes.c_int64)),
                ("label", ctypes.POINTER(ctypes.c_int32))]


class PlanOpts(ctypes.Structure):
    _fields_ = [("path", ctypes.c_int32), ("tile_m", ctypes.c_int32), ("tile_n", ctypes.c_int32),
                ("tile_k", ctypes.c_int32), ("stages", ctypes.c_int32), ("split_k", ctypes.c_int32),
                ("epilogue", ctypes.c_int32), ("flags", ctypes.c_int32),
                ("wait_limit_us", ctypes.c_int32), ("experiment", ctypes.c_int32),
                ("search", ctypes.c_int32), ("reserved", ctypes.c_int32 * 5)]


class PlanInfo(ctypes.Structure):
    _fields_ = [("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("n_m", ctypes.c_int32), ("n_n", ctypes.c_int32), ("n_k", ctypes.c_int32),
                ("labels_m", ctypes.c_int32 * GETT_MAX_MODES),
                ("labels_n", ctypes.c_int32 * GETT_MAX_MODES),
                ("labels_k", ctypes.c_int32 * GETT_MAX_MODES),
                ("merged_m", ctypes.c_int32), ("merged_n", ctypes.c_int32),
                ("merged_k", ctypes.c_int32),
                ("path", ctypes.c_int32), ("loader_a", ctypes.c_int32),
                ("loader_b", ctypes.c_int32), ("epilogue", ctypes.c_int32),
                ("tile_m", ctypes.c_int32), ("tile_n", ctypes.c_int32), ("tile_k", ctypes.c_int32),
                ("stages", ctypes.c_int32), ("split_k", ctypes.c_int32),
                ("grid", ctypes.c_int32), ("block", ctypes.c_int32), ("smem_bytes", ctypes.c_int32),
                ("digits_m", ctypes.c_int32), ("digits_n", ctypes.c_int32),
                ("digits_k", ctypes.c_int32),
                ("workspace_bytes", ctypes.c_int64), ("tiles", ctypes.c_int64),
                ("device", ctypes.c_int32), ("swapped", ctypes.c_int32),
                ("candidates", ctypes.c_int32), ("model_rank", ctypes.c_int32), ("timed", ctypes.c_int32),
                ("model_us", ctypes.c_float), ("timed_us", ctypes.c_float),
                ("stream_k", ctypes.c_int32)]

    def as_dict(self) -> Dict[str, object]:
        out = {}
        for name, _ in self._fields_:
            if name == "reserved":
                continue
            v = getattr(self, name)
            if name.startswith("labels_"):
                n = getattr(self, "n_" + name[-1])
                v = list(v)[:n]
            out[name] = v
        return out


def _load() -> ctypes.CDLL:
    path = library_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: run `python -m paper_1607_00145_b200.build` "
                          "(there is no fallback implementation)")
    lib = ctypes.CDLL(path)
    dp = ctypes.POINTER(_Desc)
    lib.gett_plan_create.restype = ctypes.c_int
    lib.gett_plan_create.argtypes = [ctypes.POINTER(ctypes.c_void_p), dp, dp, dp, ctypes.c_int,
                                     ctypes.POINTER(PlanOpts)]
    lib.gett_contract.restype = ctypes.c_int
    lib.gett_contract.argtypes = [ctypes.c_void_p, ctypes.c_float, ctypes.c_void_p,
                                  ctypes.c_void_p, ctypes.c_float, ctypes.c_void_p,
                                  ctypes.c_void_p]
    lib.gett_plan_destroy.restype = ctypes.c_int
    lib.gett_plan_destroy.argtypes = [ctypes.c_void_p]
    lib.gett_plan_get_info.restype = ctypes.c_int
    lib.gett_plan_get_info.argtypes = [ctypes.c_void_p, ctypes.POINTER(PlanInfo)]
    lib.gett_plan_get_table.restype = ctypes.c_int
    lib.gett_plan_get_table.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p,
                                        ctypes.c_size_t]
    lib.gett_plan_last_device_status.restype = ctypes.c_int
    lib.gett_plan_last_device_status.argtypes = [ctypes.c_void_p]
    dp2 = ctypes.POINTER(_Desc)
    lib.gett_contract_noalloc.restype = ctypes.c_int
    lib.gett_contract_noalloc.argtypes = [dp2, dp2, dp2, ctypes.c_int, ctypes.c_int32, ctypes.c_float,
                                          ctypes.c_void_p, ctypes.c_void_p, ctypes.c_float,
                                          ctypes.c_void_p, ctypes.c_void_p]
    lib.gett_plan_model.restype = ctypes.c_int
    lib.gett_plan_model.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
    lib.gett_status_string.restype = ctypes.c_char_p
    lib.gett_status_string.argtypes = [ctypes.c_int]
    return lib


class _LazyLibrary:
    """The shared library, loaded at the first call (so that importing the package -- and its
    `build` submodule on a fresh checkout -- does not need it).  A missing library raises
    ImportError at that first call: there is no fallback implementation."""
    _cdll = None

    def __getattr__(self, name):
        if _LazyLibrary._cdll is None:
            _LazyLibrary._cdll = _load()
        return getattr(_LazyLibrary._cdll, name)


_lib = _LazyLibrary()


class GettError(RuntimeError):
    def __init__(self, status: int, where: str):
        super().__init__(f"{where}: {gett_status_string(status)} (status {status})")
        self.status = status


def gett_status_string(status: int) -> str:
    return _lib.gett_status_string(int(status)).decode()


def _desc(labels: Sequence[int], extents: Sequence[int], strides: Optional[Sequence[int]]):
    n = len(labels)
    ext = (ctypes.c_int64 * max(n, 1))(*extents)
    lab = (ctypes.c_int32 * max(n, 1))(*labels)
    st = (ctypes.c_int64 * max(n, 1))(*strides) if strides is not None else None
    d = _Desc(n, ext, st if st is not None else ctypes.POINTER(ctypes.c_int64)(), lab)
    return d, (ext, lab, st)


def gett_plan_create(A, B, C, dtype: int, opts: Optional[PlanOpts] = None) -> int:
    """A, B, C: objects with .labels/.extents/.strides (strides may be None = packed).
    Returns the plan handle (an integer address)."""
    da, ka = _desc(A.labels, A.extents, A.strides)
    db, kb = _desc(B.labels, B.extents, B.strides)
    dc, kc = _desc(C.labels, C.extents, C.strides)
    out = ctypes.c_void_p()
    rc = _lib.gett_plan_create(ctypes.byref(out), ctypes.byref(da), ctypes.byref(db),
                               ctypes.byref(dc), int(dtype),
                               ctypes.byref(opts) if opts is not None else None)
    if rc:
        raise GettError(rc, "gett_plan_create")
    return out.value


def _ptr(x) -> int:
    return x.data_ptr() if hasattr(x, "data_ptr") else int(x)


def gett_contract(plan: int, alpha: float, A, B, beta: float, C, stream=None) -> None:
    """A, B, C: torch CUDA tensors (or raw device addresses).  stream: a
    torch.cuda.Stream, a raw cudaStream_t value, or None for torch's current stream."""
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    elif hasattr(stream, "cuda_stream"):
        stream = stream.cuda_stream
    rc = _lib.gett_contract(plan, float(alpha), _ptr(A), _ptr(B), float(beta), _ptr(C),
                            ctypes.c_void_p(int(stream)))
    if rc:
        raise GettError(rc, "gett_contract")


GETT_NOALLOC_WORKSPACE_BYTES = 16 << 20


def gett_contract_noalloc(A, B, C, dtype: int, split_k: int, alpha: float, A_data, B_data,
                          beta: float, C_data, stream=None) -> None:
    """The contraction without any device allocation (no plan): descriptors in, launch out.
    split_k * M * N * 4 bytes must fit GETT_NOALLOC_WORKSPACE_BYTES."""
    da, ka = _desc(A.labels, A.extents, A.strides)
    db, kb = _desc(B.labels, B.extents, B.strides)
    dc, kc = _desc(C.labels, C.extents, C.strides)
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    elif hasattr(stream, "cuda_stream"):
        stream = stream.cuda_stream
    rc = _lib.gett_contract_noalloc(ctypes.byref(da), ctypes.byref(db), ctypes.byref(dc), int(dtype),
                                    int(split_k), float(alpha), _ptr(A_data), _ptr(B_data),
                                    float(beta), _ptr(C_data), ctypes.c_void_p(int(stream)))
    if rc:
        raise GettError(rc, "gett_contract_noalloc")


def gett_plan_destroy(plan: Optional[int]) -> None:
    if plan:
        _lib.gett_plan_destroy(plan)


def gett_plan_get_info(plan: int) -> PlanInfo:
    info = PlanInfo()
    rc = _lib.gett_plan_get_info(plan, ctypes.byref(info))
    if rc:
        raise GettError(rc, "gett_plan_get_info")
    return info


def gett_plan_get_table(plan: int, which: int) -> np.ndarray:
    info = gett_plan_get_info(plan)
    n = {0: info.M, 1: info.K, 2: info.N, 3: info.K, 4: info.M, 5: info.N}[int(which)]
    dst = np.empty(n, dtype=np.int64)
    rc = _lib.gett_plan_get_table(plan, int(which), dst.ctypes.data, n)
    if rc:
        raise GettError(rc, "gett_plan_get_table")
    return dst


def gett_plan_model(plan: int):
    """(total_us, [macro, A, B, C] in us): the performance model's estimate for the plan."""
    total = ctypes.c_double()
    terms = (ctypes.c_double * 4)()
    rc = _lib.gett_plan_model(plan, ctypes.byref(total), terms)
    if rc:
        raise GettError(rc, "gett_plan_model")
    return float(total.value), [float(x) for x in terms]


def gett_plan_last_device_status(plan: int) -> int:
    return int(_lib.gett_plan_last_device_status(plan))


class Plan:
    """Owns one plan handle; `plan(alpha, A, B, beta, C)` runs the contraction."""

    def __init__(self, con, dtype: int, **opts):
        o = None
        if opts:
            o = PlanOpts()
            for k, v in opts.items():
                if k not in dict(PlanOpts._fields_) or k == "reserved":
                    raise TypeError(f"unknown plan option {k!r}")
                setattr(o, k, int(v))
        self.handle = gett_plan_create(con.A, con.B, con.C, dtype, o)
        self.info = gett_plan_get_info(self.handle)

    def __call__(self, alpha, A, B, beta, C, stream=None) -> None:
        gett_contract(self.handle, alpha, A, B, beta, C, stream)

    def table(self, name: str) -> np.ndarray:
        return gett_plan_get_table(self.handle, TABLE_NAMES.index(name))

    def device_status(self) -> int:
        return gett_plan_last_device_status(self.handle)

    def model(self):
        return gett_plan_model(self.handle)

    def close(self) -> None:
        gett_plan_destroy(self.handle)
        self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

"""Oracle side of the integer part of the method: the index sets and the six
offset tables, computed directly by div/mod (test infrastructure).

Sec. 2.2: a label carried by A and C is free in A (I_m), by B and C free in B
(I_n), by A and B contracted (I_k).  Extent-1 modes address nothing and are
dropped.  The paper leaves the order of modes inside a set open (every
permutation is a candidate); the order fixed here, so that tables can be
compared bit for bit, is: I_m and I_n ascending by stride in C, I_k ascending
by stride in A, ties by position in that tensor.  The fused index runs first
mode fastest:  i = sum_j idx_j * prod_{l<j} extent_l, and a table entry is
sum_j idx_j * stride_j in the tensor concerned.  Merging adjacent modes into a
super-index (Sec. 6, stage 1) never changes these tables.
"""
from __future__ import annotations

from typing import Dict, List, Tuple

import numpy as np

TABLES = ("A_M", "A_K", "B_N", "B_K", "C_M", "C_N")


def classify(con) -> Tuple[List[int], List[int], List[int]]:
    """(I_m, I_n, I_k) in canonical order, extent-1 modes dropped."""
    A, B, C = con.A, con.B, con.C
    sA = dict(zip(A.labels, A.strides))
    sC = dict(zip(C.labels, C.strides))
    ext: Dict[int, int] = {}
    for t in (A, B, C):
        for l, e in zip(t.labels, t.extents):
            ext[l] = e
    im = [l for l in C.labels if l in A.labels and ext[l] > 1]
    in_ = [l for l in C.labels if l in B.labels and ext[l] > 1]
    ik = [l for l in A.labels if l in B.labels and ext[l] > 1]
    im.sort(key=lambda l: (sC[l], C.labels.index(l)))
    in_.sort(key=lambda l: (sC[l], C.labels.index(l)))
    ik.sort(key=lambda l: (sA[l], A.labels.index(l)))
    return im, in_, ik


def _table(modes: List[int], ext: Dict[int, int], stride: Dict[int, int]) -> np.ndarray:
    size = 1
    for l in modes:
        size *= ext[l]
    fused = np.arange(size, dtype=np.int64)
    rem = fused.copy()
    off = np.zeros(size, dtype=np.int64)
    for l in modes:
        idx = rem % ext[l]
        rem = rem // ext[l]
        off += idx * stride[l]
    return off


def canonical_tables(con) -> Dict[str, np.ndarray]:
    """{"A_M": offA_M[M], "A_K": ..., "B_N", "B_K", "C_M", "C_N"} as int64."""
    im, in_, ik = classify(con)
    ext: Dict[int, int] = {}
    for t in (con.A, con.B, con.C):
        for l, e in zip(t.labels, t.extents):
            ext[l] = e
    sA = dict(zip(con.A.labels, con.A.strides))
    sB = dict(zip(con.B.labels, con.B.strides))
    sC = dict(zip(con.C.labels, con.C.strides))
    return {"A_M": _table(im, ext, sA), "A_K": _table(ik, ext, sA),
            "B_N": _table(in_, ext, sB), "B_K": _table(ik, ext, sB),
            "C_M": _table(im, ext, sC), "C_N": _table(in_, ext, sC)}


def merged_extents(con) -> Tuple[List[int], List[int], List[int]]:
    """Extents of the super-indices after merging modes that are adjacent in the
    canonical order and contiguous (stride_j = stride_i * extent_i) in both
    tensors that carry them (Sec. 6, footnote on merged indices)."""
    im, in_, ik = classify(con)
    ext: Dict[int, int] = {}
    for t in (con.A, con.B, con.C):
        for l, e in zip(t.labels, t.extents):
            ext[l] = e
    sA = dict(zip(con.A.labels, con.A.strides))
    sB = dict(zip(con.B.labels, con.B.strides))
    sC = dict(zip(con.C.labels, con.C.strides))

    def merge(modes, s1, s2):
        out: List[int] = []
        prev = None
        for l in modes:
            if prev is not None and s1[l] == s1[prev] * ext[prev] and s2[l] == s2[prev] * ext[prev]:
                out[-1] *= ext[l]
            else:
                out.append(ext[l])
            prev = l
        return out

    return merge(im, sA, sC), merge(in_, sB, sC), merge(ik, sA, sB)

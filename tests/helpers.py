"""Shared test helpers: independent re-computations used to pin the oracle, and
random contraction generators for the fuzz tests.  No code from the CUDA
library and none from oracle/ lives here."""
from __future__ import annotations

import itertools
from typing import Dict, List, Optional, Tuple

import numpy as np
from numpy.lib.stride_tricks import as_strided

from workloads import Contraction, TensorSpec, packed_strides


def nd_view(flat: np.ndarray, spec: TensorSpec) -> np.ndarray:
    """Strided nd view of a flat storage array, one axis per mode of `spec`."""
    item = flat.dtype.itemsize
    return as_strided(flat, shape=tuple(spec.extents),
                      strides=tuple(s * item for s in spec.strides), writeable=False)


def flatten_to_matrix(con: Contraction, A: np.ndarray, B: np.ndarray):
    """Gather A into an M x K matrix and B into K x N by explicit transposition
    (the TTGT view of the same contraction), in float64.  Mode order inside each
    fused dimension: order of appearance in A (for m, k) and in B (for n)."""
    im, in_, ik = con.index_sets()
    a = nd_view(A, con.A).astype(np.float64)
    b = nd_view(B, con.B).astype(np.float64)
    a = np.transpose(a, [con.A.labels.index(l) for l in im + ik])
    b = np.transpose(b, [con.B.labels.index(l) for l in ik + in_])
    ext = con.extent_of()
    M = int(np.prod([ext[l] for l in im], dtype=np.int64)) if im else 1
    N = int(np.prod([ext[l] for l in in_], dtype=np.int64)) if in_ else 1
    K = int(np.prod([ext[l] for l in ik], dtype=np.int64)) if ik else 1
    return a.reshape(M, K), b.reshape(K, N), (im, in_, ik)


def brute_force(con: Contraction, A, B, alpha, beta, C_old) -> np.ndarray:
    """alpha * (A_mat @ B_mat) scattered into C's storage + beta * C_old, float64.
    The matrix product is a plain triple loop when tiny, else a float64 matmul."""
    am, bm, (im, in_, ik) = flatten_to_matrix(con, A, B)
    M, K = am.shape
    N = bm.shape[1]
    if M * N * K <= 4096:
        prod = np.zeros((M, N))
        for i in range(M):
            for j in range(N):
                t = 0.0
                for k in range(K):
                    t += am[i, k] * bm[k, j]
                prod[i, j] = t
    else:
        prod = am @ bm
    ext = con.extent_of()
    prod = prod.reshape([ext[l] for l in im] + [ext[l] for l in in_])
    order = im + in_
    prod = np.transpose(prod, [order.index(l) for l in con.C.labels])
    out = np.zeros(con.C.span, dtype=np.float64)
    sC = con.C.strides
    for idx in itertools.product(*[range(e) for e in con.C.extents]):
        off = sum(i * s for i, s in zip(idx, sC))
        v = alpha * prod[idx]
        if beta != 0.0:
            v += beta * float(C_old[off])
        out[off] = v
    return out


def einsum_ref(con: Contraction, A, B) -> np.ndarray:
    """np.einsum over strided views, float64, returned as an nd array in C's mode order."""
    a = nd_view(A, con.A).astype(np.float64)
    b = nd_view(B, con.B).astype(np.float64)
    return np.einsum(a, con.A.labels, b, con.B.labels, con.C.labels)


def scatter_nd(nd: np.ndarray, spec: TensorSpec) -> np.ndarray:
    out = np.zeros(spec.span, dtype=nd.dtype)
    w = as_strided(out, shape=tuple(spec.extents),
                   strides=tuple(s * out.dtype.itemsize for s in spec.strides))
    w[...] = nd
    return out


def random_contraction(rng: np.random.Generator, max_rank: int = 6, max_extent: int = 9,
                       pad: bool = True, min_each: int = 1,
                       extent_choices: Optional[List[int]] = None) -> Contraction:
    """Random |I_m|,|I_n|,|I_k| >= min_each with d_A,d_B,d_C <= max_rank, random
    extents, random mode permutations, optionally padded (non-packed) strides."""
    while True:
        nm, nn, nk = (int(rng.integers(min_each, 4)) for _ in range(3))
        if nm + nk <= max_rank and nn + nk <= max_rank and nm + nn <= max_rank \
                and nm + nn + nk > 0:
            break
    labels = list(range(nm + nn + nk))
    im, in_, ik = labels[:nm], labels[nm:nm + nn], labels[nm + nn:]
    if extent_choices:
        ext = {l: int(rng.choice(extent_choices)) for l in labels}
    else:
        ext = {l: int(rng.integers(1, max_extent + 1)) for l in labels}

    def spec(ls: List[int]) -> TensorSpec:
        ls = list(rng.permutation(ls)) if ls else []
        ls = [int(x) for x in ls]
        e = [ext[l] for l in ls]
        st, s = [], 1
        for x in e:
            st.append(s)
            s *= x
            if pad and rng.random() < 0.3:
                s += int(rng.integers(1, 4))
        return TensorSpec(ls, e, st)

    return Contraction("fuzz", spec(im + ik), spec(ik + in_), spec(im + in_))

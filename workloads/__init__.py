"""Seeded synthetic inputs and the named workloads.

This module holds no contraction arithmetic.  It only describes tensors
(labels, extents, strides) and fills them with reproducible pseudo-random
numbers, so that the CPU oracle and the CUDA path read identical bits.

Layout convention (Sec. 2.2 of the paper): the FIRST listed mode of a tensor is
its stride-1 mode ("Fortran" order generalised to d modes).

Random numbers are a counter-based hash, so an element's value depends only on
(seed, tensor id, storage offset) and never on generation order:

    h        = splitmix64(seed * GOLDEN + tensor_id * MIX + offset)
    uniform  = ((h >> 40) - 2^23) / 2^23        exact in fp32, in [-1, 1)
    normal   = sqrt(-2 ln u1) cos(2 pi u2)      Box-Muller in fp64, rounded to fp32
               u1 = ((h >> 11) + 1) / 2^53,  u2 from the hash of tensor_id + 16

bf16 / fp16 operands are the round-to-nearest-even conversion of that fp32 draw,
done once here; both sides receive the same 16-bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

F32, BF16_F32, F16_F32, F64 = 0, 1, 2, 3
DTYPE_NAMES = {F32: "f32", BF16_F32: "bf16", F16_F32: "f16", F64: "f64"}

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_MIX = np.uint64(0xBF58476D1CE4E5B9)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
TENSOR_ID = {"A": 1, "B": 2, "C": 3}


def splitmix64(x: np.ndarray) -> np.ndarray:
    """The splitmix64 output function applied to each uint64 of `x`."""
    with np.errstate(over="ignore"):
        z = x + _GOLDEN
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def _hash(seed: int, tensor_id: int, offsets: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        base = np.uint64(seed) * _GOLDEN + np.uint64(tensor_id) * _MIX
        return splitmix64(offsets.astype(np.uint64) + base)


def uniform_pm1(seed: int, tensor_id: int, n: int, chunk: int = 1 << 24) -> np.ndarray:
    """n fp32 values in [-1, 1), element i drawn from storage offset i."""
    out = np.empty(n, dtype=np.float32)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        h = _hash(seed, tensor_id, np.arange(s, e, dtype=np.uint64))
        v = (h >> np.uint64(40)).astype(np.int64) - (1 << 23)
        out[s:e] = (v.astype(np.float64) / float(1 << 23)).astype(np.float32)
    return out


def uniform_pm1_f64(seed: int, tensor_id: int, n: int, chunk: int = 1 << 24) -> np.ndarray:
    """n fp64 values in [-1, 1) with 53 random bits each: ((h >> 11) - 2^52) / 2^52."""
    out = np.empty(n, dtype=np.float64)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        h = _hash(seed, tensor_id, np.arange(s, e, dtype=np.uint64))
        v = (h >> np.uint64(11)).astype(np.int64) - (1 << 52)
        out[s:e] = v.astype(np.float64) / float(1 << 52)
    return out


def normal01(seed: int, tensor_id: int, n: int, chunk: int = 1 << 23) -> np.ndarray:
    """n fp32 values ~ N(0, 1) via Box-Muller on two hashed uniforms."""
    out = np.empty(n, dtype=np.float32)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        off = np.arange(s, e, dtype=np.uint64)
        h1 = _hash(seed, tensor_id, off)
        h2 = _hash(seed, tensor_id + 16, off)
        u1 = ((h1 >> np.uint64(11)).astype(np.float64) + 1.0) / float(1 << 53)
        u2 = (h2 >> np.uint64(11)).astype(np.float64) / float(1 << 53)
        out[s:e] = (np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)).astype(np.float32)
    return out


def small_ints(seed: int, tensor_id: int, n: int, lo: int = -3, hi: int = 3) -> np.ndarray:
    """n fp32 values that are integers in [lo, hi]; sums of products stay exact."""
    h = _hash(seed, tensor_id, np.arange(n, dtype=np.uint64))
    span = np.uint64(hi - lo + 1)
    return ((h >> np.uint64(33)) % span).astype(np.int64).astype(np.float32) + np.float32(lo)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def f32_to_f16_bits(x: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(x, dtype=np.float32).astype(np.float16).view(np.uint16)


def f16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return b.view(np.float16).astype(np.float32)


def encode_operand(x_f32: np.ndarray, dtype: int) -> np.ndarray:
    """The stored form of an A/B operand for `dtype` (fp32 array or uint16 bits)."""
    if dtype == F32:
        return np.ascontiguousarray(x_f32, dtype=np.float32)
    if dtype == BF16_F32:
        return f32_to_bf16_bits(x_f32)
    if dtype == F16_F32:
        return f32_to_f16_bits(x_f32)
    raise ValueError(f"unknown dtype {dtype}")


def decode_operand(stored: np.ndarray, dtype: int) -> np.ndarray:
    """fp32 view of the stored operand values (exact widening)."""
    if dtype == F32:
        return stored
    if dtype == BF16_F32:
        return bf16_bits_to_f32(stored)
    if dtype == F16_F32:
        return f16_bits_to_f32(stored)
    raise ValueError(f"unknown dtype {dtype}")


# --------------------------------------------------------------------------- #
# Tensor and contraction descriptions
# --------------------------------------------------------------------------- #
@dataclass
class TensorSpec:
    """labels[i] has extents[i] and strides[i] (elements).  labels are ints."""
    labels: List[int]
    extents: List[int]
    strides: List[int]

    @property
    def span(self) -> int:
        """Number of storage elements the tensor covers: 1 + sum (extent-1)*stride."""
        return 1 + sum((e - 1) * s for e, s in zip(self.extents, self.strides))

    @property
    def numel(self) -> int:
        n = 1
        for e in self.extents:
            n *= e
        return n


def packed_strides(extents: Sequence[int]) -> List[int]:
    """First-mode-fastest packed strides."""
    out, s = [], 1
    for e in extents:
        out.append(s)
        s *= e
    return out


@dataclass
class Contraction:
    """C[..] = alpha * sum_k A[..] * B[..] + beta * C[..]  with named modes."""
    name: str
    A: TensorSpec
    B: TensorSpec
    C: TensorSpec
    label_names: Dict[int, str] = field(default_factory=dict)

    def extent_of(self) -> Dict[int, int]:
        ext: Dict[int, int] = {}
        for t in (self.A, self.B, self.C):
            for l, e in zip(t.labels, t.extents):
                ext[l] = e
        return ext

    def index_sets(self) -> Tuple[List[int], List[int], List[int]]:
        """(I_m, I_n, I_k) as label lists, in order of first appearance."""
        a, b, c = set(self.A.labels), set(self.B.labels), set(self.C.labels)
        im = [l for l in self.A.labels if l in c]
        in_ = [l for l in self.B.labels if l in c]
        ik = [l for l in self.A.labels if l in b]
        return im, in_, ik

    def mnk(self) -> Tuple[int, int, int]:
        ext = self.extent_of()
        im, in_, ik = self.index_sets()
        prod = lambda ls: int(np.prod([ext[l] for l in ls], dtype=np.int64)) if ls else 1
        return prod(im), prod(in_), prod(ik)

    def flops(self) -> int:
        m, n, k = self.mnk()
        return 2 * m * n * k

    def is_plain_gemm(self) -> bool:
        """Packed A[m,k], B[k,n], C[m,n]: already the equal-sized GEMM of its own comparison."""
        a, b, c = self.A, self.B, self.C
        return (len(a.labels) == 2 and len(b.labels) == 2 and len(c.labels) == 2
                and c.labels == [a.labels[0], b.labels[1]] and a.labels[1] == b.labels[0]
                and all(t.strides == packed_strides(t.extents) for t in (a, b, c)))

    def compulsory_bytes(self, dtype: int, beta: float) -> int:
        """|A| + |B| + |C| * (1 + [beta != 0]) with fp32 C."""
        ab = 4 if dtype == F32 else 8 if dtype == F64 else 2
        c = self.C.numel * (8 if dtype == F64 else 4)
        return self.A.numel * ab + self.B.numel * ab + c * (2 if beta != 0.0 else 1)


def parse_spec(spec: str, sizes: Dict[str, int], name: str = "",
               strides: Optional[Dict[str, Sequence[int]]] = None) -> Contraction:
    """Parse "C[a,b,i] = A[i,m,a] * B[m,b]" with a size per mode name.

    Modes are listed stride-1 first.  `strides` may give explicit element strides
    per tensor name ("A", "B", "C"); otherwise tensors are packed.
    """
    lhs, rhs = spec.split("=")
    ta, tb = rhs.split("*")

    def modes(txt: str) -> Tuple[str, List[str]]:
        txt = txt.strip()
        nm, rest = txt.split("[")
        body = rest.rstrip("]").strip()
        return nm.strip(), [m.strip() for m in body.split(",") if m.strip()]

    ids: Dict[str, int] = {}

    def spec_of(txt: str) -> TensorSpec:
        nm, ms = modes(txt)
        for m in ms:
            ids.setdefault(m, len(ids))
        ext = [int(sizes[m]) for m in ms]
        st = list(strides[nm]) if strides and nm in strides else packed_strides(ext)
        return TensorSpec([ids[m] for m in ms], ext, [int(s) for s in st])

    c = spec_of(lhs)
    a = spec_of(ta)
    b = spec_of(tb)
    return Contraction(name or spec.strip(), a, b, c, {v: k for k, v in ids.items()})


# --------------------------------------------------------------------------- #
# The five named workloads (shapes echo the paper's benchmark families:
# the Fig. 3 example, the GEMM control, a tensor-times-matrix case, the
# all-72 4-D family and the 6-D coupled-cluster family).
# --------------------------------------------------------------------------- #
@dataclass
class Workload:
    key: str
    contraction: Contraction
    dtypes: Tuple[int, ...]
    dist: str            # "uniform" or "normal"
    seed: int
    alpha: float
    beta: float
    bound: str           # "latency", "compute", "hbm"


def _wl(key, spec, sizes, dtypes, dist, seed, alpha, beta, bound) -> Workload:
    return Workload(key, parse_spec(spec, sizes, key), dtypes, dist, seed, alpha, beta, bound)


def workload(key: str, scale: Optional[Dict[str, int]] = None) -> Workload:
    """One of cfg1..cfg5, or the split-K shape "splitk"; `scale` overrides extents."""
    table = {
        "cfg1": ("C[m0,n0,m1] = A[m0,k,m1] * B[k,n0]",
                 dict(m0=24, m1=32, n0=40, k=48), (F32,), "uniform", 0, 1.0, 0.0, "latency"),
        "cfg2": ("C[m,n] = A[m,k] * B[k,n]",
                 dict(m=8192, n=8192, k=8192), (F32, BF16_F32), "uniform", 1, 1.0, 0.5, "compute"),
        "cfg3": ("C[m0,m1,n0] = A[k,m0,m1] * B[n0,k]",
                 dict(m0=1024, m1=1024, n0=24, k=24), (F32,), "uniform", 2, 1.0, 0.0, "hbm"),
        "cfg4": ("C[m0,n0,m1,n1] = A[m0,k0,m1,k1] * B[n1,k1,n0,k0]",
                 dict(m0=72, m1=72, n0=72, n1=72, k0=72, k1=72), (BF16_F32, F32), "normal", 3,
                 1.0, 0.0, "compute"),
        "cfg5": ("C[n0,m2,m1,n2,m0,n1] = A[m1,k,m0,m2] * B[n2,n0,k,n1]",
                 dict(m0=24, m1=24, m2=24, n0=24, n1=24, n2=24, k=64), (F32, BF16_F32),
                 "uniform", 4, 1.0, 1.0, "hbm"),
        # small output, long contraction: the shape where splitting I_k pays
        "splitk": ("C[a,b] = A[c,a,d] * B[d,c,b]",
                   dict(a=384, b=376, c=384, d=384), (F32, BF16_F32), "uniform", 5, 1.0, 0.0,
                   "compute"),
        # the same sizes with layouts the vector kernels can gather (K merges to one mode)
        "splitk_vec": ("C[a,b] = A[a,c,d] * B[c,d,b]",
                       dict(a=384, b=376, c=384, d=384), (F32, BF16_F32), "uniform", 5, 1.0, 0.0,
                       "compute"),
    }
    spec, sizes, dtypes, dist, seed, alpha, beta, bound = table[key]
    sizes = dict(sizes)
    if scale:
        sizes.update(scale)
    return _wl(key, spec, sizes, dtypes, dist, seed, alpha, beta, bound)


WORKLOAD_KEYS = ("cfg1", "cfg2", "cfg3", "cfg4", "cfg5")


def pool(seed: int = 2016, per_family: int = 5) -> List[Workload]:
    """A seeded pool of synthetic contractions with random mode orders, one family per kind of
    shape the paper's benchmark contains (its own contraction strings and input files are not
    reproduced here): plain matrices in the four transposition variants, a large tensor times
    a small matrix, 4-D tensors with two free and two contracted modes each, the 6-D / 4-D / 4-D
    coupled-cluster shape with one contracted mode, and mixed 3- to 5-D cases.  Extents are
    drawn from the values the paper's families use (24, 48, 72, 96, 312, ...).  Every tensor
    is packed with its first listed mode stride-1; the order of the modes inside A, B and C
    is a random permutation, so the pool exercises every loader / epilogue combination."""
    rng = np.random.default_rng(seed)
    out: List[Workload] = []

    def emit(family: str, m: Dict[str, int], n: Dict[str, int], k: Dict[str, int], beta: float):
        sizes = {**m, **n, **k}
        am, bn, cm = list(m) + list(k), list(k) + list(n), list(m) + list(n)
        for lst in (am, bn, cm):
            rng.shuffle(lst)
        spec = f"C[{','.join(cm)}] = A[{','.join(am)}] * B[{','.join(bn)}]"
        key = f"{family}{sum(1 for w in out if w.key.startswith(family))}"
        w = _wl(key, spec, sizes, (F32, BF16_F32), "uniform", 100 + len(out), 1.0, beta, "pool")
        w.contraction.name = spec + "  " + ",".join(f"{k_}={v}" for k_, v in sizes.items())
        out.append(w)

    pick = lambda vals: int(rng.choice(vals))
    for i in range(per_family):
        # plain matrices
        emit("gemm", {"m": pick([2048, 3072, 4096])}, {"n": pick([2048, 3072, 4096])},
             {"k": pick([1024, 2048, 4096])}, float(i % 2))
        # tensor times small matrix (either operand may be the small one after the shuffle)
        e = pick([24, 32, 48])
        emit("ttm", {"a": pick([312, 296, 256]), "b": pick([312, 296, 256]), "c": pick([8, 16, 24])},
             {"u": e}, {"k": pick([24, 32, 48])}, 0.0)
        # two free and two contracted modes per operand, one extent
        e = pick([48, 72, 96])
        emit("d4", {"a": e, "b": e}, {"c": e, "d": e}, {"k": e, "l": e}, 0.0)
        # coupled-cluster shape: three free modes per operand, one contracted mode
        e = pick([16, 24])
        emit("cc", {"a": e, "b": e, "c": e}, {"i": e, "j": e, "l": e}, {"k": pick([24, 48, 64])},
             float((i + 1) % 2))
        # mixed ranks and extents
        emit("mix", {"a": pick([40, 72, 120]), "b": pick([24, 56, 64])},
             {"c": pick([48, 96, 312])} if i % 2 else {"c": pick([48, 96]), "d": pick([8, 24, 40])},
             {"k": pick([32, 72, 200]), "l": pick([8, 24])}, 0.0)
    return out


_DRAW_CACHE: Dict[Tuple[str, int, str, int], np.ndarray] = {}


def draw_cached(dist: str, seed: int, tensor: str, n: int, keep: int = 8) -> np.ndarray:
    """draw() with the last few results kept (an element depends only on seed, tensor and storage
    offset, so contractions that differ only in the order of their modes share their arrays).
    The returned array is shared: callers must not write to it."""
    key = (dist, seed, tensor, n)
    if key not in _DRAW_CACHE:
        while len(_DRAW_CACHE) >= keep:
            _DRAW_CACHE.pop(next(iter(_DRAW_CACHE)))
        _DRAW_CACHE[key] = draw(dist, seed, tensor, n)
    return _DRAW_CACHE[key]


def draw(dist: str, seed: int, tensor: str, n: int) -> np.ndarray:
    tid = TENSOR_ID[tensor]
    if dist == "uniform":
        return uniform_pm1(seed, tid, n)
    if dist == "normal":
        return normal01(seed, tid, n)
    if dist == "ints":
        return small_ints(seed, tid, n)
    raise ValueError(dist)


def make_inputs(con: Contraction, dtype: int, dist: str, seed: int, beta: float, cache: bool = False):
    """(A_stored, B_stored, C_old) flat storage arrays of each tensor's span.

    A and B are fp32 or uint16 bit patterns depending on dtype; C_old is fp32
    (drawn uniform[-1,1) when beta != 0, zeros otherwise, as the workloads say).
    cache: reuse the fp32 draws of earlier calls with the same seed and span (read-only arrays).
    """
    if dtype == F64:  # double precision throughout: A, B and C are fp64 with 53-bit draws
        a = uniform_pm1_f64(seed, TENSOR_ID["A"], con.A.span)
        b = uniform_pm1_f64(seed, TENSOR_ID["B"], con.B.span)
        c = uniform_pm1_f64(seed, TENSOR_ID["C"], con.C.span) if beta != 0.0 else np.zeros(con.C.span, dtype=np.float64)
        return a, b, c
    d = draw_cached if cache else draw
    a = encode_operand(d(dist, seed, "A", con.A.span), dtype)
    b = encode_operand(d(dist, seed, "B", con.B.span), dtype)
    if beta != 0.0:
        c = uniform_pm1(seed, TENSOR_ID["C"], con.C.span)
    else:
        c = np.zeros(con.C.span, dtype=np.float32)
    return a, b, c

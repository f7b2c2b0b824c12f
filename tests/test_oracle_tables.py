"""Pins for the oracle's integer side: index-set classification, canonical
order, merged super-indices and the six offset tables."""
import numpy as np
import pytest

from oracle import tables as T
from workloads import parse_spec, workload


def _names(con, labels):
    return [con.label_names[l] for l in labels]


def test_classification_and_canonical_order_of_the_workloads():
    want = {
        "cfg1": (["m0", "m1"], ["n0"], ["k"]),
        "cfg2": (["m"], ["n"], ["k"]),
        "cfg3": (["m0", "m1"], ["n0"], ["k"]),
        "cfg4": (["m0", "m1"], ["n0", "n1"], ["k0", "k1"]),
        "cfg5": (["m2", "m1", "m0"], ["n0", "n2", "n1"], ["k"]),
    }
    for key, (m, n, k) in want.items():
        con = workload(key).contraction
        im, in_, ik = T.classify(con)
        assert (_names(con, im), _names(con, in_), _names(con, ik)) == (m, n, k), key


def test_fused_sizes_of_the_workloads():
    want = {"cfg1": (768, 40, 48), "cfg2": (8192, 8192, 8192), "cfg3": (1048576, 24, 24),
            "cfg4": (5184, 5184, 5184), "cfg5": (13824, 13824, 64)}
    for key, mnk in want.items():
        assert workload(key).contraction.mnk() == mnk


def test_merged_super_indices():
    # cfg3: m0, m1 are adjacent and contiguous in both A and C -> one super-index
    assert T.merged_extents(workload("cfg3").contraction) == ([1048576], [24], [24])
    # cfg4 / cfg5: nothing merges
    assert T.merged_extents(workload("cfg4").contraction) == ([72, 72], [72, 72], [72, 72])
    assert T.merged_extents(workload("cfg5").contraction) == ([24] * 3, [24] * 3, [64])
    # the paper's loops-over-GEMM example (Listing 8): (i,j) -> 576 and (a,b) -> 576
    con = parse_spec("C[a,b,c,i,j,k] = A[i,j,m,c] * B[m,k,a,b]",
                     dict(a=24, b=24, c=24, i=24, j=24, k=24, m=24))
    im, in_, ik = T.classify(con)
    assert _names(con, im) == ["c", "i", "j"] and _names(con, in_) == ["a", "b", "k"]
    assert T.merged_extents(con) == ([24, 576], [576, 24], [24])


def _golden(name):
    import os
    out = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", name)) as f:
        for line in f:
            line = line.split("#")[0].split()
            if line:
                out[line[0]] = int(line[1])
    return out


def test_listing8_constants_follow_from_first_mode_fastest_strides():
    """The numbers the paper prints for its merged-index example (fixture with the citation)."""
    gold = _golden("listing8_constants.txt")
    con = parse_spec("C[a,b,c,i,j,k] = A[i,j,m,c] * B[m,k,a,b]",
                     dict(a=24, b=24, c=24, i=24, j=24, k=24, m=24))
    sA = dict(zip(_names(con, con.A.labels), con.A.strides))
    sB = dict(zip(_names(con, con.B.labels), con.B.strides))
    sC = dict(zip(_names(con, con.C.labels), con.C.strides))
    m_ext, n_ext, k_ext = T.merged_extents(con)
    # I_m = {c, (i,j)}, I_n = {(a,b), k}, I_k = {m}: the merged extents are the example's *_UP
    assert m_ext == [gold["c_UP"], gold["i_UP"]] and n_ext == [gold["a_UP"], gold["k_UP"]]
    assert k_ext == [gold["m_UP"]]
    assert sB["a"] == gold["lda"] == gold["m_UP"] * gold["k_UP"]          # B as m x (ab) per k
    assert sA["m"] == gold["ldb"] == gold["i_UP"]                         # A as (ij) x m
    assert sC["i"] == gold["ldc"] == gold["a_UP"] * gold["c_UP"]
    assert sB["k"] == gold["B_per_k"] == gold["m_UP"]
    assert sA["c"] == gold["A_per_c"] == gold["i_UP"] * gold["m_UP"]
    assert sC["c"] == gold["C_per_c"] == gold["a_UP"]
    assert sC["k"] == gold["C_per_k"] == gold["a_UP"] * gold["c_UP"] * gold["i_UP"]


def _grid(*axes):
    """first axis fastest"""
    out = np.zeros(1, dtype=np.int64)
    for ext, stride in axes:
        out = (np.arange(ext, dtype=np.int64)[:, None] * stride + out[None, :]).reshape(-1)
    return out


def test_closed_form_tables_cfg1():
    t = T.canonical_tables(workload("cfg1").contraction)
    assert np.array_equal(t["A_M"], _grid((24, 1), (32, 1152)))
    assert np.array_equal(t["A_K"], 24 * np.arange(48))
    assert np.array_equal(t["B_N"], 48 * np.arange(40))
    assert np.array_equal(t["B_K"], np.arange(48))
    assert np.array_equal(t["C_M"], _grid((24, 1), (32, 960)))
    assert np.array_equal(t["C_N"], 24 * np.arange(40))


def test_closed_form_tables_cfg2_cfg3():
    t = T.canonical_tables(workload("cfg2").contraction)
    r = np.arange(8192, dtype=np.int64)
    for name, mult in [("A_M", 1), ("A_K", 8192), ("B_N", 8192), ("B_K", 1), ("C_M", 1),
                       ("C_N", 8192)]:
        assert np.array_equal(t[name], mult * r)
    t = T.canonical_tables(workload("cfg3").contraction)
    m = np.arange(1048576, dtype=np.int64)
    assert np.array_equal(t["A_M"], 24 * m) and np.array_equal(t["C_M"], m)
    assert np.array_equal(t["A_K"], np.arange(24)) and np.array_equal(t["B_K"], 24 * np.arange(24))
    assert np.array_equal(t["B_N"], np.arange(24))
    assert np.array_equal(t["C_N"], 1048576 * np.arange(24))


def test_closed_form_tables_cfg4_cfg5():
    t = T.canonical_tables(workload("cfg4").contraction)
    assert np.array_equal(t["A_M"], _grid((72, 1), (72, 5184)))
    assert np.array_equal(t["A_K"], _grid((72, 72), (72, 373248)))
    assert np.array_equal(t["B_N"], _grid((72, 5184), (72, 1)))
    assert np.array_equal(t["B_K"], _grid((72, 373248), (72, 72)))
    assert np.array_equal(t["C_M"], _grid((72, 1), (72, 5184)))
    assert np.array_equal(t["C_N"], _grid((72, 72), (72, 373248)))
    t = T.canonical_tables(workload("cfg5").contraction)
    assert np.array_equal(t["A_M"], _grid((24, 36864), (24, 1), (24, 1536)))
    assert np.array_equal(t["A_K"], 24 * np.arange(64))
    assert np.array_equal(t["B_N"], _grid((24, 24), (24, 1), (24, 36864)))
    assert np.array_equal(t["B_K"], 576 * np.arange(64))
    assert np.array_equal(t["C_M"], _grid((24, 24), (24, 576), (24, 331776)))
    assert np.array_equal(t["C_N"], _grid((24, 1), (24, 13824), (24, 7962624)))


@pytest.mark.parametrize("key", ["cfg1", "cfg4", "cfg5"])
def test_c_offsets_are_injective_and_inside_the_span(key):
    scale = None if key == "cfg1" else {k: 6 for k in
                                        ("m0", "m1", "m2", "n0", "n1", "n2", "k0", "k1")}
    if key == "cfg4" and scale:
        scale = {k: v for k, v in scale.items() if k in ("m0", "m1", "n0", "n1", "k0", "k1")}
    con = workload(key, scale).contraction
    t = T.canonical_tables(con)
    c = (t["C_M"][:, None] + t["C_N"][None, :]).reshape(-1)
    assert np.unique(c).size == c.size == con.C.numel
    assert c.min() == 0 and c.max() == con.C.span - 1
    assert t["A_M"].max() + t["A_K"].max() == con.A.span - 1
    assert t["B_N"].max() + t["B_K"].max() == con.B.span - 1


def test_extent_one_modes_are_dropped_and_padded_strides_kept():
    con = parse_spec("C[m,u,n] = A[k,m,u] * B[n,k]", dict(m=3, u=1, n=2, k=4),
                     strides={"A": [2, 9, 40], "B": [1, 3], "C": [1, 5, 5]})
    im, in_, ik = T.classify(con)
    assert _names(con, im) == ["m"] and _names(con, in_) == ["n"] and _names(con, ik) == ["k"]
    t = T.canonical_tables(con)
    assert t["A_M"].tolist() == [0, 9, 18] and t["A_K"].tolist() == [0, 2, 4, 6]
    assert t["C_N"].tolist() == [0, 5]

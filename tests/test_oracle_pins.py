"""Pins for the CPU oracle's value path: what the paper and the mathematics fix,
computed by routes that share nothing with oracle/gett_oracle.c."""
import itertools

import numpy as np
import pytest

import oracle
from helpers import brute_force, einsum_ref, nd_view, random_contraction, scatter_nd
from workloads import (BF16_F32, F16_F32, F32, Contraction, TensorSpec, bf16_bits_to_f32,
                       encode_operand, packed_strides, parse_spec, small_ints, uniform_pm1,
                       workload)


def _ints(con, seed=7):
    a = small_ints(seed, 1, con.A.span)
    b = small_ints(seed, 2, con.B.span)
    c = small_ints(seed, 3, con.C.span)
    return a, b, c


# ---- brute force: flatten to matrices in a different loop structure (exact) ----
@pytest.mark.parametrize("seed", range(40))
def test_matches_flatten_to_matrix_exactly_on_small_integers(seed):
    rng = np.random.default_rng(seed)
    con = random_contraction(rng, max_rank=5, max_extent=5)
    a, b, c = _ints(con, seed)
    alpha, beta = [(1.0, 0.0), (2.0, -1.0), (-3.0, 2.0), (1.0, 1.0)][seed % 4]
    ref = brute_force(con, a, b, alpha, beta, c)
    got, absacc = oracle.contract(con, F32, alpha, a, b, beta, c, threads=1 + seed % 3)
    assert np.array_equal(got, ref)
    a_m, b_m, _ = __import__("helpers").flatten_to_matrix(con, np.abs(a), np.abs(b))
    assert np.isclose(absacc.max(), (a_m @ b_m).max())


@pytest.mark.parametrize("seed", range(10))
def test_matches_einsum_on_uniform_inputs(seed):
    rng = np.random.default_rng(100 + seed)
    con = random_contraction(rng, max_rank=6, max_extent=7)
    a = uniform_pm1(seed, 1, con.A.span)
    b = uniform_pm1(seed, 2, con.B.span)
    ref = scatter_nd(einsum_ref(con, a, b), con.C)
    got, _ = oracle.contract(con, F32, 1.0, a, b, 0.0, None, threads=2)
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)


# ---- the 2-D case is Listing 1 (naive matrix multiply, column-major) ----
def test_two_d_case_is_naive_gemm():
    M, N, K = 5, 4, 6
    con = parse_spec("C[m,n] = A[m,k] * B[k,n]", dict(m=M, n=N, k=K))
    a = uniform_pm1(3, 1, M * K)
    b = uniform_pm1(3, 2, K * N)
    c = uniform_pm1(3, 3, M * N)
    alpha, beta = 1.5, -0.25
    ref = np.zeros(M * N)
    for j in range(N):
        for i in range(M):
            tmp = 0.0
            for k in range(K):
                tmp += float(a[i + M * k]) * float(b[k + K * j])
            ref[i + M * j] = alpha * tmp + beta * float(c[i + M * j])
    got, _ = oracle.contract(con, F32, alpha, a, b, beta, c)
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-15)


# ---- closed forms ----
@pytest.mark.parametrize("key,scale,expect", [
    ("cfg1", None, 48),
    ("cfg4", dict(m0=3, m1=2, n0=2, n1=3, k0=5, k1=7), 35),
    ("cfg5", dict(m0=2, m1=3, m2=2, n0=3, n1=2, n2=2, k=64), 64),
])
def test_all_ones_gives_product_of_contracted_extents(key, scale, expect):
    con = workload(key, scale).contraction
    a = np.ones(con.A.span, np.float32)
    b = np.ones(con.B.span, np.float32)
    got, absacc = oracle.contract(con, F32, 1.0, a, b, 0.0, None, threads=2)
    off = oracle.c_offsets(con)
    assert np.all(got[off] == expect) and np.all(absacc[off] == expect)


def test_identity_b_reproduces_a_permuted():
    # C[n, m1, m0] = sum_k A[m0, k, m1] * delta[k, n]  -> a pure transposition (Eq. 4)
    con = parse_spec("C[n,m1,m0] = A[m0,k,m1] * B[k,n]", dict(m0=3, m1=4, k=5, n=5))
    a = uniform_pm1(11, 1, con.A.span)
    b = np.eye(5, dtype=np.float32).reshape(-1)
    got, _ = oracle.contract(con, F32, 1.0, a, b, 0.0, None)
    a_nd = nd_view(a, con.A)                       # [m0, k, m1]
    want = np.transpose(a_nd, (1, 2, 0))           # [n(=k), m1, m0]
    assert np.array_equal(nd_view(got, con.C), want.astype(np.float64))


def test_rank_one_operands_closed_form():
    # A = u_m0 (x) u_k0 (x) u_m1 (x) u_k1, B likewise: C = prod <u_k, v_k> * outer(free vectors)
    con = workload("cfg4", dict(m0=3, m1=4, n0=2, n1=5, k0=3, k1=2)).contraction
    ext = con.extent_of()
    vec = {l: np.arange(1, ext[l] + 1, dtype=np.float64) * (l + 2) for l in ext}   # per-mode, distinct
    wec = {l: np.arange(2, ext[l] + 2, dtype=np.float64) - (l % 3) for l in ext}

    def outer(labels, table):
        out = np.ones(())
        for l in labels:
            out = np.multiply.outer(out, table[l])
        return out

    a = scatter_nd(outer(con.A.labels, vec), con.A).astype(np.float32)
    b = scatter_nd(outer(con.B.labels, wec), con.B).astype(np.float32)
    im, in_, ik = con.index_sets()
    scalar = np.prod([np.dot(vec[l], wec[l]) for l in ik])
    free = {l: (vec[l] if l in im else wec[l]) for l in con.C.labels}
    want = scalar * outer(con.C.labels, free)
    got, _ = oracle.contract(con, F32, 1.0, a, b, 0.0, None, threads=3)
    assert np.array_equal(nd_view(got, con.C), want)


def test_index_encoding_lands_at_the_right_offsets():
    # A[idx] = sum_j digit_j * 10^j ; B one-hot at (k0*, n*) picks A[:, k0*, :] into C[.., n*]
    con = parse_spec("C[n,m1,m0] = A[m0,k,m1] * B[n,k]", dict(m0=3, m1=4, k=5, n=2))
    a_nd = np.zeros((3, 5, 4))
    for m0, k, m1 in itertools.product(range(3), range(5), range(4)):
        a_nd[m0, k, m1] = m0 + 10 * k + 100 * m1
    a = scatter_nd(a_nd, con.A).astype(np.float32)
    b_nd = np.zeros((2, 5))
    b_nd[1, 3] = 1.0
    b = scatter_nd(b_nd, con.B).astype(np.float32)
    got, _ = oracle.contract(con, F32, 1.0, a, b, 0.0, None)
    for m0, m1 in itertools.product(range(3), range(4)):
        assert got[1 + 2 * m1 + 8 * m0] == m0 + 30 + 100 * m1       # n = 1
        assert got[0 + 2 * m1 + 8 * m0] == 0.0                      # n = 0


# ---- invariants ----
def _perm_storage(spec: TensorSpec, flat: np.ndarray, perm):
    """Same logical tensor stored with its modes in another order (packed)."""
    nd = nd_view(flat, spec)
    labels = [spec.labels[p] for p in perm]
    ext = [spec.extents[p] for p in perm]
    new = TensorSpec(labels, ext, packed_strides(ext))
    return new, scatter_nd(np.transpose(nd, perm), new)


@pytest.mark.parametrize("seed", range(6))
def test_relabelling_and_storage_permutation_invariance(seed):
    rng = np.random.default_rng(200 + seed)
    con = random_contraction(rng, max_rank=5, max_extent=4, pad=False)
    a, b, c = _ints(con, seed)
    base, _ = oracle.contract(con, F32, 2.0, a, b, 1.0, c)
    # consistent relabelling changes nothing
    m = {l: 50 - 3 * l for l in con.extent_of()}
    rel = Contraction("r", *[TensorSpec([m[l] for l in t.labels], t.extents, t.strides)
                             for t in (con.A, con.B, con.C)])
    again, _ = oracle.contract(rel, F32, 2.0, a, b, 1.0, c)
    assert np.array_equal(base, again)
    # permuting storage order of A and B together with their data: same C
    pa = list(rng.permutation(len(con.A.labels)))
    pb = list(rng.permutation(len(con.B.labels)))
    A2, a2 = _perm_storage(con.A, a, pa)
    B2, b2 = _perm_storage(con.B, b, pb)
    same, _ = oracle.contract(Contraction("p", A2, B2, con.C), F32, 2.0, a2, b2, 1.0, c)
    assert np.array_equal(base, same)
    # permuting C's storage permutes the result
    pc = list(rng.permutation(len(con.C.labels)))
    C2, c2 = _perm_storage(con.C, c, pc)
    moved, _ = oracle.contract(Contraction("q", con.A, con.B, C2), F32, 2.0, a, b, 1.0, c2)
    assert np.array_equal(nd_view(moved, C2), np.transpose(nd_view(base, con.C), pc))
    # swapping the roles of A and B (I_m <-> I_n) gives the same C
    swapped, _ = oracle.contract(Contraction("s", con.B, con.A, con.C), F32, 2.0, b, a, 1.0, c)
    assert np.array_equal(base, swapped)


def test_linearity_in_alpha_and_beta():
    con = workload("cfg1", dict(m0=4, m1=3, n0=5, k=6)).contraction
    a, b, c = _ints(con, 9)
    off = oracle.c_offsets(con)
    p10, _ = oracle.contract(con, F32, 1.0, a, b, 0.0, None)
    for alpha, beta in [(2.0, 0.0), (0.0, 3.0), (-1.5, 0.5), (4.0, -2.0)]:
        got, _ = oracle.contract(con, F32, alpha, a, b, beta, c)
        assert np.array_equal(got[off], alpha * p10[off] + beta * c[off].astype(np.float64))


def test_beta_zero_does_not_read_c_and_alpha_zero_scales_c():
    con = workload("cfg1", dict(m0=4, m1=3, n0=5, k=6)).contraction
    a, b, c = _ints(con, 10)
    nan_c = np.full(con.C.span, np.nan, np.float32)
    got, _ = oracle.contract(con, F32, 1.0, a, b, 0.0, nan_c)
    assert np.all(np.isfinite(got))
    got0, _ = oracle.contract(con, F32, 0.0, a, b, 2.0, c)
    assert np.array_equal(got0, 2.0 * c.astype(np.float64))


# ---- degenerate index sets and padded strides ----
def test_empty_index_sets():
    # no contracted mode: outer product
    con = parse_spec("C[m,n] = A[m] * B[n]", dict(m=3, n=4))
    a, b, _ = _ints(con, 1)
    got, _ = oracle.contract(con, F32, 1.0, a, b, 0.0, None)
    assert np.array_equal(got.reshape(4, 3), np.outer(b, a).astype(np.float64))
    # no free mode in B: matrix-vector
    con = parse_spec("C[m] = A[m,k] * B[k]", dict(m=3, k=5))
    a, b, _ = _ints(con, 2)
    got, _ = oracle.contract(con, F32, 1.0, a, b, 0.0, None)
    assert np.array_equal(got, (a.reshape(5, 3).T.astype(np.float64) @ b.astype(np.float64)))
    # no free mode at all: dot product
    con = parse_spec("C[] = A[k] * B[k]", dict(k=7))
    a, b, _ = _ints(con, 3)
    got, absacc = oracle.contract(con, F32, 1.0, a, b, 0.0, None)
    assert got[0] == float(np.dot(a.astype(np.float64), b.astype(np.float64)))
    assert absacc[0] == float(np.dot(np.abs(a).astype(np.float64), np.abs(b).astype(np.float64)))


def test_padded_strides_leave_gaps_untouched():
    con = parse_spec("C[m,n] = A[k,m] * B[n,k]", dict(m=3, n=2, k=4),
                     strides={"A": [2, 9], "B": [1, 3], "C": [1, 5]})
    a, b, c = _ints(con, 4)
    got, _ = oracle.contract(con, F32, 1.0, a, b, 1.0, c)
    ref = brute_force(con, a, b, 1.0, 1.0, c)
    assert np.array_equal(got, ref)
    touched = set(oracle.c_offsets(con).tolist())
    assert all(got[o] == 0.0 for o in range(con.C.span) if o not in touched)


# ---- 16-bit operands are widened exactly ----
@pytest.mark.parametrize("dtype", [BF16_F32, F16_F32])
def test_sixteen_bit_operands_widen_exactly(dtype):
    con = workload("cfg1", dict(m0=4, m1=3, n0=5, k=6)).contraction
    a32 = uniform_pm1(5, 1, con.A.span)
    b32 = uniform_pm1(5, 2, con.B.span)
    a16, b16 = encode_operand(a32, dtype), encode_operand(b32, dtype)
    if dtype == BF16_F32:
        aw, bw = bf16_bits_to_f32(a16), bf16_bits_to_f32(b16)
    else:
        aw, bw = a16.view(np.float16).astype(np.float32), b16.view(np.float16).astype(np.float32)
    got, _ = oracle.contract(con, dtype, 1.0, a16, b16, 0.0, None)
    want, _ = oracle.contract(con, F32, 1.0, aw, bw, 0.0, None)
    assert np.array_equal(got, want)
    # every 16-bit pattern of a half widens to numpy's value (subnormals, inf included)
    if dtype == F16_F32:
        allbits = np.arange(65536, dtype=np.uint16)
        finite = np.isfinite(allbits.view(np.float16))
        bits = allbits[finite]
        one = parse_spec("C[m] = A[m,k] * B[k]", dict(m=bits.size, k=1))
        ones = encode_operand(np.ones(1, np.float32), dtype)
        g, _ = oracle.contract(one, dtype, 1.0, bits, ones, 0.0, None)
        assert np.array_equal(g, bits.view(np.float16).astype(np.float64))


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, 1.0 + 2 ** -8 + 2 ** -20, -0.3, 3.0e38], np.float32)
    got = bf16_bits_to_f32(encode_operand(x, BF16_F32))
    # ties: 1 + 2^-8 is halfway between 1 and 1 + 2^-7 -> even (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    assert got[0] == 1.0 and got[1] == 1.0 and got[2] == 1.015625 and got[3] == 1.0078125
    assert abs(got[4] - (-0.3)) <= 2 ** -9 * 0.3 * 2


# ---- points() is the same computation as contract() ----
def test_points_equal_full_contraction():
    con = workload("cfg5", dict(m0=2, m1=3, m2=2, n0=3, n1=2, n2=2, k=5)).contraction
    a = uniform_pm1(6, 1, con.A.span)
    b = uniform_pm1(6, 2, con.B.span)
    c = uniform_pm1(6, 3, con.C.span)
    full, fabs = oracle.contract(con, F32, 1.0, a, b, 1.0, c, threads=2)
    rng = np.random.default_rng(0)
    pts = np.stack([rng.integers(0, e, 50) for e in con.C.extents], axis=1)
    vals, pabs = oracle.points(con, F32, 1.0, a, b, 1.0, c, pts, threads=2)
    off = (pts * np.array(con.C.strides)).sum(axis=1)
    assert np.array_equal(vals, full[off]) and np.array_equal(pabs, fabs[off])


# ---- preconditions (Sec. 2.2, footnote on indices in all three tensors) ----
@pytest.mark.parametrize("spec,sizes,code", [
    ("C[m,n,b] = A[m,k,b] * B[k,n,b]", dict(m=2, n=2, k=2, b=2), 2),   # batch label
    ("C[m,n] = A[m,k,x] * B[k,n]", dict(m=2, n=2, k=2, x=2), 2),       # label only in A
    ("C[m,n,y] = A[m,k] * B[k,n]", dict(m=2, n=2, k=2, y=2), 2),       # label only in C
])
def test_bad_labels_are_rejected(spec, sizes, code):
    con = parse_spec(spec, sizes)
    a, b, c = _ints(con)
    with pytest.raises(oracle.OracleError) as e:
        oracle.contract(con, F32, 1.0, a, b, 0.0, None)
    assert e.value.code == code


def test_repeated_label_and_extent_mismatch_are_rejected():
    t = TensorSpec([0, 0], [2, 2], [1, 2])
    con = Contraction("x", t, TensorSpec([0, 1], [2, 2], [1, 2]), TensorSpec([1], [2], [1]))
    with pytest.raises(oracle.OracleError) as e:
        oracle.contract(con, F32, 1.0, np.zeros(4, np.float32), np.zeros(4, np.float32), 0.0, None)
    assert e.value.code == 2
    con = Contraction("y", TensorSpec([0, 2], [2, 3], [1, 2]), TensorSpec([2, 1], [4, 2], [1, 4]),
                      TensorSpec([0, 1], [2, 2], [1, 2]))
    with pytest.raises(oracle.OracleError) as e:
        oracle.contract(con, F32, 1.0, np.zeros(6, np.float32), np.zeros(8, np.float32), 0.0, None)
    assert e.value.code == 3


# ---- fp64 operands (the precision of the paper's Table IV): same loop nest, double storage ----
@pytest.mark.parametrize("seed", range(12))
def test_fp64_operands_match_brute_force_exactly_and_einsum(seed):
    from workloads import F64, uniform_pm1_f64
    rng = np.random.default_rng(300 + seed)
    con = random_contraction(rng, max_rank=5, max_extent=5)
    # small integers stored as double: the flatten-to-matrix brute force is exact
    a, b, c = (x.astype(np.float64) for x in _ints(con, seed))
    alpha, beta = [(1.0, 0.0), (2.0, -1.0), (-3.0, 2.0)][seed % 3]
    got, _ = oracle.contract(con, F64, alpha, a, b, beta, c, threads=1 + seed % 3)
    assert np.array_equal(got, brute_force(con, a, b, alpha, beta, c))
    # 53-bit draws: the old C really is read as double (a float read would lose the low bits)
    a, b, c = (uniform_pm1_f64(seed, t, n) for t, n in ((1, con.A.span), (2, con.B.span), (3, con.C.span)))
    got, absacc = oracle.contract(con, F64, 1.0, a, b, 1.0, c)
    ref = scatter_nd(einsum_ref(con, a, b), con.C)
    off = oracle.c_offsets(con)
    np.testing.assert_allclose(got[off], ref[off] + c[off], rtol=0, atol=4e-15 * max(1.0, absacc.max()))
    only_c, _ = oracle.contract(con, F64, 0.0, a, b, 1.0, c)
    assert np.array_equal(only_c[off], c[off])          # bit-exact doubles, not floats
    pts = np.stack([rng.integers(0, e, 20) for e in con.C.extents], axis=1) if con.C.extents else np.zeros((1, 0), int)
    pv, _ = oracle.points(con, F64, 1.0, a, b, 1.0, c, pts)
    poff = (pts * np.array(con.C.strides, dtype=np.int64)).sum(axis=1) if con.C.extents else np.zeros(1, int)
    assert np.array_equal(pv, got[poff])

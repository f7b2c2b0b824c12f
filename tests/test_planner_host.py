"""Host planner through the C ABI (no GPU needed): classification, canonical
order, merging, the offset tables bit-exact against the oracle's div/mod
tables, and the error codes of the boundary."""
import numpy as np
import pytest

import paper_1607_00145_b200 as g
from helpers import random_contraction
from oracle import tables as T
from workloads import Contraction, TensorSpec, parse_spec, workload


def _tables_match(con, dtype=g.GETT_F32, **opts):
    p = g.Plan(con, dtype, **opts)
    want = T.canonical_tables(con)
    for name in g.TABLE_NAMES:
        got = p.table(name)
        assert got.dtype == np.int64
        assert np.array_equal(got, want[name]), name
    return p


@pytest.mark.parametrize("key", ["cfg1", "cfg2", "cfg4", "cfg5"])
@pytest.mark.parametrize("dtype", [g.GETT_F32, g.GETT_BF16_F32])
def test_workload_tables_bit_exact(key, dtype):
    con = workload(key).contraction
    p = _tables_match(con, dtype)
    assert (p.info.M, p.info.N, p.info.K) == con.mnk()
    im, in_, ik = T.classify(con)
    d = p.info.as_dict()
    assert (d["labels_m"], d["labels_n"], d["labels_k"]) == (im, in_, ik)
    mm, mn, mk = T.merged_extents(con)
    assert (p.info.merged_m, p.info.merged_n, p.info.merged_k) == (len(mm), len(mn), len(mk))


def test_cfg3_merges_to_one_m_digit_and_tables_match_on_a_scaled_copy():
    p = g.Plan(workload("cfg3").contraction, g.GETT_F32)
    assert (p.info.M, p.info.N, p.info.K) == (1048576, 24, 24)
    assert p.info.merged_m == 1 and p.info.digits_m == 1
    _tables_match(workload("cfg3", dict(m0=64, m1=48)).contraction)


@pytest.mark.parametrize("seed", range(60))
def test_fuzz_tables_bit_exact(seed):
    rng = np.random.default_rng(1000 + seed)
    con = random_contraction(rng, max_rank=6, max_extent=9, min_each=0 if seed % 5 == 0 else 1)
    _tables_match(con, [g.GETT_F32, g.GETT_BF16_F32, g.GETT_F16_F32][seed % 3])


def test_listing8_example_merges_like_the_paper():
    con = parse_spec("C[a,b,c,i,j,k] = A[i,j,m,c] * B[m,k,a,b]",
                     dict(a=24, b=24, c=24, i=24, j=24, k=24, m=24))
    p = _tables_match(con)
    assert (p.info.merged_m, p.info.merged_n, p.info.merged_k) == (2, 2, 1)
    assert (p.info.M, p.info.N, p.info.K) == (24 * 576, 576 * 24, 24)


def test_extent_one_and_empty_sets():
    con = parse_spec("C[m,u,n] = A[k,m,u] * B[n,k,v]", dict(m=3, u=1, n=2, k=4, v=1))
    # v is carried by B only but has extent 1: still a label error (it is in one tensor only)
    with pytest.raises(g.GettError) as e:
        g.Plan(con, g.GETT_F32)
    assert e.value.status == 2
    con = parse_spec("C[m,u,n] = A[k,m,u] * B[n,k]", dict(m=3, u=1, n=2, k=4))
    p = _tables_match(con)
    assert p.info.n_m == 1
    for spec, sizes, mnk in [("C[m,n] = A[m] * B[n]", dict(m=3, n=4), (3, 4, 1)),
                             ("C[m] = A[m,k] * B[k]", dict(m=3, k=5), (3, 1, 5)),
                             ("C[] = A[k] * B[k]", dict(k=7), (1, 1, 7))]:
        p = _tables_match(parse_spec(spec, sizes))
        assert (p.info.M, p.info.N, p.info.K) == mnk


@pytest.mark.parametrize("spec,sizes,status", [
    ("C[m,n,b] = A[m,k,b] * B[k,n,b]", dict(m=2, n=2, k=2, b=2), 2),
    ("C[m,n] = A[m,k,x] * B[k,n]", dict(m=2, n=2, k=2, x=2), 2),
    ("C[m,n,y] = A[m,k] * B[k,n]", dict(m=2, n=2, k=2, y=2), 2),
])
def test_bad_labels(spec, sizes, status):
    with pytest.raises(g.GettError) as e:
        g.Plan(parse_spec(spec, sizes), g.GETT_F32)
    assert e.value.status == status


def test_other_error_codes():
    ok = parse_spec("C[m,n] = A[m,k] * B[k,n]", dict(m=2, n=2, k=2))
    # repeated label
    bad = Contraction("x", TensorSpec([0, 0], [2, 2], [1, 2]), ok.B, ok.C)
    with pytest.raises(g.GettError) as e:
        g.Plan(bad, g.GETT_F32)
    assert e.value.status == 2
    # extent mismatch
    bad = Contraction("x", TensorSpec([0, 2], [2, 3], [1, 2]), ok.B, ok.C)
    with pytest.raises(g.GettError) as e:
        g.Plan(bad, g.GETT_F32)
    assert e.value.status == 3
    # zero stride, zero extent
    for t in (TensorSpec([0, 2], [2, 2], [0, 2]), TensorSpec([0, 2], [0, 2], [1, 2])):
        with pytest.raises(g.GettError) as e:
            g.Plan(Contraction("x", t, ok.B, ok.C), g.GETT_F32)
        assert e.value.status == 1
    # self-overlapping C
    bad = Contraction("x", ok.A, ok.B, TensorSpec([0, 1], [2, 2], [1, 1]))
    with pytest.raises(g.GettError) as e:
        g.Plan(bad, g.GETT_F32)
    assert e.value.status == 1
    # unknown dtype, too many modes
    with pytest.raises(g.GettError) as e:
        g.Plan(ok, 7)
    assert e.value.status == 4
    many = TensorSpec(list(range(13)), [1] * 13, [1] * 13)
    with pytest.raises(g.GettError) as e:
        g.Plan(Contraction("x", many, ok.B, ok.C), g.GETT_F32)
    assert e.value.status == 1


def test_null_strides_mean_packed_first_mode_fastest():
    con = workload("cfg5", dict(m0=2, m1=3, m2=4, n0=5, n1=2, n2=3, k=6)).contraction
    packed = Contraction("p", *[TensorSpec(t.labels, t.extents, None) for t in (con.A, con.B, con.C)])
    p = g.Plan(packed, g.GETT_F32)
    want = T.canonical_tables(con)
    for name in g.TABLE_NAMES:
        assert np.array_equal(p.table(name), want[name])


def test_contract_without_device_reports_cuda_error_not_a_crash():
    import torch
    if torch.cuda.is_available():
        pytest.skip("has a device")
    p = g.Plan(workload("cfg1").contraction, g.GETT_F32)
    assert p.info.device == -1
    with pytest.raises(g.GettError) as e:
        g.gett_contract(p.handle, 1.0, 16, 16, 0.0, 16, stream=0)
    assert e.value.status == 7


def test_operands_are_exchanged_when_c_runs_along_a_mode_of_a_that_is_not_a_s_own():
    # C's stride-1 mode `a` belongs to A, whose own stride-1 mode is `b`
    con = parse_spec("C[a,b,j,l,c,i] = A[b,c,k,a] * B[j,i,k,l]",
                     dict(a=24, b=24, c=8, i=8, j=24, l=8, k=40))
    for dtype in (g.GETT_BF16_F32, g.GETT_F32):
        p = _tables_match(con, dtype)          # the tables stay the caller's, bit for bit
        i = p.info
        assert i.swapped == 1 and (i.M, i.N, i.K) == con.mnk()
        im, in_, ik = T.classify(con)
        assert i.as_dict()["labels_m"] == im and i.as_dict()["labels_n"] == in_
        assert i.loader_a == g.GETT_LOAD_VEC_FREE and i.epilogue == g.GETT_EPI_STAGED
        # asked for direct stores there is nothing to gain from the exchange
        assert g.Plan(con, dtype, epilogue=g.GETT_EPI_DIRECT).info.swapped == 0
    # A's stride-1 mode is also C's: rows already run along C, no exchange
    assert g.Plan(workload("cfg4").contraction, g.GETT_BF16_F32).info.swapped == 0
    assert g.Plan(workload("cfg3").contraction, g.GETT_F32).info.swapped == 0


def test_short_16_bit_contractions_move_c_s_mode_to_the_column_side():
    """C runs along A's own stride-1 mode and the contraction is short: each thread of the tensor-core
    kernel would update its row of C element by element with no main loop to hide that behind, so the
    operands change places and C goes through the staged unpacking.  Long contractions, fp32 and
    plans with the flag keep their sides."""
    spec = "C[m0,n0,m1,n1] = A[m0,k0,m1,k1] * B[n1,k1,n0,k0]"
    short = parse_spec(spec, dict(m0=96, m1=16, n0=16, n1=96, k0=8, k1=32))      # K = 256
    i = _tables_match(short, g.GETT_BF16_F32).info
    assert i.swapped == 1 and i.epilogue == g.GETT_EPI_STAGED and (i.M, i.N, i.K) == short.mnk()
    assert g.Plan(short, g.GETT_BF16_F32, flags=g.GETT_OPT_NO_EXCHANGE).info.swapped == 0
    assert g.Plan(short, g.GETT_BF16_F32, epilogue=g.GETT_EPI_DIRECT).info.swapped == 0
    assert g.Plan(short, g.GETT_F32).info.swapped == 0
    long_ = parse_spec(spec, dict(m0=96, m1=16, n0=16, n1=96, k0=8, k1=128))     # K = 1024
    assert g.Plan(long_, g.GETT_BF16_F32).info.swapped == 0
    # a mode of C whose stride is not a multiple of four elements rules the 16-byte vectors out
    # A's own stride-1 mode is a contracted one: I_m is ordered for C anyway, the same applies
    kmaj = parse_spec("C[a,b,c,d,e,f] = A[g,d,a,b] * B[e,f,g,c]", dict(a=24, b=16, c=16, d=24, e=24, f=16, g=24))
    i = _tables_match(kmaj, g.GETT_BF16_F32).info
    assert i.swapped == 1 and i.epilogue == g.GETT_EPI_STAGED
    assert g.Plan(kmaj, g.GETT_BF16_F32, flags=g.GETT_OPT_NO_EXCHANGE).info.epilogue == g.GETT_EPI_DIRECT
    gemm = parse_spec("C[m,n] = A[m,k] * B[k,n]", dict(m=96, n=64, k=64))
    assert g.Plan(gemm, g.GETT_BF16_F32).info.swapped == 1
    padded = parse_spec("C[m,n] = A[m,k] * B[k,n]", dict(m=96, n=64, k=64), strides={"C": [1, 98]})
    assert g.Plan(padded, g.GETT_BF16_F32).info.swapped == 0


def test_split_k_planning():
    con = workload("splitk").contraction
    auto = g.Plan(con, g.GETT_F32)
    assert auto.info.split_k > 1 and auto.info.workspace_bytes == auto.info.split_k * 384 * 376 * 4
    never = g.Plan(con, g.GETT_F32, split_k=1)
    assert never.info.split_k == 1 and never.info.workspace_bytes == 0
    forced = g.Plan(workload("cfg4").contraction, g.GETT_F32, split_k=2)
    assert forced.info.split_k == 2 and forced.info.workspace_bytes == 2 * 5184 * 5184 * 4
    # cfg3's whole contracted range (24) is a single K slab: it cannot be sliced
    assert g.Plan(workload("cfg3").contraction, g.GETT_F32, split_k=2).info.split_k == 1
    assert g.Plan(workload("cfg3").contraction, g.GETT_F32, path=g.GETT_PATH_SIMT,
                  split_k=2).info.split_k == 2
    assert g.Plan(workload("cfg3").contraction, g.GETT_F32).info.split_k == 1


def test_sliced_contractions_take_the_tile_that_moves_the_fewest_operand_bytes():
    """384 x 376 x 147456 is cut along K until every SM has a piece, so the tile shape only decides how
    often A and B are delivered: 128 x 192 tiles deliver (2 + 3) x 384 rows of K, 128 x 64 tiles
    (6 + 3) x 384, 256 x 256 tiles (2 + 2) x 512."""
    for key in ("splitk", "splitk_vec"):
        i = g.Plan(workload(key).contraction, g.GETT_BF16_F32).info
        assert (i.tile_m, i.tile_n) == (128, 192) and i.tiles == 6 and i.split_k == 24 and i.grid == 144
        # an explicit width is kept
        assert g.Plan(workload(key).contraction, g.GETT_BF16_F32, tile_n=64).info.tile_n == 64
    # square 512 x 512: 256 x 256 tiles deliver (2 + 2) x 512 rows, 128 x 256 (2 + 4) x 512
    con = parse_spec("C[m,n] = A[k,m] * B[k,n]", dict(m=512, n=512, k=65536))
    i = g.Plan(con, g.GETT_BF16_F32).info
    assert (i.tile_m, i.tile_n, i.tiles) == (256, 256, 4) and i.split_k > 1
    # with enough tiles for the machine the rule stays out of it
    assert g.Plan(workload("cfg4").contraction, g.GETT_BF16_F32).info.split_k == 1


def test_fp32_tile_height_follows_the_rows_there_are():
    """Strict fp32: 64-row tiles when all rows fit them (a 24-row output in a 128-row tile is 81 %
    padding, in a 64-row tile 62 %), 128-row tiles when 64-row tiles would not pad less."""
    ttm = parse_spec("C[a,b,c] = A[b,d,a] * B[d,c]", dict(a=384, b=384, c=24, d=384))      # abc-bda-dc
    i = g.Plan(ttm, g.GETT_F32).info
    assert i.swapped == 1 and (i.tile_m, i.tile_n) == (64, 128)
    wide = parse_spec("C[a,b,c,d] = A[e,a] * B[e,b,c,d]", dict(a=96, b=84, c=84, d=84, e=96))  # abcd-ea-ebcd
    assert g.Plan(wide, g.GETT_F32).info.tile_m == 128
    assert g.Plan(workload("cfg5").contraction, g.GETT_F32).info.tile_m == 64


def test_paths_loaders_and_epilogues_chosen_for_the_workloads():
    want = {  # key, dtype -> (path, loader_a, loader_b, epilogue)
        # cfg1: N = 40, K = 48 -> the small-N kernel (A staged MN-major, B read once element by element)
        ("cfg1", g.GETT_F32): (g.GETT_PATH_FFMA, g.GETT_LOAD_VEC_FREE, g.GETT_LOAD_SCALAR, g.GETT_EPI_DIRECT),
        # cfg2: plain matrices, every tile is a box of a 2-D tensor map -> TMA
        ("cfg2", g.GETT_BF16_F32): (g.GETT_PATH_UMMA, g.GETT_LOAD_TMA_FREE, g.GETT_LOAD_TMA_K, g.GETT_EPI_DIRECT),
        # cfg3: small N and K -> B is read once into shared memory, element by element
        ("cfg3", g.GETT_F32): (g.GETT_PATH_FFMA, g.GETT_LOAD_VEC_K, g.GETT_LOAD_SCALAR, g.GETT_EPI_DIRECT),
        # cfg4: tiles straddle the 72-wide modes (72 = 64 + 8: the remainder is too narrow for atoms) -> gathers
        ("cfg4", g.GETT_BF16_F32): (g.GETT_PATH_UMMA, g.GETT_LOAD_VEC_FREE, g.GETT_LOAD_VEC_FREE, g.GETT_EPI_DIRECT),
        ("cfg5", g.GETT_BF16_F32): (g.GETT_PATH_UMMA, g.GETT_LOAD_VEC_FREE, g.GETT_LOAD_VEC_FREE, g.GETT_EPI_STAGED),
    }
    for (key, dtype), exp in want.items():
        i = g.Plan(workload(key).contraction, dtype).info
        assert (i.path, i.loader_a, i.loader_b, i.epilogue) == exp, key
    # cfg5: the tile is all 8-wide pieces of B's stride-1 mode x the whole of C's stride-1 mode
    i = g.Plan(workload("cfg5").contraction, g.GETT_BF16_F32).info
    assert (i.tile_m, i.tile_n, i.tile_k) == (128, 192, 64) and i.digits_n == 4
    # cfg5 fp32: B's mode is cut into 4-wide pieces (one 16-byte vector of fp32) around C's mode,
    # the unpacking goes through the slot-permuted transpose, short K -> 64-row tiles
    i = g.Plan(workload("cfg5").contraction, g.GETT_F32).info
    assert (i.path, i.loader_a, i.loader_b, i.epilogue) == \
        (g.GETT_PATH_FFMA, g.GETT_LOAD_VEC_FREE, g.GETT_LOAD_VEC_FREE, g.GETT_EPI_STAGED)
    assert (i.tile_m, i.tile_n, i.tile_k, i.block) == (64, 128, 32, 128) and i.digits_n == 4
    # ... asked for direct stores, the split is off and the N order follows C: B goes scalar
    i = g.Plan(workload("cfg5").contraction, g.GETT_F32, epilogue=g.GETT_EPI_DIRECT).info
    assert (i.loader_b, i.epilogue) == (g.GETT_LOAD_SCALAR, g.GETT_EPI_DIRECT)
    # ... and when a stride of C is not a multiple of four the split would not pay off either
    w5 = workload("cfg5", dict(m0=3, m1=8, m2=5, n0=8, n1=3, n2=8, k=40)).contraction
    padded = Contraction(w5.name, w5.A, w5.B,
                         TensorSpec(w5.C.labels, w5.C.extents, [1, 9, 9 * 5, 9 * 5 * 8, 9 * 5 * 8 * 8, 9 * 5 * 8 * 8 * 3]),
                         w5.label_names)
    i = g.Plan(padded, g.GETT_F32).info
    assert (i.loader_b, i.epilogue) == (g.GETT_LOAD_SCALAR, g.GETT_EPI_DIRECT)
    # 80-wide lead modes (80 = 64 + 16): tiles of 64 x 64 atoms -- 64 lead indices, or the last 16
    # x 4 indices of the next mode, alternating with period 80 * 4 -- and slabs of 8 x 8 contracted
    # indices (I_k ordered 8 x 72 x 9): the 64-wide atoms come by TMA, the others are gathered
    at = parse_spec("C[m0,n0,m1,n1] = A[m0,k0,m1,k1] * B[n1,k1,n0,k0]",
                    dict(m0=80, m1=64, n0=64, n1=80, k0=72, k1=72))
    i = g.Plan(at, g.GETT_BF16_F32).info
    assert (i.loader_a, i.loader_b) == (g.GETT_LOAD_TMA_FREE, g.GETT_LOAD_TMA_FREE)
    assert (i.digits_m, i.digits_n, i.digits_k) == (5, 5, 3) and (i.M, i.N, i.K) == (5120, 5120, 5184)
    _tables_match(at, g.GETT_BF16_F32)
    i = g.Plan(at, g.GETT_BF16_F32, flags=g.GETT_OPT_NO_ATOMS).info
    assert (i.loader_a, i.loader_b) == (g.GETT_LOAD_VEC_FREE, g.GETT_LOAD_VEC_FREE)
    # ... a lead extent whose remainder does not divide 64 (40 = 0 * 64 + 40) keeps the gather
    nob = parse_spec("C[m0,n0,m1,n1] = A[m0,k0,m1,k1] * B[n1,k1,n0,k0]",
                     dict(m0=40, m1=8, n0=8, n1=96, k0=72, k1=8))
    i = g.Plan(nob, g.GETT_BF16_F32).info
    assert (i.loader_a, i.loader_b) == (g.GETT_LOAD_VEC_FREE, g.GETT_LOAD_TMA_FREE)
    # a 4-D operand whose leading extents are multiples of the tile is a box of a 4-D tensor map
    boxy = parse_spec("C[m0,n0,m1,n1] = A[m0,k0,m1,k1] * B[n1,k1,n0,k0]",
                      dict(m0=128, m1=3, n0=5, n1=256, k0=64, k1=3))
    i = g.Plan(boxy, g.GETT_BF16_F32).info
    assert (i.loader_a, i.loader_b) == (g.GETT_LOAD_TMA_FREE, g.GETT_LOAD_TMA_FREE)
    # odd extents cannot be gathered in 16-byte vectors: scalar path
    odd = parse_spec("C[m,n] = A[m,k] * B[k,n]", dict(m=7, n=5, k=3))
    assert g.Plan(odd, g.GETT_BF16_F32).info.path == g.GETT_PATH_SIMT
    with pytest.raises(g.GettError) as e:
        g.Plan(odd, g.GETT_BF16_F32, path=g.GETT_PATH_UMMA)
    assert e.value.status == 4


def test_operands_beyond_32_bit_offsets_go_to_the_scalar_kernel():
    """The vector kernels keep operand offsets in 32 bits; a (padded) operand that spans more is
    planned for the scalar-gather kernel, and forcing a vector path is refused.  No memory is
    allocated: only the plan is made."""
    huge = 1 << 33  # elements between consecutive columns of A: 32 GiB of fp32
    for dtype, vec_path in ((g.GETT_F32, g.GETT_PATH_FFMA), (g.GETT_BF16_F32, g.GETT_PATH_UMMA)):
        stride = huge if dtype == g.GETT_F32 else huge * 8
        con = Contraction("wide", TensorSpec([0, 2], [128, 64], [1, stride]), TensorSpec([2, 1], [64, 128], [1, 64]),
                          TensorSpec([0, 1], [128, 128], [1, 128]))
        i = g.Plan(con, dtype).info
        assert i.path == g.GETT_PATH_SIMT
        with pytest.raises(g.GettError) as e:
            g.Plan(con, dtype, path=vec_path)
        assert e.value.status == 4
        # just below the limit the vector path is still taken
        small = Contraction("ok", TensorSpec([0, 2], [128, 64], [1, 1 << 20]), con.B, con.C)
        assert g.Plan(small, dtype).info.path == vec_path


def test_pair_variant_guard_rule():
    """The CTA-pair variant may only see operands that are ordinary device memory of the plan's own GPU."""
    import ctypes
    lib = ctypes.CDLL(g.library_path())
    f = lib.gett_internal_pointer_is_local
    f.restype = ctypes.c_int
    f.argtypes = [ctypes.c_int] * 3
    DEVICE, HOST, MANAGED, UNREGISTERED = 2, 1, 3, 0
    assert f(DEVICE, 0, 0) == 1 and f(DEVICE, 3, 3) == 1
    assert f(DEVICE, 1, 0) == 0          # a peer GPU's memory
    assert f(HOST, 0, 0) == 0 and f(MANAGED, 0, 0) == 0 and f(UNREGISTERED, 0, 0) == 0
    assert f(DEVICE, -1, -1) == 0        # a plan without a device


def test_stream_k_is_chosen_when_the_last_round_of_tiles_would_be_mostly_empty():
    """896 tiles on 148 SMs = six whole rounds + 8 tiles: the 8 are cut along K and shared by all SMs.
    512 tiles = three rounds + 68: the idle time saved would not pay for the pieces' trip through memory."""
    big = parse_spec("C[a,b,c,d] = A[a,e,b,f] * B[f,d,e,c]", dict(a=96, b=84, c=84, d=84, e=84, f=96))
    i = g.Plan(big, g.GETT_BF16_F32).info
    if i.grid == 148:   # (the rule depends on the SM count; without a device 148 is assumed)
        assert i.stream_k == 1 and i.split_k == 1 and i.tiles == 896 and i.workspace_bytes > 0
    assert g.Plan(big, g.GETT_BF16_F32, flags=g.GETT_OPT_NO_STREAMK).info.stream_k == 0
    mid = parse_spec("C[m,n] = A[m,k] * B[k,n]", dict(m=4096, n=4096, k=2048))
    assert g.Plan(mid, g.GETT_BF16_F32).info.stream_k == 0
    assert g.Plan(mid, g.GETT_BF16_F32, flags=g.GETT_OPT_STREAMK).info.stream_k == 1
    # never with K slices, never with fewer tiles than SMs
    assert g.Plan(workload("splitk_vec").contraction, g.GETT_BF16_F32, flags=g.GETT_OPT_STREAMK).info.stream_k == 0

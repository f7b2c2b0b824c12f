"""GPU parity: the CUDA library (through the C ABI) against the CPU oracle,
element by element on the same seeded inputs."""
import numpy as np
import pytest

import paper_1607_00145_b200 as g
from gpu_util import TOL, parity_case
from helpers import random_contraction
from workloads import BF16_F32, F16_F32, F32, F64, parse_spec, workload

pytestmark = pytest.mark.gpu

DTYPES = [F32, BF16_F32, F16_F32]


def test_cfg1_reference_case():
    w = workload("cfg1")
    ratio, info = parity_case(w.contraction, F32, w.dist, w.seed, w.alpha, w.beta, repeat=2)
    assert (info.M, info.N, info.K) == (768, 40, 48)


# Reduced copies of the other workloads: several tiles in M and N plus a ragged
# tail, several K slabs, sized so the oracle finishes in seconds.
SMALL = {
    "cfg2": dict(m=200, n=136, k=88),
    "cfg3": dict(m0=40, m1=33, n0=24, k=24),
    "cfg4": dict(m0=24, m1=9, n0=7, n1=24, k0=8, k1=11),
    "cfg5": dict(m0=3, m1=8, m2=6, n0=8, n1=3, n2=8, k=40),
}


@pytest.mark.parametrize("key", sorted(SMALL))
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("path", [g.GETT_PATH_AUTO, g.GETT_PATH_SIMT])
def test_reduced_workloads(key, dtype, path):
    w = workload(key, SMALL[key])
    parity_case(w.contraction, dtype, w.dist, w.seed, w.alpha, w.beta, repeat=2, path=path)


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("epilogue", [g.GETT_EPI_AUTO, g.GETT_EPI_DIRECT])
def test_cfg5_shape_with_split_stride_one_mode(dtype, epilogue):
    """B's stride-1 mode (16) is split into pieces of one 16-byte vector around C's stride-1
    mode (12): exercises the staged epilogues against the direct ones."""
    w = workload("cfg5", dict(m0=2, m1=16, m2=5, n0=12, n1=3, n2=16, k=72))
    ratio, info = parity_case(w.contraction, dtype, w.dist, w.seed, w.alpha, w.beta, repeat=2,
                              epilogue=epilogue)
    if epilogue == g.GETT_EPI_AUTO: # fp32 too: 4-wide pieces of B's mode, slots through shared memory
        assert info.epilogue == g.GETT_EPI_STAGED
        assert info.loader_b == g.GETT_LOAD_VEC_FREE
    parity_case(w.contraction, dtype, w.dist, w.seed, -0.5, 0.0, epilogue=epilogue)


@pytest.mark.parametrize("tile_n", [64, 128, 192, 256])
@pytest.mark.parametrize("n0", [8, 24, 28])
def test_staged_epilogue_strided_chunks_every_tile_width(tile_n, n0):
    """Column = a + 8 p: every tile width (8, 16, 24, 32 values of p per tile), with C's stride-1
    extent smaller than, equal to and not dividing the tile's p range; ragged M, N and K."""
    w = workload("cfg5", dict(m0=3, m1=8, m2=7, n0=n0, n1=2, n2=24, k=72))
    for dtype in (BF16_F32, F16_F32):
        for alpha, beta in [(1.0, 1.0), (2.0, 0.0)]:
            ratio, info = parity_case(w.contraction, dtype, w.dist, w.seed, alpha, beta, repeat=2, tile_n=tile_n)
            assert info.epilogue == g.GETT_EPI_STAGED and info.tile_n == tile_n
    parity_case(w.contraction, BF16_F32, w.dist, w.seed, 1.0, 0.5, tile_n=tile_n, split_k=2)


@pytest.mark.parametrize("n2,tile_m", [(12, 128), (12, 64), (24, 128), (40, 64)])
def test_fp32_split_of_b_mode(n2, tile_m):
    """fp32: B's stride-1 mode is cut into pieces of 4 (one 16-byte vector) around C's stride-1 mode."""
    w = workload("cfg5", dict(m0=3, m1=16, m2=4, n0=12, n1=2, n2=n2, k=40))
    for alpha, beta in [(1.0, 1.0), (-0.5, 0.0)]:
        ratio, info = parity_case(w.contraction, F32, w.dist, w.seed, alpha, beta, repeat=2, tile_m=tile_m)
        assert info.epilogue == g.GETT_EPI_STAGED and info.loader_b == g.GETT_LOAD_VEC_FREE


def test_staged_epilogue_when_columns_already_run_along_c():
    # B is K-major, C's stride-1 mode is a mode of I_n: slots are the columns themselves
    con = parse_spec("C[n0,m,n1] = A[m,k] * B[k,n1,n0]", dict(m=136, n0=24, n1=7, k=80))
    for dtype in (BF16_F32, F16_F32):
        ratio, info = parity_case(con, dtype, "uniform", 11, 1.0, 1.0, repeat=2)
        assert info.epilogue == g.GETT_EPI_STAGED and info.path == g.GETT_PATH_UMMA


@pytest.mark.parametrize("spec,sizes", [
    ("C[m,n] = A[m,k] * B[k,n]", dict(m=392, n=264, k=200)),                      # 2-D maps, ragged M, N, K
    ("C[m,n] = A[k,m] * B[n,k]", dict(m=256, n=320, k=136)),                      # K-major A, N-major B
    ("C[m0,n0,m1,n1] = A[m0,k0,m1,k1] * B[n1,k1,n0,k0]",
     dict(m0=128, m1=3, n0=2, n1=128, k0=64, k1=3)),                              # 4-D maps
    ("C[m0,m1,n0,n1] = A[k0,m0,k1,m1] * B[k0,k1,n0,n1]",
     dict(m0=256, m1=2, n0=128, n1=3, k0=64, k1=2)),                              # K-major, 4-D maps
])
def test_tma_loader_against_gather_loader_and_oracle(spec, sizes):
    """Tiles that are boxes of a tensor map go through TMA; the same plan with the
    gather loader (GETT_OPT_NO_TMA) must give the same C, and both the oracle's."""
    con = parse_spec(spec, sizes)
    for dtype in (BF16_F32, F16_F32):
        ratio, info = parity_case(con, dtype, "normal", 21, 1.0, 0.5, repeat=2)
        assert info.path == g.GETT_PATH_UMMA
        assert info.loader_a in (g.GETT_LOAD_TMA_FREE, g.GETT_LOAD_TMA_K)
        assert info.loader_b in (g.GETT_LOAD_TMA_FREE, g.GETT_LOAD_TMA_K)
        ratio2, info2 = parity_case(con, dtype, "normal", 21, 1.0, 0.5, flags=g.GETT_OPT_NO_TMA)
        assert info2.loader_a in (g.GETT_LOAD_VEC_FREE, g.GETT_LOAD_VEC_K)
        parity_case(con, dtype, "normal", 21, 1.0, 0.0, split_k=2)


@pytest.mark.parametrize("spec,sizes", [
    ("C[m,n] = A[m,k] * B[k,n]", dict(m=648, n=520, k=200)),                     # TMA, ragged 256-row tiles
    ("C[m0,n0,m1,n1] = A[m0,k0,m1,k1] * B[n1,k1,n0,k0]",
     dict(m0=24, m1=23, n0=11, n1=24, k0=8, k1=19)),                             # gathers, MN-major both
    ("C[m,n] = A[k,m] * B[n,k]", dict(m=520, n=264, k=136)),                     # K-major A, N-major B
])
def test_256_row_tiles(spec, sizes):
    """One tile in both accumulator buffers (tile_m = 256), forced, against the oracle."""
    con = parse_spec(spec, sizes)
    for dtype in (BF16_F32, F16_F32):
        for extra in ({}, {"flags": g.GETT_OPT_NO_TMA}, {"split_k": 2}):
            ratio, info = parity_case(con, dtype, "normal", 33, 1.0, 0.5, repeat=2, tile_m=256,
                                      tile_n=256, **extra)
            assert info.tile_m == 256 and info.path == g.GETT_PATH_UMMA


@pytest.mark.parametrize("spec,sizes", [
    ("C[m,n] = A[m,k] * B[k,n]", dict(m=264, n=200, k=88)),
    ("C[m,n] = A[m,k] * B[n,k]", dict(m=136, n=328, k=200)),
    ("C[m0,n0,m1,n1] = A[m0,k0,m1,k1] * B[n1,k1,n0,k0]", dict(m0=24, m1=9, n0=7, n1=24, k0=8, k1=11)),
])
def test_short_contractions_unpack_through_the_column_side(spec, sizes):
    """C runs along A's own stride-1 mode and K is short: the operands change places so that C goes
    through the staged unpacking; with the sides kept (direct stores, old values of C fetched one
    group of columns ahead) the result must pass as well."""
    con = parse_spec(spec, sizes)
    for dtype in (BF16_F32, F16_F32):
        for alpha, beta in [(1.0, 0.0), (0.5, -2.0)]:
            ratio, info = parity_case(con, dtype, "normal", 23, alpha, beta, repeat=2)
            assert info.swapped == 1 and info.epilogue == g.GETT_EPI_STAGED and info.path == g.GETT_PATH_UMMA
            ratio, info = parity_case(con, dtype, "normal", 23, alpha, beta, repeat=2, flags=g.GETT_OPT_NO_EXCHANGE)
            assert info.swapped == 0 and info.epilogue == g.GETT_EPI_DIRECT


@pytest.mark.parametrize("spec,sizes", [
    ("C[m,n] = A[m,k] * B[k,n]", dict(m=200, n=136, k=88)),                        # A free-major, B K-major
    ("C[m,n] = A[k,m] * B[n,k]", dict(m=136, n=264, k=72)),                        # A K-major, B free-major
    ("C[n0,m2,m1,n2,m0,n1] = A[m1,k,m0,m2] * B[n2,n0,k,n1]",
     dict(m0=2, m1=16, m2=5, n0=12, n1=3, n2=16, k=72)),                           # slots through shared memory
    ("C[m0,n0,m1] = A[m0,k,m1] * B[k,n0]", dict(m0=24, m1=7, n0=40, k=48)),        # rows along C
    ("C[a,b] = A[c,a,d] * B[d,c,b]", dict(a=90, b=70, c=5, d=7)),                  # scalar gathers
])
def test_fp32_64_row_tiles(spec, sizes):
    """The strict-fp32 kernel with 64-row tiles (128 threads, four CTAs per SM), forced."""
    con = parse_spec(spec, sizes)
    for alpha, beta in [(1.0, 0.0), (0.5, 2.0)]:
        ratio, info = parity_case(con, F32, "uniform", 17, alpha, beta, repeat=2, tile_m=64)
        assert info.path == g.GETT_PATH_FFMA and info.tile_m == 64
    parity_case(con, F32, "uniform", 17, 1.0, 0.5, tile_m=64, split_k=2)


ATOM_SPEC = "C[m0,n0,m1,n1] = A[m0,k0,m1,k1] * B[n1,k1,n0,k0]"


@pytest.mark.parametrize("spec,sizes", [
    # 80 = 64 + 16: atoms of 64 (TMA) and atoms of 16 x 4 (gathered) on both sides, slabs of 8 x 8 contracted indices
    (ATOM_SPEC, dict(m0=80, m1=8, n0=16, n1=80, k0=72, k1=8)),
    # 96 = 64 + 32 (atoms of 32 x 2) against 16 = 0 * 64 + 16 (no atoms: gathered); slab = 16 x 4
    (ATOM_SPEC, dict(m0=96, m1=6, n0=12, n1=16, k0=48, k1=12)),
    # 128-wide and 192-wide lead modes (64-wide atoms only), a contracted mode that is a multiple of 64 goes first
    (ATOM_SPEC, dict(m0=128, m1=3, n0=3, n1=192, k0=24, k1=64)),
    # one side keeps the gather (40 = 0 * 64 + 40 does not divide into atoms), the other uses atoms
    (ATOM_SPEC, dict(m0=40, m1=8, n0=8, n1=96, k0=72, k1=8)),
    # a single contracted mode that is not a multiple of 64: the last slab is zero-filled (TMA and gathered atoms alike)
    ("C[m0,n0,m1,n1] = A[m0,k,m1] * B[n1,k,n0]", dict(m0=80, m1=8, n0=8, n1=24, k=200)),
    # three free modes on one side (five map dimensions), the partner is the second mode of the order
    ("C[m0,n0,m1,m2] = A[m0,k0,m2,m1,k1] * B[n0,k1,k0]", dict(m0=96, m1=8, m2=3, n0=136, k0=8, k1=24)),
])
def test_atom_tma_loader_against_gather_loader_and_oracle(spec, sizes):
    """Operands whose tiles are not boxes but lists of 64 x 64 atoms that are (the 72-wide family):
    TMA atom by atom, against the oracle, against the gather loader, with split-K, with 256-row
    tiles, and with a ragged last tile in both directions."""
    con = parse_spec(spec, sizes)
    for dtype in (BF16_F32, F16_F32):
        # (a short contraction whose C runs along A's stride-1 mode would exchange its operands for
        #  the staged unpacking, which keeps the gather: the atoms are tested with the sides kept)
        ratio, info = parity_case(con, dtype, "normal", 51, 1.0, 0.5, repeat=2, flags=g.GETT_OPT_NO_EXCHANGE)
        assert info.path == g.GETT_PATH_UMMA
        assert g.GETT_LOAD_TMA_FREE in (info.loader_a, info.loader_b)
        parity_case(con, dtype, "normal", 51, 1.0, 0.5)
        ratio2, info2 = parity_case(con, dtype, "normal", 51, 1.0, 0.5, flags=g.GETT_OPT_NO_TMA)
        assert info2.loader_a == g.GETT_LOAD_VEC_FREE and info2.loader_b == g.GETT_LOAD_VEC_FREE
    parity_case(con, BF16_F32, "normal", 51, -0.5, 0.0, repeat=2, split_k=2)
    parity_case(con, BF16_F32, "normal", 51, 1.0, 1.0, repeat=2, tile_m=256, tile_n=256)
    parity_case(con, BF16_F32, "normal", 51, 1.0, 0.0, tile_n=64)


@pytest.mark.parametrize("spec,sizes", [
    ("C[m,n] = A[m,k] * B[k,n]", dict(m=648, n=1000, k=200)),    # A in boxes of 64 rows, ragged M, N and K
    ("C[m,n] = A[k,m] * B[n,k]", dict(m=520, n=520, k=136)),     # K-major A: half-height boxes
])
def test_cta_pair_variant_equals_the_single_cta_kernel(spec, sizes):
    """Two CTAs per pair of 256 x 256 tiles sharing the A tile (used when its library is there and
    the number of tile columns is even) against the oracle and, bit for bit, against the ordinary
    kernel (same arithmetic, same order)."""
    import torch
    from workloads import make_inputs
    con = parse_spec(spec, sizes)
    for dtype in (BF16_F32, F16_F32):
        parity_case(con, dtype, "normal", 41, 1.0, 0.5, repeat=2, tile_m=256, tile_n=256)
        a, b, c = make_inputs(con, dtype, "normal", 41, 0.5)
        outs = []
        for switch in (0, g.GETT_OPT_NO_PAIR):
            da = torch.from_numpy(a.view(np.int16)).cuda()
            db = torch.from_numpy(b.view(np.int16)).cuda()
            dc = torch.from_numpy(c).cuda()
            p = g.Plan(con, dtype, tile_m=256, tile_n=256, flags=switch)
            p(1.0, da, db, 0.5, dc)
            torch.cuda.synchronize()
            assert p.device_status() == 0
            outs.append(dc.cpu())
        assert torch.equal(outs[0], outs[1])


@pytest.mark.parametrize("sizes", [dict(m0=40, m1=33, n0=24, k=24), dict(m0=300, m1=7, n0=5, k=12),
                                   dict(m0=64, m1=9, n0=32, k=64), dict(m0=17, m1=3, n0=1, k=4)])
def test_tensor_times_small_matrix_kernel(sizes):
    """cfg3's shape family: B resident in shared memory, A streamed (fp32 only)."""
    w = workload("cfg3", sizes)
    for alpha, beta in [(1.0, 0.0), (0.5, 2.0)]:
        ratio, info = parity_case(w.contraction, F32, w.dist, w.seed, alpha, beta, repeat=2)
        assert info.path == g.GETT_PATH_FFMA and info.tile_m == 256
    # the same contraction through the general fp32 kernel, where B can be vector-gathered too
    if sizes["n0"] % 4 == 0:
        ratio, info = parity_case(w.contraction, F32, w.dist, w.seed, 1.0, 1.0, tile_m=128)
        assert info.tile_m == 128


@pytest.mark.parametrize("sizes", [dict(m0=40, m1=33, n0=24, k=24), dict(m0=36, m1=9, n0=50, k=64)])
def test_tensor_times_small_matrix_kernel_scalar_stores(sizes):
    """The K-major small-N kernel when C does not run along the rows (rows q, q + 64, ... per thread)."""
    con = parse_spec("C[n0,m0,m1] = A[k,m0,m1] * B[n0,k]", sizes)
    for alpha, beta in [(1.0, 0.0), (0.5, 2.0)]:
        ratio, info = parity_case(con, F32, "uniform", 29, alpha, beta, repeat=2, epilogue=g.GETT_EPI_DIRECT)
        assert info.path == g.GETT_PATH_FFMA and info.tile_m == 256 and info.loader_a == g.GETT_LOAD_VEC_K


@pytest.mark.parametrize("spec,sizes,vec_rows", [
    ("C[m0,m1,n0] = A[m0,k,m1] * B[n0,k]", dict(m0=72, m1=11, n0=24, k=24), True),     # rows run along C
    ("C[m0,n0,m1] = A[m0,m1,k] * B[k,n0]", dict(m0=40, m1=29, n0=17, k=48), True),     # odd N
    ("C[n0,m0,m1] = A[m0,k,m1] * B[k,n0]", dict(m0=24, m1=37, n0=8, k=20), False),     # C runs along n0
    ("C[m0,m1,n0] = A[m0,k,m1] * B[n0,k]", dict(m0=256, m1=5, n0=32, k=64), True),     # widest N and K
    ("C[m0,m1,n0] = A[m0,k,m1] * B[n0,k]", dict(m0=8, m1=300, n0=12, k=7), True),      # K not a multiple of 4
    ("C[m1,m0,n0] = A[m0,k,m1] * B[n0,k]", dict(m0=8, m1=300, n0=12, k=7), False),     # C runs along another mode of A:
    ("C[b,u,a,c] = A[c,k,a,b] * B[k,u]", dict(a=19, b=40, c=12, u=48, k=48), False),   # ... A's mode is split around it
])
def test_tensor_times_small_matrix_kernel_a_free_major(spec, sizes, vec_rows):
    """The small-N, small-K fp32 kernel with A staged MN-major (A's stride-1 mode is free)."""
    con = parse_spec(spec, sizes)
    for alpha, beta in [(1.0, 0.0), (0.5, 2.0)]:
        ratio, info = parity_case(con, F32, "uniform", 23, alpha, beta, repeat=2, epilogue=g.GETT_EPI_DIRECT)
        assert info.path == g.GETT_PATH_FFMA and info.tile_m == 256 and info.loader_a == g.GETT_LOAD_VEC_FREE


@pytest.mark.parametrize("spec,sizes", [
    ("C[a,b] = A[c,a,d] * B[d,c,b]", dict(a=200, b=136, c=24, d=40)),              # the paper's ab-cad-dcb layout
    ("C[a,b,c,d] = A[e,a,f,b] * B[f,d,e,c]", dict(a=24, b=9, c=7, d=24, e=16, f=24)),  # abcd-eafb-fdec
    ("C[a,b] = A[c,a,d,e] * B[d,e,c,b]", dict(a=136, b=72, c=8, d=16, e=5)),       # a third contracted mode, u of extent 8
])
def test_transposing_loader_for_two_different_contracted_stride1_modes(spec, sizes):
    """16-bit operands whose stride-1 modes are two different contracted modes: B is read along its
    own stride-1 mode and transposed in 8 x 8 blocks on the way to shared memory, so the
    tensor-core kernel applies (every tile width, split-K, both 16-bit types, ragged tiles)."""
    con = parse_spec(spec, sizes)
    for dtype in (BF16_F32, F16_F32):
        ratio, info = parity_case(con, dtype, "normal", 61, 1.0, 0.5, repeat=2)
        assert info.path == g.GETT_PATH_UMMA
        assert (info.loader_a, info.loader_b) == (g.GETT_LOAD_VEC_K, g.GETT_LOAD_VEC_KT)
    for tile_n in (64, 128, 192, 256):
        parity_case(con, BF16_F32, "normal", 61, -0.5, 0.0, repeat=2, tile_n=tile_n)
    parity_case(con, BF16_F32, "normal", 61, 1.0, 1.0, repeat=2, tile_m=256, tile_n=256)
    parity_case(con, BF16_F32, "normal", 61, 1.0, 0.0, repeat=2, split_k=3)
    parity_case(con, BF16_F32, "normal", 61, 1.0, 0.0, path=g.GETT_PATH_SIMT)


@pytest.mark.parametrize("spec,sizes", [
    ("C[a,b] = A[c,a,d] * B[d,c,b]", dict(a=136, b=72, c=24, d=40)),               # ab-cad-dcb
    ("C[a,b,c,d] = A[e,a,f,b] * B[f,d,e,c]", dict(a=24, b=9, c=7, d=24, e=12, f=24)),  # abcd-eafb-fdec, u = 3 blocks of 4
    ("C[a,b] = A[c,a,d,e] * B[d,e,c,b]", dict(a=136, b=72, c=4, d=16, e=5)),       # a third contracted mode, u of extent 4
    ("C[a,b] = A[c,a,d] * B[d,c,b]", dict(a=40, b=136, c=64, d=8)),                # eight blocks of u per block of v
])
def test_fp32_transposing_loader(spec, sizes):
    """fp32 operands whose stride-1 modes are two different contracted modes: slabs of 4 x 8 indices
    of the two modes, B read in 16-byte pieces along its own mode and transposed in 4 x 4 blocks in
    shared memory (both tile heights, narrow tiles, split-K, ragged tiles), against the oracle and
    against the element-wise gather."""
    con = parse_spec(spec, sizes)
    for alpha, beta in [(1.0, 0.5), (-0.5, 0.0)]:
        ratio, info = parity_case(con, F32, "normal", 67, alpha, beta, repeat=2)
        assert info.path == g.GETT_PATH_FFMA
        assert (info.loader_a, info.loader_b) == (g.GETT_LOAD_VEC_K, g.GETT_LOAD_VEC_KT)
    parity_case(con, F32, "normal", 67, 1.0, 0.0, repeat=2, tile_m=64)
    parity_case(con, F32, "normal", 67, 1.0, 0.0, repeat=2, tile_n=32)
    parity_case(con, F32, "normal", 67, 1.0, 1.0, repeat=2, split_k=3)
    parity_case(con, F32, "normal", 67, 1.0, 0.0, path=g.GETT_PATH_SIMT)


@pytest.mark.parametrize("spec,sizes,opts", [
    # 15 x 11 = 165 tiles of 128 x 64 on 148 SMs, 5 slabs (the last one ragged): TMA boxes
    ("C[m,n] = A[m,k] * B[k,n]", dict(m=1904, n=696, k=296), dict(tile_m=128, tile_n=64)),
    # gathered operands, 4-D, several modes per dimension
    ("C[m0,n0,m1,n1] = A[m0,k0,m1,k1] * B[n1,k1,n0,k0]", dict(m0=24, m1=80, n0=30, n1=24, k0=8, k1=20),
     dict(tile_m=128, tile_n=64)),
    # 256-row tiles (both accumulator buffers per tile): 3 x 53 = 159 tiles
    ("C[m,n] = A[k,m] * B[n,k]", dict(m=600, n=13504, k=200), dict(tile_m=256, tile_n=256)),
])
def test_stream_k_shares_of_the_tile_slab_space(spec, sizes, opts):
    """Stream-K, forced: every CTA takes an equal share of the tiles x slabs space, tiles shared by
    two CTAs go through the workspace and the fix-up kernel; against the oracle, twice (fixed
    order of the pieces: bit-reproducible), with and without the old C."""
    con = parse_spec(spec, sizes)
    for dtype in (BF16_F32, F16_F32):
        for alpha, beta in [(1.0, 0.5), (-0.5, 0.0)]:
            # (sides kept: these short contractions would otherwise take the staged unpacking, which has no pieces)
            ratio, info = parity_case(con, dtype, "normal", 71, alpha, beta, repeat=2,
                                      flags=g.GETT_OPT_STREAMK | g.GETT_OPT_NO_EXCHANGE, **opts)
            assert info.stream_k == 1 and info.split_k == 1 and info.workspace_bytes > 0
    ratio, info = parity_case(con, BF16_F32, "normal", 71, 1.0, 0.5,
                              flags=g.GETT_OPT_NO_STREAMK | g.GETT_OPT_NO_EXCHANGE, **opts)
    assert info.stream_k == 0


@pytest.mark.parametrize("key", sorted(SMALL))
def test_double_precision_path(key):
    """GETT_F64 (the precision of the paper's Table IV): fp64 operands, fp64 FMAs, fp64 C, through the
    scalar-gather kernel; against the oracle to 1e-13 of the scale, twice, and with beta = 0 on NaN."""
    w = workload(key, SMALL[key])
    ratio, info = parity_case(w.contraction, F64, w.dist, w.seed, w.alpha, w.beta, repeat=2)
    assert info.path == g.GETT_PATH_SIMT and info.split_k == 1
    parity_case(w.contraction, F64, w.dist, w.seed, -0.5, 0.0)
    with pytest.raises(g.GettError) as e:   # no K slices, no vector kernels in double precision
        g.Plan(w.contraction, F64, split_k=2)
    assert e.value.status == 4
    with pytest.raises(g.GettError) as e:
        g.Plan(w.contraction, F64, path=g.GETT_PATH_FFMA)
    assert e.value.status == 4


@pytest.mark.parametrize("seed", range(12))
def test_double_precision_fuzz(seed):
    rng = np.random.default_rng(9000 + seed)
    con = random_contraction(rng, max_rank=6, max_extent=9, min_each=0 if seed % 6 == 0 else 1)
    alpha, beta = [(1.0, 0.0), (1.0, 1.0), (-0.5, 2.0)][seed % 3]
    parity_case(con, F64, "uniform", seed, alpha, beta)


@pytest.mark.parametrize("seed", range(48))
def test_fuzz_random_contractions(seed):
    rng = np.random.default_rng(5000 + seed)
    con = random_contraction(rng, max_rank=6, max_extent=9, min_each=0 if seed % 6 == 0 else 1)
    dtype = DTYPES[seed % 3]
    alpha, beta = [(1.0, 0.0), (1.0, 1.0), (-0.5, 2.0), (2.0, -0.5), (0.0, 1.0), (0.0, 0.0)][seed % 6]
    parity_case(con, dtype, "uniform", seed, alpha, beta)


@pytest.mark.parametrize("seed", range(12))
def test_fuzz_vector_friendly_extents(seed):
    """Extents that are multiples of 8 (and 4), so the vectorised loaders engage."""
    rng = np.random.default_rng(7000 + seed)
    con = random_contraction(rng, max_rank=5, pad=False, extent_choices=[8, 16, 24, 40])
    dtype = DTYPES[seed % 3]
    alpha, beta = [(1.0, 0.0), (1.5, -1.0)][seed % 2]
    parity_case(con, dtype, "normal", seed, alpha, beta)


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("split", [2, 3, 7])
def test_forced_split_k(dtype, split):
    con = workload("splitk", dict(a=72, b=40, c=24, d=40)).contraction
    ratio, info = parity_case(con, dtype, "uniform", 5, 1.0, 0.5, repeat=2, split_k=split)
    assert info.split_k > 1 and info.workspace_bytes > 0


def test_auto_split_k_engages_on_small_outputs():
    con = workload("splitk", dict(a=64, b=48, c=64, d=64)).contraction
    ratio, info = parity_case(con, F32, "uniform", 5, 1.0, 0.0)
    assert info.split_k > 1


def test_degenerate_index_sets():
    for spec, sizes in [("C[m,n] = A[m] * B[n]", dict(m=70, n=9)),
                        ("C[m] = A[m,k] * B[k]", dict(m=130, k=77)),
                        ("C[n] = A[k] * B[k,n]", dict(n=65, k=33)),
                        ("C[] = A[k] * B[k]", dict(k=1000))]:
        for dtype in DTYPES:
            parity_case(parse_spec(spec, sizes), dtype, "uniform", 3, 2.0, 1.0)


def test_padded_strides_and_gaps():
    con = parse_spec("C[m,n,p] = A[k,m,p] * B[n,k]", dict(m=37, n=10, p=5, k=19),
                     strides={"A": [2, 41, 1600], "B": [1, 13], "C": [1, 40, 420]})
    for dtype in DTYPES:
        parity_case(con, dtype, "uniform", 8, 1.0, 1.0)
        parity_case(con, dtype, "uniform", 8, 1.0, 0.0)


def test_unaligned_bases_fall_back_to_scalar_loads():
    import torch
    from oracle import contract, c_offsets, tolerance_ratio
    from workloads import make_inputs
    con = workload("cfg4", SMALL["cfg4"]).contraction
    for dtype in DTYPES:
        a, b, c = make_inputs(con, dtype, "normal", 3, 0.0)
        conv = (lambda x: torch.from_numpy(x.view(np.int16))) if dtype != F32 else torch.from_numpy
        ta = torch.empty(a.size + 1, dtype=conv(a).dtype, device="cuda")
        tb = torch.empty(b.size + 1, dtype=conv(b).dtype, device="cuda")
        ta[1:].copy_(conv(a))
        tb[1:].copy_(conv(b))
        tc = torch.zeros(c.size + 1, dtype=torch.float32, device="cuda")
        p = g.Plan(con, dtype)
        p(1.0, ta[1:], tb[1:], 0.0, tc[1:])
        torch.cuda.synchronize()
        ref, absacc = contract(con, dtype, 1.0, a, b, 0.0, None, threads=4)
        got = tc[1:].cpu().numpy()
        assert tolerance_ratio(got, ref, absacc, 1.0, 0.0, None, c_offsets(con)) <= TOL

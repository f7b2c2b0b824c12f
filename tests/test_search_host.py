"""Candidate enumeration and the performance model (Sec. 3.3 / 3.4 re-parameterised for the GPU):
the model's ordering on cases that can be checked by hand, and the search's bookkeeping.
Host only: ranking needs no device (timing the best candidates does, see the GPU tests)."""
import pytest

import paper_1607_00145_b200 as g
from workloads import parse_spec, workload


def _model(con, dtype, **opts):
    p = g.Plan(con, dtype, **opts)
    total, terms = p.model()
    info = p.info
    p.close()
    return total, terms, info


def test_macro_term_is_the_flops_at_the_tensor_rate_up_to_whole_waves():
    con = workload("cfg2").contraction
    total, terms, info = _model(con, g.GETT_BF16_F32)
    ideal_us = con.flops() / 1670e12 * 1e6
    waves = -(-info.tiles // 148)
    assert ideal_us <= terms[0] <= ideal_us * waves * 148 / info.tiles * 1.02
    assert total >= max(terms[0], terms[3])
    assert abs(info.model_us - total) < 1e-3 * total


def test_larger_tiles_move_fewer_operand_bytes():
    con = workload("cfg2").contraction
    big = _model(con, g.GETT_BF16_F32, tile_m=256, tile_n=256)
    small = _model(con, g.GETT_BF16_F32, tile_m=128, tile_n=64)
    assert big[1][1] + big[1][2] < small[1][1] + small[1][2]   # Time_A + Time_B
    assert big[0] < small[0]


def test_tma_boxes_rank_above_gathers_and_gathers_above_the_scalar_kernel():
    con = workload("cfg2").contraction
    tma = _model(con, g.GETT_BF16_F32)[0]
    gather = _model(con, g.GETT_BF16_F32, flags=g.GETT_OPT_NO_TMA)[0]
    scalar = _model(con, g.GETT_BF16_F32, path=g.GETT_PATH_SIMT)[0]
    assert tma < gather < scalar


def test_splitting_k_wins_on_a_small_output_and_loses_on_a_large_one():
    small_out = workload("splitk_vec").contraction   # 384 x 376 outputs, K = 147456
    assert _model(small_out, g.GETT_BF16_F32, split_k=16)[0] < _model(small_out, g.GETT_BF16_F32, split_k=1)[0]
    large_out = workload("cfg4").contraction
    assert _model(large_out, g.GETT_BF16_F32, split_k=1)[0] < _model(large_out, g.GETT_BF16_F32, split_k=4)[0]


def test_stores_along_c_rank_above_scattered_stores():
    # C's stride-1 mode belongs to B: the staged epilogue stores 16-byte vectors along it, the direct
    # one scatters 4-byte stores
    con = parse_spec("C[n0,m,n1] = A[m,k] * B[k,n1,n0]", dict(m=4096, n0=64, n1=64, k=64))
    staged = _model(con, g.GETT_BF16_F32)
    direct = _model(con, g.GETT_BF16_F32, epilogue=g.GETT_EPI_DIRECT)
    assert staged[2].epilogue == g.GETT_EPI_STAGED and direct[2].epilogue == g.GETT_EPI_DIRECT
    assert staged[1][3] < direct[1][3] and staged[0] < direct[0]


@pytest.mark.parametrize("key,dtype", [("cfg2", g.GETT_BF16_F32), ("cfg4", g.GETT_BF16_F32), ("cfg5", g.GETT_F32),
                                       ("splitk", g.GETT_BF16_F32), ("cfg3", g.GETT_F32)])
def test_search_takes_the_models_best_candidate(key, dtype):
    con = workload(key).contraction
    rule = g.Plan(con, dtype)
    found = g.Plan(con, dtype, search=1)
    assert found.info.candidates >= 1 and found.info.model_rank == 0 and found.info.timed == 0
    assert found.info.model_us <= rule.info.model_us * (1 + 1e-6)   # the rule-based plan is one of the candidates
    assert (found.info.M, found.info.N, found.info.K) == (rule.info.M, rule.info.N, rule.info.K)
    # the choice is remembered: the same request again is served without enumerating
    again = g.Plan(con, dtype, search=1)
    assert again.info.candidates == 0
    assert (again.info.tile_m, again.info.tile_n, again.info.split_k, again.info.epilogue) == \
        (found.info.tile_m, found.info.tile_n, found.info.split_k, found.info.epilogue)
    # caller-fixed fields are respected by every candidate
    fixed = g.Plan(con, dtype, search=1, split_k=1)
    assert fixed.info.split_k == 1


def test_search_reports_errors_like_the_plain_call():
    bad = parse_spec("C[m,n,b] = A[m,k,b] * B[k,n,b]", dict(m=2, n=2, k=2, b=2))
    with pytest.raises(g.GettError) as e:
        g.Plan(bad, g.GETT_F32, search=2)
    assert e.value.status == 2

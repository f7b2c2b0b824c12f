"""gett_contract_noalloc: the entry point for callers that may not allocate device
memory (stream capture, pooled or fixed device heaps, callbacks).  Its split-K partial
sums live in an array built into the library, so it must give the same C as the
plan-based call, call after call, although every call reuses that one array.

Collected last on purpose: a failure here cannot hide results of the other tests."""
import numpy as np
import pytest

import paper_1607_00145_b200 as g
from workloads import BF16_F32, F32, make_inputs, workload

pytestmark = pytest.mark.gpu
TOL = 1e-5


def _dev(x, torch):
    return torch.from_numpy(x.view(np.int16) if x.dtype == np.uint16 else x).cuda()


@pytest.mark.parametrize("dtype", [F32, BF16_F32])
def test_noalloc_matches_plan_based_contract_twice_in_a_row(dtype):
    import torch
    import oracle

    w = workload("splitk", dict(a=72, b=40, c=24, d=40))
    con, split = w.contraction, 5
    a, b, c0 = make_inputs(con, dtype, "uniform", 5, 0.5)
    da, db = _dev(a, torch), _dev(b, torch)
    # reference: the existing entry point, same kernel family and slicing
    plan = g.Plan(con, dtype, path=g.GETT_PATH_SIMT, split_k=split)
    assert plan.info.split_k == split and plan.info.workspace_bytes <= g.GETT_NOALLOC_WORKSPACE_BYTES
    want = _dev(c0, torch)
    plan(1.0, da, db, 0.5, want)
    torch.cuda.synchronize()
    want = want.cpu().numpy()
    scale = float(np.max(oracle.contract(con, dtype, 1.0, a, b, 0.5, c0, threads=4)[1])) + 0.5

    for call in range(2):  # the second call finds the first call's partial sums in the array
        got = _dev(c0, torch)
        g.gett_contract_noalloc(con.A, con.B, con.C, dtype, split, 1.0, da, db, 0.5, got)
        torch.cuda.synchronize()
        err = float(np.max(np.abs(got.cpu().numpy().astype(np.float64) - want))) / scale
        assert err <= TOL, (call, err)

    # a different, smaller problem in between must not be disturbed by what the array holds
    w2 = workload("cfg1", dict(m0=8, m1=5, n0=6, k=64))
    a2, b2, c2 = make_inputs(w2.contraction, dtype, "uniform", 9, 0.0)
    got2 = torch.full((c2.size,), float("nan"), device="cuda")
    g.gett_contract_noalloc(w2.contraction.A, w2.contraction.B, w2.contraction.C, dtype, 4, 2.0,
                            _dev(a2, torch), _dev(b2, torch), 0.0, got2)
    torch.cuda.synchronize()
    ref, absacc = oracle.contract(w2.contraction, dtype, 2.0, a2, b2, 0.0, None, threads=2)
    assert oracle.tolerance_ratio(got2.cpu().numpy(), ref, absacc, 2.0, 0.0, None,
                                  oracle.c_offsets(w2.contraction)) <= TOL


def test_noalloc_rejects_problems_beyond_its_built_in_workspace():
    import torch
    con = workload("cfg4", dict(m0=72, m1=32, n0=72, n1=32, k0=8, k1=8)).contraction   # M = N = 2304
    assert 2 * 2304 * 2304 * 4 > g.GETT_NOALLOC_WORKSPACE_BYTES
    x = torch.zeros(16, device="cuda")
    with pytest.raises(g.GettError) as e:
        g.gett_contract_noalloc(con.A, con.B, con.C, F32, 2, 1.0, x, x, 0.0, x)
    assert e.value.status == 4

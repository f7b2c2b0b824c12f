"""The give-up path of the tensor-core kernel's bounded waits, without any fault injection:
a plan whose wait limit is far shorter than one tile's main loop makes the waiting warps give
up; the kernel must return by itself, report GETT_ERR_TIMEOUT in the plan's status word and
leave the context usable.  Nothing here waits without a bound."""
import numpy as np
import pytest

import oracle
import paper_1607_00145_b200 as g
from workloads import BF16_F32, make_inputs, parse_spec

pytestmark = pytest.mark.gpu


def test_short_wait_limit_gives_up_cleanly_and_the_next_plan_is_correct():
    import torch
    # one 256 x 256 output tile, 1024 slabs of 64: the unpacking warps wait ~1 ms for the accumulator
    con = parse_spec("C[m,n] = A[m,k] * B[k,n]", dict(m=256, n=256, k=65536))
    a, b, c = make_inputs(con, BF16_F32, "uniform", 77, 0.0)
    da = torch.from_numpy(a.view(np.int16)).cuda()
    db = torch.from_numpy(b.view(np.int16)).cuda()
    dc = torch.zeros(c.size, dtype=torch.float32, device="cuda")
    # gathered operands (the limit is honoured only there: their copies are drained on exit)
    short = g.Plan(con, BF16_F32, flags=g.GETT_OPT_NO_TMA, split_k=1, wait_limit_us=1)
    assert short.info.loader_a == g.GETT_LOAD_VEC_FREE and short.info.split_k == 1
    short(1.0, da, db, 0.0, dc)
    torch.cuda.synchronize()                      # the kernel came back by itself
    assert short.device_status() == 8             # GETT_ERR_TIMEOUT
    assert g.gett_status_string(8) == "device-side wait timed out"
    short.close()
    # the context is intact: the same problem with the default limit matches the oracle
    plan = g.Plan(con, BF16_F32, flags=g.GETT_OPT_NO_TMA, split_k=1)
    dc.fill_(float("nan"))
    plan(1.0, da, db, 0.0, dc)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    rng = np.random.default_rng(3)
    pts = np.stack([rng.integers(0, e, 1500) for e in con.C.extents], axis=1)
    off = (pts * np.array(con.C.strides, dtype=np.int64)).sum(axis=1)
    ref, absacc = oracle.points(con, BF16_F32, 1.0, a, b, 0.0, None, pts, threads=oracle.default_threads())
    got = dc[torch.from_numpy(off).cuda()].cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got))
    assert float(np.max(np.abs(got - ref)) / np.max(absacc)) <= 1e-5
    # a TMA-fed plan ignores a shortened limit (its copies cannot be waited for on exit)
    tma = g.Plan(con, BF16_F32, split_k=1, wait_limit_us=1)
    tma(1.0, da, db, 0.0, dc)
    torch.cuda.synchronize()
    assert tma.device_status() == 0
    plan.close()
    tma.close()

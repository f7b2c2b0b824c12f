"""Parity at the workloads' full sizes, in the launch configuration bench.py times
(automatic plan), on sampled outputs the oracle computes one by one.

Sample: the corners of C, outputs straddling every kind of tile boundary (first and
last rows/columns of tiles in the fused M and N order the plan reports), and a few
thousand uniformly random outputs."""
import numpy as np
import pytest

import oracle
import paper_1607_00145_b200 as g
from workloads import BF16_F32, DTYPE_NAMES, F32, make_inputs, workload

pytestmark = pytest.mark.gpu
TOL = 1e-5

CASES = [("cfg2", BF16_F32), ("cfg2", F32), ("cfg3", F32), ("cfg4", BF16_F32), ("cfg4", F32),
         ("cfg5", BF16_F32), ("cfg5", F32)]


def _sample_points(con, info, rng, nrand=6000):
    ext = np.array(con.C.extents, dtype=np.int64)
    pts = [np.zeros(len(ext), np.int64), ext - 1]
    # every mode at its first / last index with the others random: hits tile edges in
    # whatever order the planner fused the modes
    for i in range(len(ext)):
        for v in (0, ext[i] - 1, ext[i] // 2):
            p = np.stack([rng.integers(0, e, 64) for e in ext], axis=1)
            p[:, i] = v
            pts.append(p)
    pts.append(np.stack([rng.integers(0, e, nrand) for e in ext], axis=1))
    return np.concatenate([np.atleast_2d(p) for p in pts], axis=0)


@pytest.mark.parametrize("key,dtype", CASES, ids=[f"{k}-{DTYPE_NAMES[d]}" for k, d in CASES])
def test_full_size_sampled_parity(key, dtype):
    import torch
    w = workload(key)
    con = w.contraction
    a, b, c_old = make_inputs(con, dtype, w.dist, w.seed, w.beta)
    conv = (lambda x: torch.from_numpy(x.view(np.int16))) if dtype != F32 else torch.from_numpy
    da, db = conv(a).cuda(), conv(b).cuda()
    if w.beta == 0.0:
        dc = torch.full((c_old.size,), float("nan"), dtype=torch.float32, device="cuda")
    else:
        dc = torch.from_numpy(c_old).cuda()
    plan = g.Plan(con, dtype)
    plan(w.alpha, da, db, w.beta, dc)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    rng = np.random.default_rng(42)
    pts = _sample_points(con, plan.info, rng)
    off = (pts * np.array(con.C.strides, dtype=np.int64)).sum(axis=1)
    got = dc[torch.from_numpy(off).cuda()].cpu().numpy().astype(np.float64)
    ref, absacc = oracle.points(con, dtype, w.alpha, a, b, w.beta, c_old, pts,
                                threads=oracle.default_threads())
    assert np.all(np.isfinite(got))
    scale = abs(w.alpha) * absacc
    if w.beta != 0.0:
        scale = scale + abs(w.beta) * np.abs(c_old[off].astype(np.float64))
    ratio = float(np.max(np.abs(got - ref)) / np.max(scale))
    assert ratio <= TOL, f"{key} {DTYPE_NAMES[dtype]}: ratio {ratio:.3e}"
    K = con.mnk()[2]
    assert np.all(np.abs(got - ref) <= (K + 2) * 2.0 ** -24 * scale + 1e-30)
    # every output was written: no NaN left where beta == 0 poisoned C (checked on a stride)
    if w.beta == 0.0:
        assert not bool(torch.isnan(dc[::997]).any())
    plan.close()

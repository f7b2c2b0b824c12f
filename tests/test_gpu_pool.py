"""Parity over the seeded pool of synthetic contractions (workloads.pool): random mode orders
of the paper's shape families at realistic sizes, automatic plans, sampled outputs computed
one by one by the oracle."""
import numpy as np
import pytest

import oracle
import paper_1607_00145_b200 as g
from workloads import BF16_F32, DTYPE_NAMES, F32, make_inputs, pool

pytestmark = pytest.mark.gpu
TOL = 1e-5
POOL = pool()


def _points(con, rng, nrand=3000):
    ext = np.array(con.C.extents, dtype=np.int64)
    pts = [np.zeros((1, len(ext)), np.int64), (ext - 1)[None, :]]
    for i in range(len(ext)):  # every mode at its first / last / middle index, the others random
        for v in (0, ext[i] - 1, ext[i] // 2):
            p = np.stack([rng.integers(0, e, 48) for e in ext], axis=1)
            p[:, i] = v
            pts.append(p)
    pts.append(np.stack([rng.integers(0, e, nrand) for e in ext], axis=1))
    return np.concatenate(pts, axis=0)


@pytest.mark.parametrize("dtype", [BF16_F32, F32], ids=lambda d: DTYPE_NAMES[d])
@pytest.mark.parametrize("w", POOL, ids=[w.key for w in POOL])
def test_pool_item_sampled_parity(w, dtype):
    import torch
    con = w.contraction
    a, b, c_old = make_inputs(con, dtype, w.dist, w.seed, w.beta)
    conv = (lambda x: torch.from_numpy(x.view(np.int16))) if dtype != F32 else torch.from_numpy
    da, db = conv(a).cuda(), conv(b).cuda()
    if w.beta == 0.0:  # beta = 0 must not read C: poison it
        dc = torch.full((c_old.size,), float("nan"), dtype=torch.float32, device="cuda")
    else:
        dc = torch.from_numpy(c_old).cuda()
    plan = g.Plan(con, dtype)
    plan(w.alpha, da, db, w.beta, dc)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    pts = _points(con, np.random.default_rng(7))
    off = (pts * np.array(con.C.strides, dtype=np.int64)).sum(axis=1)
    got = dc[torch.from_numpy(off).cuda()].cpu().numpy().astype(np.float64)
    ref, absacc = oracle.points(con, dtype, w.alpha, a, b, w.beta, c_old, pts,
                                threads=oracle.default_threads())
    assert np.all(np.isfinite(got)), con.name
    scale = abs(w.alpha) * absacc
    if w.beta != 0.0:
        scale = scale + abs(w.beta) * np.abs(c_old[off].astype(np.float64))
    ratio = float(np.max(np.abs(got - ref)) / np.max(scale))
    assert ratio <= TOL, f"{con.name} {DTYPE_NAMES[dtype]}: ratio {ratio:.3e}"
    if w.beta == 0.0:
        assert not bool(torch.isnan(dc[::991]).any())
    plan.close()

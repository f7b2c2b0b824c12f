"""Parity over the paper's own benchmark shapes: the 48 contractions of its Appendix A with
their single-precision extents (Table III) and the k-sweep of its Fig. 11, automatic plans,
both dtypes, sampled outputs computed one by one by the oracle.  Inputs are this package's
seeded synthetic numbers (the paper's input files are not used)."""
import numpy as np
import pytest

import oracle
import paper_1607_00145_b200 as g
from workloads import BF16_F32, DTYPE_NAMES, F32, make_inputs
from workloads.paper_benchmark import fig11_sweep, paper_pool

pytestmark = pytest.mark.gpu
TOL = 1e-5
ITEMS = paper_pool("sp") + fig11_sweep()


def _points(con, rng, budget_macs=1.5e8):
    ext = np.array(con.C.extents, dtype=np.int64)
    K = con.mnk()[2]
    nrand = int(max(64, min(1500, budget_macs // K)))
    pts = [np.zeros((1, len(ext)), np.int64), (ext - 1)[None, :]]
    for i in range(len(ext)):  # every mode at its first / last index, the others random
        for v in (0, ext[i] - 1):
            p = np.stack([rng.integers(0, e, 8) for e in ext], axis=1)
            p[:, i] = v
            pts.append(p)
    pts.append(np.stack([rng.integers(0, e, nrand) for e in ext], axis=1))
    return np.concatenate(pts, axis=0)


@pytest.mark.parametrize("dtype", [BF16_F32, F32], ids=lambda d: DTYPE_NAMES[d])
@pytest.mark.parametrize("w", ITEMS, ids=[w.key.replace(" ", "_") for w in ITEMS])
def test_paper_item_sampled_parity(w, dtype):
    import torch
    con = w.contraction
    a, b, c_old = make_inputs(con, dtype, w.dist, w.seed, w.beta, cache=True)
    conv = (lambda x: torch.from_numpy(x.view(np.int16))) if dtype != F32 else torch.from_numpy
    da, db = conv(a).cuda(), conv(b).cuda()
    dc = torch.full((con.C.span,), float("nan"), dtype=torch.float32, device="cuda")  # beta = 0: C is not read
    plan = g.Plan(con, dtype)
    plan(w.alpha, da, db, w.beta, dc)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    pts = _points(con, np.random.default_rng(11))
    off = (pts * np.array(con.C.strides, dtype=np.int64)).sum(axis=1)
    got = dc[torch.from_numpy(off).cuda()].cpu().numpy().astype(np.float64)
    ref, absacc = oracle.points(con, dtype, w.alpha, a, b, w.beta, None, pts, threads=oracle.default_threads())
    assert np.all(np.isfinite(got)), w.key
    ratio = float(np.max(np.abs(got - ref)) / np.max(abs(w.alpha) * absacc))
    assert ratio <= TOL, f"{w.key} {DTYPE_NAMES[dtype]}: ratio {ratio:.3e}"
    assert not bool(torch.isnan(dc[::991]).any())
    plan.close()

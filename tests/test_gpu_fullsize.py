"""Parity at the workloads' full sizes, in the launch configuration bench.py times
(automatic plan), on sampled outputs the oracle computes one by one.

Sample (stratified, so that every row band and every column band of every tile is hit): for
every block of 64 consecutive fused m one random m with ALL n, for every block of 64
consecutive fused n one random n with ALL m (fused in the canonical order the plan reports),
the four 128 x 128 corner blocks, 2^16 uniformly random outputs, and every mode at its first
and last index.  Plans that do not split K must also give bit-identical results twice."""
import numpy as np
import pytest

import oracle
import paper_1607_00145_b200 as g
from workloads import BF16_F32, DTYPE_NAMES, F32, make_inputs, workload

pytestmark = pytest.mark.gpu
TOL = 1e-5

CASES = [("cfg2", BF16_F32), ("cfg2", F32), ("cfg3", F32), ("cfg4", BF16_F32), ("cfg4", F32),
         ("cfg5", BF16_F32), ("cfg5", F32)]


def _fused_to_points(con, labels_m, labels_n, m_idx, n_idx):
    """C index tuples of the (m, n) pairs: m and n are fused over labels_m / labels_n with the
    first label fastest (the canonical order gett_plan_get_info reports)."""
    ext = dict(zip(con.C.labels, con.C.extents))
    pos = {l: i for i, l in enumerate(con.C.labels)}
    pts = np.zeros((len(m_idx), len(con.C.labels)), dtype=np.int64)
    for labels, idx in ((labels_m, np.asarray(m_idx, dtype=np.int64)), (labels_n, np.asarray(n_idx, dtype=np.int64))):
        rem = idx.copy()
        for l in labels:
            pts[:, pos[l]] = rem % ext[l]
            rem //= ext[l]
    return pts


def _sample_points(con, info, rng, nrand=1 << 16, budget_macs=2.5e10):
    d = info.as_dict()
    lm, ln = d["labels_m"], d["labels_n"]
    M, N, K = con.mnk()
    ext = np.array(con.C.extents, dtype=np.int64)
    # thin the bands out if the oracle's work would exceed the budget (cfg2: 2 x 128 bands x 8192 x K)
    full = (-(-M // 64)) * N + (-(-N // 64)) * M
    step = int(max(1, np.ceil(full * K / budget_macs)))
    pts = []
    m_pick = [b * 64 + int(rng.integers(0, min(64, M - b * 64))) for b in range(0, -(-M // 64), step)]
    n_pick = [b * 64 + int(rng.integers(0, min(64, N - b * 64))) for b in range(0, -(-N // 64), step)]
    all_m, all_n = np.arange(M, dtype=np.int64), np.arange(N, dtype=np.int64)
    for m in m_pick:   # one row of every 64-band of fused m, all n
        pts.append(_fused_to_points(con, lm, ln, np.full(N, m), all_n))
    for n in n_pick:   # one column of every 64-band of fused n, all m
        pts.append(_fused_to_points(con, lm, ln, all_m, np.full(M, n)))
    cm, cn = min(128, M), min(128, N)
    for m0 in (0, M - cm):  # the four corner blocks
        for n0 in (0, N - cn):
            mm, nn = np.meshgrid(np.arange(m0, m0 + cm), np.arange(n0, n0 + cn), indexing="ij")
            pts.append(_fused_to_points(con, lm, ln, mm.ravel(), nn.ravel()))
    for i in range(len(ext)):  # every mode at its first / last index, the others random
        for v in (0, ext[i] - 1):
            p = np.stack([rng.integers(0, e, 64) for e in ext], axis=1)
            p[:, i] = v
            pts.append(p)
    pts.append(np.stack([rng.integers(0, e, nrand) for e in ext], axis=1))
    return np.concatenate(pts, axis=0)


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
    # every output was written: no NaN left where beta == 0 poisoned C
    if w.beta == 0.0:
        assert not bool(torch.isnan(dc).any())
    # run-to-run reproducibility at full size (a race would show here): same inputs, same bits
    first = dc.clone()
    if w.beta == 0.0:
        dc.fill_(float("nan"))
    else:
        dc.copy_(torch.from_numpy(c_old))
    plan(w.alpha, da, db, w.beta, dc)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    assert torch.equal(first.view(torch.int32), dc.view(torch.int32)), "not reproducible"
    plan.close()

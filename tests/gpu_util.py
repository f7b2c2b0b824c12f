"""Helpers for the GPU parity tests: guard-banded device buffers and the
acceptance ratio.  Calls the library only through the ctypes binding."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_1607_00145_b200 as g
from workloads import F32, F64, make_inputs

GUARD = 1024  # elements before and after each tensor
TOL = 1e-5    # max|C_gpu - C_ref| / max(|alpha| sum|a||b| + |beta||C_old|)


def _guarded(host: np.ndarray, fill) -> "tuple[torch.Tensor, torch.Tensor]":
    """Device buffer [guard | data | guard]; returns (whole, data view)."""
    n = host.size
    whole = np.empty(n + 2 * GUARD, dtype=host.dtype)
    whole[:GUARD] = fill
    whole[GUARD + n:] = fill
    whole[GUARD:GUARD + n] = host
    if host.dtype == np.uint16:
        t = torch.from_numpy(whole.view(np.int16)).cuda()
    else:
        t = torch.from_numpy(whole).cuda()
    return t, t[GUARD:GUARD + n]


def run_gpu(con, dtype, alpha, beta, a, b, c_old, plan=None, repeat=1, **opts):
    """Run the contraction on the device with NaN guards around A and B and a
    sentinel guard around C that must come back untouched.  Returns (C, info)."""
    own = plan is None
    if own:
        plan = g.Plan(con, dtype, **opts)
    ctype = np.float64 if dtype == F64 else np.float32  # C's element type
    nan16 = np.float64(np.nan) if dtype == F64 else np.uint16(0x7FC0) if dtype != F32 else np.float32(np.nan)
    ta, va = _guarded(a, nan16)
    tb, vb = _guarded(b, nan16)
    sentinel = ctype(-12345.678)
    tc, vc = _guarded(c_old.astype(ctype), sentinel)
    outs = []
    for _ in range(repeat):
        vc.copy_(torch.from_numpy(c_old.astype(ctype)))
        plan(alpha, va, vb, beta, vc)
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        whole = tc.cpu().numpy()
        assert np.all(whole[:GUARD] == sentinel) and np.all(whole[-GUARD:] == sentinel), \
            "write outside C"
        outs.append(whole[GUARD:-GUARD].copy())
    for o in outs[1:]:
        assert np.array_equal(o.view(np.uint8), outs[0].view(np.uint8)), "not reproducible"
    info = plan.info
    if own:
        plan.close()
    return outs[0], info


def check_against_oracle(con, dtype, alpha, beta, a, b, c_old, c_gpu, threads=None):
    """Full element-by-element comparison; returns the acceptance ratio."""
    threads = threads or oracle.default_threads()
    ref, absacc = oracle.contract(con, dtype, alpha, a, b, beta, c_old, threads=threads)
    off = oracle.c_offsets(con)
    assert np.all(np.isfinite(c_gpu[off])), "non-finite output"
    ratio = oracle.tolerance_ratio(c_gpu, ref, absacc, alpha, beta,
                                   c_old if beta != 0.0 else None, off)
    # storage that C's modes do not address must be untouched
    mask = np.ones(con.C.span, dtype=bool)
    mask[off] = False
    if mask.any():
        assert np.array_equal(c_gpu[mask], c_old.astype(c_gpu.dtype)[mask]), "gap overwritten"
    # per-element sanity ceiling: |err| <= (K + 2) * 2^-24 * scale (2^-53 for fp64 arithmetic)
    K = con.mnk()[2]
    scale = abs(alpha) * absacc[off]
    if beta != 0.0:
        scale = scale + abs(beta) * np.abs(c_old[off].astype(np.float64))
    err = np.abs(c_gpu[off].astype(np.float64) - ref[off])
    eps = 2.0 ** -53 if dtype == F64 else 2.0 ** -24
    assert np.all(err <= (K + 2) * eps * scale + 1e-30), "per-element bound"
    if dtype == F64:  # double precision end to end: far inside the fp32 acceptance figure
        assert ratio <= 1e-13, f"fp64 ratio {ratio:.3e}"
    return ratio


def parity_case(con, dtype, dist, seed, alpha, beta, repeat=1, **opts):
    """Seeded inputs -> device run (guarded) -> full comparison with the oracle."""
    a, b, c_old = make_inputs(con, dtype, dist, seed, beta)
    if beta == 0.0:
        # beta = 0 must not read C: poison every addressed element with NaN and
        # give the gaps a finite value that must survive
        off = oracle.c_offsets(con)
        c_old = np.full(con.C.span, 7.0, dtype=np.float64 if dtype == F64 else np.float32)
        c_old[off] = np.nan
    c_gpu, info = run_gpu(con, dtype, alpha, beta, a, b, c_old, repeat=repeat, **opts)
    ratio = check_against_oracle(con, dtype, alpha, beta, a, b, c_old, c_gpu)
    assert ratio <= TOL, f"ratio {ratio:.3e}"
    return ratio, info

"""Plan search on the device (Sec. 7.3: time the few candidates the model ranks best): the
search returns a working plan, reports what it timed, and the chosen plan matches the oracle."""
import numpy as np
import pytest

import paper_1607_00145_b200 as g
from gpu_util import parity_case
from workloads import BF16_F32, F32, parse_spec, workload

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("spec,sizes,dtype", [
    ("C[m0,n0,m1,n1] = A[m0,k0,m1,k1] * B[n1,k1,n0,k0]", dict(m0=24, m1=9, n0=7, n1=24, k0=8, k1=11), BF16_F32),
    ("C[n0,m2,m1,n2,m0,n1] = A[m1,k,m0,m2] * B[n2,n0,k,n1]", dict(m0=3, m1=8, m2=6, n0=8, n1=3, n2=8, k=40), F32),
    ("C[a,b] = A[c,a,d] * B[d,c,b]", dict(a=72, b=40, c=24, d=40), BF16_F32),
])
def test_timed_search_returns_a_correct_plan(spec, sizes, dtype):
    con = parse_spec(spec, sizes)
    ratio, info = parity_case(con, dtype, "uniform", 9, 1.0, 0.5, repeat=2, search=3)
    assert info.candidates >= 1 and 1 <= info.timed <= 4  # the 3 best of the model and the rule-based plan
    assert info.timed_us > 0.0 and 0 <= info.model_rank < info.candidates
    # the remembered choice gives the same plan
    p = g.Plan(con, dtype, search=3)
    assert p.info.candidates == 0
    assert (p.info.tile_m, p.info.tile_n, p.info.split_k, p.info.path) == \
        (info.tile_m, info.tile_n, info.split_k, info.path)
    p.close()

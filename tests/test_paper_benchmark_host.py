"""The paper's benchmark shapes (Appendix A, Tables III / IV; Fig. 11) as this package stores them,
and the host planner on them (no GPU)."""
import numpy as np
import pytest

import paper_1607_00145_b200 as g
from oracle import tables as T
from workloads.paper_benchmark import FIG11_K, fig11_sweep, paper_pool, paper_table


def test_the_table_has_the_papers_48_contractions():
    sp, dp = paper_table("sp"), paper_table("dp")
    assert len(sp) == 48 and len(dp) == 48 and [n for n, _ in sp] == [n for n, _ in dp]
    # spot values as printed in Table III / Table IV
    assert sp[0] == ("abc-bda-dc", dict(a=384, c=24, b=384, d=384))
    assert sp[11] == ("ab-ac-cb", dict(a=7248, c=7248, b=7240))
    assert dp[11] == ("ab-ac-cb", dict(a=5136, c=5136, b=5120))
    assert sp[13] == ("ab-cad-dcb", dict(a=384, c=384, b=376, d=384))
    assert dp[20][1] == dict(a=72, c=72, b=72, e=72, d=72, f=72)
    assert sp[47] == ("abcdef-gfbc-dega", dict(a=24, c=20, b=20, e=20, d=24, g=24, f=20))
    # every contraction of the benchmark occupies at least 200 MiB in single precision (Sec. 7.1)
    for w in paper_pool("sp"):
        con = w.contraction
        assert 4 * (con.A.numel + con.B.numel + con.C.numel) >= 200 * 2 ** 20 * 0.95, w.key


def test_fig11_sweep_sizes():
    sw = fig11_sweep()
    assert len(sw) == 2 * len(FIG11_K)
    for w in sw:
        M, N, K = w.contraction.mnk()
        assert (M, N) == (1152, 1152) and K in FIG11_K


@pytest.mark.parametrize("dtype", [g.GETT_F32, g.GETT_BF16_F32])
def test_every_item_plans_and_reports_its_index_sets(dtype):
    for w in paper_pool("sp") + paper_pool("dp") + fig11_sweep():
        con = w.contraction
        p = g.Plan(con, dtype)
        assert (p.info.M, p.info.N, p.info.K) == con.mnk(), w.key
        im, in_, ik = T.classify(con)
        d = p.info.as_dict()
        assert (d["labels_m"], d["labels_n"], d["labels_k"]) == (im, in_, ik), w.key
        p.close()


@pytest.mark.parametrize("name", ["abcdef-dega-gfbc", "abcdef-gdab-efgc", "abc-adec-ebd", "abcd-aebf-dfce"])
def test_tables_bit_exact_on_paper_items(name):
    w = [x for x in paper_pool("dp") if x.key == name][0]
    for dtype in (g.GETT_F32, g.GETT_BF16_F32):
        p = g.Plan(w.contraction, dtype)
        want = T.canonical_tables(w.contraction)
        for t in g.TABLE_NAMES:
            assert np.array_equal(p.table(t), want[t]), (name, t)
        p.close()

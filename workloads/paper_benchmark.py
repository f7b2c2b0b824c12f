"""The paper's own benchmark shapes (Sec. 7.1, Appendix A) and the k-sweep of Fig. 11.

TABLE lists, as the paper's Tables III and IV print them, the 48 contraction strings with
their single-precision and double-precision extents.  A string "abc-bda-dc" reads C-A-B:
C[a,b,c] = A[b,d,a] * B[d,c], every tensor packed with its first listed mode stride-1
(Sec. 2.2).  Only the shapes are taken from the paper; the tensors are filled with the seeded
synthetic numbers of this package, and the paper's own input files are not used.

The paper does not print alpha and beta for its benchmark: alpha = 1, beta = 0 is used here.
For Fig. 11 it prints S_Im = S_In = 1152 and S_Ik = 8 ... 1024 but not the factors of 1152;
48 x 24 is used for (i1, i2) and (j1, j2).
"""
from __future__ import annotations

from typing import Dict, List, Tuple

from . import BF16_F32, F32, Workload, parse_spec

# contraction (C-A-B), extents of Table III (single precision), extents of Table IV (double precision)
TABLE = """
abc-bda-dc           a:384;c:24;b:384;d:384;                      a:312;c:24;b:312;d:312;
abc-dca-bd           a:384;c:376;b:24;d:384;                      a:312;c:296;b:24;d:312;
abcd-dbea-ec         a:96;c:24;b:84;e:96;d:96;                    a:72;c:24;b:72;e:72;d:72;
abcd-deca-be         a:96;c:84;b:24;e:84;d:96;                    a:72;c:72;b:24;e:72;d:72;
abcd-ebad-ce         a:96;c:24;b:84;e:96;d:84;                    a:72;c:24;b:72;e:72;d:72;
abcde-efbad-cf       a:48;c:24;b:36;e:48;d:36;f:36;               a:48;c:24;b:32;e:48;d:32;f:32;
abcde-ecbfa-fd       a:48;c:36;b:36;e:48;d:24;f:48;               a:48;c:32;b:32;e:48;d:24;f:48;
abcde-efcad-bf       a:48;c:36;b:24;e:48;d:36;f:36;               a:48;c:32;b:24;e:48;d:32;f:32;
abcd-ea-ebcd         a:96;c:84;b:84;e:96;d:84;                    a:72;c:72;b:72;e:72;d:72;
abcd-eb-aecd         a:96;c:84;b:84;e:96;d:84;                    a:72;c:72;b:72;e:72;d:72;
abcd-ec-abed         a:96;c:84;b:84;e:96;d:84;                    a:72;c:72;b:72;e:72;d:72;
ab-ac-cb             a:7248;c:7248;b:7240;                        a:5136;c:5136;b:5120;
ab-acd-dbc           a:384;c:376;b:376;d:384;                     a:312;c:296;b:296;d:312;
ab-cad-dcb           a:384;c:384;b:376;d:384;                     a:312;c:312;b:296;d:312;
abc-acd-db           a:384;c:376;b:376;d:384;                     a:312;c:296;b:296;d:312;
abc-ad-bdc           a:384;c:376;b:384;d:376;                     a:312;c:296;b:312;d:296;
abc-adc-bd           a:384;c:376;b:384;d:376;                     a:312;c:296;b:312;d:296;
abc-adc-db           a:384;c:376;b:376;d:384;                     a:312;c:296;b:296;d:312;
abc-adec-ebd         a:96;c:84;b:84;e:96;d:84;                    a:72;c:72;b:72;e:72;d:72;
abcd-aebf-dfce       a:96;c:84;b:84;e:84;d:96;f:84;               a:72;c:72;b:72;e:72;d:72;f:72;
abcd-aebf-fdec       a:96;c:84;b:84;e:84;d:84;f:96;               a:72;c:72;b:72;e:72;d:72;f:72;
abcd-aecf-bfde       a:96;c:84;b:96;e:84;d:84;f:84;               a:72;c:72;b:72;e:72;d:72;f:72;
abcd-aecf-fbed       a:96;c:84;b:84;e:84;d:84;f:96;               a:72;c:72;b:72;e:72;d:72;f:72;
abcd-aedf-bfce       a:96;c:84;b:96;e:84;d:84;f:84;               a:72;c:72;b:72;e:72;d:72;f:72;
abcd-aedf-fbec       a:96;c:84;b:84;e:84;d:84;f:96;               a:72;c:72;b:72;e:72;d:72;f:72;
abcd-aefb-fdce       a:96;c:84;b:84;e:84;d:84;f:96;               a:72;c:72;b:72;e:72;d:72;f:72;
abcd-aefc-fbed       a:96;c:84;b:84;e:84;d:84;f:96;               a:72;c:72;b:72;e:72;d:72;f:72;
abcd-eafb-fdec       a:96;c:84;b:84;e:96;d:84;f:96;               a:72;c:72;b:72;e:72;d:72;f:72;
abcd-eafc-bfde       a:96;c:84;b:96;e:96;d:84;f:84;               a:72;c:72;b:72;e:72;d:72;f:72;
abcd-eafd-fbec       a:96;c:84;b:84;e:96;d:84;f:96;               a:72;c:72;b:72;e:72;d:72;f:72;
abcdef-dega-gfbc     a:24;c:20;b:20;e:20;d:24;g:24;f:20;          a:24;c:16;b:16;e:16;d:24;g:24;f:16;
abcdef-degb-gfac     a:24;c:20;b:20;e:20;d:24;g:24;f:20;          a:24;c:16;b:16;e:16;d:24;g:24;f:16;
abcdef-degc-gfab     a:24;c:20;b:20;e:20;d:24;g:24;f:20;          a:24;c:16;b:16;e:16;d:24;g:24;f:16;
abcdef-dfga-gebc     a:24;c:20;b:20;e:20;d:24;g:24;f:20;          a:24;c:16;b:16;e:16;d:24;g:24;f:16;
abcdef-dfgb-geac     a:24;c:20;b:20;e:20;d:24;g:24;f:20;          a:24;c:16;b:16;e:16;d:24;g:24;f:16;
abcdef-dfgc-geab     a:24;c:20;b:20;e:20;d:24;g:24;f:20;          a:24;c:16;b:16;e:16;d:24;g:24;f:16;
abcdef-efga-gdbc     a:24;c:20;b:20;e:24;d:20;g:24;f:20;          a:24;c:16;b:16;e:24;d:16;g:24;f:16;
abcdef-efgb-gdac     a:24;c:20;b:20;e:24;d:20;g:24;f:20;          a:24;c:16;b:16;e:24;d:16;g:24;f:16;
abcdef-efgc-gdab     a:24;c:20;b:20;e:24;d:20;g:24;f:20;          a:24;c:16;b:16;e:24;d:16;g:24;f:16;
abcdef-gdab-efgc     a:24;c:20;b:20;e:24;d:20;g:24;f:20;          a:24;c:16;b:16;e:24;d:16;g:24;f:16;
abcdef-gdac-efgb     a:24;c:20;b:20;e:24;d:20;g:24;f:20;          a:24;c:16;b:16;e:24;d:16;g:24;f:16;
abcdef-gdbc-efga     a:24;c:20;b:20;e:24;d:20;g:24;f:20;          a:24;c:16;b:16;e:24;d:16;g:24;f:16;
abcdef-geab-dfgc     a:24;c:20;b:20;e:20;d:24;g:24;f:20;          a:24;c:16;b:16;e:16;d:24;g:24;f:16;
abcdef-geac-dfgb     a:24;c:20;b:20;e:20;d:24;g:24;f:20;          a:24;c:16;b:16;e:16;d:24;g:24;f:16;
abcdef-gebc-dfga     a:24;c:20;b:20;e:20;d:24;g:24;f:20;          a:24;c:16;b:16;e:16;d:24;g:24;f:16;
abcdef-gfab-degc     a:24;c:20;b:20;e:20;d:24;g:24;f:20;          a:24;c:16;b:16;e:16;d:24;g:24;f:16;
abcdef-gfac-degb     a:24;c:20;b:20;e:20;d:24;g:24;f:20;          a:24;c:16;b:16;e:16;d:24;g:24;f:16;
abcdef-gfbc-dega     a:24;c:20;b:20;e:20;d:24;g:24;f:20;          a:24;c:16;b:16;e:16;d:24;g:24;f:16;
"""


def _sizes(txt: str) -> Dict[str, int]:
    return {kv.split(":")[0]: int(kv.split(":")[1]) for kv in txt.split(";") if kv}


def _spec(name: str) -> str:
    c, a, b = name.split("-")
    return f"C[{','.join(c)}] = A[{','.join(a)}] * B[{','.join(b)}]"


def paper_table(precision: str = "sp") -> List[Tuple[str, Dict[str, int]]]:
    """[(contraction string, {mode: extent})] in the order of the paper's tables."""
    out = []
    for line in TABLE.strip().splitlines():
        name, sp, dp = line.split()
        out.append((name, _sizes(sp if precision == "sp" else dp)))
    return out


def paper_pool(precision: str = "sp") -> List[Workload]:
    """The 48 contractions as workloads (uniform[-1, 1) inputs, one seed for all: an element's
    value depends on its storage offset only, so items with equal tensor sizes share their draws)."""
    out = []
    for name, sizes in paper_table(precision):
        w = Workload(name, parse_spec(_spec(name), sizes, name), (F32, BF16_F32), "uniform", 200, 1.0, 0.0,
                     "paper")
        out.append(w)
    return out


FIG11_K = (8, 16, 32, 64, 128, 256, 512, 1024)


def fig11_sweep() -> List[Workload]:
    """The two contractions of Fig. 11 with S_Im = S_In = 1152 and S_Ik from 8 to 1024."""
    out = []
    for k in FIG11_K:
        out.append(Workload(f"i1ji2-i1ki2-jk k={k}",
                            parse_spec("C[i1,j,i2] = A[i1,k,i2] * B[j,k]", dict(i1=48, i2=24, j=1152, k=k)),
                            (F32, BF16_F32), "uniform", 300, 1.0, 0.0, "fig11"))
        out.append(Workload(f"i1j1i2j2-i1ki2-j1kj2 k={k}",
                            parse_spec("C[i1,j1,i2,j2] = A[i1,k,i2] * B[j1,k,j2]",
                                       dict(i1=48, i2=24, j1=48, j2=24, k=k)),
                            (F32, BF16_F32), "uniform", 300, 1.0, 0.0, "fig11"))
    return out

"""B200 (sm_100a) GEMM-like tensor-tensor multiplication: thin ctypes binding
over libgett_b200.so.  Every step of the contraction runs in the CUDA library;
this package only marshals arguments.  There is no CPU fallback: importing
`binding` raises if the shared library has not been built."""
from .binding import (GettError, Plan, gett_contract, gett_plan_create, gett_plan_destroy,  # noqa: F401
                      gett_plan_get_info, gett_plan_get_table, gett_plan_last_device_status, gett_plan_model,
                      gett_status_string, library_path, PlanOpts, PlanInfo,
                      gett_contract_noalloc, GETT_NOALLOC_WORKSPACE_BYTES)
from .binding import (GETT_F32, GETT_BF16_F32, GETT_F16_F32, GETT_F64, GETT_PATH_AUTO, GETT_PATH_SIMT,  # noqa: F401
                      GETT_PATH_FFMA, GETT_PATH_UMMA, GETT_EPI_AUTO, GETT_EPI_DIRECT,
                      GETT_EPI_STAGED, GETT_LOAD_SCALAR, GETT_LOAD_VEC_FREE, GETT_LOAD_VEC_K,
                      GETT_LOAD_TMA_FREE, GETT_LOAD_TMA_K, GETT_LOAD_VEC_KT,
                      GETT_OPT_NO_TMA, GETT_OPT_NO_PAIR, GETT_OPT_NO_EXCHANGE, GETT_OPT_NO_ATOMS,
                      GETT_OPT_STREAMK, GETT_OPT_NO_STREAMK,
                      TABLE_NAMES)

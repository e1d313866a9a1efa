"""B200-native SpGEMM (gMAGNUS hot path): thin Python binding over the C ABI in include/gmagnus.h.

Every step of the computation runs in the CUDA library; this package only marshals arguments.
torch is used for device memory and streams.
"""
from .binding import (  # noqa: F401
    GmError,
    PlanOpts,
    Plan,
    DeviceCSR,
    planner_params,
    planner_batches,
    spgemm_plan,
    row_products_noalloc,
    NOALLOC_MAX_NNZ_A,
    spgemm_execute,
    spgemm,
    spgemm_host,
    load_library,
    EXPORTED_SYMBOLS,
)

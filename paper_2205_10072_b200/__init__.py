"""B200 (sm_100a) construction of round-optimal circulant-graph broadcast schedules
(arXiv 2205.10072, Section 2): a C-ABI CUDA library plus this thin binding.

The names mirror include/bcs.h.  Every computation runs in the CUDA kernels of
libbcs.so; this package only marshals arguments (PyTorch supplies device memory
and streams).  There is no CPU fallback: importing the binding without the built
library raises.
"""
from .binding import (  # noqa: F401
    BcsError,
    BatchPlan,
    bcs_allgather_tables,
    bcs_batch_plan,
    bcs_build,
    bcs_build_batch,
    bcs_build_batch_workspace_bytes,
    bcs_build_prepared,
    bcs_build_rooted,
    bcs_build_rooted_workspace_bytes,
    bcs_build_static,
    bcs_build_workspace_bytes,
    bcs_build_to_host,
    bcs_checksum,
    bcs_circulant_rounds,
    bcs_expand,
    bcs_prepare,
    bcs_prepare_codes,
    bcs_prepare_rows,
    bcs_prepare_workspace_bytes,
    bcs_q,
    bcs_simulate,
    bcs_skips,
    bcs_status_str,
    bcs_validate,
    bcs_wait_expired,
    lib,
    lib_path,
)

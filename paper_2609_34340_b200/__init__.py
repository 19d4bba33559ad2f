"""B200-native VarioPath online scheduler and send-buffer pack (CUDA, sm_100a).

Thin Python binding over the C-ABI library ``libvariopath.so`` (see
``include/variopath.h``): argument marshalling only; every step of the path
runs in the library's CUDA kernels.  There is no CPU fallback: if the library
has not been built, every call raises.
"""
from .binding import (  # noqa: F401
    VpError,
    Catalog,
    Plan,
    SchedParams,
    load_catalog,
    catalog_argmax_classes,
    build_catalog,
    build_template_catalog,
    prune_paths,
    schedule_workspace_bytes,
    schedule_batch,
    schedule_batch_host,
    pack_workspace_bytes,
    pack,
    pack_host,
    pack_static,
    PACK_STATIC_SCRATCH_BYTES,
    unpack_workspace_bytes,
    unpack,
    unpack_tokens,
    kernel_launch_count,
    plan_time,
    sweep_plan_time,
    demand_from_routing,
    schedule_read_stats,
    schedule_launch_info,
    microbench,
    exchange_put,
    exchange_wait,
    gather_exchange_tables,
    memset_probe,
    profile_enable,
    profile_read,
    library_path,
    ST_NEGATIVE, ST_OVERFLOW_RISK, ST_DIAG_NONZERO, ST_NOT_GRANULE, ST_BAD_TAU, ST_UNCOVERED,
    ST_NO_PROGRESS, ST_STEP_LIMIT, ST_PACK_MISMATCH, ST_PACK_CAPACITY, ST_EXCHANGE_TIMEOUT, ST_INTERNAL_TIMEOUT,
    E_BAD_ARG, E_BAD_CATALOG, E_NOMEM, E_CUDA, E_WORKSPACE, E_UNSUPPORTED,
)

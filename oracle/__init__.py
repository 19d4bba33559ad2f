"""CPU oracle for the VarioPath scheduler and pack: TEST INFRASTRUCTURE ONLY.

A thin ctypes wrapper over ``vp_oracle.c`` (plain C, compiled with gcc -O2).
Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library and its Python binding never do.
"""
from .vp_oracle import (  # noqa: F401
    build,
    OracleCatalog,
    demand_from_routing,
    ST_NEGATIVE, ST_OVERFLOW, ST_DIAG, ST_GRANULE, ST_BAD_TAU, ST_UNCOVERED,
    ST_NO_PROGRESS, ST_STEP_LIMIT, ST_PACK_MISMATCH, ST_PACK_CAPACITY,
)

"""Seeded synthetic inputs for the VarioPath online scheduler and pack.

This package only *produces inputs*: topology/catalog blobs (the offline
analyzer of Section 4.1 run as an input generator), demand matrices, routing
indices and token rows.  It contains none of the online method's arithmetic
(Algorithm 2, offsets, pack); both the CPU oracle and the CUDA library consume
its byte blobs and tensors and share nothing else.
"""
from .topology import (  # noqa: F401
    Topology,
    Catalog,
    tree_topology,
    ring_topology,
    crossbar_topology,
    complete_catalog,
    node_template_catalog,
    crossbar_catalog,
)
from .demand import (  # noqa: F401
    moe_demand,
    moe_routing,
    sp_demand,
    uniform_demand,
)
from .configs import CONFIGS, build_config, build_pack_case, SchedParams  # noqa: F401

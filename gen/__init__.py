"""Seeded synthetic inputs for the placement-scoring path.

This package only draws random numbers and packs them into the binary layouts
that both the CUDA library and the CPU oracle consume.  It holds none of the
method's arithmetic (no simulation, no distributor rule, no scoring), so it may
be imported by tests, the benchmark, the oracle wrapper and the product binding
alike without coupling the two implementations.
"""
from .formats import (REQUEST_DTYPE, SLO_DTYPE, RESULT_DTYPE, SLO_NONE, WMAX,
                      MAX_INSTANCES, pack_inst, unpack_inst, make_classes)
from .profiles import profile_tiny, profile_node, profile_multimodel, profile_decay, STRATEGIES_NODE
from .traces import make_trace, trace_from_rows, shrinking_prompts_trace
from .candidates import (enumerate_tiny, enumerate_node, sample_candidates,
                         candidates_from_lists)
from .configs import make_config, make_table1_config, CONFIG_NAMES, TABLE1

__all__ = [
    "REQUEST_DTYPE", "SLO_DTYPE", "RESULT_DTYPE", "SLO_NONE", "WMAX", "MAX_INSTANCES",
    "pack_inst", "unpack_inst", "make_classes",
    "profile_tiny", "profile_node", "profile_multimodel", "STRATEGIES_NODE",
    "make_trace", "trace_from_rows", "shrinking_prompts_trace", "enumerate_tiny", "enumerate_node", "sample_candidates",
    "candidates_from_lists", "make_config", "CONFIG_NAMES", "profile_decay", "make_table1_config", "TABLE1",
]

"""B200-native fused graph-attention aggregation with attention rematerialisation (SAR,
arXiv 2111.06483): Python face of the C-ABI library libsar.so.

    binding  - one function per C entry point (argument marshalling only)
    api      - allocation helpers that chain those calls
    build    - compiles the library in-tree with nvcc for sm_100a
"""
from . import api, binding  # noqa: F401
from .api import Graph, gat_backward, gat_forward, spmm_sum  # noqa: F401

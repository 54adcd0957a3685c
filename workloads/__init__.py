"""Seeded synthetic inputs shared by the oracle-side tests and the CUDA-side tests/benchmark.

This module holds NONE of the method's arithmetic: it only draws graphs (edge lists) and
node tensors from counter-based hashes, so that the same arrays can be handed to the CPU
oracle and to the CUDA library.  Everything is a pure function of (shape, seed); integer
outputs are bit-identical on CPU and CUDA devices (integer hashing + exact table lookups),
floating outputs are generated once on one device and copied wherever they are needed.
"""
from .generators import (  # noqa: F401
    ChungLuSpec,
    chung_lu_edges,
    chung_lu_r0,
    hash64,
    normal_tensor,
    uniform01,
    uniform_edges,
)
from .configs import CONFIGS, WorkloadConfig, make_graph, make_node_inputs  # noqa: F401

"""The five named workloads (graph shape, tensor shapes, dtype, partition count).

They stand in for the graphs the paper measures on (ogbn-products: 2.5 M nodes, 124 M edges;
ogbn-papers100M: 111 M nodes, 3.2 B edges; Table 1), which are not available offline: node and
edge counts, feature widths and head counts are taken from the paper's experiments (Sec. 4.1:
one GAT layer on ogbn-products; Sec. 4.2: 3-layer GAT, hidden 128, 4 heads; 3-layer GraphSage,
hidden 256), the degree distribution is a power law with exponent 2.1.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional

import torch

from .generators import ChungLuSpec, chung_lu_edges, normal_tensor, uniform_edges


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    n: int
    e: int                      # edges drawn (config 1 adds n self-loops on top)
    heads: int
    feat: int                   # features per head
    k: int                      # sequential source partitions
    dtypes: tuple               # storage types of feat/out/gout/dfeat exercised
    graph: str                  # "uniform" or "chung_lu"
    seed: int
    gamma: float = 2.1
    d_max: float = 0.0
    self_loops: bool = False
    layers: int = 1
    spmm_feat: int = 0          # row width of the sum-aggregation case (0 = none)
    slope: float = 0.2

    def scaled(self, factor: float, name: Optional[str] = None) -> "WorkloadConfig":
        """Same recipe with node and edge counts multiplied by `factor` (d_max scales too)."""
        return replace(self, name=name or f"{self.name}@{factor:g}", n=max(8, int(self.n * factor)),
                       e=max(8, int(self.e * factor)), d_max=max(4.0, self.d_max * factor))


CONFIGS = {
    "tiny": WorkloadConfig("tiny", n=2_000, e=20_000, heads=4, feat=16, k=1, dtypes=("f32",),
                           graph="uniform", seed=0, self_loops=True),
    "seqpart": WorkloadConfig("seqpart", n=100_000, e=2_000_000, heads=4, feat=32, k=8, dtypes=("f32",),
                              graph="chung_lu", seed=1, d_max=2_000.0),
    "medium": WorkloadConfig("medium", n=2_450_000, e=62_000_000, heads=4, feat=64, k=4,
                             dtypes=("f32", "bf16"), graph="chung_lu", seed=2, d_max=17_000.0,
                             spmm_feat=256),
    "dense": WorkloadConfig("dense", n=1_000_000, e=200_000_000, heads=8, feat=32, k=8, dtypes=("bf16",),
                            graph="chung_lu", seed=3, d_max=50_000.0),
    "large": WorkloadConfig("large", n=20_000_000, e=300_000_000, heads=4, feat=32, k=16,
                            dtypes=("bf16",), graph="chung_lu", seed=4, d_max=100_000.0, layers=3),
}


def make_graph(cfg: WorkloadConfig, device="cpu", permute: bool = True):
    """(src, dst) int32 edge list of the workload on `device`.  permute=False keeps node id = degree
    rank (hubs first): the locality ablation of the power-law workloads."""
    if cfg.graph == "uniform":
        return uniform_edges(cfg.n, cfg.e, cfg.seed, cfg.self_loops, device=device)
    spec = ChungLuSpec(n=cfg.n, e=cfg.e, gamma=cfg.gamma, d_max=cfg.d_max, seed=cfg.seed, permute=permute)
    return chung_lu_edges(spec, device=device)


def make_node_inputs(n: int, heads: int, feat: int, seed: int, dtype: str = "f32", device="cpu", layer: int = 0):
    """feat[n,H,F], gout[n,H,F] in the storage dtype; el[n,H], er[n,H] float32; all ~ N(0,1)."""
    tdt = {"f32": torch.float32, "bf16": torch.bfloat16}[dtype]
    base = 16 * layer
    return {
        "feat": normal_tensor((n, heads, feat), seed, base + 10, device=device, dtype=tdt),
        "gout": normal_tensor((n, heads, feat), seed, base + 11, device=device, dtype=tdt),
        "el": normal_tensor((n, heads), seed, base + 12, device=device, dtype=torch.float32),
        "er": normal_tensor((n, heads), seed, base + 13, device=device, dtype=torch.float32),
    }

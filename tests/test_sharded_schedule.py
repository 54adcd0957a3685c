"""The multi-worker schedule of Algorithm 1 / Algorithm 2 (who fetches which partition when, the return of the
errors to their owners, the order of accumulation) on CPU: world_size 2 and 3 over gloo, with the arithmetic
of each step done by a plain torch float64 reference, against the oracle on the whole graph."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

import oracle
from helpers import small_problem
from sharded_helpers import TorchRefBackend, rank_edges


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, prob, bounds, ret):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2111_06483_b200.sharded import ShardedGatLayer, TorchDistComm
    lo, hi = bounds[rank], bounds[rank + 1]
    be = TorchRefBackend(rank_edges(bounds, rank, prob["src"], prob["dst"]), hi - lo, prob["H"], prob["F"], 0.2)
    layer = ShardedGatLayer(TorchDistComm(), bounds, be)
    t = lambda k: torch.from_numpy(prob[k][lo:hi]).double()
    out = layer.forward(t("feat"), t("el"), t("er"))
    dfeat, del_, der = layer.backward(t("gout"))
    ret[rank] = tuple(x.numpy() for x in (out, be.m, be.d, dfeat, del_, der))
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_layer_equals_the_whole_graph(world):
    p = small_problem(90, 700, 2, 4, 23, self_loops=True, empty_rows=4)
    bounds = [int(b) for b in oracle.partition_bounds(90, world)]
    ret = mp.Manager().dict()
    prob = {k: p[k] for k in ("src", "dst", "feat", "el", "er", "gout", "H", "F")}
    mp.spawn(_worker, args=(world, _free_port(), prob, bounds, ret), nprocs=world, join=True)
    f = oracle.gat_fwd(p["indptr"], p["indices"], p["feat"], p["el"], p["er"], 0.2)
    b = oracle.gat_bwd(p["indptr"], p["indices"], p["feat"], p["el"], p["er"], f.alpha, p["gout"], 0.2)
    cat = lambda i: np.concatenate([ret[r][i] for r in range(world)])
    assert np.allclose(cat(0), f.out, rtol=1e-10, atol=1e-12)
    assert np.array_equal(cat(1), f.m)
    assert np.allclose(cat(2), f.d, rtol=1e-10)
    assert np.allclose(cat(3), b.dfeat, rtol=1e-9, atol=1e-11)
    assert np.allclose(cat(4), b.del_, rtol=1e-9, atol=1e-11)
    assert np.allclose(cat(5), b.der, rtol=1e-9, atol=1e-11)

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


def test_a_worker_never_holds_more_than_two_remote_partitions():
    """The point of the sequential schedule (Sec. 3.1): besides its own rows a worker holds the partition it is
    working on and the one being prefetched - however many workers there are - and in the backward pass at
    most one more buffer of returned errors.  Emulated workers as threads; receive buffers are counted from
    the moment they are posted until the last reference to what arrived is dropped."""
    import gc
    import threading
    import weakref
    from paper_2111_06483_b200.sharded import ShardedGatLayer
    from sharded_helpers import ThreadComm

    world = 6
    p = small_problem(120, 1500, 2, 4, 29, self_loops=True)
    bounds = [int(b) for b in oracle.partition_bounds(120, world)]
    mail = ThreadComm.mailboxes(world)
    peaks, errors = {}, []

    class CountingComm(ThreadComm):
        def __init__(self, *a):
            super().__init__(*a)
            self.live, self.peak, self.lock = 0, 0, threading.Lock()

        def _add(self, k):
            with self.lock:
                self.live += k
                self.peak = max(self.peak, self.live)

        def start(self, send_to, tensors, recv_from, like):
            inner = super().start(send_to, tensors, recv_from, like)
            self._add(1)  # a receive buffer is posted
            comm = self

            class _H:
                def wait(self_inner):
                    got = inner.wait()
                    weakref.finalize(got[0], comm._add, -1)  # released when the features / errors are dropped
                    return got
            return _H()

    class Collecting(TorchRefBackend):  # drop garbage promptly so that the count follows the references
        def fwd_step(self, *a):
            gc.collect()
            return super().fwd_step(*a)

        def bwd_step(self, *a):
            gc.collect()
            return super().bwd_step(*a)

    def run(rank):
        try:
            lo, hi = bounds[rank], bounds[rank + 1]
            comm = CountingComm(rank, world, mail)
            be = Collecting(rank_edges(bounds, rank, p["src"], p["dst"]), hi - lo, p["H"], p["F"], 0.2)
            layer = ShardedGatLayer(comm, bounds, be)
            t = lambda k: torch.from_numpy(p[k][lo:hi]).double()
            layer.forward(t("feat"), t("el"), t("er"))
            fwd_peak = comm.peak
            layer.backward(t("gout"))
            peaks[rank] = (fwd_peak, comm.peak)
        except Exception as exc:  # surfaced below
            errors.append(exc)

    threads = [threading.Thread(target=run, args=(r,)) for r in range(world)]
    for th in threads:
        th.start()
    for th in threads:
        th.join(timeout=300)
    assert not errors, errors
    assert len(peaks) == world
    for rank, (fwd_peak, all_peak) in peaks.items():
        assert fwd_peak <= 2, (rank, fwd_peak)   # current + prefetched
        assert all_peak <= 3, (rank, all_peak)   # + the errors coming back for its own rows

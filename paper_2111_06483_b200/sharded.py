"""Sequential aggregation over several workers (Algorithm 1 and Algorithm 2): each worker owns a contiguous
range of nodes - their output rows and their input features - and visits the source partitions one after
the other, fetching partition q's features from its owner just before it needs them and keeping only the
running softmax state in between.  In the backward pass the features are fetched again (the attention is
rebuilt, Sec. 3.3) and every partition's error is returned to its owner, who adds the contributions up.

This module is plumbing: the schedule, the point-to-point exchanges and their double buffering.  Every
arithmetic step is a call of the C-ABI library (`CudaGatBackend`); the communication goes through
torch.distributed (`TorchDistComm`: NCCL between GPUs, gloo on CPU for the tests of the schedule).
Worker p visits the partitions in the order p, p+1, ... (mod K), so that at every step each worker serves
exactly one other worker and is served by exactly one: no collective, K-1 exchanges per pass.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import api
from . import binding as B


# ----------------------------------------------------------------------------------------------
# communication
# ----------------------------------------------------------------------------------------------

class _Pending:
    def __init__(self, reqs, received, sent):
        self._reqs, self._received, self._sent = reqs, received, sent  # `sent` stays alive until the wait

    def wait(self):
        for r in self._reqs:
            r.wait()
        return self._received


class TorchDistComm:
    """Point-to-point exchanges over a torch.distributed process group."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self._dist, self._group = dist, group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)

    def start(self, send_to: int, tensors: Sequence[torch.Tensor], recv_from: int, like: Sequence[torch.Tensor]):
        """Posts the sends of `tensors` to `send_to` and the receives (shaped like `like`) from `recv_from`;
        returns a handle whose wait() gives the received tensors."""
        dist = self._dist
        received = [torch.empty_like(t) for t in like]
        peer = (lambda r: dist.get_global_rank(self._group, r)) if self._group is not None else (lambda r: r)
        sent = [t.contiguous() for t in tensors]
        ops = [dist.P2POp(dist.isend, t, peer(send_to), self._group) for t in sent]
        ops += [dist.P2POp(dist.irecv, t, peer(recv_from), self._group) for t in received]
        return _Pending(dist.batch_isend_irecv(ops) if ops else [], received, sent)


# ----------------------------------------------------------------------------------------------
# the arithmetic: calls of the library on this worker's sub-graphs G_{p,q}
# ----------------------------------------------------------------------------------------------

def build_rank_parts(n: int, bounds: Sequence[int], p: int, src: torch.Tensor, dst: torch.Tensor,
                     threshold: int = api.DEFAULT_THRESHOLD) -> List[B.Part]:
    """The K sub-graphs of worker p: edges whose destination lies in [bounds[p], bounds[p+1]), destinations
    renumbered from 0, cut by source partition with local source ids.  src, dst: global int32 ids (CUDA)."""
    lo, hi = int(bounds[p]), int(bounds[p + 1])
    keep = (dst >= lo) & (dst < hi)
    s, d = src[keep].contiguous(), (dst[keep] - lo).to(torch.int32).contiguous()
    rows, nnz, dev = hi - lo, int(s.numel()), src.device
    ws = api._workspace(B.sar_graph_workspace_bytes(nnz, max(rows, n)), dev)
    indptr = torch.empty(rows + 1, dtype=torch.int64, device=dev)
    indices = torch.empty(nnz, dtype=torch.int32, device=dev)
    B.sar_csr_from_coo(rows, n, d, s, indptr, indices, ws)
    t_indptr = torch.empty(n + 1, dtype=torch.int64, device=dev)
    t_indices = torch.empty(nnz, dtype=torch.int32, device=dev)
    B.sar_csr_from_coo(n, rows, s, d, t_indptr, t_indices, ws)
    whole = B.Part(rows, n, indptr, indices, t_indptr, t_indices)
    return api.split_parts(whole, [int(b) for b in bounds], threshold, ws)


class CudaGatBackend:
    """The steps of Algorithms 1 and 2 for one worker, on its GPU, through the C-ABI."""

    def __init__(self, parts: List[B.Part], H: int, F: int, slope: float, dtype: torch.dtype):
        self.parts, self.H, self.F, self.slope, self.dtype = parts, H, F, slope, dtype
        self.rows = parts[0].n_dst
        self.k = len(parts)
        code = B.SAR_BF16 if dtype == torch.bfloat16 else B.SAR_F32
        dev = parts[0].indptr.device
        self.ws = api._workspace(max(B.sar_gat_workspace_bytes(pt, H, F, code) for pt in parts), dev)
        self.dev = dev

    def fwd_begin(self, el: torch.Tensor):
        r, H, F = self.rows, self.H, self.F
        self.el = el
        self.m = torch.empty((r, H), dtype=torch.float32, device=self.dev)
        self.d = torch.empty((r, H), dtype=torch.float32, device=self.dev)
        self.acc = torch.empty((r, H, F), dtype=torch.float32, device=self.dev) if self.k > 1 else None
        self.out = torch.empty((r, H, F), dtype=self.dtype, device=self.dev)

    def fwd_step(self, q: int, feat_q: torch.Tensor, er_q: torch.Tensor, first: bool, last: bool):
        flags = (B.SAR_FIRST if first else 0) | (B.SAR_LAST if last else 0)
        if last and self.k > 1:   # the complete float32 numerator stays in acc: the row dot of the backward pass
            flags |= B.SAR_KEEP_NUMERATOR   # is formed from it, not from the rounded out
        B.sar_gat_fwd(self.parts[q], feat_q, self.el, er_q, self.H, self.F, self.slope, flags, self.acc, self.m, self.d,
                      self.out, self.ws)

    def fwd_end(self):
        return self.out

    def bwd_begin(self, gout: torch.Tensor):
        self.gout = gout
        self.del_ = torch.empty((self.rows, self.H), dtype=torch.float32, device=self.dev)
        if self.k > 1:  # the row dot D = <gout, numerator> / d every partition's step needs
            B.sar_gat_bwd_prepare(self.rows, self.H, self.F, self.acc, True, gout, self.el, self.m, self.d, None, self.ws)

    def bwd_step(self, q: int, feat_q: torch.Tensor, er_q: torch.Tensor, first: bool, last: bool):
        flags = (B.SAR_FIRST if first else 0) | (B.SAR_LAST if last else 0)
        dfeat_q = torch.empty_like(feat_q)
        der_q = torch.empty_like(er_q)
        B.sar_gat_bwd(self.parts[q], feat_q, self.el, er_q, self.m, self.d, self.gout, self.H, self.F, self.slope, flags,
                      dfeat_q, self.del_, der_q, self.ws)
        return dfeat_q, der_q

    def bwd_end(self):
        return self.del_

    # the sums of the error contributions other workers return (Algorithm 2), formed in float32
    def sum_begin(self, x: torch.Tensor) -> torch.Tensor:
        acc = torch.empty(x.shape, dtype=torch.float32, device=x.device)
        B.sar_accumulate(x, acc, first=True)
        return acc

    def sum_add(self, acc: torch.Tensor, x: torch.Tensor) -> None:
        B.sar_accumulate(x, acc)

    def sum_end(self, acc: torch.Tensor, like: torch.Tensor) -> torch.Tensor:
        if like.dtype == torch.float32:
            return acc
        y = torch.empty(acc.shape, dtype=like.dtype, device=acc.device)
        B.sar_round_to(acc, y)
        return y


# ----------------------------------------------------------------------------------------------
# the schedule
# ----------------------------------------------------------------------------------------------

class ShardedGatLayer:
    """One attention aggregation layer over the workers of `comm`.  `bounds` (K+1 entries) are the node ranges,
    worker p owning [bounds[p], bounds[p+1]).  `backend` does the arithmetic (CudaGatBackend on a GPU)."""

    def __init__(self, comm, bounds: Sequence[int], backend):
        self.comm, self.bounds, self.be = comm, [int(b) for b in bounds], backend
        self.p, self.K = comm.rank, comm.world
        assert len(self.bounds) == self.K + 1

    def _like(self, q: int, feat: torch.Tensor, er: torch.Tensor):
        nq = self.bounds[q + 1] - self.bounds[q]
        return [feat.new_empty((nq,) + tuple(feat.shape[1:])), er.new_empty((nq,) + tuple(er.shape[1:]))]

    def _fetch(self, s: int, feat: torch.Tensor, er: torch.Tensor):
        """Step s: this worker needs partition (p+s) mod K from its owner, and worker (p-s) mod K needs ours."""
        q, r = (self.p + s) % self.K, (self.p - s) % self.K
        return self.comm.start(r, [feat, er], q, self._like(q, feat, er))

    def forward(self, feat: torch.Tensor, el: torch.Tensor, er: torch.Tensor) -> torch.Tensor:
        """feat [n_p,H,F], el, er [n_p,H]: this worker's rows.  Returns out [n_p,H,F] (Algorithm 1)."""
        K, p, be = self.K, self.p, self.be
        self._saved = (feat, er)
        be.fwd_begin(el)
        pending = self._fetch(1, feat, er) if K > 1 else None
        cur = (feat, er)
        for s in range(K):
            be.fwd_step((p + s) % K, cur[0], cur[1], s == 0, s == K - 1)  # asynchronous on the GPU
            if s + 1 < K:
                cur = pending.wait()                                            # partition of step s+1 has arrived
                pending = self._fetch(s + 2, feat, er) if s + 2 < K else None   # the one after travels meanwhile
        return be.fwd_end()

    def backward(self, gout: torch.Tensor):
        """gout [n_p,H,F].  Returns (dfeat [n_p,H,F], del [n_p,H], der [n_p,H]) of this worker's rows
        (Algorithm 2): the features are fetched again, every partition's error goes back to its owner."""
        K, p, be = self.K, self.p, self.be
        feat, er = self._saved
        be.bwd_begin(gout)
        pending = self._fetch(1, feat, er) if K > 1 else None
        cur = (feat, er)
        dfeat_acc = der_acc = None  # sums of K terms, kept by the backend in a wide type
        returning = None
        for s in range(K):
            q = (p + s) % K
            dfeat_q, der_q = be.bwd_step(q, cur[0], cur[1], s == 0, s == K - 1)
            if returning is not None:  # the error exchanged during the previous step, added in step order
                got = returning.wait()
                be.sum_add(dfeat_acc, got[0])
                be.sum_add(der_acc, got[1])
                returning = got = None  # the receive buffer is released before the next one is posted
            if s == 0:
                dfeat_acc, der_acc = be.sum_begin(dfeat_q), be.sum_begin(der_q)
            else:
                # our error for partition q goes to its owner; worker (p-s) mod K holds the error for our sources
                returning = self.comm.start(q, [dfeat_q, der_q], (p - s) % K, [feat, er])
            if s + 1 < K:
                cur = pending.wait()
                pending = self._fetch(s + 2, feat, er) if s + 2 < K else None
        if returning is not None:
            got = returning.wait()
            be.sum_add(dfeat_acc, got[0])
            be.sum_add(der_acc, got[1])
        return be.sum_end(dfeat_acc, feat), be.bwd_end(), be.sum_end(der_acc, er)

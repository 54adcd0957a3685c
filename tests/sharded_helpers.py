"""Test-only pieces for the sharded driver: a reference backend in plain torch float64 (the arithmetic of
one worker's steps written from Algorithm 1 / Algorithm 2, on edge lists) and an in-process communicator
that lets several emulated workers run as threads."""
import queue

import numpy as np
import torch


def leaky(s, slope):
    return torch.where(s > 0, s, slope * s)


class TorchRefBackend:
    """edges[q] = (src_local, dst_local) int64 tensors of G_{p,q}."""

    def __init__(self, edges, rows, H, F, slope):
        self.edges, self.rows, self.H, self.F, self.slope = edges, rows, H, F, slope

    def fwd_begin(self, el):
        self.el = el.double()
        self.m = torch.full((self.rows, self.H), -np.inf, dtype=torch.float64)
        self.d = torch.zeros((self.rows, self.H), dtype=torch.float64)
        self.acc = torch.zeros((self.rows, self.H, self.F), dtype=torch.float64)

    def fwd_step(self, q, feat_q, er_q, first, last):
        src, dst = self.edges[q]
        if src.numel() == 0:
            return
        e = leaky(self.el[dst] + er_q.double()[src], self.slope)
        mq = torch.full_like(self.m, -np.inf).scatter_reduce(0, dst[:, None].expand(-1, self.H), e, "amax", include_self=True)
        mn = torch.maximum(self.m, mq)
        safe = torch.where(torch.isinf(mn), torch.zeros_like(mn), mn)
        c_old = torch.where(torch.isinf(self.m), torch.zeros_like(mn), torch.exp(self.m - safe))
        w = torch.exp(e - safe[dst])
        self.acc = self.acc * c_old[:, :, None]
        self.acc.index_add_(0, dst, w[:, :, None] * feat_q.double()[src])
        self.d = self.d * c_old
        self.d.index_add_(0, dst, w)
        self.m = mn

    def fwd_end(self):
        self.out = torch.where(self.d[:, :, None] > 0, self.acc / torch.where(self.d > 0, self.d, torch.ones_like(self.d))[:, :, None],
                               torch.zeros_like(self.acc))
        return self.out

    def bwd_begin(self, gout):
        self.gout = gout.double()
        self.D = (self.gout * self.out).sum(-1)
        self.del_ = torch.zeros((self.rows, self.H), dtype=torch.float64)

    def bwd_step(self, q, feat_q, er_q, first, last):
        src, dst = self.edges[q]
        f, er = feat_q.double(), er_q.double()
        dfeat = torch.zeros_like(f)
        der = torch.zeros_like(er)
        if src.numel():
            s = self.el[dst] + er[src]
            alpha = torch.exp(leaky(s, self.slope) - self.m[dst]) / self.d[dst]
            dalpha = (self.gout[dst] * f[src]).sum(-1)
            ds = alpha * (dalpha - self.D[dst]) * torch.where(s > 0, torch.ones_like(s), torch.full_like(s, self.slope))
            dfeat.index_add_(0, src, alpha[:, :, None] * self.gout[dst])
            der.index_add_(0, src, ds)
            self.del_.index_add_(0, dst, ds)
        return dfeat, der

    def bwd_end(self):
        return self.del_

    def sum_begin(self, x):
        return x.double().clone()

    def sum_add(self, acc, x):
        acc += x.double()

    def sum_end(self, acc, like):
        return acc.to(like.dtype)


class ThreadComm:
    """Emulated workers as threads of one process: mail[(a, b)] carries the messages from a to b in order."""

    def __init__(self, rank, world, mail):
        self.rank, self.world, self.mail = rank, world, mail

    @staticmethod
    def mailboxes(world):
        return {(a, b): queue.Queue() for a in range(world) for b in range(world)}

    def start(self, send_to, tensors, recv_from, like):
        self.mail[(self.rank, send_to)].put([t.clone() for t in tensors])
        mail, me = self.mail, self.rank

        class _H:
            def wait(self_inner):
                return mail[(recv_from, me)].get(timeout=120)
        return _H()


def rank_edges(bounds, p, src, dst):
    """(src_local, dst_local) per source partition q for worker p, from global numpy edge arrays."""
    lo, hi = bounds[p], bounds[p + 1]
    out = []
    for q in range(len(bounds) - 1):
        k = (dst >= lo) & (dst < hi) & (src >= bounds[q]) & (src < bounds[q + 1])
        out.append((torch.from_numpy(src[k] - bounds[q]).long(), torch.from_numpy(dst[k] - lo).long()))
    return out

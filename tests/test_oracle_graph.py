"""Pins for the oracle's integer side (CSR build, transpose, partition split) and for the
seeded generators (CPU only)."""
import numpy as np
import pytest
import torch

import oracle
import workloads


def _edges(n, e, seed):
    s, d = workloads.uniform_edges(n, e, seed, self_loops=True)
    return s.numpy(), d.numpy()


def test_csr_from_coo_matches_lexsort_and_keeps_duplicates():
    n = 300
    src, dst = _edges(n, 5000, 31)
    src = np.concatenate([src, src[:200]])           # force duplicates
    dst = np.concatenate([dst, dst[:200]])
    indptr, indices = oracle.csr_from_coo(n, n, src, dst)
    order = np.lexsort((src, dst))
    assert np.array_equal(indices, src[order])
    assert np.array_equal(indptr, np.concatenate([[0], np.cumsum(np.bincount(dst, minlength=n))]))
    # round trip: the CSR holds exactly the input multiset of edges
    back_dst = np.repeat(np.arange(n), np.diff(indptr))
    a = np.sort(back_dst.astype(np.int64) * n + indices)
    b = np.sort(dst.astype(np.int64) * n + src)
    assert np.array_equal(a, b)


def test_transpose_is_an_involution_and_matches_lexsort():
    n = 257
    src, dst = _edges(n, 4000, 32)
    indptr, indices = oracle.csr_from_coo(n, n, src, dst)
    t_indptr, t_indices = oracle.csr_transpose(n, n, indptr, indices)
    order = np.lexsort((dst, src))
    assert np.array_equal(t_indices, dst[order])
    assert np.array_equal(t_indptr, np.concatenate([[0], np.cumsum(np.bincount(src, minlength=n))]))
    tt_indptr, tt_indices = oracle.csr_transpose(n, n, t_indptr, t_indices)
    assert np.array_equal(tt_indptr, indptr) and np.array_equal(tt_indices, indices)


@pytest.mark.parametrize("n,k", [(10, 3), (257, 8), (100, 100), (5, 1), (1000, 16)])
def test_partition_bounds_and_split(n, k):
    bounds = oracle.partition_bounds(n, k)
    assert bounds[0] == 0 and bounds[-1] == n and np.all(np.diff(bounds) >= 0)
    assert np.array_equal(bounds, [q * n // k for q in range(k + 1)])
    src, dst = _edges(n, 20 * n, 33)
    indptr, indices = oracle.csr_from_coo(n, n, src, dst)
    sp = oracle.csr_split(n, indptr, indices, bounds)
    assert sp.nnz_off[-1] == len(indices)
    # concatenating the K sub-rows (global ids) re-creates each row
    for i in range(0, n, max(1, n // 50)):
        row = []
        for q in range(k):
            ip, idx = sp.part(q)
            loc = idx[ip[i]:ip[i + 1]]
            assert np.all((loc >= 0) & (loc < bounds[q + 1] - bounds[q]))
            row.append(loc.astype(np.int64) + bounds[q])
        assert np.array_equal(np.concatenate(row), indices[indptr[i]:indptr[i + 1]])
    for q in range(k):
        ip, idx = sp.part(q)
        assert ip[0] == 0 and ip[-1] == len(idx)


def test_generators_are_deterministic_and_shaped():
    cfg = workloads.CONFIGS["seqpart"].scaled(0.05)
    s1, d1 = workloads.make_graph(cfg)
    s2, d2 = workloads.make_graph(cfg)
    assert torch.equal(s1, s2) and torch.equal(d1, d2)
    assert s1.dtype == torch.int32 and s1.shape == (cfg.e,)
    assert int(s1.min()) >= 0 and int(s1.max()) < cfg.n
    deg = torch.bincount(d1.long(), minlength=cfg.n)
    assert abs(float(deg.float().mean()) - cfg.e / cfg.n) < 1e-6
    # heavy tail: the top destination is near d_max, the median is far below the mean
    assert 0.6 * cfg.d_max < int(deg.max()) < 1.5 * cfg.d_max
    assert int(deg.median()) < cfg.e / cfg.n
    t = workloads.make_node_inputs(1000, 4, 16, seed=0)
    assert abs(float(t["feat"].mean())) < 0.02 and abs(float(t["feat"].std()) - 1) < 0.02
    tb = workloads.make_node_inputs(1000, 4, 16, seed=0, dtype="bf16")
    assert tb["feat"].dtype == torch.bfloat16 and tb["el"].dtype == torch.float32
    assert torch.equal(tb["feat"], t["feat"].to(torch.bfloat16))


def test_tiny_config_edge_count():
    cfg = workloads.CONFIGS["tiny"]
    s, d = workloads.make_graph(cfg)
    assert s.shape[0] == cfg.e + cfg.n                      # 20,000 random edges + one self-loop per node
    assert int((s[: cfg.e] == d[: cfg.e]).sum()) == 0
    assert torch.equal(s[cfg.e:], d[cfg.e:])

"""Pins for the oracle's batch normalisation (Sec. 3.4) and for the host logic that combines the workers'
statistics, CPU only: torch's batch_norm (forward and autograd backward) in float64, and a two-rank gloo
run whose combined statistics must equal those of the concatenated rows."""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp

import oracle


def test_forward_and_backward_match_torch_batch_norm():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((300, 7)) * 3.0 + 5.0
    gamma, beta = rng.standard_normal(7), rng.standard_normal(7)
    gy = rng.standard_normal((300, 7))
    xt = torch.tensor(x, requires_grad=True)
    gt, bt = torch.tensor(gamma, requires_grad=True), torch.tensor(beta, requires_grad=True)
    yt = torch.nn.functional.batch_norm(xt, None, None, gt, bt, training=True, eps=1e-5)
    (yt * torch.tensor(gy)).sum().backward()
    y, mean, rstd = oracle.bn_forward(x, 1e-5, gamma, beta)
    assert np.allclose(y, yt.detach().numpy(), rtol=1e-12, atol=1e-12)
    gx, dgamma, dbeta = oracle.bn_backward(x, gy, 1e-5, gamma)
    assert np.allclose(gx, xt.grad.numpy(), rtol=1e-10, atol=1e-12)
    assert np.allclose(dgamma, gt.grad.numpy(), rtol=1e-10, atol=1e-12)
    assert np.allclose(dbeta, bt.grad.numpy(), rtol=1e-10, atol=1e-12)
    # normalised columns: mean 0, variance 1 - eps * rstd^2
    yh, _, _ = oracle.bn_forward(x, 1e-5)
    assert np.allclose(yh.mean(axis=0), 0, atol=1e-12) and np.allclose(yh.var(axis=0), 1 - 1e-5 * rstd ** 2, rtol=1e-10)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, x_parts, gy_parts, ret):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2111_06483_b200 import api
    x, gy = x_parts[rank], gy_parts[rank]
    mean_l, m2_l = oracle.bn_moments(x.numpy())
    n_all, mean, m2 = api.combine_moments(x.shape[0], torch.tensor(mean_l, dtype=torch.float32),
                                          torch.tensor(m2_l, dtype=torch.float32), group=dist.group.WORLD)
    rstd = torch.rsqrt(m2 / n_all + 1e-5)
    xhat = (x - mean) * rstd
    s0, s1 = api.combine_sums([gy.sum(0), (gy * xhat).sum(0)], group=dist.group.WORLD)
    gx = rstd * (gy - s0 / n_all - xhat * s1 / n_all)
    ret[rank] = (n_all, mean, m2, gx)
    dist.destroy_process_group()


def test_two_workers_combine_to_the_statistics_of_all_rows():
    rng = np.random.default_rng(1)
    xa = torch.tensor(rng.standard_normal((130, 5)) + 2.0, dtype=torch.float32)
    xb = torch.tensor(rng.standard_normal((70, 5)) * 2.0 - 1.0, dtype=torch.float32)  # different size, different moments
    ga = torch.tensor(rng.standard_normal((130, 5)), dtype=torch.float32)
    gb = torch.tensor(rng.standard_normal((70, 5)), dtype=torch.float32)
    ret = mp.Manager().dict()
    mp.spawn(_worker, args=(2, _free_port(), [xa, xb], [ga, gb], ret), nprocs=2, join=True)
    x_all, g_all = torch.cat([xa, xb]).numpy(), torch.cat([ga, gb]).numpy()
    mean, m2 = oracle.bn_moments(x_all)
    gx_all, _, _ = oracle.bn_backward(x_all, g_all, 1e-5)
    for rank, rows in ((0, slice(0, 130)), (1, slice(130, 200))):
        n_all, mean_r, m2_r, gx = ret[rank]
        assert n_all == 200
        assert np.allclose(mean_r.numpy(), mean, rtol=1e-6, atol=1e-6)
        assert np.allclose(m2_r.numpy(), m2, rtol=1e-5)
        # each worker's gradient rows are the rows of the gradient computed over all rows at once
        assert np.allclose(gx.numpy(), gx_all[rows], rtol=1e-4, atol=1e-5)


def test_splitmix64_known_answers_and_dropout_statistics():
    # the generator's published first outputs for seed 0
    assert [hex(int(v)) for v in oracle.splitmix64(0, 4)] == ["0xe220a8397b1dcdaf", "0x6e789e6aa1b965f4",
                                                              "0x6c45d188009454f", "0xf88bb8a8724c81ec"]
    x = np.ones((1000, 200))
    for p in (0.0, 0.1, 0.5, 0.9):
        y, keep = oracle.dropout(x, p, 12345)
        n = x.size
        assert abs(keep.mean() - (1 - p)) <= 4 * np.sqrt(p * (1 - p) / n) + 1e-7   # binomial, 4 sigma
        assert np.allclose(y[keep], 1 / (1 - p), rtol=1e-6) and np.all(y[~keep] == 0)
        assert abs(y.mean() - 1.0) <= 4 * np.sqrt(p / (1 - p) / n) + 1e-6            # expectation preserved
    a, _ = oracle.dropout(x, 0.5, 1)
    b, _ = oracle.dropout(x, 0.5, 2)
    c, _ = oracle.dropout(x, 0.5, 1)
    assert np.array_equal(a, c) and not np.array_equal(a, b)
    # neighbouring elements are not correlated: the lag-1 agreement rate of the mask is 1/2 at p = 1/2
    k = oracle.dropout(np.ones(200000), 0.5, 7)[1]
    assert abs((k[1:] == k[:-1]).mean() - 0.5) < 0.01

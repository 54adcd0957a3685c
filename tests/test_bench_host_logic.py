"""CPU tests of bench.py's host logic: byte model, pass grouping, clock parsing, and the max-over-ranks
reduction of the replicas-only multi-GPU mode (two gloo ranks on CPU)."""
import os
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_compulsory_byte_model_matches_the_scope_table():
    # 'large': N = 20 M, E = 300 M, H*F = 128, bf16 -> forward 12.88 GB; 'medium' float32 forward 5.44 GB
    assert abs(bench.bytes_fwd(20_000_000, 300_000_000, 4, 32, 2) / 1e9 - 12.88) < 0.01
    assert abs(bench.bytes_fwd(2_450_000, 62_000_000, 4, 64, 4) / 1e9 - 5.44) < 0.01
    # every array once per layer: 3 x index + 4 feature-sized arrays + the [N,H] vectors
    n, e, H, F, b = 1000, 5000, 4, 16, 2
    idx = 8 * (n + 1) + 4 * e
    assert bench.bytes_layer_fwd_bwd(n, e, H, F, b) == 3 * idx + 4 * n * H * F * b + 10 * n * H * 4
    assert bench.bytes_bwd_dst(n, e, H, F, b) + bench.bytes_bwd_src(n, e, H, F, b) > bench.bytes_fwd(n, e, H, F, b)


def test_pass_grouping_and_clock_parsing():
    k = {"gat_fwd": {"avg_ms": 2.0}, "gat_fwd_seg": {"avg_ms": 1.0}, "gat_fwd_merge": {"avg_ms": 0.5},
         "gat_bwd_src": {"avg_ms": 3.0}}
    p = bench.group_passes(k)
    assert p["gat_fwd"]["ms"] == 3.5 and sorted(p["gat_fwd"]["launches"]) == ["gat_fwd", "gat_fwd_merge", "gat_fwd_seg"]
    assert p["gat_bwd_src"]["ms"] == 3.0
    lines = ["1965, 1965, 410.2, Not Active, Not Active, Not Active, Not Active",
             "1500, 1965, 990.0, Not Active, Not Active, Not Active, Active",
             "1800, 1965, 700.0, Not Active, Not Active, Not Active, Not Active", "garbage"]
    c = bench.ClockSampler.parse(lines)
    assert c["sm_mhz"] == 1800.0 and c["sm_max_mhz"] == 1965.0 and c["reasons"] == ["sw_power_cap"] and c["samples"] == 3


def _rank(rank, world, port, out):
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    got = bench.max_over_ranks(10.0 + 5.0 * rank, dist)     # rank 1 is the slow replica
    out.put((rank, got))
    dist.destroy_process_group()


def test_max_over_ranks_with_two_gloo_ranks():
    assert bench.max_over_ranks(3.5) == 3.5
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == {0: 15.0, 1: 15.0}                        # every rank reports the slowest replica's time

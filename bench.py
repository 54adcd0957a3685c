#!/usr/bin/env python
"""Benchmark of the fused GAT aggregation (forward + backward with attention rematerialisation).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One STEP is one pass of the whole hot path over one batch of synthetic node tensors: for each of
the workload's layers the forward over the K source partitions, then for each layer the
rematerialising backward (destination-major and source-major passes).  Two SCHEDULES of the K
partitions are timed on the same inputs:

  fused       one row-stationary walk per pass over the un-split graph: sources ascend within a row, so
              a row meets the partitions in order and the running state never leaves the registers.  The
              kernels see ONE partition (the K bounds only describe where the partitions lie);
  sequential  Algorithm 1 / Algorithm 2 call by call: K calls of sar_gat_fwd with the running numerator,
              max and normaliser in device memory, then sar_gat_bwd_prepare and K calls of sar_gat_bwd.

`value` comes from the schedule named in `config.schedule` (--schedule, default fused); both are
reported under `schedules`.  The graph (CSR, CSC, per-partition sub-graphs, long-row plans) is
prepared once by the library before the timed region and its time is reported as `prep_ms`; a graph
is fixed across the training steps the paper times (its partitioning is an offline step).

The default run (workload large, one GPU) also times, briefly, the other named workloads
(`workloads`), the sum aggregation on the headline graph with the same row width as a measured
ceiling for any gather kernel on this input (`gather_ceiling`), a deliberately plain variant that
stores the attention coefficients (`storing_baseline`), the end-to-end path through host buffers
(`e2e`) and the CPU oracle (`cpu_baseline`).

Prints ONE JSON line (rank 0).  `value` = edges x layers processed per second by all ranks (each
rank runs an independent replica: the path does not shard, so scaling is "weak" with no
collective on the data path).
"""
from __future__ import annotations

import argparse
import gc
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "gat_fwd_bwd_edges_per_sec"
UNIT = "edges/s"
TARGET_FRAC = 0.60  # of the HBM roofline, on the largest single-GPU graph


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large", help="tiny | seqpart | medium | dense | large")
    ap.add_argument("--dtype", default=None, help="f32 | bf16 (default: the workload's last listed dtype)")
    ap.add_argument("--scale", type=float, default=1.0, help="shrink the workload (debugging and profiling)")
    ap.add_argument("--threshold", type=int, default=None, help="long-row split threshold")
    ap.add_argument("--t-threshold", type=int, default=None, help="long-row split threshold of the CSC (default: the same)")
    ap.add_argument("--schedule", default="fused", choices=["fused", "sequential"],
                    help="which schedule of the K partitions `value` is taken from (both are timed)")
    ap.add_argument("--only-schedule", action="store_true", help="time only the schedule named by --schedule")
    ap.add_argument("--glue", action="store_true",
                    help="also run the rest of the layer each step: dense projection z = h W (bf16 workloads), score "
                         "projections, ReLU, and their backward passes (default: aggregation kernels only)")
    ap.add_argument("--ids", default="permuted", choices=["permuted", "degree_sorted"],
                    help="node numbering of the power-law graph: seeded random permutation (the workload) or "
                         "degree rank = id (locality ablation)")
    ap.add_argument("--bn-dropout", action="store_true",
                    help="with --glue on a bf16 workload: batch normalisation over the nodes and dropout (p = 0.5) "
                         "between the layers, as in the paper's networks (Sec. 4.2), forward and backward")
    ap.add_argument("--spmm", action="store_true",
                    help="time the sum aggregation (sar_spmm_agg forward + its backward on the transposed graph) "
                         "on the workload's graph instead of the attention stack; its own metric, not the headline")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the other workloads, the gather ceiling and the storing baseline")
    ap.add_argument("--cpu-sample", type=float, default=0.05, help="fraction of the workload the oracle is timed on")
    return ap.parse_args()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# --------------------------------------------------------------------------------------------------
# algorithmic (compulsory) bytes: every distinct input byte read once, every output byte written once
# --------------------------------------------------------------------------------------------------

def idx_bytes(n, e):
    return 8 * (n + 1) + 4 * e


def bytes_fwd(n, e, H, F, b):
    return idx_bytes(n, e) + 2 * n * H * F * b + 4 * n * H * 4          # feat, out; el, er, m, d


def bytes_bwd_dst(n, e, H, F, b):
    # CSR, gathered feat, gout row; el, er, m, d read; del and the 16-byte record written
    return idx_bytes(n, e) + 2 * n * H * F * b + 4 * n * H * 4 + n * H * 4 + n * H * 16


def bytes_bwd_src(n, e, H, F, b):
    # CSC, gathered gout, feat row, dfeat written; er and the record read; der written
    return idx_bytes(n, e) + 3 * n * H * F * b + n * H * 4 + n * H * 16 + n * H * 4


def bytes_layer_fwd_bwd(n, e, H, F, b):
    # the whole layer, each array once: 3x index (CSR fwd, CSR + CSC bwd), feat, out, gout, dfeat,
    # el, er, m, d (written then read), del, der
    return 3 * idx_bytes(n, e) + 4 * n * H * F * b + 10 * n * H * 4


def bytes_spmm(n, e, F, b):
    # one direction of the sum aggregation: indices, every input row once, every output row once
    return idx_bytes(n, e) + 2 * n * F * b


def state_bytes_sequential(n, H, F, K, L):
    """Bytes of running state (float32 numerator, max, normaliser) the call-by-call forward writes and
    reads back between partitions, per step: every partition but the last writes it, every one but the
    first reads it (Algorithm 1 keeps it in the worker's memory)."""
    per = n * H * F * 4 + 2 * n * H * 4
    return L * 2 * max(K - 1, 0) * per


KERNEL_BYTES = {"gat_fwd": bytes_fwd, "gat_bwd_dst": bytes_bwd_dst, "gat_bwd_src": bytes_bwd_src}

# DRAM traffic of one pass (rows + segments + merge launches), dram__bytes_read.sum + dram__bytes_write.sum from one-pass
# ncu captures of the kernels of this tree at full size, nine forward and six backward launches at a time (commands and
# per-launch figures: profiles/gat_kernels_large_launch_list_and_dram.md).  A constant of that capture, not of this run.
# `traffic_rate_frac` = that traffic / the pass's measured time / the peak: how close the pass runs to the copy
# bandwidth for the bytes it really moves (the compulsory-byte fraction `frac` counts every row once).
NCU_TRAFFIC_SOURCE = ("ncu one-pass capture of these kernels at full size (profiles/gat_kernels_large_launch_list_and_dram.md), "
                      "not measured in this run")
NCU_TRAFFIC = {
    # (workload, storage dtype, pass): bytes per full-size pass
    ("large", "bf16", "gat_fwd"): 82.36e9,
    ("large", "bf16", "gat_bwd_dst"): 84.37e9,
    ("large", "bf16", "gat_bwd_src"): 89.50e9,
}


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """Largest `value` over all ranks (the job is as slow as its slowest replica); identity without dist."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def group_passes(kernels: dict) -> dict:
    """Launch names -> passes: 'gat_fwd', 'gat_fwd_seg', 'gat_fwd_merge' (and, call by call, the 'gat_fwd_finalize' that
    divides after the last partition) together are one pass over the edges.
    `ms` adds the launches' average durations (one launch of each per pass: the fused schedule); `total_ms`
    adds everything the pass's launches took inside the timed region (any schedule)."""
    passes = {}
    for name, v in kernels.items():
        base = name
        for suffix in ("_seg", "_merge", "_finalize"):
            if name.endswith(suffix):
                base = name[:-len(suffix)]
        p_ = passes.setdefault(base, {"ms": 0.0, "total_ms": 0.0, "launches": []})
        p_["ms"] += v["avg_ms"]
        p_["total_ms"] += v.get("total_ms", v["avg_ms"] * v.get("launches", 1))
        p_["launches"].append(name)
    return passes


def pass_table(kernels, passes_per_run, n, e, H, F, b, peak):
    """Per pass over the E edges: milliseconds (all its launches, averaged over the passes of the timed
    region), edges/s and the fraction of the compulsory-byte roofline."""
    out = {}
    for name, p_ in group_passes(kernels).items():
        if name not in KERNEL_BYTES or passes_per_run <= 0:
            continue
        ms = p_["total_ms"] / passes_per_run
        alg = KERNEL_BYTES[name](n, e, H, F, b)
        out[name] = {"ms": ms, "edges_per_sec": e / (ms * 1e-3), "algorithmic_bytes": alg,
                     "frac_of_roofline": alg / (ms * 1e-3) / 1e9 / peak, "launches": sorted(p_["launches"])}
    return out


# --------------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.path = tempfile.mktemp(prefix="clocks_", suffix=".csv")
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(gpu_index)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()       # the exact child started above
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        try:
            out = self.parse(open(self.path).read().splitlines())
            os.unlink(self.path)
        except OSError:
            pass
        return out

    @staticmethod
    def parse(lines):
        """nvidia-smi CSV lines -> median SM clock under load, max clock, throttle reasons seen Active."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for nme, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nme)
        if sm:
            sm.sort()
            out.update(sm_mhz=sm[len(sm) // 2], sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def gpu_index_of(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
    if vis.replace(",", "").isdigit():
        return int(vis.split(",")[local_rank])
    return local_rank


# --------------------------------------------------------------------------------------------------
# the CPU oracle as a timed baseline (reference arm and cpu_baseline leg)
# --------------------------------------------------------------------------------------------------

def oracle_sample(cfg, dtype, fraction):
    """Inputs of a bounded sample of the workload for the oracle: the same recipe with node and edge
    counts multiplied by `fraction`, one layer."""
    import workloads
    small = cfg.scaled(fraction) if fraction < 1.0 else cfg
    src, dst = workloads.make_graph(small)
    t = workloads.make_node_inputs(small.n, small.heads, small.feat, small.seed, dtype=dtype)
    return small, src.numpy(), dst.numpy(), {k: v.float().numpy() for k, v in t.items()}


def oracle_step(small, src, dst, h, slope):
    """One layer forward + backward of the oracle as it stands (CSR given); returns seconds."""
    import oracle
    indptr, indices = oracle.csr_from_coo(small.n, small.n, src, dst)
    t0 = time.perf_counter()
    f = oracle.gat_fwd(indptr, indices, h["feat"], h["el"], h["er"], slope)
    oracle.gat_bwd(indptr, indices, h["feat"], h["el"], h["er"], f.alpha, h["gout"], slope)
    return time.perf_counter() - t0


def run_reference(args, rank):
    """--impl reference: the oracle, as it stands, on the host cores, on a bounded sample."""
    if rank != 0:
        return
    import oracle
    import workloads
    cfg = workloads.CONFIGS[args.workload]
    dtype = args.dtype or cfg.dtypes[-1]
    # a smaller sample than the cpu_baseline leg: warmup + steps passes must end within minutes
    small, src, dst, h = oracle_sample(cfg, dtype, min(1.0, 0.4 * args.cpu_sample * args.scale))
    for _ in range(args.warmup):
        oracle_step(small, src, dst, h, cfg.slope)
    secs = [oracle_step(small, src, dst, h, cfg.slope) for _ in range(args.steps)]
    total = sum(secs)
    value = small.e * args.steps / total
    sample = f"{small.name}: n={small.n} e={small.e} H={small.heads} F={small.feat}, one layer fwd+bwd per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "sample": sample, "storage_dtype": dtype},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def cpu_baseline_leg(cfg_name, dtype, fraction, slope):
    """The oracle as it stands on the host cores: all cores on a `fraction` sample of the workload, and
    one thread on a sample an eighth of that (so that both end within seconds)."""
    import oracle
    import workloads
    cfg = workloads.CONFIGS[cfg_name]
    small, s_src, s_dst, h = oracle_sample(cfg, dtype, min(1.0, fraction))
    cores = oracle.num_threads()
    secs = oracle_step(small, s_src, s_dst, h, slope)
    out = {"value": small.e / secs, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": f"{small.name}: n={small.n} e={small.e} H={small.heads} F={small.feat}, one layer fwd+bwd, "
                     f"{secs:.1f} s"}
    tiny, t_src, t_dst, th = oracle_sample(cfg, dtype, min(1.0, fraction / 8))
    oracle.set_num_threads(1)
    try:
        secs1 = oracle_step(tiny, t_src, t_dst, th, slope)
    finally:
        oracle.set_num_threads(cores)
    out["single_thread"] = {"value": tiny.e / secs1, "unit": UNIT, "cores": 1,
                            "sample": f"{tiny.name}: n={tiny.n} e={tiny.e}, one layer fwd+bwd, {secs1:.1f} s"}
    return out


# --------------------------------------------------------------------------------------------------
# the aggregation stack on the device
# --------------------------------------------------------------------------------------------------

class AggStack:
    """L chained aggregation layers of one workload: the graph and every node tensor on the device.

    feat^{l+1} = out^l with seeded el^l, er^l; the backward pass feeds dfeat^{l+1} as gout of layer l."""

    def __init__(self, cfg, dtype, dev, ids="permuted", threshold=None, parts=True, t_threshold=None, reorder=None):
        import torch
        import workloads
        from paper_2111_06483_b200 import api, binding as B
        self.B, self.api, self.torch = B, api, torch
        self.cfg, self.dtype, self.dev = cfg, dtype, dev
        self.tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
        self.b = 2 if dtype == "bf16" else 4
        n, H, F, L, K = cfg.n, cfg.heads, cfg.feat, cfg.layers, cfg.k
        self.n, self.H, self.F, self.L, self.K = n, H, F, L, K
        self.threshold = threshold if threshold is not None else api.DEFAULT_THRESHOLD
        src, dst = workloads.make_graph(cfg, device=dev, permute=ids == "permuted")
        self.e = src.numel()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        self.g = api.Graph.from_coo(n, src, dst, k=K, threshold=self.threshold, build_parts=parts and K > 1,
                                    t_threshold=t_threshold, reorder=reorder)
        torch.cuda.synchronize()
        self.prep_ms = 1e3 * (time.perf_counter() - t0)
        del src, dst
        tdt = self.tdt
        self.feats = [workloads.normal_tensor((n, H, F), cfg.seed, 10, device=dev, dtype=tdt)]
        self.feats += [torch.empty((n, H, F), dtype=tdt, device=dev) for _ in range(L)]
        self.els = [workloads.normal_tensor((n, H), cfg.seed, 16 * l + 12, device=dev) for l in range(L)]
        self.ers = [workloads.normal_tensor((n, H), cfg.seed, 16 * l + 13, device=dev) for l in range(L)]
        self.gout = workloads.normal_tensor((n, H, F), cfg.seed, 11, device=dev, dtype=tdt)
        if reorder:   # the node arrays enter the graph's numbering once, before the timed region
            self.feats[0] = self.g.to_internal(self.feats[0])
            self.els = [self.g.to_internal(x) for x in self.els]
            self.ers = [self.g.to_internal(x) for x in self.ers]
            self.gout = self.g.to_internal(self.gout)
        self.gbuf = [torch.empty((n, H, F), dtype=tdt, device=dev) for _ in range(2)]
        f32 = lambda: torch.empty((n, H), dtype=torch.float32, device=dev)
        self.ms, self.ds = [f32() for _ in range(L)], [f32() for _ in range(L)]
        self.dels, self.ders = [f32() for _ in range(L)], [f32() for _ in range(L)]
        g = self.g
        nbytes = B.sar_gat_workspace_bytes(g.whole, H, F, B._dtype(self.feats[0]))
        for p in g.parts:
            nbytes = max(nbytes, B.sar_gat_workspace_bytes(p, H, F, B._dtype(self.feats[0])))
        self.ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=dev)
        self.acc = None

    def can_run_sequential(self):
        return self.K == 1 or bool(self.g.parts)

    def step_fused(self):
        B, g, c = self.B, self.g, self.cfg
        H, F, L = self.H, self.F, self.L
        for l in range(L):
            B.sar_gat_fwd_fused(g.whole, g.bounds, self.feats[l], self.els[l], self.ers[l], H, F, c.slope, self.ms[l],
                                self.ds[l], self.feats[l + 1], self.ws)
        gin = self.gout
        for i, l in enumerate(reversed(range(L))):
            B.sar_gat_bwd_fused(g.whole, g.bounds, self.feats[l], self.els[l], self.ers[l], self.ms[l], self.ds[l], gin,
                                H, F, c.slope, self.gbuf[i % 2], self.dels[l], self.ders[l], self.ws)
            gin = self.gbuf[i % 2]

    def step_sequential(self):
        """Algorithm 1 and Algorithm 2 call by call: the running state (numerator, max, normaliser) lives in
        device memory between the K forward calls; the backward pass rebuilds each partition's attention."""
        B, g, c, torch = self.B, self.g, self.cfg, self.torch
        H, F, L, K, n = self.H, self.F, self.L, self.K, self.n
        parts = g.parts if K > 1 else [g.whole]
        if K > 1 and self.acc is None:
            self.acc = torch.empty((n, H, F), dtype=torch.float32, device=self.dev)
        for l in range(L):
            for q, part in enumerate(parts):
                flags = (B.SAR_FIRST if q == 0 else 0) | (B.SAR_LAST if q == K - 1 else 0)
                s0, s1 = g.bounds[q], g.bounds[q + 1]
                B.sar_gat_fwd(part, self.feats[l][s0:s1], self.els[l], self.ers[l][s0:s1], H, F, c.slope, flags, self.acc,
                              self.ms[l], self.ds[l], self.feats[l + 1], self.ws)
        gin = self.gout
        for i, l in enumerate(reversed(range(L))):
            if K > 1:
                B.sar_gat_bwd_prepare(n, H, F, self.feats[l + 1], False, gin, self.els[l], self.ms[l], self.ds[l], None,
                                      self.ws)
            for q, part in enumerate(parts):
                flags = (B.SAR_FIRST if q == 0 else 0) | (B.SAR_LAST if q == K - 1 else 0)
                s0, s1 = g.bounds[q], g.bounds[q + 1]
                B.sar_gat_bwd(part, self.feats[l][s0:s1], self.els[l], self.ers[l][s0:s1], self.ms[l], self.ds[l], gin, H,
                              F, c.slope, flags, self.gbuf[i % 2][s0:s1], self.dels[l], self.ders[l][s0:s1], self.ws)
            gin = self.gbuf[i % 2]

    def step(self, schedule):
        return self.step_fused if schedule == "fused" else self.step_sequential


def measure(step, steps, warmup, dist=None, dev=None, clocks_gpu=None):
    """`warmup` untimed steps, then exactly `steps` steps between a barrier + synchronize on both sides,
    timed with CUDA events on the launching stream; per-kernel times from the library's launch observer."""
    import torch
    from paper_2111_06483_b200 import binding as B
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(clocks_gpu) if clocks_gpu is not None else None
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with B.LaunchTimer() as lt:
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    elapsed_ms = max_over_ranks(e0.elapsed_time(e1), dist, dev)
    clocks = sampler.stop() if sampler else None
    kernels = lt.summary()
    return {"ms_per_step": elapsed_ms / steps, "kernels": kernels, "clocks": clocks,
            "launches": sum(v["launches"] for v in kernels.values())}


def schedule_entry(st: AggStack, schedule, r, steps, peak):
    n, e, H, F, b, L, K = st.n, st.e, st.H, st.F, st.b, st.L, st.K
    entry = {
        "ms_per_step": r["ms_per_step"], "steps": steps, "edges_per_sec": L * e / (r["ms_per_step"] * 1e-3),
        "partitions_seen_by_the_kernels": 1 if schedule == "fused" else K,
        "launches_per_step": r["launches"] // max(steps, 1),
        "passes": pass_table(r["kernels"], steps * L, n, e, H, F, b, peak),
        "step_frac_of_roofline": L * bytes_layer_fwd_bwd(n, e, H, F, b) / (r["ms_per_step"] * 1e-3) / 1e9 / peak,
    }
    if schedule == "sequential":
        # what the forward calls really move: the first call writes every row's state, a middle call reads and writes
        # the rows that have edges in its partition (the kernel skips the others), the last call reads every row's
        entry["state_bytes_upper_bound"] = state_bytes_sequential(n, H, F, K, L)
        if st.g.parts and K > 1:
            touched = [int(((p_.indptr[1:] - p_.indptr[:-1]) > 0).sum().item()) for p_ in st.g.parts[1:-1]]
            per = H * F * 4 + 2 * H * 4
            entry["state_bytes_per_step"] = L * per * (2 * n + 2 * sum(touched))
            entry["rows_with_edges_per_middle_partition"] = sum(touched) / max(len(touched), 1) / n
        else:
            entry["state_bytes_per_step"] = entry["state_bytes_upper_bound"]
        entry["calls"] = f"{K} x sar_gat_fwd, sar_gat_bwd_prepare + {K} x sar_gat_bwd per layer"
    else:
        entry["calls"] = "sar_gat_fwd_fused, sar_gat_bwd_fused per layer (one walk over the un-split graph)"
    if r.get("clocks"):
        entry["clocks"] = r["clocks"]
    return entry


# --------------------------------------------------------------------------------------------------
# legs of the default run
# --------------------------------------------------------------------------------------------------

def time_spmm(g, x, gout, steps, warmup, peak, n, e, b):
    """Sum aggregation forward (CSR) + its backward (the same call on the transposed graph)."""
    import torch
    from paper_2111_06483_b200 import binding as B
    F = x.shape[1]
    out, dx = torch.empty_like(x), torch.empty_like(x)
    fwd, bwd = g.whole, g.whole.transposed()
    ws = torch.empty(max(B.sar_spmm_workspace_bytes(fwd, F, B._dtype(x)), B.sar_spmm_workspace_bytes(bwd, F, B._dtype(x)), 256),
                     dtype=torch.uint8, device=x.device)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    f_ms = b_ms = 0.0
    for it in range(warmup + steps):
        ev[0].record()
        B.sar_spmm_agg(fwd, x, F, B.SAR_FIRST | B.SAR_LAST, None, out, ws)
        ev[1].record()
        B.sar_spmm_agg(bwd, gout, F, B.SAR_FIRST | B.SAR_LAST, None, dx, ws)
        ev[2].record()
        torch.cuda.synchronize()
        if it >= warmup:
            f_ms += ev[0].elapsed_time(ev[1]) / steps
            b_ms += ev[1].elapsed_time(ev[2]) / steps
    alg = bytes_spmm(n, e, F, b)
    return {"columns": F, "csr_ms": f_ms, "csc_ms": b_ms, "ms_per_step": f_ms + b_ms,
            "edges_per_sec": e / ((f_ms + b_ms) * 1e-3), "algorithmic_bytes_per_direction": alg,
            "frac_of_roofline": 2 * alg / ((f_ms + b_ms) * 1e-3) / 1e9 / peak,
            "gathered_bytes_per_direction": e * F * b}


def storing_leg(st: AggStack, steps=2, warmup=1):
    """The non-rematerialising baseline on the same stack: every layer's forward pass writes its attention
    coefficients alpha[E,H] (kept until that layer's backward pass reads them).  Reports its step time and the
    device memory both variants hold at their peak, measured by the allocator during one step each."""
    import torch
    B, g, cfg = st.B, st.g, st.cfg
    n, H, F, L, e = st.n, st.H, st.F, st.L, st.e
    torch.cuda.synchronize()
    torch.cuda.reset_peak_memory_stats()
    st.step_fused()
    torch.cuda.synchronize()
    remat_peak = torch.cuda.max_memory_allocated()
    held = torch.cuda.memory_allocated()
    need = L * e * H * 4 + B.sar_gat_storing_workspace_bytes(g.whole, H)
    free = torch.cuda.mem_get_info()[0]
    if need > 0.9 * free:
        return {"skipped": f"needs {need} more bytes, {free} free", "remat_peak_mem_bytes": remat_peak}
    torch.cuda.reset_peak_memory_stats()
    alphas = [torch.empty((e, H), dtype=torch.float32, device=st.dev) for _ in range(L)]
    ws = torch.empty(B.sar_gat_storing_workspace_bytes(g.whole, H), dtype=torch.uint8, device=st.dev)

    def step():
        for l in range(L):
            B.sar_gat_fwd_storing(g.whole, st.feats[l], st.els[l], st.ers[l], H, F, cfg.slope, alphas[l], st.feats[l + 1])
        gin = st.gout
        for i, l in enumerate(reversed(range(L))):
            B.sar_gat_bwd_storing(g.whole, st.feats[l], st.els[l], st.ers[l], alphas[l], gin, H, F, cfg.slope,
                                  st.gbuf[i % 2], st.dels[l], st.ders[l], ws)
            gin = st.gbuf[i % 2]

    r = measure(step, steps, warmup)
    storing_peak = torch.cuda.max_memory_allocated()
    del alphas, ws
    return {"ms_per_step": r["ms_per_step"], "steps": steps, "warmup": warmup,
            "kernels": {k: v["avg_ms"] for k, v in r["kernels"].items()},
            "peak_mem_bytes": storing_peak, "remat_peak_mem_bytes": remat_peak,
            "extra_bytes_over_remat": storing_peak - remat_peak,
            "attention_bytes_kept": L * e * H * 4, "stats_bytes_kept_by_remat": L * 2 * n * H * 4,
            "held_before_bytes": held,
            "kind": "plain two-step kernels, one warp per row, not tuned (sar_gat_fwd_storing / sar_gat_bwd_storing)"}


def extra_workloads(dev, peak, args):
    """The other named workloads, a few steps each (configs 2-4 and the sum aggregation of config 3)."""
    import torch
    import workloads
    from paper_2111_06483_b200 import api
    out = {}
    plan = [("seqpart", "f32", ("fused", "sequential")), ("medium", "f32", ("fused",)),
            ("medium", "bf16", ("fused", "sequential")), ("dense", "bf16", ("fused", "sequential"))]
    steps, warmup = 5, 3
    for name, dtype, schedules in plan:
        cfg = workloads.CONFIGS[name]
        need = (6 * cfg.n * cfg.heads * cfg.feat * (2 if dtype == "bf16" else 4) + 4 * cfg.n * cfg.heads * cfg.feat
                + 40 * cfg.e) * 1.3
        if torch.cuda.get_device_properties(dev).total_memory < need:
            out[f"{name}_{dtype}"] = {"skipped": "not enough device memory"}
            continue
        st = AggStack(cfg, dtype, dev, ids=args.ids, parts="sequential" in schedules)
        entry = {"n": st.n, "e": st.e, "heads": st.H, "feat_per_head": st.F, "layers": st.L, "partitions": st.K,
                 "storage_dtype": dtype, "prep_ms": st.prep_ms, "schedules": {}}
        for sch in schedules:
            r = measure(st.step(sch), steps, warmup, clocks_gpu=None)
            entry["schedules"][sch] = schedule_entry(st, sch, r, steps, peak)
        if name == "dense":
            entry["storing_baseline"] = storing_leg(st)
            entry["storing_baseline"]["remat_ms_per_step"] = entry["schedules"]["fused"]["ms_per_step"]
        out[f"{name}_{dtype}"] = entry
        if name == "medium" and cfg.spmm_feat:
            x = workloads.normal_tensor((st.n, cfg.spmm_feat), cfg.seed, 20, device=dev, dtype=st.tdt)
            go = workloads.normal_tensor((st.n, cfg.spmm_feat), cfg.seed, 21, device=dev, dtype=st.tdt)
            out[f"spmm_{name}_{dtype}"] = time_spmm(st.g, x, go, steps, warmup, peak, st.n, st.e, st.b)
            del x, go
        del st
        gc.collect()
        torch.cuda.empty_cache()
    return out


def make_glue_step(args, st: AggStack):
    """--glue: the rest of the layer around the aggregation (fused schedule only)."""
    import torch
    import workloads
    B, g, cfg, dev = st.B, st.g, st.cfg, st.dev
    n, H, F, L, tdt = st.n, st.H, st.F, st.L, st.tdt
    feats, els, ers, ms, ds, dels, ders = st.feats, st.els, st.ers, st.ms, st.ds, st.dels, st.ders
    gout, gbuf, ws = st.gout, st.gbuf, st.ws
    a_ls = [workloads.normal_tensor((H, F), cfg.seed, 16 * l + 14, device=dev) / F ** 0.5 for l in range(L)]
    a_rs = [workloads.normal_tensor((H, F), cfg.seed, 16 * l + 15, device=dev) / F ** 0.5 for l in range(L)]
    da_l, da_r = torch.empty((H, F), device=dev), torch.empty((H, F), device=dev)
    pws = torch.empty(B.sar_gat_project_workspace_bytes(H, F), dtype=torch.uint8, device=dev)

    if tdt == torch.bfloat16 and (H * F) % 8 == 0:
        # the whole layer: dense projection z = h W on the tensor cores, scores, aggregation, ReLU
        D = H * F
        Ws = [(workloads.normal_tensor((D, D), cfg.seed, 16 * l + 9, device=dev) / D ** 0.5).to(tdt) for l in range(L)]
        zs = [torch.empty((n, H, F), dtype=tdt, device=dev) for _ in range(L)]
        dW = torch.empty((D, D), dtype=torch.float32, device=dev)
        lws = torch.empty(B.sar_linear_workspace_bytes(n, D, D), dtype=torch.uint8, device=dev)
        flat = lambda x: x.view(n, D)

        if args.bn_dropout:
            # layer l's aggregation output stays in feats[l+1] (batch normalisation needs it again in the backward
            # pass); hs[l+1] = dropout(ReLU(BN(feats[l+1]))) is the next layer's input
            hs = [feats[0]] + [torch.empty((n, H, F), dtype=tdt, device=dev) for _ in range(L - 1)]
            bn_mean = [torch.empty(D, dtype=torch.float32, device=dev) for _ in range(L)]
            bn_m2 = [torch.empty(D, dtype=torch.float32, device=dev) for _ in range(L)]
            bn_rstd = [torch.empty(D, dtype=torch.float32, device=dev) for _ in range(L)]
            bn_s0, bn_s1 = torch.empty(D, dtype=torch.float32, device=dev), torch.empty(D, dtype=torch.float32, device=dev)
            bws = torch.empty(B.sar_bn_workspace_bytes(D), dtype=torch.uint8, device=dev)
            p_drop, seeds = 0.5, [1000 + l for l in range(L)]
            act = B.SAR_GLUE_RELU | B.SAR_GLUE_DROPOUT  # y = dropout(relu(bn(x))) in one pass over the node array
            gx_bn = torch.empty((n, H, F), dtype=tdt, device=dev)  # gradient w.r.t. a layer's aggregation output

            def step():
                for l in range(L):
                    B.sar_linear_project(flat(hs[l]), Ws[l], a_ls[l], a_rs[l], flat(zs[l]), els[l], ers[l], lws)
                    B.sar_gat_fwd_fused(g.whole, g.bounds, zs[l], els[l], ers[l], H, F, cfg.slope, ms[l], ds[l],
                                        feats[l + 1], ws)
                    if l + 1 < L:
                        x = flat(feats[l + 1])
                        B.sar_bn_stats(x, bn_mean[l], bn_m2[l], bws)
                        B.sar_bn_rstd(bn_m2[l], n, 1e-5, bn_rstd[l])
                        B.sar_bn_apply_act(x, bn_mean[l], bn_rstd[l], None, None, act, p_drop, seeds[l], flat(hs[l + 1]))
                gin = gout
                for l in reversed(range(L)):
                    B.sar_gat_bwd_fused(g.whole, g.bounds, zs[l], els[l], ers[l], ms[l], ds[l], gin, H, F, cfg.slope,
                                        gbuf[0], dels[l], ders[l], ws)
                    B.sar_gat_project_bwd(zs[l], a_ls[l], a_rs[l], dels[l], ders[l], gbuf[0], da_l, da_r, pws, 0)
                    B.sar_linear_bwd_weight(flat(hs[l]), flat(gbuf[0]), dW, lws)
                    B.sar_linear_bwd_input(flat(gbuf[0]), Ws[l], flat(gbuf[1]), lws)
                    if l > 0:
                        gh = flat(gbuf[1])      # gradient w.r.t. hs[l]; the two calls take it back through the dropout
                        x = flat(feats[l])      # and the ReLU (hs[l] > 0 where both let it pass) on the fly
                        B.sar_bn_bwd_stats_act(x, bn_mean[l - 1], bn_rstd[l - 1], gh, flat(hs[l]), act, p_drop, seeds[l - 1],
                                               bn_s0, bn_s1, bws)
                        B.sar_bn_bwd_apply_act(x, bn_mean[l - 1], bn_rstd[l - 1], None, gh, flat(hs[l]), act, p_drop,
                                               seeds[l - 1], bn_s0, bn_s1, 1.0 / n, flat(gx_bn))
                        gin = gx_bn
            return step

        def step_plain():
            relu_flags = B.SAR_FIRST | B.SAR_LAST | B.SAR_RELU_OUT
            for l in range(L):   # the ReLU that closes a layer is applied where its aggregate is finalised
                B.sar_linear_project(flat(feats[l]), Ws[l], a_ls[l], a_rs[l], flat(zs[l]), els[l], ers[l], lws)
                B.sar_gat_fwd(g.whole, zs[l], els[l], ers[l], H, F, cfg.slope, relu_flags, None, ms[l], ds[l],
                              feats[l + 1], ws)
            gin = gout
            B.sar_relu_bwd(feats[L], gin)  # masks gout in place on the first pass; the same mask every step
            for l in reversed(range(L)):
                # gbuf[0]: gradient w.r.t. z of this layer, gbuf[1]: w.r.t. the layer's input
                B.sar_gat_bwd_fused(g.whole, g.bounds, zs[l], els[l], ers[l], ms[l], ds[l], gin, H, F, cfg.slope,
                                        gbuf[0], dels[l], ders[l], ws)
                B.sar_gat_project_bwd(zs[l], a_ls[l], a_rs[l], dels[l], ders[l], gbuf[0], da_l, da_r, pws, 0)
                B.sar_linear_bwd_weight(flat(feats[l]), flat(gbuf[0]), dW, lws)
                if l > 0:   # the backward of the ReLU that produced this layer's input, in the GEMM's epilogue
                    B.sar_linear_bwd_input_relu(flat(gbuf[0]), Ws[l], flat(feats[l]), flat(gbuf[1]), lws)
                else:
                    B.sar_linear_bwd_input(flat(gbuf[0]), Ws[l], flat(gbuf[1]), lws)
                gin = gbuf[1]
        return step_plain

    def step():
        for l in range(L):  # the ReLU closing layer l-1 runs inside layer l's projection
            B.sar_gat_project(feats[l], a_ls[l], a_rs[l], els[l], ers[l], B.SAR_GLUE_RELU if l > 0 else 0)
            B.sar_gat_fwd_fused(g.whole, g.bounds, feats[l], els[l], ers[l], H, F, cfg.slope, ms[l], ds[l],
                                feats[l + 1], ws)
        B.sar_relu(feats[L])
        gin = gout
        B.sar_relu_bwd(feats[L], gin)  # masks gout in place on the first pass; the same mask every step
        for i, l in enumerate(reversed(range(L))):
            B.sar_gat_bwd_fused(g.whole, g.bounds, feats[l], els[l], ers[l], ms[l], ds[l], gin, H, F, cfg.slope,
                                gbuf[i % 2], dels[l], ders[l], ws)
            gin = gbuf[i % 2]
            B.sar_gat_project_bwd(feats[l], a_ls[l], a_rs[l], dels[l], ders[l], gin, da_l, da_r, pws,
                                  B.SAR_GLUE_RELU if l > 0 else 0)
    return step


def time_e2e(st: AggStack, args, dist, world):
    """The same metric through sar_gat_stack_host with pinned HOST buffers: every step copies all its inputs in
    and all its results out inside the timed region."""
    import torch
    import workloads
    B, g, cfg, dev = st.B, st.g, st.cfg, st.dev
    n, H, F, L, tdt, b = st.n, st.H, st.F, st.L, st.tdt, st.b
    pin = lambda shape, dt: torch.empty(shape, dtype=dt).pin_memory()
    h_feat0 = pin((n, H, F), tdt)
    h_gout = pin((n, H, F), tdt)
    h_out, h_dfeat = pin((n, H, F), tdt), pin((n, H, F), tdt)
    h_el = [pin((n, H), torch.float32) for _ in range(L)]
    h_er = [pin((n, H), torch.float32) for _ in range(L)]
    h_del = [pin((n, H), torch.float32) for _ in range(L)]
    h_der = [pin((n, H), torch.float32) for _ in range(L)]
    h_feat0.copy_(workloads.normal_tensor((n, H, F), cfg.seed, 10, device=dev, dtype=tdt))
    h_gout.copy_(workloads.normal_tensor((n, H, F), cfg.seed, 11, device=dev, dtype=tdt))
    for l in range(L):
        h_el[l].copy_(st.els[l])
        h_er[l].copy_(st.ers[l])
    # two working sets: the pipelined mode overlaps the copies of step t+1 with the kernels of step t
    one = (B.sar_gat_stack_arena_bytes(g.whole, L, H, F, B._dtype(h_feat0)) + 255) // 256 * 256
    arena = torch.empty(2 * one, dtype=torch.uint8, device=dev)

    def host_step():
        B.sar_gat_stack_host(g.whole, g.bounds, H, F, cfg.slope, h_feat0, h_el, h_er, h_gout, h_out, h_dfeat,
                             h_del, h_der, arena, pipelined=True)

    for _ in range(3):
        host_step()
    B.sar_gat_stack_host_wait()
    torch.cuda.synchronize()
    n_e2e = max(1, min(args.steps, 10))
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(n_e2e):
        host_step()
    B.sar_gat_stack_host_wait()
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    dt = max_over_ranks(dt, dist, dev)
    h2d = 2 * n * H * F * b + 2 * L * n * H * 4
    d2h = 2 * n * H * F * b + 2 * L * n * H * 4
    return {"value": world * L * st.e * n_e2e / dt, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "ms_per_step": 1e3 * dt / n_e2e, "steps": n_e2e, "warmup": 3,
            "entry_point": "sar_gat_stack_host, pipelined (every step copies all its inputs in and all its results out)"}


# --------------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------------

def run_ours(args, rank, world, local_rank):
    import torch
    import workloads

    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    dev = torch.device(f"cuda:{local_rank}")
    torch.cuda.set_device(dev)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    cfg = workloads.CONFIGS[args.workload]
    if args.scale != 1.0:
        cfg = cfg.scaled(args.scale)
    dtype = args.dtype or cfg.dtypes[-1]
    peak, peak_src = load_peaks()
    glue = args.glue
    schedules = [args.schedule] if (args.only_schedule or glue) else ["fused", "sequential"]
    if glue:
        schedules = ["fused"]
    st = AggStack(cfg, dtype, dev, ids=args.ids, threshold=args.threshold, parts="sequential" in schedules,
                  t_threshold=args.t_threshold)
    n, e, H, F, b, L, K = st.n, st.e, st.H, st.F, st.b, st.L, st.K
    main_sched = "fused" if glue else args.schedule
    gpu_index = gpu_index_of(local_rank)
    prep_ms, threshold = st.prep_ms, st.threshold

    torch.cuda.reset_peak_memory_stats()
    results = {}
    for sch in schedules:
        step = make_glue_step(args, st) if glue else st.step(sch)
        is_main = sch == main_sched
        steps = args.steps if is_main else max(1, min(args.steps, 3))
        results[sch] = measure(step, steps, args.warmup, dist, dev, clocks_gpu=gpu_index if (is_main and rank == 0) else None)
        results[sch]["steps"] = steps
    peak_mem = torch.cuda.max_memory_allocated()
    main = results[main_sched]
    ms_per_step = main["ms_per_step"]
    value = world * L * e / (ms_per_step * 1e-3)
    kernels = main["kernels"]
    sched_out = {sch: schedule_entry(st, sch, r, r["steps"], peak) for sch, r in results.items()}

    # ---- roofline of the dominant pass ---------------------------------------------------------------
    # A pass over the E edges is the launches of the library that together visit every edge once (rows,
    # long-row segments, merge; K times as many in the sequential schedule); its algorithmic bytes are
    # divided by the CUDA-event time those launches took per pass.
    passes = sched_out[main_sched]["passes"]
    roofline = None
    if passes:
        dom = max(passes, key=lambda k_: passes[k_]["ms"])
        alg = passes[dom]["algorithmic_bytes"]
        achieved = alg / (passes[dom]["ms"] * 1e-3) / 1e9
        default_plan = args.threshold is None and args.t_threshold is None and args.ids == "permuted"
        traffic = (NCU_TRAFFIC.get((args.workload, dtype, dom))
                   if (args.scale == 1.0 and main_sched == "fused" and default_plan) else None)
        roofline = {"bound": "hbm", "kernel": dom, "launches": passes[dom]["launches"], "achieved": achieved,
                    "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src,
                    "traffic": traffic, "traffic_source": NCU_TRAFFIC_SOURCE if traffic else None,
                    "traffic_rate_frac": (traffic / (passes[dom]["ms"] * 1e-3) / 1e9 / peak) if traffic else None,
                    "algorithmic_bytes_per_launch": alg, "avg_launch_ms": passes[dom]["ms"],
                    "target_frac": TARGET_FRAC, "target_met": bool(achieved / peak >= TARGET_FRAC)}
    step_bytes = L * bytes_layer_fwd_bwd(n, e, H, F, b)
    step_frac = step_bytes / (ms_per_step * 1e-3) / 1e9 / peak

    extras = (not args.no_extras) and world == 1 and not glue and args.scale == 1.0 and args.workload == "large"
    ceiling = None
    if extras:
        # what ANY gather kernel can reach on this graph with this row width: the sum aggregation (no scores, no
        # softmax, one accumulator), CSR and CSC direction
        x = st.feats[0].view(n, H * F)
        ceiling = time_spmm(st.g, x, st.gout.view(n, H * F), 5, 3, peak, n, e, b)
        for name, p_ in passes.items():
            ref = ceiling["csc_ms"] if name == "gat_bwd_src" else ceiling["csr_ms"]
            p_["frac_of_gather_ceiling"] = ref / p_["ms"]

    storing = None
    if extras:
        storing = storing_leg(st)
        storing["remat_ms_per_step"] = sched_out["fused"]["ms_per_step"] if "fused" in sched_out else None

    e2e = None
    if not args.no_e2e and not glue:
        st.feats, st.gbuf, st.gout, st.acc = None, None, None, None
        gc.collect()
        torch.cuda.empty_cache()
        e2e = time_e2e(st, args, dist, world)

    others = None
    if extras:
        step = None   # the bound method keeps the stack alive
        del st
        gc.collect()
        torch.cuda.empty_cache()
        others = extra_workloads(dev, peak, args)
        if args.ids == "permuted":
            # the same workload (ids a seeded permutation) with the library's renumbering by degree in graph preparation
            # (sar_degree_order: hubs next to each other, rows of similar length in a span); the node arrays are
            # carried into the new numbering once, outside the timed region; fused schedule, five steps
            st2 = AggStack(cfg, dtype, dev, ids="permuted", parts=False, reorder="degree")
            r2 = measure(st2.step("fused"), 5, 3, clocks_gpu=None)
            others["large_renumbered_by_degree"] = {"ms_per_step": r2["ms_per_step"], "steps": 5, "prep_ms": st2.prep_ms,
                                                   "edges_per_sec": L * e / (r2["ms_per_step"] * 1e-3),
                                                   "passes_ms": {k: v["ms"] for k, v in pass_table(r2["kernels"], 5 * L, n, e, H, F, b, peak).items()},
                                                   "note": "graph preparation with reorder='degree' (sar_degree_order, sar_relabel, sar_permute_rows); "
                                                           "`value` above is measured without it"}
            del st2
            gc.collect()
            torch.cuda.empty_cache()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline_leg(args.workload, dtype, args.cpu_sample * args.scale, cfg.slope)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {
                "workload": cfg.name, "n": n, "e": e, "heads": H, "feat_per_head": F, "layers": L,
                "schedule": main_sched, "partitions": sched_out[main_sched]["partitions_seen_by_the_kernels"],
                "partitions_configured": K, "storage_dtype": dtype, "layer_glue": bool(glue),
                "bn_dropout": bool(glue and args.bn_dropout), "ids": args.ids,
                "l2": "inputs_exceed_l2" if n * H * F * b > 126e6 else "inputs_fit_l2",
                "long_row_threshold": threshold, "parallelism": f"replicas x{world}",
                "edges_x_heads_x_feat_per_sec": value * H * F,
            },
            "roofline": roofline,
            "step_roofline": {"compulsory_bytes_per_step": step_bytes, "frac_of_peak": step_frac, "peak": peak,
                              "peak_source": peak_src},
            "schedules": sched_out, "passes": passes, "kernels": kernels, "gpu_launches": main["launches"],
            "prep_ms": prep_ms,
            "peak_mem_bytes": peak_mem,
            "attention_bytes_if_stored": {"value": L * e * H * 4, "kind": "computed: 4 bytes x E x H x layers"},
            "stats_bytes_kept": L * 2 * n * H * 4,
            "gather_ceiling": ceiling, "storing_baseline": storing, "workloads": others,
            "clocks": main["clocks"] or {}, "e2e": e2e, "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


def run_spmm(args, local_rank):
    """--spmm: one step = out = A x (CSR) and dx = A^T gout (the same call on the transposed partition), Eq. 2's
    aggregation with F columns per node.  One GPU; prints its own JSON line (metric spmm_fwd_bwd_edges_per_sec)."""
    import torch
    import workloads
    from paper_2111_06483_b200 import api, binding as B

    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    dev = torch.device(f"cuda:{local_rank}")
    torch.cuda.set_device(dev)
    cfg = workloads.CONFIGS[args.workload]
    if args.scale != 1.0:
        cfg = cfg.scaled(args.scale)
    dtype = args.dtype or cfg.dtypes[-1]
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    b = 2 if dtype == "bf16" else 4
    n, F = cfg.n, cfg.spmm_feat or cfg.heads * cfg.feat
    threshold = args.threshold if args.threshold is not None else api.DEFAULT_THRESHOLD
    src, dst = workloads.make_graph(cfg, device=dev, permute=args.ids == "permuted")
    e = src.numel()
    g = api.Graph.from_coo(n, src, dst, k=1, threshold=threshold)
    del src, dst
    x = workloads.normal_tensor((n, F), cfg.seed, 20, device=dev, dtype=tdt)
    gout = workloads.normal_tensor((n, F), cfg.seed, 21, device=dev, dtype=tdt)
    out, dx = torch.empty_like(x), torch.empty_like(x)
    fwd, bwd = g.whole, g.whole.transposed()
    ws = torch.empty(max(B.sar_spmm_workspace_bytes(fwd, F, B._dtype(x)), B.sar_spmm_workspace_bytes(bwd, F, B._dtype(x))),
                     dtype=torch.uint8, device=dev)

    def step():
        B.sar_spmm_agg(fwd, x, F, B.SAR_FIRST | B.SAR_LAST, None, out, ws)
        B.sar_spmm_agg(bwd, gout, F, B.SAR_FIRST | B.SAR_LAST, None, dx, ws)

    r = measure(step, args.steps, args.warmup, clocks_gpu=gpu_index_of(local_rank))
    ms_per_step = r["ms_per_step"]
    peak, peak_src = load_peaks()
    alg = bytes_spmm(n, e, F, b)  # per direction
    achieved = 2 * alg / (ms_per_step * 1e-3) / 1e9
    line = {
        "metric": "spmm_fwd_bwd_edges_per_sec", "value": e / (ms_per_step * 1e-3), "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": cfg.name, "n": n, "e": e, "columns": F, "storage_dtype": dtype, "ids": args.ids,
                   "l2": "inputs_exceed_l2" if n * F * b > 126e6 else "inputs_fit_l2", "long_row_threshold": threshold},
        "roofline": {"bound": "hbm", "kernel": "spmm (forward + transposed)", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src, "traffic": None,
                     "algorithmic_bytes_per_step": 2 * alg, "gathered_bytes_per_step": 2 * e * F * b},
        "kernels": r["kernels"], "gpu_launches": r["launches"], "clocks": r["clocks"],
    }
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.spmm:
        if rank == 0:
            run_spmm(args, local_rank)
        return
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()

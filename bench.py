#!/usr/bin/env python
"""Benchmark of the fused GAT aggregation (forward + backward with attention rematerialisation).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One STEP is one pass of the whole hot path over one batch of synthetic node tensors: for each of
the workload's layers the fused forward over the K source partitions, then for each layer the
rematerialising backward (destination-major and source-major passes).  The graph (CSR, CSC,
long-row plan) is prepared once by the library before the timed region and its time is reported
as `prep_ms`; a graph is fixed across the training steps the paper times (its partitioning is an
offline step).

Prints ONE JSON line (rank 0).  `value` = edges x layers processed per second by all ranks (each
rank runs an independent replica: the path does not shard, so scaling is "weak" with no
collective on the data path).
"""
from __future__ import annotations

import argparse
import json
import math
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


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large", help="tiny | seqpart | medium | dense | large")
    ap.add_argument("--dtype", default=None, help="f32 | bf16 (default: the workload's last listed dtype)")
    ap.add_argument("--scale", type=float, default=1.0, help="shrink the workload (debugging only)")
    ap.add_argument("--threshold", type=int, default=None, help="long-row split threshold")
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


KERNEL_BYTES = {"gat_fwd": bytes_fwd, "gat_bwd_dst": bytes_bwd_dst, "gat_bwd_src": bytes_bwd_src}

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one pass (rows + segments + merge launches),
# from the one-pass ncu capture at full size whose launch list is summarised under profiles/.
NCU_TRAFFIC_BYTES = {
    ("large", "bf16", "gat_fwd"): 81.89e9,
    ("large", "bf16", "gat_bwd_dst"): 84.07e9,
    ("large", "bf16", "gat_bwd_src"): 89.08e9,
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
    """Launch names -> passes: 'gat_fwd', 'gat_fwd_seg', 'gat_fwd_merge' together are one pass over the edges."""
    passes = {}
    for name, v in kernels.items():
        base = name
        for suffix in ("_seg", "_merge"):
            if name.endswith(suffix):
                base = name[:-len(suffix)]
        p_ = passes.setdefault(base, {"ms": 0.0, "launches": []})
        p_["ms"] += v["avg_ms"]
        p_["launches"].append(name)
    return passes


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


# --------------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------------

def run_ours(args, rank, world, local_rank):
    import torch
    import workloads
    from paper_2111_06483_b200 import api, binding as B

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
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    b = 2 if dtype == "bf16" else 4
    n, H, F, L, K = cfg.n, cfg.heads, cfg.feat, cfg.layers, cfg.k
    threshold = args.threshold if args.threshold is not None else api.DEFAULT_THRESHOLD

    # ---- inputs (seeded, generated on the device; same recipe as the parity tests) --------------
    src, dst = workloads.make_graph(cfg, device=dev, permute=args.ids == "permuted")
    e = src.numel()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    g = api.Graph.from_coo(n, src, dst, k=K, threshold=threshold)
    torch.cuda.synchronize()
    prep_ms = 1e3 * (time.perf_counter() - t0)
    del src, dst
    feats = [workloads.normal_tensor((n, H, F), cfg.seed, 10, device=dev, dtype=tdt)]
    feats += [torch.empty((n, H, F), dtype=tdt, device=dev) for _ in range(L)]
    els = [workloads.normal_tensor((n, H), cfg.seed, 16 * l + 12, device=dev) for l in range(L)]
    ers = [workloads.normal_tensor((n, H), cfg.seed, 16 * l + 13, device=dev) for l in range(L)]
    gout = workloads.normal_tensor((n, H, F), cfg.seed, 11, device=dev, dtype=tdt)
    gbuf = [torch.empty((n, H, F), dtype=tdt, device=dev) for _ in range(2)]
    ms = [torch.empty((n, H), dtype=torch.float32, device=dev) for _ in range(L)]
    ds = [torch.empty((n, H), dtype=torch.float32, device=dev) for _ in range(L)]
    dels = [torch.empty((n, H), dtype=torch.float32, device=dev) for _ in range(L)]
    ders = [torch.empty((n, H), dtype=torch.float32, device=dev) for _ in range(L)]
    ws = api.gat_workspace(g.whole, H, F, tdt)
    cut = lambda t: [t[g.bounds[q]:] for q in range(K)]
    feat_q = [cut(f) for f in feats]
    er_q = [cut(x) for x in ers]
    der_q = [cut(x) for x in ders]
    gbuf_q = [cut(x) for x in gbuf]

    glue = args.glue
    if glue:
        a_ls = [workloads.normal_tensor((H, F), cfg.seed, 16 * l + 14, device=dev) / F ** 0.5 for l in range(L)]
        a_rs = [workloads.normal_tensor((H, F), cfg.seed, 16 * l + 15, device=dev) / F ** 0.5 for l in range(L)]
        da_l, da_r = torch.empty((H, F), device=dev), torch.empty((H, F), device=dev)
        pws = torch.empty(B.sar_gat_project_workspace_bytes(H, F), dtype=torch.uint8, device=dev)

    if glue and tdt == torch.bfloat16 and (H * F) % 8 == 0:
        # the whole layer: dense projection z = h W on the tensor cores, scores, aggregation, ReLU
        D = H * F
        Ws = [(workloads.normal_tensor((D, D), cfg.seed, 16 * l + 9, device=dev) / D ** 0.5).to(tdt) for l in range(L)]
        zs = [torch.empty((n, H, F), dtype=tdt, device=dev) for _ in range(L)]
        z_q = [cut(z) for z in zs]
        dW = torch.empty((D, D), dtype=torch.float32, device=dev)
        lws = torch.empty(B.sar_linear_workspace_bytes(n, D, D), dtype=torch.uint8, device=dev)
        flat = lambda x: x.view(n, D)

        bnd = args.bn_dropout
        if bnd:
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
                    B.sar_linear(flat(hs[l]), Ws[l], flat(zs[l]), lws)
                    B.sar_gat_project(zs[l], a_ls[l], a_rs[l], els[l], ers[l], 0)
                    B.sar_gat_fwd_fused(g.whole, g.bounds, z_q[l], els[l], er_q[l], H, F, cfg.slope, ms[l], ds[l],
                                        feats[l + 1], ws)
                    if l + 1 < L:
                        x = flat(feats[l + 1])
                        B.sar_bn_stats(x, bn_mean[l], bn_m2[l], bws)
                        B.sar_bn_rstd(bn_m2[l], n, 1e-5, bn_rstd[l])
                        B.sar_bn_apply_act(x, bn_mean[l], bn_rstd[l], None, None, act, p_drop, seeds[l], flat(hs[l + 1]))
                gin = gout
                for l in reversed(range(L)):
                    B.sar_gat_bwd_fused(g.whole, g.bounds, z_q[l], els[l], er_q[l], ms[l], ds[l], gin, H, F, cfg.slope,
                                        gbuf_q[0], dels[l], der_q[l], ws)
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

        def step_plain():
            for l in range(L):
                if l > 0:
                    B.sar_relu(feats[l])
                B.sar_linear(flat(feats[l]), Ws[l], flat(zs[l]), lws)
                B.sar_gat_project(zs[l], a_ls[l], a_rs[l], els[l], ers[l], 0)
                B.sar_gat_fwd_fused(g.whole, g.bounds, z_q[l], els[l], er_q[l], H, F, cfg.slope, ms[l], ds[l],
                                    feats[l + 1], ws)
            B.sar_relu(feats[L])
            gin = gout
            B.sar_relu_bwd(feats[L], gin)  # masks gout in place on the first pass; the same mask every step
            for l in reversed(range(L)):
                # gbuf[0]: gradient w.r.t. z of this layer, gbuf[1]: w.r.t. the layer's input
                B.sar_gat_bwd_fused(g.whole, g.bounds, z_q[l], els[l], er_q[l], ms[l], ds[l], gin, H, F, cfg.slope,
                                    gbuf_q[0], dels[l], der_q[l], ws)
                B.sar_gat_project_bwd(zs[l], a_ls[l], a_rs[l], dels[l], ders[l], gbuf[0], da_l, da_r, pws, 0)
                B.sar_linear_bwd_weight(flat(feats[l]), flat(gbuf[0]), dW, lws)
                B.sar_linear_bwd_input(flat(gbuf[0]), Ws[l], flat(gbuf[1]), lws)
                if l > 0:
                    B.sar_relu_bwd(feats[l], gbuf[1])
                gin = gbuf[1]

        if not bnd:
            step = step_plain
    else:
        def step():
            for l in range(L):
                if glue:  # the ReLU closing layer l-1 runs inside layer l's projection
                    B.sar_gat_project(feats[l], a_ls[l], a_rs[l], els[l], ers[l], B.SAR_GLUE_RELU if l > 0 else 0)
                B.sar_gat_fwd_fused(g.whole, g.bounds, feat_q[l], els[l], er_q[l], H, F, cfg.slope, ms[l], ds[l],
                                    feats[l + 1], ws)
            if glue:
                B.sar_relu(feats[L])
            gin = gout
            if glue:
                B.sar_relu_bwd(feats[L], gin)  # masks gout in place on the first pass; the same mask every step
            for i, l in enumerate(reversed(range(L))):
                B.sar_gat_bwd_fused(g.whole, g.bounds, feat_q[l], els[l], er_q[l], ms[l], ds[l], gin, H, F, cfg.slope,
                                    gbuf_q[i % 2], dels[l], der_q[l], ws)
                gin = gbuf[i % 2]
                if glue:
                    B.sar_gat_project_bwd(feats[l], a_ls[l], a_rs[l], dels[l], ders[l], gin, da_l, da_r, pws,
                                          B.SAR_GLUE_RELU if l > 0 else 0)

    torch.cuda.reset_peak_memory_stats()
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    peak_mem = torch.cuda.max_memory_allocated()

    # ---- timed region ----------------------------------------------------------------------------
    gpu_index = int(os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",")[local_rank]) \
        if os.environ.get("CUDA_VISIBLE_DEVICES", "").replace(",", "").isdigit() else local_rank
    sampler = ClockSampler(gpu_index) if rank == 0 else None
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with B.LaunchTimer() as lt:
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    elapsed_ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if sampler else {}
    elapsed_ms = max_over_ranks(elapsed_ms, dist, dev)
    kernels = lt.summary()
    launches = sum(v["launches"] for v in kernels.values())
    ms_per_step = elapsed_ms / args.steps
    value = world * L * e / (ms_per_step * 1e-3)

    # ---- roofline of the dominant pass ---------------------------------------------------------------
    # A pass over the E edges is up to three launches of the library (rows, long-row segments, merge);
    # its algorithmic bytes are divided by the sum of their average CUDA-event durations.
    peak, peak_src = load_peaks()
    passes = group_passes(kernels)
    dom = max(passes, key=lambda k_: passes[k_]["ms"])
    roofline = None
    if dom in KERNEL_BYTES:
        alg = KERNEL_BYTES[dom](n, e, H, F, b)
        achieved = alg / (passes[dom]["ms"] * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": dom, "launches": passes[dom]["launches"], "achieved": achieved,
                    "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src,
                    "traffic": NCU_TRAFFIC_BYTES.get((args.workload, dtype, dom)) if args.scale == 1.0 else None,
                    "algorithmic_bytes_per_launch": alg, "avg_launch_ms": passes[dom]["ms"]}
    pass_ms = {k_: v["ms"] for k_, v in passes.items() if k_ in KERNEL_BYTES}
    per_pass = {k_: {"ms": ms_, "edges_per_sec": e / (ms_ * 1e-3),
                     "frac_of_roofline": KERNEL_BYTES[k_](n, e, H, F, b) / (ms_ * 1e-3) / 1e9 / peak}
                for k_, ms_ in pass_ms.items()}
    step_bytes = L * bytes_layer_fwd_bwd(n, e, H, F, b)
    step_frac = step_bytes / (ms_per_step * 1e-3) / 1e9 / peak

    # ---- end to end through the host-buffer entry point ---------------------------------------------
    e2e = None
    if not args.no_e2e:
        del feats, gbuf, feat_q, gbuf_q, gout
        torch.cuda.empty_cache()
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
            h_el[l].copy_(els[l])
            h_er[l].copy_(ers[l])
        # two working sets: the pipelined mode overlaps the copies of step t+1 with the kernels of step t
        one = (B.sar_gat_stack_arena_bytes(g.whole, L, H, F, B._dtype(h_feat0)) + 255) // 256 * 256
        arena = torch.empty(2 * one, dtype=torch.uint8, device=dev)

        def host_step():
            B.sar_gat_stack_host(g.whole, g.bounds, H, F, cfg.slope, h_feat0, h_el, h_er, h_gout, h_out, h_dfeat,
                                 h_del, h_der, arena, pipelined=True)

        host_step()
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
        e2e = {"value": world * L * e * n_e2e / dt, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "ms_per_step": 1e3 * dt / n_e2e, "steps": n_e2e,
               "entry_point": "sar_gat_stack_host, pipelined (every step copies all its inputs in and all its results out)"}

    # ---- the oracle on the host cores, bounded sample ------------------------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        small, s_src, s_dst, h = oracle_sample(workloads.CONFIGS[args.workload], dtype,
                                               min(1.0, args.cpu_sample * args.scale))
        secs = oracle_step(small, s_src, s_dst, h, cfg.slope)
        cpu = {"value": small.e / secs, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
               "sample": f"{small.name}: n={small.n} e={small.e} H={small.heads} F={small.feat}, one layer fwd+bwd, "
                         f"{secs:.1f} s"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {
                "workload": cfg.name, "n": n, "e": e, "heads": H, "feat_per_head": F, "layers": L, "partitions": K,
                "storage_dtype": dtype, "layer_glue": bool(args.glue), "bn_dropout": bool(args.glue and args.bn_dropout), "ids": args.ids, "schedule": "fused row-stationary (sar_gat_fwd_fused / sar_gat_bwd_fused)",
                "l2": "inputs_exceed_l2", "long_row_threshold": threshold, "parallelism": f"replicas x{world}",
                "edges_x_heads_x_feat_per_sec": value * H * F,
            },
            "roofline": roofline,
            "step_roofline": {"compulsory_bytes_per_step": step_bytes, "frac_of_peak": step_frac, "peak": peak,
                              "peak_source": peak_src},
            "passes": per_pass, "kernels": kernels, "gpu_launches": launches, "prep_ms": prep_ms,
            "peak_mem_bytes": peak_mem, "attention_bytes_if_stored": L * e * H * 4,
            "stats_bytes_kept": L * 2 * n * H * 4,
            "clocks": clocks, "e2e": e2e, "cpu_baseline": cpu,
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

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with B.LaunchTimer() as lt:
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms_per_step = e0.elapsed_time(e1) / args.steps
    kernels = lt.summary()
    peak, peak_src = load_peaks()
    alg = idx_bytes(n, e) + 2 * n * F * b  # per direction: indices, every input row once, every output row once
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
        "kernels": kernels, "gpu_launches": sum(v["launches"] for v in kernels.values()), "clocks": clocks,
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

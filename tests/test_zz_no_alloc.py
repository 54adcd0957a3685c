"""The backward entry point that needs no scratch from its caller (sar_gat_bwd_noalloc).

Some users of the library cannot allocate device memory at the point where they call it (a host
application that owns the allocator, a loop where cudaMalloc's device-wide synchronisation is not
acceptable, a fixed memory budget).  For them the library keeps a fixed scratch array of its own.
This test calls that entry point through the C-ABI twice in a row, on two different problems, and
checks each result against the ordinary entry point (same kernels, caller-provided workspace): the
second call finds the first call's leftovers in the shared array and must not be disturbed by them.
The two entry points run the same kernels in the same order, so besides the tolerance check the
results must agree bit for bit; the first problem is also compared with the CPU oracle.
It sits in a file of its own, collected last, so that a failure here cannot hide other tests.
"""
import numpy as np
import pytest
import torch

import oracle
import workloads
from helpers import allclose_report

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2111_06483_b200 import api, binding as B

DEV = "cuda"


def _problem(n, e, H, F, seed, dtype, hub):
    if hub:
        spec = workloads.ChungLuSpec(n=n, e=e, gamma=2.1, d_max=n / 8, seed=seed)
        src, dst = workloads.chung_lu_edges(spec)
    else:
        src, dst = workloads.uniform_edges(n, e, seed, self_loops=True)
    g = api.Graph.from_coo(n, src.to(DEV), dst.to(DEV), threshold=32)
    host = workloads.make_node_inputs(n, H, F, seed, dtype=dtype)
    t = {k: v.to(DEV) for k, v in host.items()}
    return g, t, H, F, (src, dst, host)


def _both_ways(g, t, H, F, slope=0.2):
    out, m, d = api.gat_forward(g, t["feat"], t["el"], t["er"], slope)
    want = api.gat_backward(g, t["feat"], t["el"], t["er"], m, d, t["gout"], slope)
    dfeat = torch.full_like(t["feat"], float("nan"))
    del_ = torch.full((g.n, H), float("nan"), device=DEV)
    der = torch.full((g.n, H), float("nan"), device=DEV)
    B.sar_gat_bwd_noalloc(g.whole, t["feat"], t["el"], t["er"], m, d, t["gout"], H, F, slope, dfeat, del_, der)
    torch.cuda.synchronize()
    return want, (dfeat, del_, der)


def _close(got, want, dtype):
    # same kernels, same launch configuration, same arithmetic order: the tolerances of the parity tests
    # (float32 gradients rtol 1e-4 / floor 1e-5, bf16 rtol 2e-2 / floor 2e-2) are met with room to spare
    rtol, atol = (2e-2, 2e-2) if dtype == "bf16" else (1e-4, 1e-5)
    for a, b, name in zip(got, want, ("dfeat", "del", "der")):
        a, b = a.float(), b.float()
        assert torch.isfinite(a).all(), name
        bad = (a - b).abs() > atol * max(1.0, float(b.pow(2).mean().sqrt())) + rtol * b.abs()
        assert not bad.any(), f"{name}: {int(bad.sum())} elements differ"


def test_two_calls_in_a_row_match_the_ordinary_entry_point():
    assert B.sar_gat_bwd_noalloc_limit() == 16 << 20
    first = _problem(6000, 60000, 4, 32, 11, "bf16", hub=True)      # long rows: records + segment partials
    second = _problem(2000, 20000, 4, 16, 12, "f32", hub=False)     # smaller: the array still holds call 1's data
    assert first[0].whole.split.n_long > 0
    for prob, dtype in ((first, "bf16"), (second, "f32")):
        want, got = _both_ways(*prob[:4])
        _close(got, want, dtype)
        for a, b, name in zip(got, want, ("dfeat", "del", "der")):
            assert torch.equal(a, b), f"{name}: same kernels, same order, yet not bit-identical"
    # the first problem against the oracle as well, with the parity tests' tolerances
    g, t, H, F, (src, dst, host) = first
    _, got = _both_ways(g, t, H, F)
    h = {k: v.float().numpy() for k, v in host.items()}
    indptr, indices = oracle.csr_from_coo(g.n, g.n, src.numpy(), dst.numpy())
    f = oracle.gat_fwd(indptr, indices, h["feat"], h["el"], h["er"], 0.2)
    b = oracle.gat_bwd(indptr, indices, h["feat"], h["el"], h["er"], f.alpha, h["gout"], 0.2)
    for a, w, name in zip(got, (b.dfeat, b.del_, b.der), ("dfeat", "del", "der")):
        scale = max(float(np.sqrt(np.mean(w * w))), 1.0)
        if name == "dfeat":   # stored in bf16: one rounding
            allclose_report(a.float().cpu().numpy(), w, 2.0 ** -7, 2.0 ** -9 * scale, f"noalloc {name} vs oracle")
        else:                 # float32 arrays
            allclose_report(a.float().cpu().numpy(), w, 1e-4, 1e-5 * scale, f"noalloc {name} vs oracle")


def test_problems_beyond_the_fixed_scratch_are_refused():
    n, H, F = 300_000, 4, 8                                         # 300k x 4 heads x 16 B > 16 MiB
    src, dst = workloads.uniform_edges(n, 2 * n, 13, self_loops=False)
    g = api.Graph.from_coo(n, src.to(DEV), dst.to(DEV))
    t = {k: v.to(DEV) for k, v in workloads.make_node_inputs(n, H, F, 13).items()}
    out, m, d = api.gat_forward(g, t["feat"], t["el"], t["er"], 0.2)
    dfeat, del_, der = torch.empty_like(t["feat"]), torch.empty((n, H), device=DEV), torch.empty((n, H), device=DEV)
    with pytest.raises(B.SarError) as ei:
        B.sar_gat_bwd_noalloc(g.whole, t["feat"], t["el"], t["er"], m, d, t["gout"], H, F, 0.2, dfeat, del_, der)
    assert ei.value.code == -4
    torch.cuda.synchronize()

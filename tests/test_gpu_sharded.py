"""The sharded driver with the CUDA backend: K workers emulated as threads of one process (the host threads
wait for each other's messages; no kernel waits for another), every arithmetic step a call of the library on
the worker's sub-graphs G_{p,q}; the concatenated results against the oracle on the whole graph."""
import threading

import numpy as np
import pytest
import torch

import oracle
import workloads
from helpers import allclose_report
from sharded_helpers import ThreadComm

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("K,dt", [(1, "f32"), (3, "f32"), (4, "bf16")])
def test_sharded_layer_on_the_gpu_equals_the_whole_graph(K, dt):
    from paper_2111_06483_b200.sharded import CudaGatBackend, ShardedGatLayer, build_rank_parts
    n, H, F = 5000, 4, 16
    s, d = workloads.chung_lu_edges(workloads.ChungLuSpec(n=n, e=60000, gamma=2.1, d_max=700.0, seed=17))
    t = workloads.make_node_inputs(n, H, F, 17, dtype=dt)
    host = {k: v.float().numpy() for k, v in t.items()}
    indptr, indices = oracle.csr_from_coo(n, n, s.numpy(), d.numpy())
    f = oracle.gat_fwd(indptr, indices, host["feat"], host["el"], host["er"], 0.2)
    b = oracle.gat_bwd(indptr, indices, host["feat"], host["el"], host["er"], f.alpha, host["gout"], 0.2)
    bounds = [int(x) for x in oracle.partition_bounds(n, K)]
    mail = ThreadComm.mailboxes(K)
    tdt = torch.bfloat16 if dt == "bf16" else torch.float32
    sd, dd = s.to("cuda"), d.to("cuda")
    results, errors = [None] * K, []

    def worker(p):
        try:
            torch.cuda.set_device(0)
            lo, hi = bounds[p], bounds[p + 1]
            parts = build_rank_parts(n, bounds, p, sd, dd, threshold=24)
            layer = ShardedGatLayer(ThreadComm(p, K, mail), bounds, CudaGatBackend(parts, H, F, 0.2, tdt))
            dev = {k: v[lo:hi].to("cuda") for k, v in t.items()}
            out = layer.forward(dev["feat"], dev["el"], dev["er"])
            dfeat, del_, der = layer.backward(dev["gout"])
            torch.cuda.synchronize()
            results[p] = [x.float().cpu().numpy() for x in (out, layer.be.m, layer.be.d, dfeat, del_, der)]
        except Exception as ex:  # surfaced in the main thread
            errors.append((p, repr(ex)))

    threads = [threading.Thread(target=worker, args=(p,)) for p in range(K)]
    for th in threads:
        th.start()
    for th in threads:
        th.join(300)
    assert not errors, errors
    cat = lambda i: np.concatenate([results[p][i] for p in range(K)])
    rms = lambda x: max(float(np.sqrt(np.mean(np.asarray(x, np.float64) ** 2))), 1.0)
    if dt == "bf16":
        allclose_report(cat(0), f.out, 2e-2, 2e-2 * rms(f.out), "out")
        # K bf16 contributions per source are rounded before they travel: a few bf16 ulps of the largest term
        allclose_report(cat(3), b.dfeat, 4e-2, 4e-2 * rms(b.dfeat), "dfeat")
        # float32 arrays computed in float32 from inputs the oracle shares exactly (the row dot comes from the float32
        # numerator the last forward step leaves behind, not from the rounded out)
        allclose_report(cat(4), b.del_, 1e-4, 1e-5 * rms(b.del_), "del")
        allclose_report(cat(5), b.der, 1e-4, 1e-5 * rms(b.der), "der")
    else:
        allclose_report(cat(0), f.out, 1e-5, 1e-6, "out")
        allclose_report(cat(3), b.dfeat, 1e-4, 1e-5 * rms(b.dfeat), "dfeat")
        allclose_report(cat(4), b.del_, 1e-4, 1e-5 * rms(b.del_), "del")
        allclose_report(cat(5), b.der, 1e-4, 1e-5 * rms(b.der), "der")
    allclose_report(cat(1), f.m, 1e-5, 1e-6, "m")   # float32 scores against the oracle's float64 ones
    allclose_report(cat(2), f.d, 1e-5, 1e-6, "d")


@pytest.mark.parametrize("n,dtype", [(1, torch.float32), (1000, torch.bfloat16), (100003, torch.bfloat16), (4096, torch.float32)])
def test_error_sums_in_float32(n, dtype):
    """acc = x0; acc += x1; acc += x2 in float32, then one rounding to the storage type: the sum of the errors
    returned by the other workers (Algorithm 2)."""
    from paper_2111_06483_b200 import binding as B
    rng = np.random.default_rng(n)
    xs = [torch.from_numpy(rng.standard_normal(n).astype(np.float32)).to(dtype).cuda() for _ in range(3)]
    acc = torch.full((n,), float("nan"), dtype=torch.float32, device="cuda")
    B.sar_accumulate(xs[0], acc, first=True)
    B.sar_accumulate(xs[1], acc)
    B.sar_accumulate(xs[2], acc)
    want = (xs[0].float() + xs[1].float()) + xs[2].float()  # the same float32 additions in the same order
    assert torch.equal(acc, want)
    y = torch.empty(n, dtype=dtype, device="cuda")
    B.sar_round_to(acc, y)
    assert torch.equal(y, want.to(dtype))  # round to nearest even
    with pytest.raises(AssertionError):  # the sum is float32 whatever the storage type
        B.sar_accumulate(xs[0], acc.double())

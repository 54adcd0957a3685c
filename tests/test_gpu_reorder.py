"""The library's node order by degree (sar_degree_order / sar_relabel / sar_permute_rows) against the oracle, bit for
bit, and the attention layer on a renumbered graph against the oracle in the caller's numbering."""
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


def _hub_edges(n, e, seed):
    spec = workloads.ChungLuSpec(n=n, e=e, gamma=2.1, d_max=min(900.0, n / 4), seed=seed)
    return workloads.chung_lu_edges(spec)


@pytest.mark.parametrize("n,e", [(5000, 60000), (257, 3000), (64, 0), (1, 3)])
def test_degree_order_and_relabel_are_bit_exact(n, e):
    if e and n == 1:
        src = dst = torch.zeros(e, dtype=torch.int32)        # self-loops of the only node
    elif e:
        src, dst = _hub_edges(n, e, 5) if n > 300 else workloads.uniform_edges(n, e, 5, False)
    else:
        src = dst = torch.zeros(0, dtype=torch.int32)
    want_order, want_rank = oracle.degree_order(n, src.numpy(), dst.numpy())
    s, d = src.to(DEV), dst.to(DEV)
    order = torch.empty(n, dtype=torch.int32, device=DEV)
    rank = torch.empty(n, dtype=torch.int32, device=DEV)
    ws = torch.empty(B.sar_degree_order_workspace_bytes(n) + 256, dtype=torch.uint8, device=DEV)
    B.sar_degree_order(n, s, d, order, rank, ws)
    assert np.array_equal(order.cpu().numpy(), want_order)
    assert np.array_equal(rank.cpu().numpy(), want_rank)
    if e:
        out = torch.empty_like(s)
        B.sar_relabel(s, rank, out)
        assert np.array_equal(out.cpu().numpy(), want_rank[src.numpy()])


@pytest.mark.parametrize("shape,dtype", [((1000, 4, 32), torch.bfloat16), ((1000, 4), torch.float32),
                                          ((333, 3), torch.bfloat16), ((50, 5), torch.uint8)])
def test_permute_rows_is_an_indexed_copy(shape, dtype):
    g = torch.Generator().manual_seed(1)
    x = torch.randint(0, 255, shape, generator=g, dtype=torch.uint8).to(dtype) if dtype == torch.uint8 else \
        torch.randn(shape, generator=g).to(dtype)
    index = torch.randperm(shape[0], generator=g).to(torch.int32)
    out = torch.empty_like(x, device=DEV)
    B.sar_permute_rows(index.to(DEV), x.to(DEV), out)
    assert torch.equal(out.cpu(), x[index.long()])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_attention_layer_on_a_renumbered_graph_matches_the_oracle(dtype):
    n, e, H, F = 6000, 70000, 4, 32
    src, dst = _hub_edges(n, e, 9)
    t = workloads.make_node_inputs(n, H, F, 31, dtype=dtype)
    host = {k: v.float().numpy() for k, v in t.items()}
    indptr, indices = oracle.csr_from_coo(n, n, src.numpy(), dst.numpy())
    f = oracle.gat_fwd(indptr, indices, host["feat"], host["el"], host["er"], 0.2)
    b = oracle.gat_bwd(indptr, indices, host["feat"], host["el"], host["er"], f.alpha, host["gout"], 0.2)

    g = api.Graph.from_coo(n, src.to(DEV), dst.to(DEV), reorder="degree")
    assert g.order is not None and int(g.whole.indptr[-1].item()) == e
    dev = {k: g.to_internal(v.to(DEV)) for k, v in t.items()}
    out, m, d = api.gat_forward(g, dev["feat"], dev["el"], dev["er"], 0.2)[:3]
    dfeat, del_, der = api.gat_backward(g, dev["feat"], dev["el"], dev["er"], m, d, dev["gout"], 0.2, out=out)
    out, m, d, dfeat, del_, der = (g.to_external(x) for x in (out, m, d, dfeat, del_, der))
    bf = dtype == "bf16"
    rms = lambda x: float(np.sqrt(np.mean(np.square(x))))
    allclose_report(out.float().cpu().numpy(), f.out, 2.0 ** -7 if bf else 1e-5, 2.0 ** -9 * max(rms(f.out), 1) if bf else 1e-6, "out[reordered]")
    allclose_report(m.cpu().numpy(), f.m, 1e-6, 1e-6, "m[reordered]")
    allclose_report(d.cpu().numpy(), f.d, 1e-5, 1e-6, "d[reordered]")
    allclose_report(dfeat.float().cpu().numpy(), b.dfeat, 2.0 ** -7 if bf else 1e-4,
                    (2.0 ** -9 if bf else 1e-5) * max(rms(b.dfeat), 1), "dfeat[reordered]")
    allclose_report(del_.cpu().numpy(), b.del_, 1e-4, 1e-5 * max(rms(b.del_), 1), "del[reordered]")
    allclose_report(der.cpu().numpy(), b.der, 1e-4, 1e-5 * max(rms(b.der), 1), "der[reordered]")
    # the degrees of the renumbered graph's nodes do not increase
    deg = (g.whole.indptr[1:] - g.whole.indptr[:-1]) + (g.whole.t_indptr[1:] - g.whole.t_indptr[:-1])
    assert bool((deg[:-1] >= deg[1:]).all())

"""GPU parity of message-flow pruning (Appendix B) with the oracle: masks and pruned CSRs bit-exact, and
the property it exists for — a pruned stack gives the labelled nodes the same outputs and the same
parameter gradients as the full stack — checked on the CUDA path itself."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from helpers import small_problem

pytestmark = pytest.mark.gpu


def _dev(x, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(x)).to("cuda")
    return t if dtype is None else t.to(dtype)


def _graph(n, src, dst, **kw):
    from paper_2111_06483_b200 import api
    return api.Graph.from_coo(n, _dev(src, torch.int32), _dev(dst, torch.int32), **kw)


@pytest.mark.parametrize("case", ["uniform", "hubs", "empty", "one_node"])
@pytest.mark.parametrize("density", [0.0, 0.01, 0.2, 1.0])
def test_frontier_and_filter_bit_exact(case, density):
    from paper_2111_06483_b200 import api, binding as B
    if case == "uniform":
        n = 3000
        p = small_problem(n, 20000, 1, 4, 21, self_loops=False, empty_rows=7)
        src, dst = p["src"], p["dst"]
    elif case == "hubs":
        n = 6000
        s, d = workloads.chung_lu_edges(workloads.ChungLuSpec(n=n, e=90000, gamma=2.1, d_max=2500.0, seed=9))
        src, dst = s.numpy(), d.numpy()
    elif case == "empty":
        n, src, dst = 500, np.zeros(0, np.int32), np.zeros(0, np.int32)
    else:
        n, src, dst = 1, np.zeros(3, np.int32), np.zeros(3, np.int32)
    indptr, indices = oracle.csr_from_coo(n, n, src, dst)
    g = _graph(n, src, dst)
    rng = np.random.default_rng(4)
    keep = (rng.random(n) < density).astype(np.uint8)
    keep_d = _dev(keep)
    need_in = torch.full((n,), 7, dtype=torch.uint8, device="cuda")
    B.sar_mfg_frontier(n, g.whole.indptr, g.whole.indices, keep_d, need_in)
    assert np.array_equal(need_in.cpu().numpy(), oracle.mfg_frontier(indptr, indices, keep))
    fg = api.filter_rows(g, keep_d)
    want_ptr, want_idx = oracle.csr_filter_rows(indptr, indices, keep)
    assert np.array_equal(fg.whole.indptr.cpu().numpy(), want_ptr)
    assert np.array_equal(fg.whole.indices.cpu().numpy(), want_idx)
    # the transposed side of the filtered graph is the transpose of the filtered CSR
    t_ptr, t_idx = oracle.csr_transpose(n, n, want_ptr, want_idx)
    assert np.array_equal(fg.whole.t_indptr.cpu().numpy(), t_ptr)
    assert np.array_equal(fg.whole.t_indices.cpu().numpy(), t_idx)


@pytest.mark.parametrize("dt", [torch.float32, torch.bfloat16])
def test_pruned_stack_equals_full_stack_on_labelled_nodes(dt):
    from paper_2111_06483_b200 import api, binding as B
    n, H, F, L = 20000, 4, 16, 3
    s, d = workloads.chung_lu_edges(workloads.ChungLuSpec(n=n, e=120000, gamma=2.1, d_max=800.0, seed=13))
    g = api.Graph.from_coo(n, s.to("cuda"), d.to("cuda"), k=2)
    labelled = torch.zeros(n, dtype=torch.uint8, device="cuda")
    labelled[torch.arange(0, n, 997, device="cuda")] = 1
    graphs, need = api.mfg_layers(g, labelled, L)
    # the pruning is real: fewer edges at every layer, most at the last
    sizes = [gr.nnz for gr in graphs]
    assert sizes[-1] < sizes[0] < g.nnz and sizes == sorted(sizes, reverse=True)
    for l in range(L):  # need[l] is what the oracle derives from need[l + 1]
        want = oracle.mfg_frontier(g.whole.indptr.cpu().numpy(), g.whole.indices.cpu().numpy(), need[l + 1].cpu().numpy())
        assert np.array_equal(need[l].cpu().numpy(), want)
    feat = workloads.normal_tensor((n, H, F), 1, 10, device="cuda", dtype=dt)
    a_l = [workloads.normal_tensor((H, F), 1, 20 + l, device="cuda") * 0.3 for l in range(L)]
    a_r = [workloads.normal_tensor((H, F), 1, 30 + l, device="cuda") * 0.3 for l in range(L)]
    gout0 = workloads.normal_tensor((n, H, F), 1, 11, device="cuda", dtype=dt)
    gout0 = gout0 * labelled.to(dt)[:, None, None]  # the loss reads only the labelled nodes

    def run(graph_of_layer):
        z = [feat.clone()]
        saved = []
        for l in range(L):
            out, sv = api.gat_layer_forward(graph_of_layer(l), z[l], a_l[l], a_r[l], 0.2, relu_input=l > 0)
            z.append(out)
            saved.append(sv)
        grad = gout0.clone()
        das = []
        for l in reversed(range(L)):
            grad, dal, dar = api.gat_layer_backward(graph_of_layer(l), z[l], a_l[l], a_r[l], saved[l], grad, 0.2,
                                                    relu_input=l > 0)
            das.append((dal, dar))
        return z[L], grad, das

    out_f, dfeat_f, das_f = run(lambda l: g)
    out_p, dfeat_p, das_p = run(lambda l: graphs[l])
    lab = labelled.bool()
    assert torch.equal(out_p[lab], out_f[lab])  # a row's arithmetic does not depend on the other rows
    # gradients: the full stack adds exact zeros for the pruned rows, in a different summation order
    tol = 2e-2 if dt == torch.bfloat16 else 1e-4
    def close(a, b):
        a, b = a.float(), b.float()
        return float((a - b).abs().max()) <= tol * max(1.0, float(b.abs().max()))
    assert close(dfeat_p, dfeat_f)
    for (pl, pr), (fl, fr) in zip(das_p, das_f):
        assert close(pl, fl) and close(pr, fr)

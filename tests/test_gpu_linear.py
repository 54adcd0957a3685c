"""GPU parity of the dense projection z = h W and its backward pass (tensor-core GEMMs) with the float64
oracle on the same bf16-rounded inputs, through the C-ABI."""
import numpy as np
import pytest
import torch

import oracle
from helpers import allclose_report
from workloads.generators import normal_tensor as _normal

pytestmark = pytest.mark.gpu


def _np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("d_in,d_out", [(128, 128), (64, 256), (8, 8), (256, 64), (40, 72)])
@pytest.mark.parametrize("n", [1, 100, 4097, 300001])
def test_projection_forward_and_backward(d_in, d_out, n):
    from paper_2111_06483_b200 import binding as B
    h = _normal((n, d_in), 91, 1).to(torch.bfloat16).cuda()
    w = (_normal((d_in, d_out), 91, 2) / d_in ** 0.5).to(torch.bfloat16).cuda()
    dz = _normal((n, d_out), 91, 3).to(torch.bfloat16).cuda()
    ws = torch.empty(B.sar_linear_workspace_bytes(n, d_in, d_out), dtype=torch.uint8, device="cuda")
    z = torch.full((n, d_out), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.sar_linear(h, w, z, ws)
    want_z = oracle.linear(_np(h), _np(w))
    # exact bf16 products, float32 accumulation of d_in terms, one rounding of the result to bf16
    allclose_report(_np(z), want_z, 2.0 ** -8, 2.0 ** -8 * 0.5, "z")
    dh = torch.full((n, d_in), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.sar_linear_bwd_input(dz, w, dh, ws)
    want_dh, want_dw = oracle.linear_bwd(_np(h), _np(w), _np(dz))
    allclose_report(_np(dh), want_dh, 2.0 ** -8, 2.0 ** -8 * 0.5, "dh")
    dw = torch.full((d_in, d_out), float("nan"), dtype=torch.float32, device="cuda")
    B.sar_linear_bwd_weight(h, dz, dw, ws)
    # float32 sums of n unit-scale products, reduced in pieces: error ~ 2^-24 * sqrt(n) * |terms|
    allclose_report(_np(dw), want_dw, 1e-4, 1e-5 * max(1.0, float(np.sqrt(n))), "dw")


@pytest.mark.parametrize("d_in,H,F", [(128, 4, 32), (64, 8, 32), (128, 2, 64), (40, 4, 16), (64, 1, 128), (128, 16, 8)])
@pytest.mark.parametrize("n", [1, 100, 4097, 300001])
def test_projection_with_scores_in_the_epilogue(d_in, H, F, n):
    """sar_linear_project = sar_linear followed by sar_gat_project, in one kernel: z bit for bit, el / er up to the
    order of the F float32 additions; both against the oracle's projection of the bf16-rounded z as well."""
    from paper_2111_06483_b200 import binding as B
    d_out = H * F
    h = _normal((n, d_in), 93, 1).to(torch.bfloat16).cuda()
    w = (_normal((d_in, d_out), 93, 2) / d_in ** 0.5).to(torch.bfloat16).cuda()
    a_l = (_normal((H, F), 93, 4) / F ** 0.5).cuda()
    a_r = (_normal((H, F), 93, 5) / F ** 0.5).cuda()
    ws = torch.empty(B.sar_linear_workspace_bytes(n, d_in, d_out), dtype=torch.uint8, device="cuda")
    z0 = torch.empty((n, d_out), dtype=torch.bfloat16, device="cuda")
    B.sar_linear(h, w, z0, ws)
    el0, er0 = torch.empty((n, H), device="cuda"), torch.empty((n, H), device="cuda")
    B.sar_gat_project(z0.view(n, H, F), a_l, a_r, el0, er0)
    z = torch.full((n, d_out), float("nan"), dtype=torch.bfloat16, device="cuda")
    el = torch.full((n, H), float("nan"), device="cuda")
    er = torch.full((n, H), float("nan"), device="cuda")
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.sar_linear_project(h, w, a_l, a_r, z, el, er, ws, flag)
    assert int(flag.item()) == 0          # every row's elements sit in one thread of the epilogue
    assert torch.equal(z, z0)
    want_el, want_er = oracle.project(_np(z0).reshape(n, H, F), _np(a_l), _np(a_r))
    for got, ref, want, what in ((el, el0, want_el, "el"), (er, er0, want_er, "er")):
        allclose_report(_np(got), want, 1e-5, 1e-6 * F ** 0.5, what + " vs oracle")
        allclose_report(_np(got), _np(ref), 1e-5, 1e-6 * F ** 0.5, what + " vs the two-call path")


@pytest.mark.parametrize("d_in,d_out", [(128, 128), (64, 256), (8, 8), (40, 72)])
@pytest.mark.parametrize("n", [1, 4097, 300001])
def test_input_gradient_with_the_relu_mask_in_the_epilogue(d_in, d_out, n):
    """sar_linear_bwd_input_relu = sar_linear_bwd_input followed by sar_relu_bwd, in one kernel, bit for bit."""
    from paper_2111_06483_b200 import binding as B
    dz = _normal((n, d_out), 95, 1).to(torch.bfloat16).cuda()
    w = (_normal((d_in, d_out), 95, 2) / d_in ** 0.5).to(torch.bfloat16).cuda()
    y = torch.clamp_min(_normal((n, d_in), 95, 3), 0).to(torch.bfloat16).cuda()   # a ReLU's output: about half zeros
    ws = torch.empty(B.sar_linear_workspace_bytes(n, d_in, d_out), dtype=torch.uint8, device="cuda")
    ref = torch.empty((n, d_in), dtype=torch.bfloat16, device="cuda")
    B.sar_linear_bwd_input(dz, w, ref, ws)
    B.sar_relu_bwd(y, ref)
    got = torch.full((n, d_in), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.sar_linear_bwd_input_relu(dz, w, y, got, ws)
    assert torch.equal(got, ref)
    want_dh, _ = oracle.linear_bwd(np.zeros((n, d_in)), _np(w), _np(dz))
    allclose_report(_np(got), np.where(_np(y) > 0, want_dh, 0.0), 2.0 ** -8, 2.0 ** -8 * 0.5, "masked dh")


def test_projection_rejects_what_it_cannot_do():
    from paper_2111_06483_b200 import binding as B
    h = torch.zeros((16, 12), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((12, 8), dtype=torch.bfloat16, device="cuda")
    z = torch.zeros((16, 8), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SarError) as ei:   # d_in not a multiple of 8
        B.sar_linear(h, w, z, ws)
    assert ei.value.code == -2
    hf = torch.zeros((16, 16), dtype=torch.float32, device="cuda")
    with pytest.raises(B.SarError) as ei:   # float32 storage
        B.sar_linear(hf, torch.zeros((16, 8), device="cuda"), torch.zeros((16, 8), device="cuda"), ws)
    assert ei.value.code == -2


def test_two_whole_layers_match_the_oracle_network():
    """Dense projection -> scores -> aggregation -> ReLU, twice, forward and backward, on bf16 storage, against
    the float64 network of the oracle, which rounds the node arrays to bf16 where the library stores them (the
    score gradients amplify a rounding of their inputs).  Compared in relative Frobenius norm."""
    from paper_2111_06483_b200 import api, binding as B
    from helpers import small_problem
    n, H, F, L = 4000, 4, 16, 2
    D = H * F
    p = small_problem(n, 50000, H, F, 61, self_loops=True, empty_rows=6)
    rng = np.random.default_rng(8)
    bf = lambda x: torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16)
    Ws = [bf(rng.standard_normal((D, D)) / np.sqrt(D)) for _ in range(L)]
    a_l = [(rng.standard_normal((H, F)) * 0.3).astype(np.float32) for _ in range(L)]
    a_r = [(rng.standard_normal((H, F)) * 0.3).astype(np.float32) for _ in range(L)]
    h0 = bf(p["feat"].reshape(n, D))
    gout = bf(p["gout"])
    as_bf16 = lambda x: torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16).double().numpy()
    want = oracle.gat_net(p["indptr"], p["indices"], _np(h0), [_np(w) for w in Ws], a_l, a_r, _np(gout), 0.2,
                          stored=as_bf16)
    g = api.Graph.from_coo(n, torch.from_numpy(p["src"]).cuda(), torch.from_numpy(p["dst"]).cuda(), k=2)
    dev = lambda x: torch.from_numpy(x).cuda()
    h = [h0.cuda()]
    saved = []
    for l in range(L):
        out, sv = api.full_layer_forward(g, h[l], Ws[l].cuda(), dev(a_l[l]), dev(a_r[l]), 0.2, relu_input=l > 0)
        h.append(out.view(n, D))
        saved.append(sv)
    B.sar_relu(h[L])
    grad = gout.cuda().clone()
    B.sar_relu_bwd(h[L].view(n, H, F), grad)
    got_dW, got_al, got_ar = [None] * L, [None] * L, [None] * L
    for l in reversed(range(L)):
        grad, got_dW[l], got_al[l], got_ar[l] = api.full_layer_backward(g, h[l], Ws[l].cuda(), dev(a_l[l]), dev(a_r[l]),
                                                                        saved[l], grad.view(n, H, F), 0.2, relu_input=l > 0)
    rel = lambda a, b: np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30)
    assert rel(_np(h[L]), want["out"]) < 2e-2
    # gradients: a unit whose pre-activation lies within the forward error of zero takes the other branch of its
    # ReLU; a wrong or missing term would show as an error of tens of percent
    errs = {"dh0": rel(_np(grad), want["dh0"])}
    for l in range(L):
        errs[f"dW{l}"] = rel(_np(got_dW[l]), want["dW"][l])
        errs[f"da_l{l}"] = rel(_np(got_al[l]), want["da_l"][l])
        errs[f"da_r{l}"] = rel(_np(got_ar[l]), want["da_r"][l])
    assert max(errs.values()) < 3e-2, errs

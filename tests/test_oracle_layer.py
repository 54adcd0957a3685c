"""Pins for the oracle's layer functions (projection, its backward, ReLU, the layer stack), CPU only:
torch CPU float64 autograd over a dense formulation of the whole stack, and closed forms."""
import numpy as np
import torch

import oracle
from helpers import allclose_report, count_matrix, dense_gat_torch, small_problem


def test_projection_matches_matmul_and_its_backward_matches_autograd():
    rng = np.random.default_rng(0)
    z = rng.standard_normal((50, 3, 5))
    a_l, a_r = rng.standard_normal((3, 5)), rng.standard_normal((3, 5))
    el, er = oracle.project(z, a_l, a_r)
    for h in range(3):
        allclose_report(el[:, h], z[:, h, :] @ a_l[h], 1e-13, 1e-14, "el")
        allclose_report(er[:, h], z[:, h, :] @ a_r[h], 1e-13, 1e-14, "er")
    gl, gr = rng.standard_normal((50, 3)), rng.standard_normal((50, 3))
    zt, alt, art = (torch.tensor(x, requires_grad=True) for x in (z, a_l, a_r))
    ((zt * alt).sum(-1) * torch.tensor(gl) + (zt * art).sum(-1) * torch.tensor(gr)).sum().backward()
    dz, dal, dar = oracle.project_bwd(z, a_l, a_r, gl, gr)
    allclose_report(dz, zt.grad.numpy(), 1e-12, 1e-14, "dz")
    allclose_report(dal, alt.grad.numpy(), 1e-12, 1e-13, "da_l")
    allclose_report(dar, art.grad.numpy(), 1e-12, 1e-13, "da_r")


def test_layer_stack_matches_torch_autograd_on_dense_formulation():
    p = small_problem(40, 300, 2, 4, 41, self_loops=True, empty_rows=2)
    rng = np.random.default_rng(1)
    L = 3
    a_l = [rng.standard_normal((2, 4)) * 0.5 for _ in range(L)]
    a_r = [rng.standard_normal((2, 4)) * 0.5 for _ in range(L)]
    got = oracle.gat_stack(p["indptr"], p["indices"], p["feat"], a_l, a_r, p["gout"], 0.2, storage=np.float64)
    C = torch.from_numpy(count_matrix(40, 40, p["src"], p["dst"]))
    z = torch.tensor(p["feat"], dtype=torch.float64, requires_grad=True)
    z0 = z
    als = [torch.tensor(x, requires_grad=True) for x in a_l]
    ars = [torch.tensor(x, requires_grad=True) for x in a_r]
    for l in range(L):
        el, er = (z * als[l]).sum(-1), (z * ars[l]).sum(-1)
        z = torch.relu(dense_gat_torch(C, z, el, er, 0.2))
    (z * torch.tensor(p["gout"], dtype=torch.float64)).sum().backward()
    # the oracle's aggregation takes float32 el/er: agreement to float32 input rounding, not to 1e-12
    allclose_report(got["out"], z.detach().numpy(), 1e-5, 1e-6, "stack out")
    allclose_report(got["dfeat0"], z0.grad.numpy(), 1e-4, 1e-5, "stack dfeat0")
    for l in range(L):
        allclose_report(got["da_l"][l], als[l].grad.numpy(), 1e-4, 1e-5, f"da_l[{l}]")
        allclose_report(got["da_r"][l], ars[l].grad.numpy(), 1e-4, 1e-5, f"da_r[{l}]")


def test_linear_is_the_definition_and_its_backward_matches_autograd():
    rng = np.random.default_rng(4)
    h, w, dz = rng.standard_normal((9, 5)), rng.standard_normal((5, 7)), rng.standard_normal((9, 7))
    z = oracle.linear(h, w)
    brute = np.array([[sum(h[i, k] * w[k, o] for k in range(5)) for o in range(7)] for i in range(9)])
    allclose_report(z, brute, 1e-13, 1e-14, "z")
    ht, wt = torch.tensor(h, requires_grad=True), torch.tensor(w, requires_grad=True)
    ((ht @ wt) * torch.tensor(dz)).sum().backward()
    dh, dw = oracle.linear_bwd(h, w, dz)
    allclose_report(dh, ht.grad.numpy(), 1e-12, 1e-13, "dh")
    allclose_report(dw, wt.grad.numpy(), 1e-12, 1e-13, "dw")


def test_whole_network_with_weights_matches_torch_autograd():
    p = small_problem(30, 200, 2, 4, 43, self_loops=True, empty_rows=2)
    rng = np.random.default_rng(6)
    L, D = 2, 8
    Ws = [rng.standard_normal((D, D)) / np.sqrt(D) for _ in range(L)]
    a_l = [rng.standard_normal((2, 4)) * 0.5 for _ in range(L)]
    a_r = [rng.standard_normal((2, 4)) * 0.5 for _ in range(L)]
    h0 = p["feat"].reshape(30, D).astype(np.float64)
    got = oracle.gat_net(p["indptr"], p["indices"], h0, Ws, a_l, a_r, p["gout"], 0.2)
    C = torch.from_numpy(count_matrix(30, 30, p["src"], p["dst"]))
    h = torch.tensor(h0, requires_grad=True)
    h_in = h
    Wt = [torch.tensor(x, requires_grad=True) for x in Ws]
    als = [torch.tensor(x, requires_grad=True) for x in a_l]
    ars = [torch.tensor(x, requires_grad=True) for x in a_r]
    for l in range(L):
        z = (h @ Wt[l]).reshape(30, 2, 4)
        h = torch.relu(dense_gat_torch(C, z, (z * als[l]).sum(-1), (z * ars[l]).sum(-1), 0.2)).reshape(30, D)
    (h * torch.tensor(p["gout"], dtype=torch.float64).reshape(30, D)).sum().backward()
    allclose_report(got["out"], h.detach().numpy(), 1e-5, 1e-6, "net out")
    allclose_report(got["dh0"], h_in.grad.numpy(), 1e-4, 1e-5, "net dh0")
    for l in range(L):
        allclose_report(got["dW"][l], Wt[l].grad.numpy(), 1e-4, 1e-5, f"dW[{l}]")
        allclose_report(got["da_l"][l], als[l].grad.numpy(), 1e-4, 1e-5, f"da_l[{l}]")
        allclose_report(got["da_r"][l], ars[l].grad.numpy(), 1e-4, 1e-5, f"da_r[{l}]")

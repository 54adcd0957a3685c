"""GPU parity of batch normalisation over the node dimension (Sec. 3.4) with the float64 oracle, through the
C-ABI: local statistics, apply, backward statistics, backward apply, vector and scalar paths."""
import numpy as np
import pytest
import torch

import oracle
from helpers import allclose_report
from workloads.generators import normal_tensor as _normal

pytestmark = pytest.mark.gpu
DT = {"f32": torch.float32, "bf16": torch.bfloat16}


def _np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("C", [128, 8, 1000, 5, 2048])
@pytest.mark.parametrize("dt", ["f32", "bf16"])
@pytest.mark.parametrize("n", [1, 1237, 60001])
@pytest.mark.parametrize("offset", [0.0, 100.0])
def test_batchnorm_forward_and_backward(C, dt, n, offset):
    from paper_2111_06483_b200 import api, binding as B
    if n == 60001 and C > 128:
        n = 20001  # keeps the float64 reference on the host quick
    x = (_normal((n, C), 77, 1) * 0.5 + offset).to(DT[dt]).to("cuda")
    gy = _normal((n, C), 77, 2).to(DT[dt]).to("cuda")
    gamma = (_normal((C,), 77, 3) * 0.3 + 1.0).to("cuda")
    beta = _normal((C,), 77, 4).to("cuda")
    x_ref, gy_ref = _np(x), _np(gy)
    # local statistics
    ws = torch.empty(B.sar_bn_workspace_bytes(C), dtype=torch.uint8, device="cuda")
    mean = torch.full((C,), float("nan"), device="cuda")
    m2 = torch.full((C,), float("nan"), device="cuda")
    B.sar_bn_stats(x, mean, m2, ws)
    want_mean, want_m2 = oracle.bn_moments(x_ref)
    # float32 partial sums of up to ~170 rows per lane group, float64 above: relative 1e-6 of the magnitudes summed
    allclose_report(_np(mean), want_mean, 2e-6, 2e-6 * (abs(offset) + 1.0), "mean")
    allclose_report(_np(m2), want_m2, 1e-4, 1e-4 * (1.0 + want_m2.max() * 1e-2), "m2")
    # forward with the oracle's definition of everything
    y, (mean_g, rstd_g, n_all) = api.bn_forward(x, 1e-5, gamma, beta)
    assert n_all == n
    want_y, _, want_rstd = oracle.bn_forward(x_ref, 1e-5, _np(gamma), _np(beta))
    if n > 1:
        allclose_report(_np(rstd_g), want_rstd, 1e-4, 0.0, "rstd")
    # x - mean cancels |offset| / std digits of a float32 input
    lost = (abs(offset) + 1.0) * 2.0 ** -23 / 0.5 * 8
    if dt == "bf16":
        allclose_report(_np(y), want_y, 2e-2, 2e-2, "y")
    else:
        allclose_report(_np(y), want_y, 1e-4, 1e-5 + lost, "y")
    # backward
    gx, dgamma, dbeta = api.bn_backward(x, gy, (mean_g, rstd_g, n_all), gamma)
    want_gx, want_dg, want_db = oracle.bn_backward(x_ref, gy_ref, 1e-5, _np(gamma))
    scale_g = max(1.0, float(np.sqrt(n)))
    if dt == "bf16":
        allclose_report(_np(gx), want_gx, 2e-2, 2e-2 * max(1.0, float(np.abs(want_gx).max()) * 0.1), "gx")
    else:
        allclose_report(_np(gx), want_gx, 1e-3, (1e-5 + lost) * max(1.0, float(np.abs(want_gx).max())), "gx")
    allclose_report(_np(dbeta), want_db, 1e-4, 1e-5 * scale_g, "dbeta")
    allclose_report(_np(dgamma), want_dg, 1e-3, (1e-5 + lost) * scale_g * 4, "dgamma")
    # in place: y may be x
    x2 = x.clone()
    B.sar_bn_apply(x2, mean_g, rstd_g, gamma, beta, x2)
    assert torch.equal(x2, y)


def test_batchnorm_empty_input_and_errors():
    from paper_2111_06483_b200 import binding as B
    C = 16
    x = torch.empty((0, C), device="cuda")
    ws = torch.empty(B.sar_bn_workspace_bytes(C), dtype=torch.uint8, device="cuda")
    mean = torch.full((C,), 3.0, device="cuda")
    m2 = torch.full((C,), 3.0, device="cuda")
    B.sar_bn_stats(x, mean, m2, ws)
    assert float(mean.abs().max()) == 0.0 and float(m2.abs().max()) == 0.0
    x = torch.ones((64, C), device="cuda")
    with pytest.raises(B.SarError) as ei:   # scratch too small for the vector path
        B.sar_bn_stats(x, mean, m2, ws[:64])
    assert ei.value.code == -4


@pytest.mark.parametrize("C,n", [(128, 5003), (8, 300), (5, 1237), (1000, 2001)])
@pytest.mark.parametrize("dt", ["f32", "bf16"])
@pytest.mark.parametrize("flags", [1, 2, 3])
def test_batchnorm_with_relu_and_dropout_folded_in(C, n, dt, flags):
    """y = dropout(relu(bn(x))) in one pass and its backward pass against the oracle's three separate steps
    (normalisation, max(., 0), counter-based dropout with the same seed)."""
    from paper_2111_06483_b200 import binding as B
    p, seed = 0.3, 4242
    x = (_normal((n, C), 78, 1) * 0.7 + 0.2).to(DT[dt]).to("cuda")
    gy = _normal((n, C), 78, 2).to(DT[dt]).to("cuda")
    gamma = (_normal((C,), 78, 3) * 0.3 + 1.0).to("cuda")
    beta = (_normal((C,), 78, 4) * 0.5).to("cuda")
    x_ref, gy_ref, ga, be = _np(x), _np(gy), _np(gamma), _np(beta)
    # the oracle's chain
    y, mean_ref, rstd_ref = oracle.bn_forward(x_ref, 1e-5, ga, be)
    relu_mask = y > 0
    if flags & 1:
        y = np.where(relu_mask, y, 0.0)
    keep = np.ones_like(relu_mask)
    scale = 1.0
    if flags & 2:
        y, keep = oracle.dropout(y, p, seed)
        scale = float(np.float32(1.0) / (np.float32(1.0) - np.float32(p)))
    g_in = gy_ref * np.where(keep, scale, 0.0)
    if flags & 1:
        g_in = np.where(relu_mask, g_in, 0.0)
    # the library, with statistics from the oracle (their own parity is tested above)
    mean = torch.from_numpy(mean_ref.astype(np.float32)).cuda()
    rstd = torch.from_numpy(rstd_ref.astype(np.float32)).cuda()
    out = torch.full_like(x, float("nan"))
    B.sar_bn_apply_act(x, mean, rstd, gamma, beta, flags, p, seed, out)
    tol = dict(rtol=2e-5, atol=2e-5) if dt == "f32" else dict(rtol=2.0 ** -7, atol=2.0 ** -7)
    got = _np(out)
    # an element within rounding of 0 before the ReLU may fall on either side; compare away from that edge
    edge = np.abs(oracle.bn_forward(x_ref, 1e-5, ga, be)[0]) < (1e-4 if dt == "f32" else 5e-2)
    allclose_report(np.where(edge, 0.0, got), np.where(edge, 0.0, y), what="y", **tol)
    assert np.array_equal((got != 0)[~edge], (y != 0)[~edge])
    # backward: the gradient that reaches the normalisation, with the library's own ReLU decisions at the edge
    g_lib = gy_ref * np.where(keep, scale, 0.0)
    if flags & 1:
        g_lib = np.where(got > 0, g_lib, 0.0)
    want_gx, want_dgamma, want_dbeta = oracle.bn_backward(x_ref, g_lib, 1e-5, ga)
    ws = torch.empty(B.sar_bn_workspace_bytes(C), dtype=torch.uint8, device="cuda")
    s0 = torch.full((C,), float("nan"), device="cuda")
    s1 = torch.full((C,), float("nan"), device="cuda")
    B.sar_bn_bwd_stats_act(x, mean, rstd, gy, out, flags, p, seed, s0, s1, ws)
    allclose_report(_np(s0), want_dbeta, 1e-4, 1e-4 * n ** 0.5, "sum gy")
    allclose_report(_np(s1), want_dgamma, 1e-4, 1e-4 * n ** 0.5, "sum gy xhat")
    gx = torch.full_like(x, float("nan"))
    B.sar_bn_bwd_apply_act(x, mean, rstd, gamma, gy, out, flags, p, seed, s0, s1, 1.0 / n, gx)
    tol_g = dict(rtol=1e-4, atol=1e-4) if dt == "f32" else dict(rtol=2.0 ** -7, atol=2.0 ** -6)
    allclose_report(_np(gx), want_gx, what="gx", **tol_g)
    if not edge.any():  # then the oracle's own chain is the same function
        allclose_report(_np(gx), oracle.bn_backward(x_ref, g_in, 1e-5, ga)[0], what="gx, oracle's masks", **tol_g)
    with pytest.raises(B.SarError):
        B.sar_bn_apply_act(x, mean, rstd, gamma, beta, 4, p, seed, out)
    if flags & 1:
        with pytest.raises(B.SarError):
            B.sar_bn_bwd_stats_act(x, mean, rstd, gy, None, flags, p, seed, s0, s1, ws)

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

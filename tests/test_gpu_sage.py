"""GPU parity of the GraphSage layer (Eq. 2: residual projection plus the mean of the neighbours' projections),
forward and backward, with the float64 oracle on the same bf16-rounded inputs, through the C-ABI."""
import numpy as np
import pytest
import torch

import oracle
from helpers import allclose_report, small_problem

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def _bf16(a):
    return torch.from_numpy(np.asarray(a, np.float32)).to(torch.bfloat16)


def _rms(a):
    return float(np.sqrt((a ** 2).mean()))


@pytest.mark.parametrize("n,e,d_in,d_out,k,empty", [
    (200, 1500, 16, 8, 1, 5),
    (200, 1500, 16, 8, 3, 5),
    (30000, 400000, 256, 256, 1, 0),
    (30000, 400000, 128, 256, 4, 100),
])
def test_sage_layer_forward_and_backward(n, e, d_in, d_out, k, empty):
    from paper_2111_06483_b200 import api
    p = small_problem(n, e, 1, 4, 31, empty_rows=empty)
    g = api.Graph.from_coo(n, torch.from_numpy(p["src"]).to(DEV), torch.from_numpy(p["dst"]).to(DEV), k=k, build_parts=k > 1)
    rng = np.random.default_rng(8)
    h = _bf16(rng.standard_normal((n, d_in))).to(DEV)
    W = _bf16(rng.standard_normal((d_in, d_out)) / d_in ** 0.5).to(DEV)
    W_res = _bf16(rng.standard_normal((d_in, d_out)) / d_in ** 0.5).to(DEV)
    gpre = _bf16(rng.standard_normal((n, d_out))).to(DEV)
    pre, saved = api.sage_layer_forward(g, h, W, W_res)
    want = oracle.sage_layer(p["indptr"], p["indices"], _np(h), _np(W), _np(W_res))
    # bf16 storage of the aggregate and of the output (written, then read and written again): a few roundings of 2^-9
    allclose_report(_np(pre), want, 2e-2, 2e-2 * _rms(want), "pre")
    dh, dW, dW_res = api.sage_layer_backward(g, h, W, W_res, saved, gpre)
    want_dh, want_dW, want_dW_res = oracle.sage_layer_bwd(p["indptr"], p["indices"], _np(h), _np(W), _np(W_res), _np(gpre))
    allclose_report(_np(dh), want_dh, 2e-2, 2e-2 * _rms(want_dh), "dh")
    allclose_report(_np(dW), want_dW, 2e-2, 2e-2 * _rms(want_dW), "dW")
    allclose_report(_np(dW_res), want_dW_res, 1e-3, 1e-3 * _rms(want_dW_res), "dW_res")
    for got, ref in ((pre, want), (dh, want_dh), (dW, want_dW)):
        assert float(np.linalg.norm(_np(got) - ref) / np.linalg.norm(ref)) < 5e-3

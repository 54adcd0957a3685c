"""GPU parity of the layer functions around the aggregation (score projections of Eq. 3, their
backward pass, the ReLU between layers) against the float64 oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

import oracle
from helpers import allclose_report, small_problem
from workloads.generators import normal_tensor as _normal


def normal_tensor(shape, stream):
    return _normal(shape, 2024, stream).numpy()

pytestmark = pytest.mark.gpu

DT = {"f32": torch.float32, "bf16": torch.bfloat16}


def _dev(x, dtype=torch.float32):
    return torch.from_numpy(np.ascontiguousarray(x)).to("cuda").to(dtype)


def _np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


# shapes: the vector path at several group widths, two vectors per lane, and shapes that only the scalar path takes
SHAPES = [(1, 4), (1, 8), (4, 32), (2, 16), (8, 8), (3, 20), (1, 256), (4, 64), (2, 3), (5, 7), (1, 1)]


@pytest.mark.parametrize("H,F", SHAPES)
@pytest.mark.parametrize("dt", ["f32", "bf16"])
@pytest.mark.parametrize("n", [0, 1, 1237, 40001])
@pytest.mark.parametrize("flags", [0, 1])
def test_projection_and_its_backward(H, F, dt, n, flags):
    from paper_2111_06483_b200 import binding as B
    if n == 40001 and H * F > 512:
        n = 9001
    z = normal_tensor((n, H, F), 11).astype(np.float32)
    a_l = normal_tensor((H, F), 12).astype(np.float32)
    a_r = normal_tensor((H, F), 13).astype(np.float32)
    gl = normal_tensor((n, H), 14).astype(np.float32)
    gr = normal_tensor((n, H), 15).astype(np.float32)
    dz0 = normal_tensor((n, H, F), 16).astype(np.float32)
    zt = _dev(z, DT[dt])
    z_ref = _np(zt)  # the values the kernel reads (bf16-rounded in the bf16 case)
    dzt = _dev(dz0, DT[dt])
    dz_ref = _np(dzt)
    el = torch.full((n, H), float("nan"), device="cuda")
    er = torch.full((n, H), float("nan"), device="cuda")
    B.sar_gat_project(zt, _dev(a_l), _dev(a_r), el, er, flags)
    if flags:  # the ReLU of the input is applied in place, exactly
        z_ref = np.maximum(z_ref, 0.0)
    assert np.array_equal(_np(zt), z_ref)
    want_el, want_er = oracle.project(z_ref, a_l, a_r)
    # float32 accumulation of F products: error <= F * 2^-24 * sum|terms|; floor from the term magnitudes
    floor = 1e-6 * max(1.0, float(np.sqrt(F)))
    allclose_report(_np(el), want_el, 1e-5, floor * 4, "el")
    allclose_report(_np(er), want_er, 1e-5, floor * 4, "er")
    da_l = torch.full((H, F), float("nan"), device="cuda")
    da_r = torch.full((H, F), float("nan"), device="cuda")
    ws = torch.empty(B.sar_gat_project_workspace_bytes(H, F), dtype=torch.uint8, device="cuda")
    B.sar_gat_project_bwd(zt, _dev(a_l), _dev(a_r), _dev(gl), _dev(gr), dzt, da_l, da_r, ws, flags)
    want_dz, want_dal, want_dar = oracle.project_bwd(z_ref, a_l, a_r, gl, gr)
    want_dz = want_dz + dz_ref
    if flags:
        want_dz = np.where(z_ref > 0, want_dz, 0.0)
        assert np.all(_np(dzt)[z_ref <= 0] == 0.0)
    if dt == "bf16":
        allclose_report(_np(dzt), want_dz, 2e-2, 2e-2, "dz")
    else:
        allclose_report(_np(dzt), want_dz, 1e-5, 2e-6, "dz")
    # a sum of n float32 products: floor scales with sqrt(n) term magnitudes
    gfloor = 1e-5 * max(1.0, float(np.sqrt(max(n, 1))))
    allclose_report(_np(da_l), want_dal, 1e-4, gfloor, "da_l")
    allclose_report(_np(da_r), want_dar, 1e-4, gfloor, "da_r")


@pytest.mark.parametrize("dt", ["f32", "bf16"])
@pytest.mark.parametrize("n", [0, 1, 5, 1023, 1 << 20, (1 << 22) + 3])
def test_relu_forward_and_backward_are_exact(dt, n):
    from paper_2111_06483_b200 import binding as B
    x = _dev(normal_tensor((n,), 3).astype(np.float32), DT[dt])
    if n > 4:
        x[1] = 0.0
        x[2] = -0.0
    want = torch.clamp_min(x.clone(), 0)
    y = x.clone()
    B.sar_relu(y)
    assert torch.equal(y, want)
    g = _dev(normal_tensor((n,), 4).astype(np.float32), DT[dt])
    wantg = torch.where(y > 0, g, torch.zeros_like(g))
    B.sar_relu_bwd(y, g)
    assert torch.equal(g, wantg)


@pytest.mark.parametrize("k", [1, 3])
def test_three_layer_stack_matches_oracle_f32(k):
    from paper_2111_06483_b200 import api, binding as B
    n, H, F, L = 3000, 2, 16, 3
    p = small_problem(n, 40000, H, F, 77, self_loops=True, empty_rows=5)
    rng = np.random.default_rng(5)
    a_l = [(rng.standard_normal((H, F)) * 0.3).astype(np.float32) for _ in range(L)]
    a_r = [(rng.standard_normal((H, F)) * 0.3).astype(np.float32) for _ in range(L)]
    want = oracle.gat_stack(p["indptr"], p["indices"], p["feat"], a_l, a_r, p["gout"], 0.2, storage=np.float32)
    g = api.Graph.from_coo(n, _dev(p["src"], torch.int32), _dev(p["dst"], torch.int32), k=k)
    z = [_dev(p["feat"])]
    saved = []
    for l in range(L):  # z[l + 1] holds layer l's output; the next layer's projection applies its ReLU in place
        out, sv = api.gat_layer_forward(g, z[l], _dev(a_l[l]), _dev(a_r[l]), 0.2, relu_input=l > 0)
        z.append(out)
        saved.append(sv)
    B.sar_relu(z[L])
    grad = _dev(p["gout"])
    B.sar_relu_bwd(z[L], grad)
    got_al, got_ar = [None] * L, [None] * L
    for l in reversed(range(L)):
        grad, got_al[l], got_ar[l] = api.gat_layer_backward(g, z[l], _dev(a_l[l]), _dev(a_r[l]), saved[l], grad, 0.2,
                                                            relu_input=l > 0)
    # three layers deep: rounding of each layer's float32 outputs feeds the next, and a unit whose
    # pre-activation is within rounding of zero may flip its ReLU mask; compare in a norm that tolerates that
    out_err = np.abs(_np(z[L]) - want["out"]).max()
    assert out_err <= 1e-4 * max(1.0, np.abs(want["out"]).max()), out_err
    def rel(a, b):
        return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30)
    assert rel(_np(grad), want["dfeat0"]) < 1e-3
    for l in range(L):
        assert rel(_np(got_al[l]), want["da_l"][l]) < 1e-3, l
        assert rel(_np(got_ar[l]), want["da_r"][l]) < 1e-3, l


@pytest.mark.parametrize("dt", ["f32", "bf16"])
@pytest.mark.parametrize("n", [0, 1, 7, 4099, (1 << 20) + 5])
@pytest.mark.parametrize("p", [0.0, 0.25, 0.5])
def test_dropout_mask_is_the_oracles_mask(dt, n, p):
    from paper_2111_06483_b200 import binding as B
    x = _dev(normal_tensor((n,), 8).astype(np.float32), DT[dt])
    y = torch.full_like(x, float("nan"))
    B.sar_dropout(x, p, 0xDEADBEEFCAFE, y)
    want, keep = oracle.dropout(_np(x), p, 0xDEADBEEFCAFE)
    got = _np(y)
    assert np.array_equal(got != 0, keep & (_np(x) != 0))          # the same elements survive
    if dt == "bf16":
        allclose_report(got, want, 2 ** -8, 0.0, "dropout")           # one rounding to bf16
    else:
        allclose_report(got, want, 2e-7, 0.0, "dropout")
    # the backward pass draws the same mask again; in place
    g = x.clone()
    B.sar_dropout(g, p, 0xDEADBEEFCAFE, g)
    assert torch.equal(g, y)
    if n > 4 and p > 0:   # an unaligned view takes the scalar path and must agree with the vector path
        xo = x[1:]
        yo = torch.empty_like(xo)
        B.sar_dropout(xo, p, 3, yo)
        assert np.array_equal(_np(yo) != 0, oracle.dropout(_np(xo), p, 3)[1] & (_np(xo) != 0))

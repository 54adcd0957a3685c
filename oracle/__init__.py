"""CPU oracle for the SAR graph-attention aggregation (arXiv 2111.06483).

TEST INFRASTRUCTURE ONLY: a plain float64 restatement of Eq. 2, Eq. 3, Algorithm 1
(with the running max of Sec. 3.4) and the chain rule behind Algorithm 2, compiled from
``sar_oracle.c`` with gcc and called through ctypes.  It imports nothing from the CUDA
package and the CUDA package imports nothing from here.  Only tests, the smoke check
and the benchmark's CPU-baseline / reference arm may use it.

All array arguments are numpy arrays; floating inputs are float32 storage (bf16 cases pass
bf16-rounded values held in float32), every result is float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sar_oracle.c")
_LIB = os.path.join(_HERE, "libsar_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile sar_oracle.c into libsar_oracle.so next to it (gcc -O2 -fopenmp)."""
    if force or (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
    return _lib


def _p(a: np.ndarray, dtype):
    assert a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    return a.ctypes.data_as(ctypes.c_void_p)


def _i64(a):
    return np.ascontiguousarray(a, dtype=np.int64)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _check(rc: int, what: str):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(ctypes.c_int(int(n)))


# --------------------------------------------------------------------------------------
# integer side (Sec. 3.2, subgraphs G_{p,q})
# --------------------------------------------------------------------------------------

def csr_from_coo(n_dst: int, n_src: int, src, dst):
    """CSR by destination of the edge list src[t] -> dst[t]; sources ascend within a row."""
    src, dst = _i32(src), _i32(dst)
    nnz = src.shape[0]
    indptr = np.empty(n_dst + 1, dtype=np.int64)
    indices = np.empty(nnz, dtype=np.int32)
    rc = _load().oracle_csr_from_coo(ctypes.c_int64(n_dst), ctypes.c_int64(n_src), ctypes.c_int64(nnz),
                                     _p(src, np.int32), _p(dst, np.int32), _p(indptr, np.int64),
                                     _p(indices, np.int32))
    _check(rc, "csr_from_coo")
    return indptr, indices


def csr_transpose(n_rows: int, n_cols: int, indptr, indices):
    indptr, indices = _i64(indptr), _i32(indices)
    t_indptr = np.empty(n_cols + 1, dtype=np.int64)
    t_indices = np.empty(indices.shape[0], dtype=np.int32)
    rc = _load().oracle_csr_transpose(ctypes.c_int64(n_rows), ctypes.c_int64(n_cols), _p(indptr, np.int64),
                                      _p(indices, np.int32), _p(t_indptr, np.int64), _p(t_indices, np.int32))
    _check(rc, "csr_transpose")
    return t_indptr, t_indices


def partition_bounds(n: int, k: int) -> np.ndarray:
    bounds = np.empty(k + 1, dtype=np.int64)
    _check(_load().oracle_partition_bounds(ctypes.c_int64(n), ctypes.c_int32(k), _p(bounds, np.int64)),
           "partition_bounds")
    return bounds


@dataclass
class SplitCSR:
    """K per-partition CSRs in one block: partition q is indptr_all[q], indices_all[nnz_off[q]:nnz_off[q+1]]."""
    n_dst: int
    k: int
    bounds: np.ndarray       # int64[k+1]
    indptr_all: np.ndarray   # int64[k, n_dst+1]
    indices_all: np.ndarray  # int32[nnz], local source ids
    nnz_off: np.ndarray      # int64[k+1]

    def part(self, q: int):
        return self.indptr_all[q], self.indices_all[self.nnz_off[q]:self.nnz_off[q + 1]]


def csr_split(n_dst: int, indptr, indices, bounds) -> SplitCSR:
    indptr, indices, bounds = _i64(indptr), _i32(indices), _i64(bounds)
    k = bounds.shape[0] - 1
    indptr_all = np.empty((k, n_dst + 1), dtype=np.int64)
    indices_all = np.empty(indices.shape[0], dtype=np.int32)
    nnz_off = np.empty(k + 1, dtype=np.int64)
    rc = _load().oracle_csr_split(ctypes.c_int64(n_dst), _p(indptr, np.int64), _p(indices, np.int32),
                                  ctypes.c_int32(k), _p(bounds, np.int64), _p(indptr_all, np.int64),
                                  _p(indices_all, np.int32), _p(nnz_off, np.int64))
    _check(rc, "csr_split")
    return SplitCSR(n_dst, k, bounds, indptr_all, indices_all, nnz_off)


# --------------------------------------------------------------------------------------
# floating side
# --------------------------------------------------------------------------------------

@dataclass
class GatForward:
    e: np.ndarray      # [nnz,H]  LeakyReLU(el_i + er_j)
    alpha: np.ndarray  # [nnz,H]  softmax over each destination's in-edges
    out: np.ndarray    # [n_dst,H,F]
    m: np.ndarray      # [n_dst,H] row max of e (-inf for empty rows)
    d: np.ndarray      # [n_dst,H] sum of exp(e - m) (0 for empty rows)


def gat_fwd(indptr, indices, feat, el, er, slope: float) -> GatForward:
    """Eq. 3 as written: per-edge scores, softmax over each in-neighbourhood, weighted sum."""
    indptr, indices = _i64(indptr), _i32(indices)
    feat, el, er = _f32(feat), _f32(el), _f32(er)
    n_dst = indptr.shape[0] - 1
    _, H, F = feat.shape
    assert el.shape == (n_dst, H) and er.shape == (feat.shape[0], H)
    nnz = indices.shape[0]
    assert int(indptr[-1]) == nnz
    if nnz:
        assert indices.min() >= 0 and indices.max() < feat.shape[0]
    e = np.empty((nnz, H), dtype=np.float64)
    alpha = np.empty((nnz, H), dtype=np.float64)
    out = np.empty((n_dst, H, F), dtype=np.float64)
    m = np.empty((n_dst, H), dtype=np.float64)
    d = np.empty((n_dst, H), dtype=np.float64)
    rc = _load().oracle_gat_fwd(ctypes.c_int64(n_dst), _p(indptr, np.int64), _p(indices, np.int32),
                                _p(feat, np.float32), _p(el, np.float32), _p(er, np.float32),
                                ctypes.c_int32(H), ctypes.c_int32(F), ctypes.c_double(slope),
                                _p(e, np.float64), _p(alpha, np.float64), _p(out, np.float64),
                                _p(m, np.float64), _p(d, np.float64))
    _check(rc, "gat_fwd")
    return GatForward(e, alpha, out, m, d)


@dataclass
class GatBackward:
    D: np.ndarray      # [n_dst,H]  sum_t alpha*dalpha
    dfeat: np.ndarray  # [n_src,H,F]
    del_: np.ndarray   # [n_dst,H]
    der: np.ndarray    # [n_src,H]


def gat_bwd(indptr, indices, feat, el, er, alpha, gout, slope: float) -> GatBackward:
    """Chain rule on Eq. 3 with the per-edge alpha of gat_fwd."""
    indptr, indices = _i64(indptr), _i32(indices)
    feat, el, er, gout = _f32(feat), _f32(el), _f32(er), _f32(gout)
    alpha = np.ascontiguousarray(alpha, dtype=np.float64)
    n_dst = indptr.shape[0] - 1
    n_src, H, F = feat.shape
    assert gout.shape == (n_dst, H, F) and alpha.shape == (indices.shape[0], H)
    D = np.empty((n_dst, H), dtype=np.float64)
    dfeat = np.empty((n_src, H, F), dtype=np.float64)
    del_ = np.empty((n_dst, H), dtype=np.float64)
    der = np.empty((n_src, H), dtype=np.float64)
    rc = _load().oracle_gat_bwd(ctypes.c_int64(n_dst), ctypes.c_int64(n_src), _p(indptr, np.int64),
                                _p(indices, np.int32), _p(feat, np.float32), _p(el, np.float32),
                                _p(er, np.float32), _p(alpha, np.float64), _p(gout, np.float32),
                                ctypes.c_int32(H), ctypes.c_int32(F), ctypes.c_double(slope),
                                _p(D, np.float64), _p(dfeat, np.float64), _p(del_, np.float64),
                                _p(der, np.float64))
    _check(rc, "gat_bwd")
    return GatBackward(D, dfeat, del_, der)


def gat_fwd_seq(split: SplitCSR, feat, el, er, slope: float, order=None):
    """Algorithm 1 + running max (Sec. 3.4): partitions visited one by one. Returns (out, m, d)."""
    feat, el, er = _f32(feat), _f32(el), _f32(er)
    n_dst, k = split.n_dst, split.k
    _, H, F = feat.shape
    order = _i32(np.arange(k) if order is None else order)
    assert sorted(order.tolist()) == list(range(k))
    out = np.empty((n_dst, H, F), dtype=np.float64)
    m = np.empty((n_dst, H), dtype=np.float64)
    d = np.empty((n_dst, H), dtype=np.float64)
    rc = _load().oracle_gat_fwd_seq(ctypes.c_int64(n_dst), ctypes.c_int32(k), _p(split.bounds, np.int64),
                                    _p(order, np.int32), _p(split.indptr_all, np.int64),
                                    _p(split.indices_all, np.int32), _p(split.nnz_off, np.int64),
                                    _p(feat, np.float32), _p(el, np.float32), _p(er, np.float32),
                                    ctypes.c_int32(H), ctypes.c_int32(F), ctypes.c_double(slope),
                                    _p(out, np.float64), _p(m, np.float64), _p(d, np.float64))
    _check(rc, "gat_fwd_seq")
    return out, m, d


def spmm(indptr, indices, feat, mean: bool = False) -> np.ndarray:
    """Eq. 2's neighbour sum (mean=True divides by the in-degree)."""
    indptr, indices = _i64(indptr), _i32(indices)
    feat = _f32(feat)
    n_dst = indptr.shape[0] - 1
    F = feat.shape[1]
    if indices.shape[0]:
        assert indices.min() >= 0 and indices.max() < feat.shape[0]
    out = np.empty((n_dst, F), dtype=np.float64)
    rc = _load().oracle_spmm(ctypes.c_int64(n_dst), _p(indptr, np.int64), _p(indices, np.int32),
                             _p(feat, np.float32), ctypes.c_int32(F), ctypes.c_int32(1 if mean else 0),
                             _p(out, np.float64))
    _check(rc, "spmm")
    return out


# --------------------------------------------------------------------------------------
# the layer around the aggregation (Eq. 3's a^T(z_i || z_j); f_node of Eq. 1 taken as a ReLU)
# plain numpy, float64
# --------------------------------------------------------------------------------------

def project(z, a_l, a_r):
    """el[i,h] = <z[i,h,:], a_l[h,:]>, er[i,h] = <z[i,h,:], a_r[h,:]>."""
    z = np.asarray(z, dtype=np.float64)
    return np.einsum("nhf,hf->nh", z, np.asarray(a_l, np.float64)), np.einsum("nhf,hf->nh", z, np.asarray(a_r, np.float64))


def project_bwd(z, a_l, a_r, del_, der):
    """Returns (dz_add[n,H,F], da_l[H,F], da_r[H,F]) of the projection for upstream del, der."""
    z, a_l, a_r = (np.asarray(x, np.float64) for x in (z, a_l, a_r))
    del_, der = np.asarray(del_, np.float64), np.asarray(der, np.float64)
    dz = del_[:, :, None] * a_l[None] + der[:, :, None] * a_r[None]
    return dz, np.einsum("nh,nhf->hf", del_, z), np.einsum("nh,nhf->hf", der, z)


def gat_stack(indptr, indices, feat0, a_l, a_r, gout, slope: float, storage=np.float32):
    """L layers z^{l+1} = ReLU(GAT(z^l, <z^l,a_l^l>, <z^l,a_r^l>)) and the gradient of <gout, z^L>.

    The aggregation functions take float32 storage, so activations are rounded to `storage` between
    layers exactly where the library stores them (z, el, er and the upstream gradient)."""
    L = len(a_l)
    z = [np.asarray(feat0, dtype=storage)]
    saved = []
    for l in range(L):
        el, er = project(z[l], a_l[l], a_r[l])
        el, er = el.astype(np.float32), er.astype(np.float32)
        f = gat_fwd(indptr, indices, z[l].astype(np.float32), el, er, slope)
        saved.append((el, er, f))
        z.append(np.maximum(f.out, 0.0).astype(storage))
    g = np.asarray(gout, dtype=np.float64)
    da_l, da_r = [None] * L, [None] * L
    for l in reversed(range(L)):
        el, er, f = saved[l]
        g = np.where(z[l + 1].astype(np.float64) > 0, g, 0.0).astype(storage)
        b = gat_bwd(indptr, indices, z[l].astype(np.float32), el, er, f.alpha, g.astype(np.float32), slope)
        dz_add, da_l[l], da_r[l] = project_bwd(z[l], a_l[l], a_r[l], b.del_.astype(np.float32), b.der.astype(np.float32))
        g = (b.dfeat.astype(storage).astype(np.float64) + dz_add)
    return dict(out=z[L].astype(np.float64), dfeat0=g, da_l=da_l, da_r=da_r)


def gat_net(indptr, indices, h0, weights, a_l, a_r, gout, slope: float, stored=None):
    """L whole layers h^{l+1} = ReLU(GAT(z, <z,a_l>, <z,a_r>)) with z = h^l W^l, and the gradient of
    <gout, h^L> with respect to h^0, every W^l, a_l^l, a_r^l.  float64 except at the aggregation
    functions' float32 inputs.  `stored(x)` (default: identity) is applied wherever an implementation with
    narrower storage keeps a node array between two steps (z, the layer outputs, dz, dh), so that a bf16
    implementation can be compared on equal inputs: the score gradients are differences of nearly equal sums
    and amplify a rounding of their inputs."""
    st = (lambda x: x) if stored is None else stored
    L = len(weights)
    h = [np.asarray(h0, dtype=np.float64)]
    saved = []
    n = h[0].shape[0]
    H, F = np.asarray(a_l[0]).shape
    for l in range(L):
        z = st(linear(h[l], weights[l])).reshape(n, H, F)
        el, er = project(z, a_l[l], a_r[l])
        f = gat_fwd(indptr, indices, z.astype(np.float32), el.astype(np.float32), er.astype(np.float32), slope)
        saved.append((z, el, er, f))
        h.append(np.maximum(st(f.out), 0.0).reshape(n, H * F))
    g = np.asarray(gout, dtype=np.float64).reshape(n, H * F)
    dW, da_l, da_r = [None] * L, [None] * L, [None] * L
    for l in reversed(range(L)):
        z, el, er, f = saved[l]
        g = np.where(h[l + 1] > 0, g, 0.0)
        b = gat_bwd(indptr, indices, z.astype(np.float32), el.astype(np.float32), er.astype(np.float32), f.alpha,
                    g.reshape(n, H, F).astype(np.float32), slope)
        dz_add, da_l[l], da_r[l] = project_bwd(z, a_l[l], a_r[l], b.del_.astype(np.float32), b.der.astype(np.float32))
        dz = st(st(b.dfeat) + dz_add).reshape(n, H * F)
        dh, dW[l] = linear_bwd(h[l], weights[l], dz)
        g = st(dh)
    return dict(out=h[L], dh0=g, dW=dW, da_l=da_l, da_r=da_r)


# --------------------------------------------------------------------------------------
# message-flow pruning (Appendix B), plain numpy / Python loops
# --------------------------------------------------------------------------------------

def mfg_frontier(indptr, indices, need_out):
    """need_in[j] = 1 if j's input to the layer can reach a needed output: j is a needed row itself
    (its features enter its own score term) or the source of an in-edge of a needed row."""
    indptr, indices = _i64(indptr), _i32(indices)
    need_out = np.asarray(need_out).astype(bool)
    need_in = need_out.copy()
    for i in np.flatnonzero(need_out):
        need_in[indices[indptr[i]:indptr[i + 1]]] = True
    return need_in.astype(np.uint8)


def csr_filter_rows(indptr, indices, keep):
    """CSR in which the rows with keep[i] == 0 are empty; kept rows keep their column ids in order."""
    indptr, indices = _i64(indptr), _i32(indices)
    keep = np.asarray(keep).astype(bool)
    n = indptr.shape[0] - 1
    out_ptr = np.zeros(n + 1, dtype=np.int64)
    rows = []
    for i in range(n):
        row = indices[indptr[i]:indptr[i + 1]] if keep[i] else indices[:0]
        rows.append(row)
        out_ptr[i + 1] = out_ptr[i] + row.shape[0]
    out_idx = np.concatenate(rows).astype(np.int32) if rows else np.zeros(0, np.int32)
    return out_ptr, out_idx


def degree_order(n: int, src, dst):
    """Node order by total degree (edges as a source + edges as a destination), descending, ties by ascending id:
    order[new] = old, rank[old] = new.  Graph preparation for locality; the paper's counterpart is its offline
    partitioning (Sec. 4.2), not one of its algorithms."""
    src, dst = _i32(src), _i32(dst)
    deg = np.zeros(n, dtype=np.int64)
    for t in range(src.shape[0]):
        deg[src[t]] += 1
        deg[dst[t]] += 1
    order = np.array(sorted(range(n), key=lambda i: (-deg[i], i)), dtype=np.int32)
    rank = np.empty(n, dtype=np.int32)
    rank[order] = np.arange(n, dtype=np.int32)
    return order, rank


def spmm_scaled(indptr, indices, feat, src_scale=None, dst_scale=None):
    """out[i,:] = dst_scale[i] * sum over the in-edges (j -> i) of src_scale[j] * feat[j,:], float64
    (the propagation X <- diag(dst_scale) A diag(src_scale) X; a missing scale is all ones)."""
    feat = np.asarray(feat, dtype=np.float64)
    x = feat if src_scale is None else feat * np.asarray(src_scale, np.float64)[:, None]
    indptr, indices = _i64(indptr), _i32(indices)
    n = indptr.shape[0] - 1
    out = np.zeros((n, feat.shape[1]), dtype=np.float64)
    for i in range(n):
        cols = indices[indptr[i]:indptr[i + 1]]
        if cols.shape[0]:
            out[i] = x[cols].sum(axis=0)
    if dst_scale is not None:
        out *= np.asarray(dst_scale, np.float64)[:, None]
    return out


# --------------------------------------------------------------------------------------
# batch normalisation over the node dimension (Sec. 3.4), plain numpy float64
# --------------------------------------------------------------------------------------

def bn_moments(x):
    """(mean[c], m2[c] = sum_i (x[i,c] - mean[c])^2) over the rows of x."""
    x = np.asarray(x, dtype=np.float64)
    mean = x.mean(axis=0) if x.shape[0] else np.zeros(x.shape[1])
    return mean, ((x - mean) ** 2).sum(axis=0)


def bn_forward(x, eps=1e-5, gamma=None, beta=None):
    x = np.asarray(x, dtype=np.float64)
    mean, m2 = bn_moments(x)
    rstd = 1.0 / np.sqrt(m2 / max(x.shape[0], 1) + eps)
    y = (x - mean) * rstd
    if gamma is not None:
        y = y * np.asarray(gamma, np.float64)
    if beta is not None:
        y = y + np.asarray(beta, np.float64)
    return y, mean, rstd


def bn_backward(x, gy, eps=1e-5, gamma=None):
    """(gx, dgamma, dbeta) of y = xhat * gamma + beta for the upstream gradient gy."""
    x, gy = np.asarray(x, np.float64), np.asarray(gy, np.float64)
    n = x.shape[0]
    _, mean, rstd = bn_forward(x, eps)
    xhat = (x - mean) * rstd
    dbeta = gy.sum(axis=0)
    dgamma = (gy * xhat).sum(axis=0)
    g = 1.0 if gamma is None else np.asarray(gamma, np.float64)
    gx = g * rstd * (gy - dbeta / n - xhat * dgamma / n)
    return gx, dgamma, dbeta


# --------------------------------------------------------------------------------------
# dropout with a counter-based mask (SplitMix64), numpy
# --------------------------------------------------------------------------------------

def splitmix64(seed: int, count: int) -> np.ndarray:
    """The first `count` outputs of the SplitMix64 generator started at `seed` (uint64)."""
    with np.errstate(over="ignore"):
        k = np.arange(1, count + 1, dtype=np.uint64)
        z = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + k * np.uint64(0x9E3779B97F4A7C15)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        return z ^ (z >> np.uint64(31))


def dropout(x, p: float, seed: int):
    """y = x / (1 - p) where the element's 24-bit draw reaches floor(p * 2^24), else 0 (flattened order)."""
    x = np.asarray(x, dtype=np.float64)
    draws = (splitmix64(seed, x.size) >> np.uint64(40)).astype(np.int64).reshape(x.shape)
    keep = draws >= int(float(np.float32(p)) * 16777216.0)
    return np.where(keep, x * float(np.float32(1.0) / (np.float32(1.0) - np.float32(p))), 0.0), keep


# --------------------------------------------------------------------------------------
# the dense projection of a layer, numpy float64
# --------------------------------------------------------------------------------------

def linear(h, w):
    """z[i, o] = sum_k h[i, k] * w[k, o]."""
    return np.asarray(h, np.float64) @ np.asarray(w, np.float64)


def linear_bwd(h, w, dz):
    """(dh, dw) of z = h w for the upstream gradient dz."""
    h, w, dz = (np.asarray(x, np.float64) for x in (h, w, dz))
    return dz @ w.T, h.T @ dz


# --------------------------------------------------------------------------------------
# relational layer (Appendix A), plain numpy float64 written from the layer's equation:
# every neighbour's features are transformed by the relation's matrix, then averaged per
# relation and summed over the relations
# --------------------------------------------------------------------------------------

def rgcn_layer(graphs, h, weights):
    """z[i,:] = sum_r (1/|N^r_i|) sum_{j in N^r_i} h[j,:] W_r  (the argument of sigma in the appendix's first
    equation).  graphs: one (indptr, indices) CSR by destination per relation; weights: [R][d_in, d_out]."""
    h = np.asarray(h, np.float64)
    n = _i64(graphs[0][0]).shape[0] - 1
    d_out = np.asarray(weights[0]).shape[1]
    z = np.zeros((n, d_out), np.float64)
    for (indptr, indices), w in zip(graphs, weights):
        indptr, indices, w = _i64(indptr), _i32(indices), np.asarray(w, np.float64)
        for i in range(n):
            nb = indices[indptr[i]:indptr[i + 1]]
            if nb.shape[0]:
                z[i] += (h[nb] @ w).sum(axis=0) / nb.shape[0]
    return z


def rgcn_layer_bwd(graphs, h, weights, gz):
    """(dh, [dW_r]) for the upstream gradient gz of rgcn_layer's result: edge by edge,
    dW_r += h_j^T gz_i / |N^r_i| and dh_j += gz_i W_r^T / |N^r_i|."""
    h, gz = np.asarray(h, np.float64), np.asarray(gz, np.float64)
    dh = np.zeros_like(h)
    dws = []
    for (indptr, indices), w in zip(graphs, weights):
        indptr, indices, w = _i64(indptr), _i32(indices), np.asarray(w, np.float64)
        dw = np.zeros_like(w)
        back = gz @ w.T
        for i in range(indptr.shape[0] - 1):
            nb = indices[indptr[i]:indptr[i + 1]]
            if nb.shape[0]:
                c = 1.0 / nb.shape[0]
                dw += c * np.outer(h[nb].sum(axis=0), gz[i])
                np.add.at(dh, nb, c * back[i])
        dws.append(dw)
    return dh, dws


def rgcn_basis(a, V):
    """W_r = sum_b a[r,b] V_b (the appendix's second equation); a [R,B], V [B, ...]."""
    a, V = np.asarray(a, np.float64), np.asarray(V, np.float64)
    W = np.zeros((a.shape[0],) + V.shape[1:], np.float64)
    for r in range(a.shape[0]):
        for b in range(a.shape[1]):
            W[r] += a[r, b] * V[b]
    return W


def rgcn_basis_bwd(a, V, dW):
    """(da, dV) for the upstream gradient dW [R, ...] of rgcn_basis's result."""
    a, V, dW = np.asarray(a, np.float64), np.asarray(V, np.float64), np.asarray(dW, np.float64)
    da = np.zeros_like(a)
    dV = np.zeros_like(V)
    for r in range(a.shape[0]):
        for b in range(a.shape[1]):
            da[r, b] = float((dW[r] * V[b]).sum())
            dV[b] += a[r, b] * dW[r]
    return da, dV


# --------------------------------------------------------------------------------------
# GraphSage layer (Eq. 2), plain numpy float64 in the equation's order: project every
# node (z = h W), average the neighbours' z, add the residual term h W_res
# --------------------------------------------------------------------------------------

def sage_layer(indptr, indices, h, w, w_res):
    """pre[i,:] = h[i,:] W_res + (1/|N(i)|) sum_{j in N(i)} (h W)[j,:]  (the argument of sigma in Eq. 2;
    the mean of an empty neighbourhood is 0)."""
    h, w, w_res = (np.asarray(x, np.float64) for x in (h, w, w_res))
    indptr, indices = _i64(indptr), _i32(indices)
    z = h @ w
    pre = h @ w_res
    for i in range(indptr.shape[0] - 1):
        nb = indices[indptr[i]:indptr[i + 1]]
        if nb.shape[0]:
            pre[i] += z[nb].sum(axis=0) / nb.shape[0]
    return pre


def sage_layer_bwd(indptr, indices, h, w, w_res, g):
    """(dh, dW, dW_res) for the upstream gradient g of sage_layer's result."""
    h, w, w_res, g = (np.asarray(x, np.float64) for x in (h, w, w_res, g))
    indptr, indices = _i64(indptr), _i32(indices)
    dz = np.zeros((h.shape[0], w.shape[1]), np.float64)  # gradient of z = h W: every in-edge hands back g_i / |N(i)|
    for i in range(indptr.shape[0] - 1):
        nb = indices[indptr[i]:indptr[i + 1]]
        if nb.shape[0]:
            np.add.at(dz, nb, g[i] / nb.shape[0])
    return g @ w_res.T + dz @ w.T, h.T @ dz, h.T @ g


def propagate(indptr, indices, x0, alpha: float, iters: int, src_scale=None, dst_scale=None):
    """X_iters of the iteration X_0 = x0, X_{t+1} = (1 - alpha) x0 + alpha S X_t with S = diag(dst_scale) A
    diag(src_scale) (the propagation of Sec. 4.2's label post-processing), float64."""
    x0 = np.asarray(x0, np.float64)
    x = x0.copy()
    for _ in range(iters):
        x = (1.0 - alpha) * x0 + alpha * spmm_scaled(indptr, indices, x, src_scale, dst_scale)
    return x

"""Convenience layer over the binding: allocates device tensors with torch and calls libsar.

Nothing is computed here; every step (graph build, transpose, split, long-row plan, forward,
backward, sum aggregation) is a call into the C-ABI library.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import torch

from . import binding as B

DEFAULT_THRESHOLD = 256    # rows of the CSR with more edges are cut into segments of this many edges
DEFAULT_T_THRESHOLD = 256  # the same for the CSC (its own knob: the two plans are independent)


def _workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def build_plan(n_rows: int, indptr: torch.Tensor, threshold: int) -> Optional[B.Split]:
    """Long-row plan of one CSR.  A plan without long rows (n_long = 0) still tells the library that no row
    is longer than `threshold`."""
    dev = indptr.device
    counts = torch.zeros(2, dtype=torch.int64, device=dev)
    n_long, n_seg = B.sar_plan_count(n_rows, indptr, threshold, counts)
    if n_long == 0:
        return B.Split(threshold, 0, 0, torch.empty(0, dtype=torch.int32, device=dev),
                       torch.zeros(1, dtype=torch.int64, device=dev))
    long_row = torch.empty(n_long, dtype=torch.int32, device=dev)
    long_seg = torch.empty(n_long + 1, dtype=torch.int64, device=dev)
    ws = _workspace(B.sar_graph_workspace_bytes(0, n_rows), dev)
    B.sar_plan_fill(n_rows, indptr, threshold, n_long, long_row, long_seg, ws)
    return B.Split(threshold, n_long, n_seg, long_row, long_seg)


@dataclass
class Graph:
    """A graph on the device: the un-split CSR/CSC (`whole`) and, optionally, its K source partitions."""
    n: int
    nnz: int
    whole: B.Part
    k: int = 1
    bounds: List[int] = field(default_factory=list)
    parts: List[B.Part] = field(default_factory=list)
    order: Optional[torch.Tensor] = None    # reorder="degree": the graph's node i is the caller's node order[i]
    rank: Optional[torch.Tensor] = None     # ... and the caller's node j is the graph's node rank[j]

    def to_internal(self, x: torch.Tensor) -> torch.Tensor:
        """A node array [n, ...] in the caller's numbering -> the graph's numbering (a copy; x itself when the graph
        keeps the caller's numbering)."""
        if self.order is None:
            return x
        out = torch.empty_like(x)
        B.sar_permute_rows(self.order, x.contiguous(), out)
        return out

    def to_external(self, x: torch.Tensor) -> torch.Tensor:
        """The inverse of to_internal."""
        if self.rank is None:
            return x
        out = torch.empty_like(x)
        B.sar_permute_rows(self.rank, x.contiguous(), out)
        return out

    @staticmethod
    def from_coo(n: int, src: torch.Tensor, dst: torch.Tensor, k: int = 1, threshold: int = DEFAULT_THRESHOLD,
                 build_parts: bool = False, t_threshold: Optional[int] = None,
                 reorder: Optional[str] = None) -> "Graph":
        """src[t] -> dst[t] int32 CUDA tensors.  Builds CSR by destination, its transpose, the long-row
        plans and (build_parts) the K per-partition sub-graphs with local source ids.
        reorder="degree": the nodes are renumbered by total degree first (sar_degree_order); every node array then
        enters through to_internal and leaves through to_external."""
        dev = src.device
        nnz = src.numel()
        order = rank = None
        if reorder == "degree":
            order = torch.empty(n, dtype=torch.int32, device=dev)
            rank = torch.empty(n, dtype=torch.int32, device=dev)
            B.sar_degree_order(n, src, dst, order, rank, _workspace(B.sar_degree_order_workspace_bytes(n), dev))
            src2, dst2 = torch.empty_like(src), torch.empty_like(dst)
            B.sar_relabel(src, rank, src2)
            B.sar_relabel(dst, rank, dst2)
            src, dst = src2, dst2
        elif reorder is not None:
            raise ValueError(f"unknown reorder {reorder!r}")
        ws = _workspace(B.sar_graph_workspace_bytes(nnz, n), dev)
        indptr = torch.empty(n + 1, dtype=torch.int64, device=dev)
        indices = torch.empty(nnz, dtype=torch.int32, device=dev)
        B.sar_csr_from_coo(n, n, dst, src, indptr, indices, ws)
        t_indptr = torch.empty(n + 1, dtype=torch.int64, device=dev)
        t_indices = torch.empty(nnz, dtype=torch.int32, device=dev)
        B.sar_csr_from_coo(n, n, src, dst, t_indptr, t_indices, ws)
        if t_threshold is None:   # the CSC's plan has its own threshold
            t_threshold = DEFAULT_T_THRESHOLD if threshold == DEFAULT_THRESHOLD else threshold
        split = build_plan(n, indptr, threshold) if threshold else None
        t_split = build_plan(n, t_indptr, t_threshold) if t_threshold else None
        whole = B.Part(n, n, indptr, indices, t_indptr, t_indices, split, t_split)
        g = Graph(n=n, nnz=nnz, whole=whole, k=k, bounds=B.sar_partition_bounds(n, k), order=order, rank=rank)
        if build_parts:
            g.parts = split_parts(whole, g.bounds, threshold, ws)
        return g


def graph_from_csr(n: int, indptr: torch.Tensor, indices: torch.Tensor, k: int = 1,
                   threshold: int = DEFAULT_THRESHOLD) -> Graph:
    """A Graph from a CSR by destination already on the device (n rows, n columns)."""
    dev = indptr.device
    nnz = indices.numel()
    ws = _workspace(B.sar_graph_workspace_bytes(nnz, n), dev)
    t_indptr = torch.empty(n + 1, dtype=torch.int64, device=dev)
    t_indices = torch.empty(nnz, dtype=torch.int32, device=dev)
    B.sar_csr_transpose(n, n, indptr, indices, t_indptr, t_indices, ws)
    split = build_plan(n, indptr, threshold) if threshold else None
    t_split = build_plan(n, t_indptr, threshold) if threshold else None
    whole = B.Part(n, n, indptr, indices, t_indptr, t_indices, split, t_split)
    return Graph(n=n, nnz=nnz, whole=whole, k=k, bounds=B.sar_partition_bounds(n, k))


def filter_rows(g: Graph, keep: torch.Tensor, threshold: int = DEFAULT_THRESHOLD) -> Graph:
    """The graph in which only the destinations with keep[i] != 0 keep their in-edges."""
    dev = keep.device
    ws = _workspace(B.sar_graph_workspace_bytes(0, g.n), dev)
    indptr = torch.empty(g.n + 1, dtype=torch.int64, device=dev)
    B.sar_csr_filter_rows_indptr(g.n, g.whole.indptr, keep, indptr, ws)
    nnz = int(indptr[-1].item())
    indices = torch.empty(nnz, dtype=torch.int32, device=dev)
    if nnz > 0:
        B.sar_csr_filter_rows_indices(g.n, g.whole.indptr, g.whole.indices, indptr, indices)
    return graph_from_csr(g.n, indptr, indices, k=g.k, threshold=threshold)


def mfg_layers(g: Graph, labelled: torch.Tensor, layers: int, threshold: int = DEFAULT_THRESHOLD):
    """Message-flow pruning for a stack of `layers` layers whose loss reads only the nodes with
    labelled[i] != 0 (uint8 [n]).  Returns (graphs, need): graphs[l] is the graph layer l aggregates over
    (only the rows whose output still matters keep their edges), need[l] marks the nodes whose input to
    layer l matters (need[layers] = labelled)."""
    need = [None] * (layers + 1)
    graphs = [None] * layers
    need[layers] = labelled.to(torch.uint8).contiguous()
    for l in reversed(range(layers)):
        graphs[l] = filter_rows(g, need[l + 1], threshold)
        need[l] = torch.empty(g.n, dtype=torch.uint8, device=labelled.device)
        B.sar_mfg_frontier(g.n, g.whole.indptr, g.whole.indices, need[l + 1], need[l])
    return graphs, need


def split_parts(whole: B.Part, bounds: List[int], threshold: int, ws: Optional[torch.Tensor] = None) -> List[B.Part]:
    """The K sub-graphs G_{p,q}: CSR with local source ids (split on the device) and CSC slices."""
    dev = whole.indptr.device
    n, k = whole.n_dst, len(bounds) - 1
    if ws is None:
        ws = _workspace(B.sar_graph_workspace_bytes(whole.nnz, n), dev)
    indptr_all = torch.empty((k, n + 1), dtype=torch.int64, device=dev)
    B.sar_csr_split_indptr(n, whole.indptr, whole.indices, bounds, indptr_all, ws)
    nnz_q = indptr_all[:, n].tolist()
    nnz_off = [0]
    for c in nnz_q:
        nnz_off.append(nnz_off[-1] + int(c))
    indices_all = torch.empty(max(nnz_off[-1], 1), dtype=torch.int32, device=dev)
    B.sar_csr_split_indices(n, whole.indptr, whole.indices, bounds, indptr_all, nnz_off, indices_all)
    parts = []
    for q in range(k):
        s0, s1 = bounds[q], bounds[q + 1]
        ip = indptr_all[q]
        idx = indices_all[nnz_off[q]:nnz_off[q + 1]]
        # CSC of partition q: the sources s0..s1 of the whole CSC, offsets counted from the slice's first edge
        t_ip = torch.empty(s1 - s0 + 1, dtype=torch.int64, device=dev)
        B.sar_csc_slice_indptr(s0, s1, whole.t_indptr, t_ip)
        e0 = int(whole.t_indptr[s0])
        t_idx = whole.t_indices[e0:e0 + nnz_q[q]]
        split = build_plan(n, ip, threshold) if threshold else None
        t_split = build_plan(s1 - s0, t_ip, threshold) if threshold else None
        parts.append(B.Part(n, s1 - s0, ip, idx, t_ip, t_idx, split, t_split, nnz=nnz_q[q]))
    return parts


# ----------------------------------------------------------------------------------------------

def gat_workspace(part: B.Part, H: int, F: int, dtype: torch.dtype) -> torch.Tensor:
    code = B.SAR_BF16 if dtype == torch.bfloat16 else B.SAR_F32
    return _workspace(B.sar_gat_workspace_bytes(part, H, F, code), part.indptr.device)


def gat_forward(g: Graph, feat: torch.Tensor, el: torch.Tensor, er: torch.Tensor, slope: float,
                workspace: Optional[torch.Tensor] = None, mode: str = "fused", keep_numerator: bool = False,
                relu_out: bool = False):
    """Forward over the K partitions.  mode "fused": one row-stationary walk over the un-split graph, the
    partitions being slices of the arrays (sar_gat_fwd_fused);
    mode "stateful": K calls of sar_gat_fwd with the running state in global memory (Algorithm 1).
    keep_numerator (stateful mode): returns (out, m, d, acc) with the complete float32 numerator in acc,
    which gat_backward can take in place of `out` for the row dot.
    relu_out: out = max(out, 0), the ReLU that closes the layer, applied where the aggregate is finalised."""
    n, H, F = feat.shape
    dev = feat.device
    m = torch.empty((g.n, H), dtype=torch.float32, device=dev)
    d = torch.empty((g.n, H), dtype=torch.float32, device=dev)
    out = torch.empty((g.n, H, F), dtype=feat.dtype, device=dev)
    if mode == "fused":
        ws = workspace if workspace is not None else gat_workspace(g.whole, H, F, feat.dtype)
        if relu_out:   # the un-split graph as one partition holding all sources
            B.sar_gat_fwd(g.whole, feat, el, er, H, F, slope, B.SAR_FIRST | B.SAR_LAST | B.SAR_RELU_OUT, None, m, d, out, ws)
        else:
            B.sar_gat_fwd_fused(g.whole, g.bounds, feat, el, er, H, F, slope, m, d, out, ws)
        return out, m, d
    assert g.parts, "stateful mode needs Graph.from_coo(..., build_parts=True)"
    acc = torch.empty((g.n, H, F), dtype=torch.float32, device=dev) if (g.k > 1 or keep_numerator) else None
    for q, part in enumerate(g.parts):
        flags = (B.SAR_FIRST if q == 0 else 0) | (B.SAR_LAST if q == g.k - 1 else 0)
        if keep_numerator and q == g.k - 1:
            flags |= B.SAR_KEEP_NUMERATOR
        if relu_out and q == g.k - 1:
            flags |= B.SAR_RELU_OUT
        ws = gat_workspace(part, H, F, feat.dtype)
        s0, s1 = g.bounds[q], g.bounds[q + 1]
        B.sar_gat_fwd(part, feat[s0:s1], el, er[s0:s1], H, F, slope, flags, acc, m, d, out, ws)
    return (out, m, d, acc) if keep_numerator else (out, m, d)


def gat_backward(g: Graph, feat: torch.Tensor, el: torch.Tensor, er: torch.Tensor, m: torch.Tensor,
                 d: torch.Tensor, gout: torch.Tensor, slope: float, out: Optional[torch.Tensor] = None,
                 workspace: Optional[torch.Tensor] = None, mode: str = "fused", acc: Optional[torch.Tensor] = None):
    """Backward over the K partitions; returns (dfeat, del, der).  "stateful" needs `out` or the complete
    float32 numerator `acc` (for the row dot) and runs sar_gat_bwd_prepare followed by K calls of sar_gat_bwd."""
    n, H, F = feat.shape
    dev = feat.device
    dfeat = torch.empty_like(feat)
    del_ = torch.empty((g.n, H), dtype=torch.float32, device=dev)
    der = torch.empty((g.n, H), dtype=torch.float32, device=dev)
    if mode == "fused":
        ws = workspace if workspace is not None else gat_workspace(g.whole, H, F, feat.dtype)
        B.sar_gat_bwd_fused(g.whole, g.bounds, feat, el, er, m, d, gout, H, F, slope, dfeat, del_, der, ws)
        return dfeat, del_, der
    assert g.parts and (out is not None or acc is not None)
    nbytes = max(B.sar_gat_workspace_bytes(p, H, F, B._dtype(feat)) for p in g.parts)
    ws = _workspace(nbytes, dev)
    if acc is not None:
        B.sar_gat_bwd_prepare(g.n, H, F, acc, True, gout, el, m, d, None, ws)
    else:
        B.sar_gat_bwd_prepare(g.n, H, F, out, False, gout, el, m, d, None, ws)
    for q, part in enumerate(g.parts):
        flags = (B.SAR_FIRST if q == 0 else 0) | (B.SAR_LAST if q == g.k - 1 else 0)
        s0, s1 = g.bounds[q], g.bounds[q + 1]
        B.sar_gat_bwd(part, feat[s0:s1], el, er[s0:s1], m, d, gout, H, F, slope, flags, dfeat[s0:s1], del_,
                      der[s0:s1], ws)
    return dfeat, del_, der


def spmm_sum(part: B.Part, feat: torch.Tensor, mean: bool = False, deg_total: Optional[torch.Tensor] = None):
    """out[i,:] = sum (or mean) of feat over the in-edges of i for one partition holding all sources."""
    F = feat.shape[1]
    out = torch.empty((part.n_dst, F), dtype=feat.dtype, device=feat.device)
    ws = _workspace(B.sar_spmm_workspace_bytes(part, F, B._dtype(feat)), feat.device)
    flags = B.SAR_FIRST | B.SAR_LAST | (B.SAR_MEAN if mean else 0)
    B.sar_spmm_agg(part, feat, F, flags, deg_total, out, ws)
    return out


# ----------------------------------------------------------------------------------------------
# the layer around the aggregation: z' = GAT(z, <z,a_l>, <z,a_r>) with z = ReLU(previous layer's
# output) (Eq. 3 with f_node of Eq. 1 taken as a ReLU); argument marshalling only, every step is a
# library call.

def gat_layer_forward(g: Graph, z: torch.Tensor, a_l: torch.Tensor, a_r: torch.Tensor, slope: float,
                      workspace: Optional[torch.Tensor] = None, relu_input: bool = False):
    """Returns (out, saved): out is the layer's aggregation output (before any activation) and
    saved = (el, er, m, d) is what the backward pass needs besides z.  relu_input=True first applies
    z = max(z, 0) in place, inside the projection kernel."""
    n, H, F = z.shape
    el = torch.empty((n, H), dtype=torch.float32, device=z.device)
    er = torch.empty_like(el)
    B.sar_gat_project(z, a_l, a_r, el, er, B.SAR_GLUE_RELU if relu_input else 0)
    out, m, d = gat_forward(g, z, el, er, slope, workspace)
    return out, (el, er, m, d)


def gat_layer_backward(g: Graph, z: torch.Tensor, a_l: torch.Tensor, a_r: torch.Tensor, saved, gout: torch.Tensor,
                       slope: float, workspace: Optional[torch.Tensor] = None, relu_input: bool = False):
    """Returns (dz, da_l, da_r); with relu_input=True dz is the gradient with respect to the input
    before its ReLU (zero where z <= 0)."""
    n, H, F = z.shape
    el, er, m, d = saved
    dz, del_, der = gat_backward(g, z, el, er, m, d, gout, slope, workspace=workspace)
    da_l = torch.empty((H, F), dtype=torch.float32, device=z.device)
    da_r = torch.empty_like(da_l)
    ws = _workspace(B.sar_gat_project_workspace_bytes(H, F), z.device)
    B.sar_gat_project_bwd(z, a_l, a_r, del_, der, dz, da_l, da_r, ws, B.SAR_GLUE_RELU if relu_input else 0)
    return dz, da_l, da_r


def spmm_scaled(part: B.Part, feat: torch.Tensor, src_scale: Optional[torch.Tensor] = None,
                dst_scale: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None, first: bool = True):
    """out[i,:] (+)= dst_scale[i] * sum over the in-edges of i of src_scale[j] * feat[j,:] (one partition)."""
    F = feat.shape[1]
    if out is None:
        out = torch.empty((part.n_dst, F), dtype=feat.dtype, device=feat.device)
    ws = _workspace(B.sar_spmm_workspace_bytes(part, F, B._dtype(feat)), feat.device)
    B.sar_spmm_agg_scaled(part, feat, F, (B.SAR_FIRST if first else 0) | B.SAR_LAST, src_scale, dst_scale, out, ws)
    return out


# ----------------------------------------------------------------------------------------------
# batch normalisation over the node dimension (Sec. 3.4); with `group` the statistics are combined across
# the workers of a torch.distributed process group (each holds some of the rows): a few floats per column.

def _gather_rows(row: torch.Tensor, group) -> torch.Tensor:
    """Every worker's copy of `row` (a flat tensor), stacked in rank order, on the HOST."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    parts = [torch.empty_like(row) for _ in range(world)]
    dist.all_gather(parts, row.contiguous(), group=group)
    return torch.stack(parts).cpu()


def combine_moments(n_local: int, mean: torch.Tensor, m2: torch.Tensor, group=None):
    """(n, mean, m2 = sum of squared deviations) of the local rows -> the same for all rows of all workers.
    torch.distributed only moves the triples; the rule of Sec. 3.4 is the library's sar_bn_combine_moments."""
    if group is None:
        return n_local, mean, m2
    n_r = _gather_rows(torch.tensor([int(n_local)], dtype=torch.int64, device=mean.device), group)[:, 0].tolist()
    rows = _gather_rows(torch.cat([mean.float(), m2.float()]), group)
    C = mean.numel()
    n_all, mean_all, m2_all = B.sar_bn_combine_moments(n_r, rows[:, :C], rows[:, C:])
    return n_all, mean_all.to(mean.device), m2_all.to(mean.device)


def combine_sums(tensors, group=None):
    """Element-wise sums over the workers (the backward statistics), by the library's sar_bn_combine_sums."""
    if group is None:
        return tensors
    rows = _gather_rows(torch.cat([t.float().flatten() for t in tensors]), group)
    flat = B.sar_bn_combine_sums(rows)
    out, o = [], 0
    for t in tensors:
        out.append(flat[o:o + t.numel()].reshape(t.shape).to(device=t.device, dtype=t.dtype))
        o += t.numel()
    return out


def bn_forward(x: torch.Tensor, eps: float = 1e-5, gamma: Optional[torch.Tensor] = None,
               beta: Optional[torch.Tensor] = None, group=None):
    """Returns (y, saved) with saved = (mean, rstd, n_all) for bn_backward.  x is [n_local, C]."""
    n, C = x.shape
    dev = x.device
    ws = _workspace(B.sar_bn_workspace_bytes(C), dev)
    mean = torch.empty(C, dtype=torch.float32, device=dev)
    m2 = torch.empty(C, dtype=torch.float32, device=dev)
    B.sar_bn_stats(x, mean, m2, ws)
    n_all, mean, m2 = combine_moments(n, mean, m2, group)
    rstd = torch.empty_like(m2)
    B.sar_bn_rstd(m2, max(n_all, 1), eps, rstd)
    y = torch.empty_like(x)
    B.sar_bn_apply(x, mean, rstd, gamma, beta, y)
    return y, (mean, rstd, n_all)


def bn_backward(x: torch.Tensor, gy: torch.Tensor, saved, gamma: Optional[torch.Tensor] = None, group=None):
    """Returns (gx, dgamma, dbeta); dgamma and dbeta are already summed over the workers."""
    n, C = x.shape
    dev = x.device
    mean, rstd, n_all = saved
    ws = _workspace(B.sar_bn_workspace_bytes(C), dev)
    s0 = torch.empty(C, dtype=torch.float32, device=dev)
    s1 = torch.empty(C, dtype=torch.float32, device=dev)
    B.sar_bn_bwd_stats(x, mean, rstd, gy, s0, s1, ws)
    s0, s1 = combine_sums([s0, s1], group)
    gx = torch.empty_like(x)
    B.sar_bn_bwd_apply(x, mean, rstd, gamma, gy, s0, s1, 1.0 / max(n_all, 1), gx)
    return gx, s1, s0


# ----------------------------------------------------------------------------------------------
# whole layers: h' = GAT(z, <z,a_l>, <z,a_r>) with z = ReLU?(h) W  (bf16; the dense projection runs on the
# tensor cores).  Marshalling only.

def full_layer_forward(g: Graph, h: torch.Tensor, W: torch.Tensor, a_l: torch.Tensor, a_r: torch.Tensor, slope: float,
                       relu_input: bool = False):
    """h [n, D_in], W [D_in, H*F] (bf16), a_l / a_r [H, F] float32.  Returns (out [n,H,F], saved).
    relu_input=True first applies h = max(h, 0) in place (the activation that closes the previous layer)."""
    n = h.shape[0]
    H, F = a_l.shape
    if relu_input:
        B.sar_relu(h)
    z = torch.empty((n, H, F), dtype=h.dtype, device=h.device)
    ws = _workspace(B.sar_linear_workspace_bytes(n, h.shape[1], H * F), h.device)
    el = torch.empty((n, H), dtype=torch.float32, device=h.device)
    er = torch.empty_like(el)
    if F % 8 == 0 and 128 % F == 0:   # the scores leave the projection's epilogue
        B.sar_linear_project(h, W, a_l, a_r, z.view(n, H * F), el, er, ws)
    else:
        B.sar_linear(h, W, z.view(n, H * F), ws)
        B.sar_gat_project(z, a_l, a_r, el, er, 0)
    out, m, d = gat_forward(g, z, el, er, slope)
    return out, (z, el, er, m, d)


def full_layer_backward(g: Graph, h: torch.Tensor, W: torch.Tensor, a_l: torch.Tensor, a_r: torch.Tensor, saved,
                        gout: torch.Tensor, slope: float, relu_input: bool = False):
    """Returns (dh [n, D_in], dW [D_in, H*F] float32, da_l, da_r); with relu_input=True dh is the gradient
    before the input's ReLU (h must be the array full_layer_forward left, i.e. already max(h, 0))."""
    n, d_in = h.shape
    H, F = a_l.shape
    z, el, er, m, d = saved
    dz, del_, der = gat_backward(g, z, el, er, m, d, gout, slope)
    da_l = torch.empty((H, F), dtype=torch.float32, device=h.device)
    da_r = torch.empty_like(da_l)
    B.sar_gat_project_bwd(z, a_l, a_r, del_, der, dz, da_l, da_r, _workspace(B.sar_gat_project_workspace_bytes(H, F), h.device), 0)
    ws = _workspace(B.sar_linear_workspace_bytes(n, d_in, H * F), h.device)
    dW = torch.empty((d_in, H * F), dtype=torch.float32, device=h.device)
    B.sar_linear_bwd_weight(h, dz.view(n, H * F), dW, ws)
    dh = torch.empty_like(h)
    if relu_input:   # the mask of the input's ReLU is applied in the GEMM's epilogue
        B.sar_linear_bwd_input_relu(dz.view(n, H * F), W, h, dh, ws)
    else:
        B.sar_linear_bwd_input(dz.view(n, H * F), W, dh, ws)
    return dh, dW, da_l, da_r


# ----------------------------------------------------------------------------------------------
# relational layer (Appendix A): z_i = sum_r (1/|N^r_i|) sum_{j in N^r_i} h_j W_r, one Graph per relation.
# Per relation the mean aggregate of h is built partition by partition and multiplied by W_r into z; the
# backward pass rebuilds the aggregate from h instead of keeping R of them.  Marshalling only.

def rgcn_inv_degrees(graphs: List[Graph]) -> List[torch.Tensor]:
    """Per relation the factor 1/|N^r_i| of every node (0 without in-edges), float32 [n]."""
    out = []
    for g in graphs:
        inv = torch.empty(g.n, dtype=torch.float32, device=g.whole.indptr.device)
        B.sar_degree_scale(g.whole.indptr, -1.0, inv)
        out.append(inv)
    return out


def _pieces(g: Graph):
    return (g.parts, g.bounds) if g.parts else ([g.whole], [0, g.n])


def _rgcn_aggregate(g: Graph, h: torch.Tensor, inv: torch.Tensor, agg: torch.Tensor) -> None:
    parts, bounds = _pieces(g)
    for q, part in enumerate(parts):
        flags = (B.SAR_FIRST if q == 0 else 0) | (B.SAR_LAST if q == len(parts) - 1 else 0)
        ws = _workspace(B.sar_spmm_workspace_bytes(part, h.shape[1], B._dtype(h)), h.device)
        B.sar_spmm_agg_scaled(part, h[bounds[q]:bounds[q + 1]], h.shape[1], flags, None, inv, agg, ws)


def rgcn_layer_forward(graphs: List[Graph], h: torch.Tensor, W: torch.Tensor, inv: Optional[List[torch.Tensor]] = None):
    """h [n, d_in] bf16, W [R, d_in, d_out] bf16.  Returns (z [n, d_out] before the activation, inv)."""
    n, d_in = h.shape
    d_out = W.shape[2]
    inv = inv if inv is not None else rgcn_inv_degrees(graphs)
    agg = torch.empty_like(h)
    z = torch.empty((n, d_out), dtype=h.dtype, device=h.device)
    ws = _workspace(B.sar_linear_workspace_bytes(n, d_in, d_out), h.device)
    for r, g in enumerate(graphs):
        _rgcn_aggregate(g, h, inv[r], agg)
        (B.sar_linear if r == 0 else B.sar_linear_accumulate)(agg, W[r], z, ws)
    return z, inv


def rgcn_layer_backward(graphs: List[Graph], h: torch.Tensor, W: torch.Tensor, inv: List[torch.Tensor], gz: torch.Tensor):
    """Returns (dh [n, d_in], dW [R, d_in, d_out] float32) for the upstream gradient gz [n, d_out]."""
    n, d_in = h.shape
    d_out = W.shape[2]
    agg = torch.empty_like(h)
    dagg = torch.empty_like(h)
    dh = torch.empty_like(h)
    dW = torch.empty((len(graphs), d_in, d_out), dtype=torch.float32, device=h.device)
    ws = _workspace(B.sar_linear_workspace_bytes(n, d_in, d_out), h.device)
    for r, g in enumerate(graphs):
        _rgcn_aggregate(g, h, inv[r], agg)  # rebuilt from the input features
        B.sar_linear_bwd_weight(agg, gz, dW[r], ws)
        B.sar_linear_bwd_input(gz, W[r], dagg, ws)
        parts, bounds = _pieces(g)
        for q, part in enumerate(parts):  # the partition's sources receive from all destinations
            tp = part.transposed()
            sws = _workspace(B.sar_spmm_workspace_bytes(tp, d_in, B._dtype(h)), h.device)
            B.sar_spmm_agg_scaled(tp, dagg, d_in, (B.SAR_FIRST if r == 0 else 0) | B.SAR_LAST, inv[r], None,
                                  dh[bounds[q]:bounds[q + 1]], sws)
    return dh, dW


def rgcn_basis_weights(a: torch.Tensor, V: torch.Tensor, dtype: torch.dtype = torch.bfloat16) -> torch.Tensor:
    """W [R, d_in, d_out] = sum_b a[r,b] V[b] from a [R,B] and V [B, d_in, d_out] (float32)."""
    W = torch.empty((a.shape[0],) + tuple(V.shape[1:]), dtype=dtype, device=V.device)
    B.sar_rgcn_basis(a, V, W)
    return W


def rgcn_basis_backward(a: torch.Tensor, V: torch.Tensor, dW: torch.Tensor):
    """(da [R,B], dV like V) from dW [R, d_in, d_out] float32."""
    da = torch.empty_like(a)
    dV = torch.empty_like(V)
    B.sar_rgcn_basis_bwd(a, V, dW, da, dV)
    return da, dV


# ----------------------------------------------------------------------------------------------
# GraphSage layer (Eq. 2): pre_i = h_i W_res + mean_{j in N(i)} h_j W.  The mean commutes with W, so the
# neighbours' raw features are averaged first (one aggregation of d_in columns) and the two projections
# accumulate into one output.  The aggregation has no parameters ("case 1" of Sec. 3.2): the backward pass
# needs no source features, only the graph.  Marshalling only.

def sage_layer_forward(g: Graph, h: torch.Tensor, W: torch.Tensor, W_res: torch.Tensor, inv: Optional[torch.Tensor] = None):
    """h [n, d_in], W and W_res [d_in, d_out] (bf16).  Returns (pre [n, d_out] before the activation, saved)."""
    n, d_in = h.shape
    d_out = W.shape[1]
    if inv is None:
        inv = rgcn_inv_degrees([g])[0]
    agg = torch.empty_like(h)
    _rgcn_aggregate(g, h, inv, agg)
    pre = torch.empty((n, d_out), dtype=h.dtype, device=h.device)
    ws = _workspace(B.sar_linear_workspace_bytes(n, d_in, d_out), h.device)
    B.sar_linear(h, W_res, pre, ws)
    B.sar_linear_accumulate(agg, W, pre, ws)
    return pre, (agg, inv)


def sage_layer_backward(g: Graph, h: torch.Tensor, W: torch.Tensor, W_res: torch.Tensor, saved, gpre: torch.Tensor):
    """Returns (dh [n, d_in], dW, dW_res [d_in, d_out] float32) for the upstream gradient gpre [n, d_out]."""
    n, d_in = h.shape
    d_out = W.shape[1]
    agg, inv = saved
    ws = _workspace(B.sar_linear_workspace_bytes(n, d_in, d_out), h.device)
    dW = torch.empty((d_in, d_out), dtype=torch.float32, device=h.device)
    dW_res = torch.empty_like(dW)
    B.sar_linear_bwd_weight(agg, gpre, dW, ws)
    B.sar_linear_bwd_weight(h, gpre, dW_res, ws)
    dh = torch.empty_like(h)
    B.sar_linear_bwd_input(gpre, W_res, dh, ws)       # the residual path
    dagg = torch.empty_like(h)
    B.sar_linear_bwd_input(gpre, W, dagg, ws)
    parts, bounds = _pieces(g)
    for q, part in enumerate(parts):                  # plus what every out-edge hands back: dagg_i / |N(i)|
        tp = part.transposed()
        sws = _workspace(B.sar_spmm_workspace_bytes(tp, d_in, B._dtype(h)), h.device)
        B.sar_spmm_agg_scaled(tp, dagg, d_in, B.SAR_LAST, inv, None, dh[bounds[q]:bounds[q + 1]], sws)
    return dh, dW, dW_res


# ----------------------------------------------------------------------------------------------
# iterated propagation X <- (1 - alpha) X0 + alpha S X with S = diag(dst_scale) A diag(src_scale): the smoothing /
# error-correction steps of the label-propagation post-processing the paper combines SAR with (Sec. 4.2).

def sym_norm_scales(g: Graph):
    """(src_scale, dst_scale) = (out-degree^-1/2, in-degree^-1/2), the symmetric normalisation (0 for degree 0)."""
    dev = g.whole.indptr.device
    dst = torch.empty(g.n, dtype=torch.float32, device=dev)
    src = torch.empty(g.n, dtype=torch.float32, device=dev)
    B.sar_degree_scale(g.whole.indptr, -0.5, dst)
    B.sar_degree_scale(g.whole.t_indptr, -0.5, src)
    return src, dst


def propagate(g: Graph, x0: torch.Tensor, alpha: float, iters: int, src_scale: Optional[torch.Tensor] = None,
              dst_scale: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Returns X_iters with X_0 = x0 and X_{t+1} = (1 - alpha) x0 + alpha S X_t; x0 [n, F]."""
    x = x0.clone()
    nxt = torch.empty_like(x0)
    parts, bounds = _pieces(g)
    F = x0.shape[1]
    for _ in range(iters):
        for q, part in enumerate(parts):
            flags = (B.SAR_FIRST if q == 0 else 0) | (B.SAR_LAST if q == len(parts) - 1 else 0)
            ws = _workspace(B.sar_spmm_workspace_bytes(part, F, B._dtype(x0)), x0.device)
            sq = None if src_scale is None else src_scale[bounds[q]:bounds[q + 1]]
            B.sar_spmm_agg_scaled(part, x[bounds[q]:bounds[q + 1]], F, flags, sq, dst_scale, nxt, ws)
        B.sar_axpby(1.0 - alpha, x0, alpha, nxt)
        x, nxt = nxt, x
    return x

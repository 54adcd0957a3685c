"""ctypes binding of libsar.so (include/sar.h): argument marshalling only.

Every function here has the name of the C entry point it calls and does nothing but turn
torch CUDA tensors into pointers (PyTorch supplies device memory and the current stream) and
check the returned status.  There is no Python or CPU fallback: if the library cannot be loaded
the import of this module's functions fails loudly.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_float, c_int32, c_int64, c_size_t, c_uint32, c_void_p
from typing import Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libsar.so")

SAR_OK = 0
SAR_F32, SAR_BF16 = 0, 1
SAR_FIRST, SAR_LAST, SAR_MEAN, SAR_KEEP_NUMERATOR, SAR_RELU_OUT = 1, 2, 4, 8, 16
SAR_MAX_PARTS = 64

EXPORTS = [
    "sar_status_string", "sar_built_for_sm", "sar_graph_workspace_bytes", "sar_csr_from_coo", "sar_csr_transpose",
    "sar_partition_bounds", "sar_csr_split_indptr", "sar_csr_split_indices", "sar_validate_part", "sar_plan_count",
    "sar_plan_fill", "sar_gat_workspace_bytes", "sar_gat_fwd", "sar_gat_fwd_fused", "sar_gat_bwd_prepare",
    "sar_gat_bwd", "sar_gat_bwd_fused", "sar_spmm_agg", "sar_spmm_workspace_bytes", "sar_set_launch_hook",
    "sar_gat_stack_arena_bytes", "sar_gat_stack_host", "sar_gat_bwd_noalloc", "sar_gat_bwd_noalloc_limit",
    "sar_gat_project_workspace_bytes", "sar_gat_project", "sar_gat_project_bwd", "sar_relu", "sar_relu_bwd",
    "sar_mfg_frontier", "sar_csr_filter_rows_indptr", "sar_csr_filter_rows_indices", "sar_spmm_agg_scaled",
    "sar_gat_stack_host_wait", "sar_bn_workspace_bytes", "sar_bn_stats", "sar_bn_apply", "sar_bn_bwd_stats",
    "sar_bn_bwd_apply", "sar_dropout", "sar_linear_workspace_bytes", "sar_linear", "sar_linear_bwd_input",
    "sar_linear_bwd_weight", "sar_linear_accumulate", "sar_degree_scale", "sar_rgcn_basis", "sar_rgcn_basis_bwd", "sar_axpby", "sar_bn_rstd", "sar_accumulate", "sar_round_to", "sar_bn_apply_act",
    "sar_bn_bwd_stats_act", "sar_bn_bwd_apply_act", "sar_csc_slice_indptr",
    "sar_gat_storing_workspace_bytes", "sar_gat_fwd_storing", "sar_gat_bwd_storing", "sar_bn_combine_moments",
    "sar_bn_combine_sums", "sar_degree_order_workspace_bytes", "sar_degree_order", "sar_relabel", "sar_permute_rows", "sar_linear_project", "sar_linear_bwd_input_relu",
]


class SarError(RuntimeError):
    def __init__(self, fn: str, code: int, text: str):
        super().__init__(f"{fn} failed: {text} (status {code})")
        self.code = code


class sar_split(Structure):
    _fields_ = [("threshold", c_int32), ("n_long", c_int32), ("n_seg", c_int64), ("long_row", c_void_p),
                ("long_seg", c_void_p)]


class sar_part(Structure):
    _fields_ = [("n_dst", c_int64), ("n_src", c_int64), ("nnz", c_int64), ("indptr", c_void_p),
                ("indices", c_void_p), ("t_indptr", c_void_p), ("t_indices", c_void_p),
                ("split", POINTER(sar_split)), ("t_split", POINTER(sar_split))]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library.  Raises if libsar.so is missing: build it with
    `python -m paper_2111_06483_b200.build` (there is no other code path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: run `python -m paper_2111_06483_b200.build` "
                               "(libsar has no CPU or PyTorch fallback)")
        L = ctypes.CDLL(LIB_PATH)
        L.sar_status_string.restype = c_char_p
        L.sar_status_string.argtypes = [ctypes.c_int]
        L.sar_built_for_sm.restype = c_int32
        for name in ("sar_graph_workspace_bytes", "sar_gat_workspace_bytes", "sar_spmm_workspace_bytes",
                     "sar_gat_stack_arena_bytes", "sar_gat_bwd_noalloc_limit", "sar_gat_project_workspace_bytes",
                     "sar_bn_workspace_bytes", "sar_linear_workspace_bytes", "sar_gat_storing_workspace_bytes",
                     "sar_degree_order_workspace_bytes"):
            getattr(L, name).restype = c_size_t
        _lib = L
    return _lib


def _check(fn: str, code: int) -> None:
    if code != SAR_OK:
        raise SarError(fn, code, lib().sar_status_string(code).decode())


def _ptr(t: Optional[torch.Tensor]) -> c_void_p:
    if t is None:
        return c_void_p(0)
    assert t.is_cuda and t.is_contiguous(), "libsar takes contiguous CUDA tensors"
    return c_void_p(t.data_ptr())


def _stream() -> c_void_p:
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _dtype(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return SAR_F32
    if t.dtype == torch.bfloat16:
        return SAR_BF16
    raise TypeError(f"unsupported storage dtype {t.dtype}")


def _ws(workspace: Optional[torch.Tensor]):
    if workspace is None:
        return c_void_p(0), c_size_t(0)
    return _ptr(workspace), c_size_t(workspace.numel() * workspace.element_size())


class Split:
    """Device arrays of a long-row plan plus the C struct that points at them."""

    def __init__(self, threshold: int, n_long: int, n_seg: int, long_row: torch.Tensor, long_seg: torch.Tensor):
        self.threshold, self.n_long, self.n_seg = threshold, n_long, n_seg
        self.long_row, self.long_seg = long_row, long_seg
        self.c = sar_split(threshold, n_long, n_seg, long_row.data_ptr(), long_seg.data_ptr())


class Part:
    """One source partition (or the whole graph): owns the index tensors and the C struct."""

    def __init__(self, n_dst: int, n_src: int, indptr: torch.Tensor, indices: torch.Tensor,
                 t_indptr: Optional[torch.Tensor] = None, t_indices: Optional[torch.Tensor] = None,
                 split: Optional[Split] = None, t_split: Optional[Split] = None, nnz: Optional[int] = None):
        assert indptr.dtype == torch.int64 and indices.dtype == torch.int32
        self.n_dst, self.n_src = int(n_dst), int(n_src)
        self.nnz = int(indices.numel() if nnz is None else nnz)
        self.indptr, self.indices, self.t_indptr, self.t_indices = indptr, indices, t_indptr, t_indices
        self.split, self.t_split = split, t_split
        self.c = sar_part(self.n_dst, self.n_src, self.nnz, indptr.data_ptr(), indices.data_ptr(),
                          t_indptr.data_ptr() if t_indptr is not None else None,
                          t_indices.data_ptr() if t_indices is not None else None,
                          ctypes.pointer(split.c) if split is not None else None,
                          ctypes.pointer(t_split.c) if t_split is not None else None)

    def transposed(self) -> "Part":
        """The same edges with the roles of rows and columns swapped (for the backward of the sum)."""
        assert self.t_indptr is not None
        return Part(self.n_src, self.n_dst, self.t_indptr, self.t_indices, self.indptr, self.indices,
                    self.t_split, self.split, nnz=self.nnz)


# ----------------------------------------------------------------------------------------------
# launch observer
# ----------------------------------------------------------------------------------------------

_HOOK_T = ctypes.CFUNCTYPE(None, c_char_p, c_int32, c_void_p, c_void_p)
_hook_keepalive = None


def sar_set_launch_hook(fn) -> None:
    """fn(kernel_name: str, phase: int) is called before (0) and after (1) every kernel launch of the
    aggregation entry points; None removes the observer."""
    global _hook_keepalive
    if fn is None:
        lib().sar_set_launch_hook(None, None)
        _hook_keepalive = None
        return
    cb = _HOOK_T(lambda name, phase, stream, user: fn(name.decode(), int(phase)))
    lib().sar_set_launch_hook(cb, None)
    _hook_keepalive = cb


class LaunchTimer:
    """Context manager: CUDA events around every kernel launch inside the block, on the current
    stream.  After the block (and a synchronize) `summary()` gives per-kernel launch counts and
    device times."""

    def __init__(self):
        self.records = []   # (name, start_event, end_event)
        self._open = {}

    def _hook(self, name, phase):
        ev = torch.cuda.Event(enable_timing=True)
        ev.record()
        if phase == 0:
            self._open[name] = ev
        else:
            self.records.append((name, self._open.pop(name), ev))

    def __enter__(self):
        sar_set_launch_hook(self._hook)
        return self

    def __exit__(self, *exc):
        sar_set_launch_hook(None)
        return False

    def summary(self):
        torch.cuda.synchronize()
        agg = {}
        for name, e0, e1 in self.records:
            n, ms = agg.get(name, (0, 0.0))
            agg[name] = (n + 1, ms + e0.elapsed_time(e1))
        return {k: {"launches": n, "total_ms": ms, "avg_ms": ms / n} for k, (n, ms) in agg.items()}


# ----------------------------------------------------------------------------------------------
# graph preparation
# ----------------------------------------------------------------------------------------------

def sar_built_for_sm() -> int:
    return int(lib().sar_built_for_sm())


def sar_graph_workspace_bytes(nnz: int, n_rows: int) -> int:
    return int(lib().sar_graph_workspace_bytes(c_int64(nnz), c_int64(n_rows)))


def sar_csr_from_coo(n_rows: int, n_cols: int, row: torch.Tensor, col: torch.Tensor, indptr: torch.Tensor,
                     indices: torch.Tensor, workspace: torch.Tensor) -> None:
    assert row.dtype == torch.int32 and col.dtype == torch.int32 and row.numel() == col.numel()
    w, wb = _ws(workspace)
    _check("sar_csr_from_coo", lib().sar_csr_from_coo(c_int64(n_rows), c_int64(n_cols), c_int64(row.numel()),
                                                      _ptr(row), _ptr(col), _ptr(indptr), _ptr(indices), w, wb,
                                                      _stream()))


def sar_csr_transpose(n_rows: int, n_cols: int, indptr: torch.Tensor, indices: torch.Tensor,
                      t_indptr: torch.Tensor, t_indices: torch.Tensor, workspace: torch.Tensor) -> None:
    w, wb = _ws(workspace)
    _check("sar_csr_transpose", lib().sar_csr_transpose(c_int64(n_rows), c_int64(n_cols), _ptr(indptr),
                                                        _ptr(indices), _ptr(t_indptr), _ptr(t_indices), w, wb,
                                                        _stream()))


def sar_partition_bounds(n: int, k: int) -> list:
    arr = (c_int64 * (k + 1))()
    _check("sar_partition_bounds", lib().sar_partition_bounds(c_int64(n), c_int32(k), arr))
    return list(arr)


def _host_i64(xs: Sequence[int]):
    return (c_int64 * len(xs))(*[int(x) for x in xs])


def sar_csr_split_indptr(n_dst: int, indptr: torch.Tensor, indices: torch.Tensor, bounds: Sequence[int],
                         indptr_all: torch.Tensor, workspace: torch.Tensor) -> None:
    k = len(bounds) - 1
    w, wb = _ws(workspace)
    _check("sar_csr_split_indptr", lib().sar_csr_split_indptr(c_int64(n_dst), _ptr(indptr), _ptr(indices),
                                                              c_int32(k), _host_i64(bounds), _ptr(indptr_all), w, wb,
                                                              _stream()))


def sar_csr_split_indices(n_dst: int, indptr: torch.Tensor, indices: torch.Tensor, bounds: Sequence[int],
                          indptr_all: torch.Tensor, nnz_off: Sequence[int], indices_all: torch.Tensor) -> None:
    k = len(bounds) - 1
    _check("sar_csr_split_indices", lib().sar_csr_split_indices(c_int64(n_dst), _ptr(indptr), _ptr(indices),
                                                                c_int32(k), _host_i64(bounds), _ptr(indptr_all),
                                                                _host_i64(nnz_off), _ptr(indices_all), _stream()))


def sar_csc_slice_indptr(s0: int, s1: int, t_indptr: torch.Tensor, t_indptr_q: torch.Tensor) -> None:
    assert t_indptr.dtype == torch.int64 and t_indptr_q.dtype == torch.int64 and t_indptr_q.numel() == s1 - s0 + 1
    _check("sar_csc_slice_indptr", lib().sar_csc_slice_indptr(c_int64(s0), c_int64(s1), _ptr(t_indptr),
                                                              _ptr(t_indptr_q), _stream()))


def sar_degree_order_workspace_bytes(n: int) -> int:
    return int(lib().sar_degree_order_workspace_bytes(c_int64(n)))


def sar_degree_order(n: int, src: torch.Tensor, dst: torch.Tensor, order: torch.Tensor, rank: torch.Tensor,
                     workspace: torch.Tensor) -> None:
    assert src.dtype == torch.int32 and dst.dtype == torch.int32 and src.numel() == dst.numel()
    assert order.dtype == torch.int32 and rank.dtype == torch.int32 and order.numel() == n and rank.numel() == n
    wp, wb = _ws(workspace)
    _check("sar_degree_order", lib().sar_degree_order(c_int64(n), c_int64(src.numel()), _ptr(src), _ptr(dst), _ptr(order),
                                                      _ptr(rank), wp, wb, _stream()))


def sar_relabel(ids: torch.Tensor, rank: torch.Tensor, out: torch.Tensor) -> None:
    assert ids.dtype == torch.int32 and rank.dtype == torch.int32 and out.dtype == torch.int32
    assert out.numel() == ids.numel()
    _check("sar_relabel", lib().sar_relabel(c_int64(ids.numel()), _ptr(ids), _ptr(rank), _ptr(out), _stream()))


def sar_permute_rows(index: torch.Tensor, x: torch.Tensor, out: torch.Tensor) -> None:
    """out row i = x row index[i]; x, out contiguous with the same shape, first dimension = index.numel()."""
    assert index.dtype == torch.int32 and x.is_contiguous() and out.is_contiguous()
    assert x.shape == out.shape and x.dtype == out.dtype and x.shape[0] == index.numel()
    n = index.numel()
    row_bytes = (x.numel() // n) * x.element_size() if n else 1
    _check("sar_permute_rows", lib().sar_permute_rows(c_int64(n), c_int64(row_bytes), _ptr(index), _ptr(x), _ptr(out),
                                                      _stream()))


def sar_mfg_frontier(n: int, indptr: torch.Tensor, indices: torch.Tensor, need_out: torch.Tensor,
                     need_in: torch.Tensor) -> None:
    _check("sar_mfg_frontier", lib().sar_mfg_frontier(c_int64(n), _ptr(indptr), _ptr(indices), _ptr(need_out),
                                                      _ptr(need_in), _stream()))


def sar_csr_filter_rows_indptr(n: int, indptr: torch.Tensor, keep: torch.Tensor, indptr_out: torch.Tensor,
                               workspace: torch.Tensor) -> None:
    w, wb = _ws(workspace)
    _check("sar_csr_filter_rows_indptr", lib().sar_csr_filter_rows_indptr(c_int64(n), _ptr(indptr), _ptr(keep),
                                                                          _ptr(indptr_out), w, wb, _stream()))


def sar_csr_filter_rows_indices(n: int, indptr: torch.Tensor, indices: torch.Tensor, indptr_out: torch.Tensor,
                                indices_out: torch.Tensor) -> None:
    _check("sar_csr_filter_rows_indices", lib().sar_csr_filter_rows_indices(c_int64(n), _ptr(indptr), _ptr(indices),
                                                                            _ptr(indptr_out), _ptr(indices_out),
                                                                            _stream()))


def sar_validate_part(part: Part, flag: torch.Tensor) -> None:
    _check("sar_validate_part", lib().sar_validate_part(byref(part.c), _ptr(flag), _stream()))


def sar_plan_count(n_rows: int, indptr: torch.Tensor, threshold: int, counts: torch.Tensor):
    n_long, n_seg = c_int32(0), c_int64(0)
    _check("sar_plan_count", lib().sar_plan_count(c_int64(n_rows), _ptr(indptr), c_int32(threshold), _ptr(counts),
                                                  byref(n_long), byref(n_seg), _stream()))
    return n_long.value, n_seg.value


def sar_plan_fill(n_rows: int, indptr: torch.Tensor, threshold: int, n_long: int, long_row: torch.Tensor,
                  long_seg: torch.Tensor, workspace: torch.Tensor) -> None:
    w, wb = _ws(workspace)
    _check("sar_plan_fill", lib().sar_plan_fill(c_int64(n_rows), _ptr(indptr), c_int32(threshold), c_int32(n_long),
                                                _ptr(long_row), _ptr(long_seg), w, wb, _stream()))


# ----------------------------------------------------------------------------------------------
# aggregation
# ----------------------------------------------------------------------------------------------

def sar_gat_workspace_bytes(part: Part, H: int, F: int, dtype: int) -> int:
    return int(lib().sar_gat_workspace_bytes(byref(part.c), c_int32(H), c_int32(F), ctypes.c_int(dtype)))


def sar_spmm_workspace_bytes(part: Part, F: int, dtype: int) -> int:
    return int(lib().sar_spmm_workspace_bytes(byref(part.c), c_int32(F), ctypes.c_int(dtype)))


def sar_gat_fwd(part: Part, feat_q: torch.Tensor, el: torch.Tensor, er_q: torch.Tensor, H: int, F: int,
                slope: float, flags: int, acc: Optional[torch.Tensor], m: torch.Tensor, d: torch.Tensor,
                out: Optional[torch.Tensor], workspace: Optional[torch.Tensor]) -> None:
    w, wb = _ws(workspace)
    _check("sar_gat_fwd", lib().sar_gat_fwd(byref(part.c), _ptr(feat_q), _ptr(el), _ptr(er_q), c_int32(H), c_int32(F),
                                            ctypes.c_int(_dtype(feat_q)), c_float(slope), c_uint32(flags), _ptr(acc),
                                            _ptr(m), _ptr(d), _ptr(out), w, wb, _stream()))


def sar_gat_fwd_fused(part: Part, bounds: Sequence[int], feat: torch.Tensor, el: torch.Tensor, er: torch.Tensor,
                      H: int, F: int, slope: float, m: torch.Tensor, d: torch.Tensor, out: torch.Tensor,
                      workspace: Optional[torch.Tensor]) -> None:
    k = len(bounds) - 1
    w, wb = _ws(workspace)
    _check("sar_gat_fwd_fused", lib().sar_gat_fwd_fused(byref(part.c), c_int32(k), _host_i64(bounds), _ptr(feat),
                                                        _ptr(el), _ptr(er), c_int32(H), c_int32(F),
                                                        ctypes.c_int(_dtype(feat)), c_float(slope), _ptr(m), _ptr(d),
                                                        _ptr(out), w, wb, _stream()))


def sar_gat_bwd_prepare(n_dst: int, H: int, F: int, out_or_acc: torch.Tensor, acc_is_numerator: bool,
                        gout: torch.Tensor, el: torch.Tensor, m: torch.Tensor, d: torch.Tensor,
                        D: Optional[torch.Tensor], workspace: torch.Tensor) -> None:
    w, wb = _ws(workspace)
    _check("sar_gat_bwd_prepare", lib().sar_gat_bwd_prepare(c_int64(n_dst), c_int32(H), c_int32(F),
                                                            ctypes.c_int(_dtype(gout)), _ptr(out_or_acc),
                                                            c_int32(1 if acc_is_numerator else 0), _ptr(gout),
                                                            _ptr(el), _ptr(m), _ptr(d), _ptr(D), w, wb, _stream()))


def sar_gat_bwd(part: Part, feat_q: torch.Tensor, el: torch.Tensor, er_q: torch.Tensor, m: torch.Tensor,
                d: torch.Tensor, gout: torch.Tensor, H: int, F: int, slope: float, flags: int,
                dfeat_q: torch.Tensor, del_: torch.Tensor, der_q: torch.Tensor, workspace: torch.Tensor) -> None:
    w, wb = _ws(workspace)
    _check("sar_gat_bwd", lib().sar_gat_bwd(byref(part.c), _ptr(feat_q), _ptr(el), _ptr(er_q), _ptr(m), _ptr(d),
                                            _ptr(gout), c_int32(H), c_int32(F), ctypes.c_int(_dtype(feat_q)),
                                            c_float(slope), c_uint32(flags), _ptr(dfeat_q), _ptr(del_), _ptr(der_q),
                                            w, wb, _stream()))


def sar_gat_bwd_fused(part: Part, bounds: Sequence[int], feat: torch.Tensor, el: torch.Tensor, er: torch.Tensor,
                      m: torch.Tensor, d: torch.Tensor, gout: torch.Tensor, H: int, F: int, slope: float,
                      dfeat: torch.Tensor, del_: torch.Tensor, der: torch.Tensor, workspace: torch.Tensor) -> None:
    k = len(bounds) - 1
    w, wb = _ws(workspace)
    _check("sar_gat_bwd_fused", lib().sar_gat_bwd_fused(byref(part.c), c_int32(k), _host_i64(bounds), _ptr(feat),
                                                        _ptr(el), _ptr(er), _ptr(m), _ptr(d), _ptr(gout), c_int32(H),
                                                        c_int32(F), ctypes.c_int(_dtype(gout)), c_float(slope),
                                                        _ptr(dfeat), _ptr(del_), _ptr(der), w, wb, _stream()))


def sar_gat_storing_workspace_bytes(part: Part, H: int) -> int:
    return int(lib().sar_gat_storing_workspace_bytes(byref(part.c), c_int32(H)))


def sar_gat_fwd_storing(part: Part, feat: torch.Tensor, el: torch.Tensor, er: torch.Tensor, H: int, F: int,
                        slope: float, alpha: torch.Tensor, out: torch.Tensor) -> None:
    """The storing baseline's forward pass: writes alpha [nnz,H] and out (measurement and tests only)."""
    _check("sar_gat_fwd_storing", lib().sar_gat_fwd_storing(byref(part.c), _ptr(feat), _ptr(el), _ptr(er), c_int32(H),
                                                            c_int32(F), ctypes.c_int(_dtype(feat)), c_float(slope),
                                                            _ptr(alpha), _ptr(out), _stream()))


def sar_gat_bwd_storing(part: Part, feat: torch.Tensor, el: torch.Tensor, er: torch.Tensor, alpha: torch.Tensor,
                        gout: torch.Tensor, H: int, F: int, slope: float, dfeat: torch.Tensor, del_: torch.Tensor,
                        der: torch.Tensor, workspace: torch.Tensor) -> None:
    w, wb = _ws(workspace)
    _check("sar_gat_bwd_storing", lib().sar_gat_bwd_storing(byref(part.c), _ptr(feat), _ptr(el), _ptr(er), _ptr(alpha),
                                                            _ptr(gout), c_int32(H), c_int32(F),
                                                            ctypes.c_int(_dtype(feat)), c_float(slope), _ptr(dfeat),
                                                            _ptr(del_), _ptr(der), w, wb, _stream()))


def sar_spmm_agg(part: Part, feat_q: torch.Tensor, F: int, flags: int, deg_total: Optional[torch.Tensor],
                 out: torch.Tensor, workspace: Optional[torch.Tensor]) -> None:
    w, wb = _ws(workspace)
    _check("sar_spmm_agg", lib().sar_spmm_agg(byref(part.c), _ptr(feat_q), c_int32(F), ctypes.c_int(_dtype(feat_q)),
                                              c_uint32(flags), _ptr(deg_total), _ptr(out), w, wb, _stream()))


def sar_spmm_agg_scaled(part: Part, feat_q: torch.Tensor, F: int, flags: int, src_scale: Optional[torch.Tensor],
                        dst_scale: Optional[torch.Tensor], out: torch.Tensor, workspace: Optional[torch.Tensor]) -> None:
    w, wb = _ws(workspace)
    _check("sar_spmm_agg_scaled", lib().sar_spmm_agg_scaled(byref(part.c), _ptr(feat_q), c_int32(F),
                                                            ctypes.c_int(_dtype(feat_q)), c_uint32(flags),
                                                            _ptr(src_scale), _ptr(dst_scale), _ptr(out), w, wb,
                                                            _stream()))


# ----------------------------------------------------------------------------------------------
# host-buffer stack
# ----------------------------------------------------------------------------------------------

class sar_stack_host_io(Structure):
    _fields_ = [("L", c_int32), ("H", c_int32), ("F", c_int32), ("t", ctypes.c_int), ("slope", c_float),
                ("feat0", c_void_p), ("el", POINTER(c_void_p)), ("er", POINTER(c_void_p)), ("gout", c_void_p),
                ("out_last", c_void_p), ("dfeat0", c_void_p), ("del_", POINTER(c_void_p)), ("der", POINTER(c_void_p)),
                ("flags", c_uint32)]


SAR_STACK_PIPELINED = 1


def sar_gat_stack_arena_bytes(part: Part, L: int, H: int, F: int, dtype: int) -> int:
    return int(lib().sar_gat_stack_arena_bytes(byref(part.c), c_int32(L), c_int32(H), c_int32(F), ctypes.c_int(dtype)))


def _host_ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert (not t.is_cuda) and t.is_contiguous(), "host buffers are contiguous CPU tensors (pin them for async copies)"
    return t.data_ptr()


def _host_ptr_array(ts):
    if ts is None:
        return None
    return (c_void_p * len(ts))(*[_host_ptr(t) for t in ts])


def sar_gat_stack_host(part: Part, bounds: Sequence[int], H: int, F: int, slope: float, feat0: torch.Tensor,
                       el: Sequence[torch.Tensor], er: Sequence[torch.Tensor], gout: torch.Tensor,
                       out_last: Optional[torch.Tensor], dfeat0: Optional[torch.Tensor],
                       del_: Optional[Sequence[torch.Tensor]], der: Optional[Sequence[torch.Tensor]],
                       arena: torch.Tensor, pipelined: bool = False) -> None:
    """L = len(el) chained aggregation layers, fwd + bwd, all node tensors in HOST memory.  pipelined=True:
    `arena` holds two working sets and successive calls overlap (finish with sar_gat_stack_host_wait)."""
    L = len(el)
    io = sar_stack_host_io(L, H, F, _dtype(feat0), slope, _host_ptr(feat0), _host_ptr_array(el), _host_ptr_array(er),
                           _host_ptr(gout), _host_ptr(out_last), _host_ptr(dfeat0), _host_ptr_array(del_),
                           _host_ptr_array(der), SAR_STACK_PIPELINED if pipelined else 0)
    w, wb = _ws(arena)
    _check("sar_gat_stack_host", lib().sar_gat_stack_host(byref(part.c), c_int32(len(bounds) - 1), _host_i64(bounds),
                                                          byref(io), w, wb, _stream()))


def sar_bn_workspace_bytes(C: int) -> int:
    return int(lib().sar_bn_workspace_bytes(c_int32(C)))


def sar_bn_combine_moments(n_r: Sequence[int], mean_r: torch.Tensor, m2_r: torch.Tensor):
    """HOST tensors mean_r, m2_r [R, C] float32 (row r: worker r's local statistics) -> (n_all, mean [C], m2 [C])."""
    R, C = mean_r.shape
    assert (not mean_r.is_cuda) and (not m2_r.is_cuda) and mean_r.dtype == torch.float32 and m2_r.dtype == torch.float32
    mean_r, m2_r = mean_r.contiguous(), m2_r.contiguous()
    mean, m2 = torch.empty(C, dtype=torch.float32), torch.empty(C, dtype=torch.float32)
    n_all = c_int64(0)
    _check("sar_bn_combine_moments", lib().sar_bn_combine_moments(c_int32(R), c_int32(C), _host_i64(n_r),
                                                                  c_void_p(mean_r.data_ptr()), c_void_p(m2_r.data_ptr()),
                                                                  byref(n_all), c_void_p(mean.data_ptr()),
                                                                  c_void_p(m2.data_ptr())))
    return int(n_all.value), mean, m2


def sar_bn_combine_sums(sums_r: torch.Tensor) -> torch.Tensor:
    """HOST tensor sums_r [R, count] float32 -> their sum over the workers [count], added in rank order."""
    assert (not sums_r.is_cuda) and sums_r.dtype == torch.float32
    sums_r = sums_r.contiguous()
    R, count = sums_r.shape
    out = torch.empty(count, dtype=torch.float32)
    _check("sar_bn_combine_sums", lib().sar_bn_combine_sums(c_int32(R), c_int64(count), c_void_p(sums_r.data_ptr()),
                                                            c_void_p(out.data_ptr())))
    return out


def sar_bn_stats(x: torch.Tensor, mean: torch.Tensor, m2: torch.Tensor, workspace: torch.Tensor) -> None:
    n, C = x.shape
    w, wb = _ws(workspace)
    _check("sar_bn_stats", lib().sar_bn_stats(c_int64(n), c_int32(C), ctypes.c_int(_dtype(x)), _ptr(x), _ptr(mean),
                                              _ptr(m2), w, wb, _stream()))


def sar_bn_rstd(m2: torch.Tensor, count: int, eps: float, rstd: torch.Tensor) -> None:
    _check("sar_bn_rstd", lib().sar_bn_rstd(c_int32(m2.numel()), _ptr(m2), c_int64(count), c_float(eps), _ptr(rstd),
                                            _stream()))


def sar_bn_apply(x: torch.Tensor, mean: torch.Tensor, rstd: torch.Tensor, gamma: Optional[torch.Tensor],
                 beta: Optional[torch.Tensor], y: torch.Tensor) -> None:
    n, C = x.shape
    _check("sar_bn_apply", lib().sar_bn_apply(c_int64(n), c_int32(C), ctypes.c_int(_dtype(x)), _ptr(x), _ptr(mean),
                                              _ptr(rstd), _ptr(gamma), _ptr(beta), _ptr(y), _stream()))


def sar_bn_bwd_stats(x: torch.Tensor, mean: torch.Tensor, rstd: torch.Tensor, gy: torch.Tensor, sum_gy: torch.Tensor,
                     sum_gy_xhat: torch.Tensor, workspace: torch.Tensor) -> None:
    n, C = x.shape
    w, wb = _ws(workspace)
    _check("sar_bn_bwd_stats", lib().sar_bn_bwd_stats(c_int64(n), c_int32(C), ctypes.c_int(_dtype(x)), _ptr(x),
                                                      _ptr(mean), _ptr(rstd), _ptr(gy), _ptr(sum_gy),
                                                      _ptr(sum_gy_xhat), w, wb, _stream()))


def sar_bn_bwd_apply(x: torch.Tensor, mean: torch.Tensor, rstd: torch.Tensor, gamma: Optional[torch.Tensor],
                     gy: torch.Tensor, sum_gy: torch.Tensor, sum_gy_xhat: torch.Tensor, inv_count: float,
                     gx: torch.Tensor) -> None:
    n, C = x.shape
    _check("sar_bn_bwd_apply", lib().sar_bn_bwd_apply(c_int64(n), c_int32(C), ctypes.c_int(_dtype(x)), _ptr(x),
                                                      _ptr(mean), _ptr(rstd), _ptr(gamma), _ptr(gy), _ptr(sum_gy),
                                                      _ptr(sum_gy_xhat), c_float(inv_count), _ptr(gx), _stream()))


def sar_bn_apply_act(x: torch.Tensor, mean: torch.Tensor, rstd: torch.Tensor, gamma: Optional[torch.Tensor],
                     beta: Optional[torch.Tensor], flags: int, p: float, seed: int, y: torch.Tensor) -> None:
    n, C = x.shape
    _check("sar_bn_apply_act", lib().sar_bn_apply_act(c_int64(n), c_int32(C), ctypes.c_int(_dtype(x)), _ptr(x), _ptr(mean),
                                                      _ptr(rstd), _ptr(gamma), _ptr(beta), c_uint32(flags), c_float(p),
                                                      ctypes.c_uint64(seed & 0xFFFFFFFFFFFFFFFF), _ptr(y), _stream()))


def sar_bn_bwd_stats_act(x: torch.Tensor, mean: torch.Tensor, rstd: torch.Tensor, gy: torch.Tensor,
                         post: Optional[torch.Tensor], flags: int, p: float, seed: int, sum_gy: torch.Tensor,
                         sum_gy_xhat: torch.Tensor, workspace: torch.Tensor) -> None:
    n, C = x.shape
    w, wb = _ws(workspace)
    _check("sar_bn_bwd_stats_act", lib().sar_bn_bwd_stats_act(
        c_int64(n), c_int32(C), ctypes.c_int(_dtype(x)), _ptr(x), _ptr(mean), _ptr(rstd), _ptr(gy), _ptr(post),
        c_uint32(flags), c_float(p), ctypes.c_uint64(seed & 0xFFFFFFFFFFFFFFFF), _ptr(sum_gy), _ptr(sum_gy_xhat), w, wb,
        _stream()))


def sar_bn_bwd_apply_act(x: torch.Tensor, mean: torch.Tensor, rstd: torch.Tensor, gamma: Optional[torch.Tensor],
                         gy: torch.Tensor, post: Optional[torch.Tensor], flags: int, p: float, seed: int,
                         sum_gy: torch.Tensor, sum_gy_xhat: torch.Tensor, inv_count: float, gx: torch.Tensor) -> None:
    n, C = x.shape
    _check("sar_bn_bwd_apply_act", lib().sar_bn_bwd_apply_act(
        c_int64(n), c_int32(C), ctypes.c_int(_dtype(x)), _ptr(x), _ptr(mean), _ptr(rstd), _ptr(gamma), _ptr(gy),
        _ptr(post), c_uint32(flags), c_float(p), ctypes.c_uint64(seed & 0xFFFFFFFFFFFFFFFF), _ptr(sum_gy),
        _ptr(sum_gy_xhat), c_float(inv_count), _ptr(gx), _stream()))


def sar_gat_stack_host_wait() -> None:
    _check("sar_gat_stack_host_wait", lib().sar_gat_stack_host_wait(_stream()))


# ----------------------------------------------------------------------------------------------
# backward pass with the library's built-in scratch
# ----------------------------------------------------------------------------------------------

def sar_gat_bwd_noalloc_limit() -> int:
    return int(lib().sar_gat_bwd_noalloc_limit())


def sar_gat_bwd_noalloc(part: Part, feat: torch.Tensor, el: torch.Tensor, er: torch.Tensor, m: torch.Tensor,
                        d: torch.Tensor, gout: torch.Tensor, H: int, F: int, slope: float, dfeat: torch.Tensor,
                        del_: torch.Tensor, der: torch.Tensor) -> None:
    """Whole-graph backward pass for callers that cannot provide scratch memory: the library uses a fixed
    array inside its own device image (problems whose scratch need exceeds it are refused).  Calls on
    one device must not overlap on the GPU; make the first call on a device outside stream capture."""
    _check("sar_gat_bwd_noalloc", lib().sar_gat_bwd_noalloc(byref(part.c), _ptr(feat), _ptr(el), _ptr(er), _ptr(m),
                                                            _ptr(d), _ptr(gout), c_int32(H), c_int32(F),
                                                            ctypes.c_int(_dtype(feat)), c_float(slope), _ptr(dfeat),
                                                            _ptr(del_), _ptr(der), _stream()))


# ----------------------------------------------------------------------------------------------
# the layer around the aggregation
# ----------------------------------------------------------------------------------------------

def sar_gat_project_workspace_bytes(H: int, F: int) -> int:
    return int(lib().sar_gat_project_workspace_bytes(c_int32(H), c_int32(F)))


SAR_GLUE_RELU = 1
SAR_GLUE_DROPOUT = 2


def sar_gat_project(z: torch.Tensor, a_l: torch.Tensor, a_r: torch.Tensor, el: torch.Tensor, er: torch.Tensor,
                    flags: int = 0) -> None:
    n, H, F = z.shape
    _check("sar_gat_project", lib().sar_gat_project(c_int64(n), c_int32(H), c_int32(F), ctypes.c_int(_dtype(z)), _ptr(z),
                                                    _ptr(a_l), _ptr(a_r), _ptr(el), _ptr(er), c_uint32(flags),
                                                    _stream()))


def sar_gat_project_bwd(z: torch.Tensor, a_l: torch.Tensor, a_r: torch.Tensor, del_: torch.Tensor, der: torch.Tensor,
                        dz: torch.Tensor, da_l: torch.Tensor, da_r: torch.Tensor, workspace: torch.Tensor,
                        flags: int = 0) -> None:
    n, H, F = z.shape
    w, wb = _ws(workspace)
    _check("sar_gat_project_bwd", lib().sar_gat_project_bwd(c_int64(n), c_int32(H), c_int32(F), ctypes.c_int(_dtype(z)),
                                                            _ptr(z), _ptr(a_l), _ptr(a_r), _ptr(del_), _ptr(der), _ptr(dz),
                                                            _ptr(da_l), _ptr(da_r), c_uint32(flags), w, wb,
                                                            _stream()))


def sar_relu(x: torch.Tensor) -> None:
    _check("sar_relu", lib().sar_relu(c_int64(x.numel()), ctypes.c_int(_dtype(x)), _ptr(x), _stream()))


def sar_linear_workspace_bytes(n: int, d_in: int, d_out: int) -> int:
    return int(lib().sar_linear_workspace_bytes(c_int64(n), c_int32(d_in), c_int32(d_out)))


def sar_linear(h: torch.Tensor, w: torch.Tensor, z: torch.Tensor, workspace: torch.Tensor) -> None:
    n, d_in = h.shape
    d_out = w.shape[1]
    ws, wb = _ws(workspace)
    _check("sar_linear", lib().sar_linear(c_int64(n), c_int32(d_in), c_int32(d_out), ctypes.c_int(_dtype(h)), _ptr(h),
                                          _ptr(w), _ptr(z), ws, wb, _stream()))


def sar_linear_bwd_input_relu(dz: torch.Tensor, w: torch.Tensor, y: torch.Tensor, dh: torch.Tensor,
                              workspace: torch.Tensor) -> None:
    """dh = (dz W^T) where y > 0, else 0 (y: the output of the ReLU that produced the layer's input)."""
    n, d_out = dz.shape
    d_in = w.shape[0]
    assert y.shape == (n, d_in) and dh.shape == (n, d_in) and y.dtype == dz.dtype
    ws, wb = _ws(workspace)
    _check("sar_linear_bwd_input_relu", lib().sar_linear_bwd_input_relu(c_int64(n), c_int32(d_in), c_int32(d_out),
                                                                        ctypes.c_int(_dtype(dz)), _ptr(dz), _ptr(w), _ptr(y),
                                                                        _ptr(dh), ws, wb, _stream()))


def sar_linear_project(h: torch.Tensor, w: torch.Tensor, a_l: torch.Tensor, a_r: torch.Tensor, z: torch.Tensor,
                       el: torch.Tensor, er: torch.Tensor, workspace: torch.Tensor,
                       flag: Optional[torch.Tensor] = None) -> None:
    """z[n,H,F] = h W and el, er [n,H] = <z, a_l>, <z, a_r> in one kernel."""
    n, d_in = h.shape
    H, F = a_l.shape
    assert w.shape == (d_in, H * F) and z.numel() == n * H * F and el.shape == (n, H) and er.shape == (n, H)
    assert a_l.dtype == torch.float32 and a_r.dtype == torch.float32 and el.dtype == torch.float32
    assert flag is None or flag.dtype == torch.int32
    ws, wb = _ws(workspace)
    _check("sar_linear_project", lib().sar_linear_project(c_int64(n), c_int32(d_in), c_int32(H), c_int32(F),
                                                          ctypes.c_int(_dtype(h)), _ptr(h), _ptr(w), _ptr(a_l), _ptr(a_r),
                                                          _ptr(z), _ptr(el), _ptr(er), _ptr(flag), ws, wb, _stream()))


def sar_linear_accumulate(h: torch.Tensor, w: torch.Tensor, z: torch.Tensor, workspace: torch.Tensor) -> None:
    n, d_in = h.shape
    d_out = w.shape[1]
    ws, wb = _ws(workspace)
    _check("sar_linear_accumulate", lib().sar_linear_accumulate(c_int64(n), c_int32(d_in), c_int32(d_out),
                                                                ctypes.c_int(_dtype(h)), _ptr(h), _ptr(w), _ptr(z), ws,
                                                                wb, _stream()))


def sar_degree_scale(indptr: torch.Tensor, power: float, scale: torch.Tensor) -> None:
    _check("sar_degree_scale", lib().sar_degree_scale(c_int64(indptr.numel() - 1), _ptr(indptr), c_float(power),
                                                      _ptr(scale), _stream()))


def sar_rgcn_basis(a: torch.Tensor, V: torch.Tensor, W: torch.Tensor) -> None:
    """a [R,B], V [B,...] float32; W [R,...] bf16 or float32."""
    R, Bn = a.shape
    size = V.numel() // Bn
    _check("sar_rgcn_basis", lib().sar_rgcn_basis(c_int32(R), c_int32(Bn), c_int64(size), ctypes.c_int(_dtype(W)),
                                                  _ptr(a), _ptr(V), _ptr(W), _stream()))


def sar_rgcn_basis_bwd(a: torch.Tensor, V: torch.Tensor, dW: torch.Tensor, da: torch.Tensor, dV: torch.Tensor) -> None:
    R, Bn = a.shape
    size = V.numel() // Bn
    _check("sar_rgcn_basis_bwd", lib().sar_rgcn_basis_bwd(c_int32(R), c_int32(Bn), c_int64(size), _ptr(a), _ptr(V),
                                                          _ptr(dW), _ptr(da), _ptr(dV), _stream()))


def sar_linear_bwd_input(dz: torch.Tensor, w: torch.Tensor, dh: torch.Tensor, workspace: torch.Tensor) -> None:
    n, d_out = dz.shape
    d_in = w.shape[0]
    ws, wb = _ws(workspace)
    _check("sar_linear_bwd_input", lib().sar_linear_bwd_input(c_int64(n), c_int32(d_in), c_int32(d_out),
                                                              ctypes.c_int(_dtype(dz)), _ptr(dz), _ptr(w), _ptr(dh), ws,
                                                              wb, _stream()))


def sar_linear_bwd_weight(h: torch.Tensor, dz: torch.Tensor, dw: torch.Tensor, workspace: torch.Tensor) -> None:
    n, d_in = h.shape
    d_out = dz.shape[1]
    ws, wb = _ws(workspace)
    _check("sar_linear_bwd_weight", lib().sar_linear_bwd_weight(c_int64(n), c_int32(d_in), c_int32(d_out),
                                                                ctypes.c_int(_dtype(h)), _ptr(h), _ptr(dz), _ptr(dw), ws,
                                                                wb, _stream()))


def sar_dropout(x: torch.Tensor, p: float, seed: int, y: torch.Tensor) -> None:
    _check("sar_dropout", lib().sar_dropout(c_int64(x.numel()), ctypes.c_int(_dtype(x)), _ptr(x), c_float(p),
                                            ctypes.c_uint64(seed & 0xFFFFFFFFFFFFFFFF), _ptr(y), _stream()))


def sar_axpby(a: float, x: torch.Tensor, b: float, y: torch.Tensor) -> None:
    """y = a*x + b*y."""
    assert x.numel() == y.numel() and x.dtype == y.dtype
    _check("sar_axpby", lib().sar_axpby(c_int64(x.numel()), ctypes.c_int(_dtype(x)), c_float(a), _ptr(x), c_float(b),
                                        _ptr(y), _stream()))


def sar_accumulate(x: torch.Tensor, acc: torch.Tensor, first: bool = False) -> None:
    """acc (float32) += x, or acc = x with first=True."""
    assert x.numel() == acc.numel() and acc.dtype == torch.float32
    _check("sar_accumulate", lib().sar_accumulate(c_int64(x.numel()), ctypes.c_int(_dtype(x)), _ptr(x), _ptr(acc),
                                                  c_uint32(SAR_FIRST if first else 0), _stream()))


def sar_round_to(acc: torch.Tensor, y: torch.Tensor) -> None:
    assert y.numel() == acc.numel() and acc.dtype == torch.float32
    _check("sar_round_to", lib().sar_round_to(c_int64(acc.numel()), ctypes.c_int(_dtype(y)), _ptr(acc), _ptr(y),
                                              _stream()))


def sar_relu_bwd(y: torch.Tensor, g: torch.Tensor) -> None:
    _check("sar_relu_bwd", lib().sar_relu_bwd(c_int64(y.numel()), ctypes.c_int(_dtype(y)), _ptr(y), _ptr(g), _stream()))

// Lean span kernels, bwd dst pass, bf16 storage (see sar_lean_kernels.cuh).
#include "sar_lean_kernels.cuh"

SAR_LEAN_TU(bwd_dst_bf16, __nv_bfloat16, sar::kBwdDst, "gat_bwd_dst", "gat_bwd_dst_seg")

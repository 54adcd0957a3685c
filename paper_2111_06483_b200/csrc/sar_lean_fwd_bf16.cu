// Lean span kernels, fwd pass, bf16 storage (see sar_lean_kernels.cuh).
#include "sar_lean_kernels.cuh"

SAR_LEAN_TU(fwd_bf16, __nv_bfloat16, sar::kFwd, "gat_fwd", "gat_fwd_seg")

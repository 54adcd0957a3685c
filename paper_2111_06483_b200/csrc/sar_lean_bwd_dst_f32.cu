// Lean span kernels, bwd dst pass, float32 storage (see sar_lean_kernels.cuh).
#include "sar_lean_kernels.cuh"

SAR_LEAN_TU(bwd_dst_f32, float, sar::kBwdDst, "gat_bwd_dst", "gat_bwd_dst_seg")

// Lean span kernels, fwd pass, float32 storage (see sar_lean_kernels.cuh).
#include "sar_lean_kernels.cuh"

SAR_LEAN_TU(fwd_f32, float, sar::kFwd, "gat_fwd", "gat_fwd_seg")

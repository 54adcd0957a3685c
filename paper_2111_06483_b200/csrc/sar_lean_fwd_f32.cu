// Lean span kernel of the forward pass, float32 storage (see sar_lean_fwd_kernels.cuh).
#include "sar_lean_fwd_kernels.cuh"

SAR_LEAN_FWD_TU(f32, float)

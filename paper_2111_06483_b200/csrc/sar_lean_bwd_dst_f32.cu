// Lean span kernel of the destination-major backward pass, float32 storage (see sar_lean_dst_kernels.cuh).
#include "sar_lean_dst_kernels.cuh"

SAR_LEAN_DST_TU(f32, float)

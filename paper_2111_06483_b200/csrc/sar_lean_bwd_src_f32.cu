// Lean span kernel of the source-major backward pass, float32 storage (see sar_lean_src_kernels.cuh).
#include "sar_lean_src_kernels.cuh"

SAR_LEAN_SRC_TU(f32, float)

// Lean span kernel of the source-major backward pass, bf16 storage (see sar_lean_src_kernels.cuh).
#include "sar_lean_src_kernels.cuh"

SAR_LEAN_SRC_TU(bf16, __nv_bfloat16)

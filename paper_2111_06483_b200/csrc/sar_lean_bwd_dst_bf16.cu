// Lean span kernel of the destination-major backward pass, bf16 storage (see sar_lean_dst_kernels.cuh).
#include "sar_lean_dst_kernels.cuh"

SAR_LEAN_DST_TU(bf16, __nv_bfloat16)

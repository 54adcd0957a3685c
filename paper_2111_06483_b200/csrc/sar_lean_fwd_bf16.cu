// Lean span kernel of the forward pass, bf16 storage (see sar_lean_fwd_kernels.cuh).
#include "sar_lean_fwd_kernels.cuh"

SAR_LEAN_FWD_TU(bf16, __nv_bfloat16)

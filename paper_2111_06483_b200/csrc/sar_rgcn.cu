// The small pieces a relational layer (Appendix A) needs besides the aggregation and the dense
// contraction: the per-relation factor 1/|N_i^r| as an array (the backward pass of the mean applies it on the
// gather side), and the basis decomposition of the relation weights, W_r = sum_b a_rb V_b, with its backward
// pass.  Contracts are in include/sar.h.  Fixed summation orders, no atomics.
#include "sar_common.cuh"

#include <cuda_bf16.h>

namespace sar {

__global__ void degree_scale_kernel(long long n, const int64_t *__restrict__ indptr, float power, float *__restrict__ scale) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        const long long deg = indptr[i + 1] - indptr[i];
        float v = 0.f;
        if (deg > 0) v = power == -1.f ? 1.f / (float)deg : (power == -0.5f ? rsqrtf((float)deg) : powf((float)deg, power));
        scale[i] = v;
    }
}

// W[r, x] = sum_b a[r, b] V[b, x]; one thread per x, b ascending
template <typename T>
__global__ void basis_kernel(int R, int Bn, long long size, const float *__restrict__ a, const float *__restrict__ V, T *__restrict__ W) {
    for (long long x = blockIdx.x * (long long)blockDim.x + threadIdx.x; x < size; x += (long long)gridDim.x * blockDim.x)
        for (int r = 0; r < R; ++r) {
            float acc = 0.f;
            for (int b = 0; b < Bn; ++b) acc = fmaf(a[r * Bn + b], V[b * size + x], acc);
            if constexpr (sizeof(T) == 4) W[r * size + x] = acc;
            else W[r * size + x] = __float2bfloat16_rn(acc);
        }
}

// dV[b, x] = sum_r a[r, b] dW[r, x]; one thread per x, r ascending
__global__ void basis_bwd_v_kernel(int R, int Bn, long long size, const float *__restrict__ a, const float *__restrict__ dW, float *__restrict__ dV) {
    for (long long x = blockIdx.x * (long long)blockDim.x + threadIdx.x; x < size; x += (long long)gridDim.x * blockDim.x)
        for (int b = 0; b < Bn; ++b) {
            float acc = 0.f;
            for (int r = 0; r < R; ++r) acc = fmaf(a[r * Bn + b], dW[r * size + x], acc);
            dV[b * size + x] = acc;
        }
}

// da[r, b] = <dW[r, :], V[b, :]>; one block per (r, b): strided partial sums in float64, a fixed tree across the block
__global__ void basis_bwd_a_kernel(int Bn, long long size, const float *__restrict__ dW, const float *__restrict__ V, float *__restrict__ da) {
    const int r = blockIdx.x / Bn, b = blockIdx.x % Bn;
    double acc = 0.0;
    for (long long x = threadIdx.x; x < size; x += blockDim.x) acc += (double)dW[r * size + x] * (double)V[b * size + x];
    __shared__ double part[256];
    part[threadIdx.x] = acc;
    __syncthreads();
    for (int off = 128; off > 0; off >>= 1) {
        if ((int)threadIdx.x < off) part[threadIdx.x] += part[threadIdx.x + off];
        __syncthreads();
    }
    if (threadIdx.x == 0) da[blockIdx.x] = (float)part[0];
}

static unsigned grid_for(long long work) {
    long long blocks = (work + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (blocks < 1) blocks = 1;
    return (unsigned)blocks;
}

}  // namespace sar

using namespace sar;

extern "C" {

sar_status sar_degree_scale(int64_t n, const int64_t *indptr, float power, float *scale, void *stream) {
    if (n < 0 || !indptr || (n > 0 && !scale)) return SAR_ERR_INVALID_ARG;
    if (!(power <= 0.f)) return SAR_ERR_INVALID_ARG;  // a normalisation: degree to a non-positive power
    if (n == 0) return SAR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SAR_LAUNCH("degree_scale", st, (degree_scale_kernel<<<grid_for(n), 256, 0, st>>>(n, indptr, power, scale)));
    return sar_after_launch();
}

sar_status sar_rgcn_basis(int32_t R, int32_t B, int64_t size, sar_dtype t, const float *a, const float *V, void *W, void *stream) {
    if (R < 1 || B < 1 || size < 0 || !a || (size > 0 && (!V || !W))) return SAR_ERR_INVALID_ARG;
    if (t != SAR_F32 && t != SAR_BF16) return SAR_ERR_INVALID_ARG;
    if (size == 0) return SAR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (t == SAR_F32)
        SAR_LAUNCH("rgcn_basis", st, (basis_kernel<float><<<grid_for(size), 256, 0, st>>>(R, B, size, a, V, static_cast<float *>(W))));
    else
        SAR_LAUNCH("rgcn_basis", st, (basis_kernel<__nv_bfloat16><<<grid_for(size), 256, 0, st>>>(R, B, size, a, V, static_cast<__nv_bfloat16 *>(W))));
    return sar_after_launch();
}

sar_status sar_rgcn_basis_bwd(int32_t R, int32_t B, int64_t size, const float *a, const float *V, const float *dW, float *da,
                              float *dV, void *stream) {
    if (R < 1 || B < 1 || size < 0 || !a || !da || (size > 0 && (!V || !dW || !dV))) return SAR_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (size == 0) return cudaMemsetAsync(da, 0, sizeof(float) * (size_t)R * B, st) == cudaSuccess ? SAR_OK : SAR_ERR_CUDA;
    SAR_LAUNCH("rgcn_basis_bwd_v", st, (basis_bwd_v_kernel<<<grid_for(size), 256, 0, st>>>(R, B, size, a, dW, dV)));
    SAR_TRY(sar_after_launch());
    SAR_LAUNCH("rgcn_basis_bwd_a", st, (basis_bwd_a_kernel<<<(unsigned)(R * B), 256, 0, st>>>(B, size, dW, V, da)));
    return sar_after_launch();
}

}  // extern "C"

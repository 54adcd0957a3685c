// The non-rematerialising baseline: a deliberately plain two-step implementation of the same layer that WRITES the
// attention coefficients alpha[E,H] in the forward pass and READS them back in the backward pass (the usual
// implementation the paper's Sec. 4.1 compares its fused kernels with; Sec. 3.3 explains what fusing avoids).
// It exists so that the memory and the run time of keeping O(E*H) attention can be MEASURED next to the
// rematerialising path; nothing else in the library calls it.  One warp per row, no staging, no tuning.
// Contracts are in include/sar.h.
#include "sar_common.cuh"

namespace sar {

struct StoringArgs {
    long long n_dst, n_src, nnz;
    const int64_t *indptr;
    const int32_t *indices;
    const int64_t *t_indptr;
    const int32_t *t_indices;
    const void *feat, *gout;
    const float *el, *er;
    float *alpha;        // [nnz,H] in CSR order
    float *ds;           // [nnz,H] per-edge score gradient, CSR order
    int32_t *eid;        // [nnz] CSC position -> CSR edge index
    void *out, *dfeat;
    float *del, *der;
    int H, F;
    float slope;
};

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}
__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}

// step 1 of the forward pass: edge scores, softmax over each destination's in-edges, coefficients to memory
__global__ void storing_alpha_kernel(const StoringArgs a) {
    const long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= a.n_dst) return;
    const long long beg = a.indptr[row], end = a.indptr[row + 1];
    for (int h = 0; h < a.H; ++h) {
        const float el_i = a.el[row * a.H + h];
        float mx = SAR_NEG_INF;
        for (long long t = beg + lane; t < end; t += 32) {
            float gr;
            mx = fmaxf(mx, leaky(el_i + a.er[(long long)a.indices[t] * a.H + h], a.slope, gr));
        }
        mx = warp_max(mx);
        float sum = 0.f;
        for (long long t = beg + lane; t < end; t += 32) {
            float gr;
            const float w = expf(leaky(el_i + a.er[(long long)a.indices[t] * a.H + h], a.slope, gr) - mx);
            a.alpha[t * a.H + h] = w;
            sum += w;
        }
        sum = warp_sum(sum);
        const float inv = sum > 0.f ? 1.f / sum : 0.f;
        for (long long t = beg + lane; t < end; t += 32) a.alpha[t * a.H + h] *= inv;   // each lane rescales what it wrote
    }
}

// step 2: out[i] = sum_t alpha[t] * feat[col_t], lanes across the H*F columns
template <typename T>
__global__ void storing_spmm_kernel(const StoringArgs a) {
    const long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= a.n_dst) return;
    const long long beg = a.indptr[row], end = a.indptr[row + 1];
    const int HF = a.H * a.F;
    const T *feat = reinterpret_cast<const T *>(a.feat);
    T *out = reinterpret_cast<T *>(a.out) + row * HF;
    for (int c0 = 0; c0 < HF; c0 += 128) {   // four columns per lane at a time
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (long long t = beg; t < end; ++t) {
            const long long j = a.indices[t];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int c = c0 + 32 * u + lane;
                if (c < HF) acc[u] = fmaf(a.alpha[t * a.H + c / a.F], Elem<T>::load1(feat + j * HF + c), acc[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int c = c0 + 32 * u + lane;
            if (c < HF) Elem<T>::store1(out + c, acc[u]);
        }
    }
}

// backward, destination-major: dalpha[t,h] = <gout_i, feat_j>, D = sum alpha*dalpha, ds = alpha*(dalpha - D)*g', del = sum ds
template <typename T>
__global__ void storing_bwd_dst_kernel(const StoringArgs a) {
    const long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= a.n_dst) return;
    const long long beg = a.indptr[row], end = a.indptr[row + 1];
    const int HF = a.H * a.F;
    const T *feat = reinterpret_cast<const T *>(a.feat);
    const T *gout = reinterpret_cast<const T *>(a.gout) + row * HF;
    for (int h = 0; h < a.H; ++h) {
        float D = 0.f;
        for (long long t = beg; t < end; ++t) {
            const long long j = a.indices[t];
            float p = 0.f;
            for (int f = lane; f < a.F; f += 32)
                p = fmaf(Elem<T>::load1(gout + h * a.F + f), Elem<T>::load1(feat + j * HF + h * a.F + f), p);
            p = warp_sum(p);
            if (lane == 0) a.ds[t * a.H + h] = p;   // dalpha for now
            D = fmaf(a.alpha[t * a.H + h], p, D);
        }
        __syncwarp();
        const float el_i = a.el[row * a.H + h];
        float sum = 0.f;
        for (long long t = beg + lane; t < end; t += 32) {
            const float s = el_i + a.er[(long long)a.indices[t] * a.H + h];
            const float v = a.alpha[t * a.H + h] * (a.ds[t * a.H + h] - D) * (s > 0.f ? 1.f : a.slope);
            a.ds[t * a.H + h] = v;
            sum += v;
        }
        sum = warp_sum(sum);
        if (lane == 0) a.del[row * a.H + h] = sum;
    }
}

__device__ __forceinline__ long long lower_bound_i32(const int32_t *__restrict__ p, long long lo, long long hi, int key) {
    while (lo < hi) {
        const long long mid = (lo + hi) >> 1;
        if (p[mid] < key) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// CSC position -> CSR edge index (the k-th copy of a duplicate edge maps to the k-th copy)
__global__ void storing_edge_map_kernel(const StoringArgs a) {
    const long long j = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (j >= a.n_src) return;
    const long long beg = a.t_indptr[j], end = a.t_indptr[j + 1];
    for (long long t = beg + lane; t < end; t += 32) {
        const int i = a.t_indices[t];
        const long long rank = t - lower_bound_i32(a.t_indices, beg, end, i);
        a.eid[t] = (int32_t)(lower_bound_i32(a.indices, a.indptr[i], a.indptr[i + 1], (int)j) + rank);
    }
}

// backward, source-major: dfeat[j] = sum_i alpha * gout_i, der[j] = sum_i ds, both read through the edge map
template <typename T>
__global__ void storing_bwd_src_kernel(const StoringArgs a) {
    const long long j = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (j >= a.n_src) return;
    const long long beg = a.t_indptr[j], end = a.t_indptr[j + 1];
    const int HF = a.H * a.F;
    const T *gout = reinterpret_cast<const T *>(a.gout);
    T *dfeat = reinterpret_cast<T *>(a.dfeat) + j * HF;
    for (int c0 = 0; c0 < HF; c0 += 128) {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (long long t = beg; t < end; ++t) {
            const long long i = a.t_indices[t], e = a.eid[t];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int c = c0 + 32 * u + lane;
                if (c < HF) acc[u] = fmaf(a.alpha[e * a.H + c / a.F], Elem<T>::load1(gout + i * HF + c), acc[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int c = c0 + 32 * u + lane;
            if (c < HF) Elem<T>::store1(dfeat + c, acc[u]);
        }
    }
    for (int h = 0; h < a.H; ++h) {
        float sum = 0.f;
        for (long long t = beg + lane; t < end; t += 32) sum += a.ds[(long long)a.eid[t] * a.H + h];
        sum = warp_sum(sum);
        if (lane == 0) a.der[j * a.H + h] = sum;
    }
}

static unsigned warp_blocks(long long rows) { return (unsigned)((rows * 32 + 255) / 256); }

}  // namespace sar

using namespace sar;

extern "C" {

size_t sar_gat_storing_workspace_bytes(const sar_part *g, int32_t H) {
    if (!g || H < 1) return 0;
    return sar_round_up((size_t)g->nnz * H * 4, 256) + sar_round_up((size_t)g->nnz * 4, 256) + 256;
}

sar_status sar_gat_fwd_storing(const sar_part *g, const void *feat, const float *el, const float *er, int32_t H,
                               int32_t F, sar_dtype t, float slope, float *alpha, void *out, void *stream) {
    if (!g || !g->indptr || H < 1 || F < 1 || !el || !out) return SAR_ERR_INVALID_ARG;
    if (t != SAR_F32 && t != SAR_BF16) return SAR_ERR_INVALID_ARG;
    if (g->nnz > 0 && (!g->indices || !feat || !er || !alpha)) return SAR_ERR_INVALID_ARG;
    if (g->n_dst == 0) return SAR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    StoringArgs a{};
    a.n_dst = g->n_dst;
    a.n_src = g->n_src;
    a.nnz = g->nnz;
    a.indptr = g->indptr;
    a.indices = g->indices;
    a.feat = feat;
    a.el = el;
    a.er = er;
    a.alpha = alpha;
    a.out = out;
    a.H = H;
    a.F = F;
    a.slope = slope;
    SAR_LAUNCH("storing_alpha", st, storing_alpha_kernel<<<warp_blocks(g->n_dst), 256, 0, st>>>(a));
    SAR_TRY(sar_after_launch());
    if (t == SAR_F32)
        SAR_LAUNCH("storing_spmm", st, storing_spmm_kernel<float><<<warp_blocks(g->n_dst), 256, 0, st>>>(a));
    else
        SAR_LAUNCH("storing_spmm", st, storing_spmm_kernel<__nv_bfloat16><<<warp_blocks(g->n_dst), 256, 0, st>>>(a));
    return sar_after_launch();
}

sar_status sar_gat_bwd_storing(const sar_part *g, const void *feat, const float *el, const float *er,
                               const float *alpha, const void *gout, int32_t H, int32_t F, sar_dtype t, float slope,
                               void *dfeat, float *del, float *der, void *workspace, size_t workspace_bytes,
                               void *stream) {
    if (!g || !g->indptr || !g->t_indptr || H < 1 || F < 1 || !el || !gout || !del) return SAR_ERR_INVALID_ARG;
    if (t != SAR_F32 && t != SAR_BF16) return SAR_ERR_INVALID_ARG;
    if (g->nnz > 0 && (!g->indices || !g->t_indices || !feat || !er || !alpha)) return SAR_ERR_INVALID_ARG;
    if (g->n_src > 0 && (!dfeat || !der)) return SAR_ERR_INVALID_ARG;
    if (g->nnz > INT32_MAX) return SAR_ERR_UNSUPPORTED;   // the edge map is 32-bit
    if (!workspace || !sar_aligned(workspace, 16) || workspace_bytes < sar_gat_storing_workspace_bytes(g, H))
        return SAR_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    StoringArgs a{};
    a.n_dst = g->n_dst;
    a.n_src = g->n_src;
    a.nnz = g->nnz;
    a.indptr = g->indptr;
    a.indices = g->indices;
    a.t_indptr = g->t_indptr;
    a.t_indices = g->t_indices;
    a.feat = feat;
    a.gout = gout;
    a.el = el;
    a.er = er;
    a.alpha = const_cast<float *>(alpha);
    a.ds = static_cast<float *>(workspace);
    a.eid = reinterpret_cast<int32_t *>(static_cast<char *>(workspace) + sar_round_up((size_t)g->nnz * H * 4, 256));
    a.dfeat = dfeat;
    a.del = del;
    a.der = der;
    a.H = H;
    a.F = F;
    a.slope = slope;
    if (g->n_dst > 0) {
        if (t == SAR_F32)
            SAR_LAUNCH("storing_bwd_dst", st, storing_bwd_dst_kernel<float><<<warp_blocks(g->n_dst), 256, 0, st>>>(a));
        else
            SAR_LAUNCH("storing_bwd_dst", st, storing_bwd_dst_kernel<__nv_bfloat16><<<warp_blocks(g->n_dst), 256, 0, st>>>(a));
        SAR_TRY(sar_after_launch());
    }
    if (g->n_src > 0) {
        SAR_LAUNCH("storing_edge_map", st, storing_edge_map_kernel<<<warp_blocks(g->n_src), 256, 0, st>>>(a));
        SAR_TRY(sar_after_launch());
        if (t == SAR_F32)
            SAR_LAUNCH("storing_bwd_src", st, storing_bwd_src_kernel<float><<<warp_blocks(g->n_src), 256, 0, st>>>(a));
        else
            SAR_LAUNCH("storing_bwd_src", st, storing_bwd_src_kernel<__nv_bfloat16><<<warp_blocks(g->n_src), 256, 0, st>>>(a));
        SAR_TRY(sar_after_launch());
    }
    return SAR_OK;
}

}  // extern "C"

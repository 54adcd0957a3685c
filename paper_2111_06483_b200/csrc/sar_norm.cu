// Batch normalisation over the node dimension (Sec. 3.4, "Batch normalization"): per-column statistics of a
// node array x[n, C], the normalisation, and its backward pass, split so that a worker that holds only some
// of the rows can combine its statistics with the other workers' before applying them.  Streaming kernels;
// contracts are in include/sar.h.
#include "sar_dispatch.cuh"
#include "sar_rowkernels.cuh"

namespace sar {

constexpr int kNormBlocks = 148 * 8;  // fixed grid of the reducing kernels: a fixed summation order

struct NormArgs {
    long long n;
    int C;
    const void *x;
    const void *gy;
    void *y;                     // apply: y; backward apply: gx
    const float *mean, *rstd;    // [C]
    const float *gamma, *beta;   // [C] or null
    const float *s0, *s1;        // backward apply: sum gy, sum gy*xhat
    float inv_count;
    float *partial;              // [blocks][2][C]
    RowGeom g;
    // optional chain after the normalisation, y = dropout(relu(bn(x))) (the paper's networks, Sec. 4.2), and its
    // mirror in front of the backward pass: the incoming gradient is masked by the dropout and the ReLU first
    unsigned act;                // bit 0 (SAR_GLUE_RELU), bit 1 (SAR_GLUE_DROPOUT)
    unsigned threshold;          // floor(p * 2^24)
    float scale;                 // 1 / (1 - p)
    unsigned long long seed;
    const void *post;            // backward: y as the forward chain left it
};

// forward chain on one element of flat index idx
// ACT (template argument of the kernels): 0 = no chain, 3 = ReLU and dropout (the networks' case, decided at compile
// time so that the backward kernels carry no generator code), 1 = whatever NormArgs::act says.
template <int ACT>
__device__ __forceinline__ float act_fwd(const NormArgs &a, float o, long long idx) {
    const unsigned act = ACT == 3 ? 3u : a.act;
    if (act & 1u) o = o > 0.f ? o : 0.f;
    if (act & 2u) o = (unsigned)(splitmix64_at(a.seed, (unsigned long long)idx) >> 40) >= a.threshold ? o * a.scale : 0.f;
    return o;
}
// the gradient that reaches the normalisation's output: through the dropout (kept and scaled, or 0) and the ReLU.
// With both, y > 0 exactly where the ReLU passed and the mask kept, so the stored y decides alone.
template <int ACT>
__device__ __forceinline__ float act_bwd(const NormArgs &a, float g, float post, long long idx) {
    if constexpr (ACT == 3) return post > 0.f ? g * a.scale : 0.f;
    if ((a.act & 3u) == 3u) return post > 0.f ? g * a.scale : 0.f;
    if (a.act & 2u) g = (unsigned)(splitmix64_at(a.seed, (unsigned long long)idx) >> 40) >= a.threshold ? g * a.scale : 0.f;
    if (a.act & 1u) g = post > 0.f ? g : 0.f;
    return g;
}

enum NormSum { kSumX = 0, kSumDev2 = 1, kSumGrad = 2 };

__device__ __forceinline__ float nrm_as_float(float x) { return x; }
__device__ __forceinline__ float nrm_as_float(__nv_bfloat16 x) { return __bfloat162float(x); }

// the EPV per-column constants that meet lane (gl, v)'s vector; `fill` where the pointer is null or out of range
template <int G, int V, int EPV>
__device__ __forceinline__ void load_cols(const float *__restrict__ p, float fill, const RowGeom &g, int gl,
                                          float (&c)[V][EPV]) {
#pragma unroll
    for (int v = 0; v < V; ++v) {
        const int vi = v * G + gl;
#pragma unroll
        for (int e = 0; e < EPV; ++e) c[v][e] = (p && vi < g.n_vec) ? __ldg(p + vi * EPV + e) : fill;
    }
}

// Column sums over the block's rows: WHAT = kSumX: sum x; kSumDev2: sum (x - mean)^2; kSumGrad: sum gy and
// sum gy * xhat with xhat = (x - mean) * rstd.  Per-block partials, no atomics.
template <typename T, int G, int V, int WHAT, int ACT = 0>
__global__ void __launch_bounds__(kThreads) norm_sums_kernel(const NormArgs a) {
    constexpr int EPV = Elem<T>::EPV;
    constexpr int RPW = 32 / G;
    constexpr int GPB = kWarpsPerBlock * RPW;
    extern __shared__ __align__(16) float smem[];  // [GPB][2][G*V*EPV]
    const LaneId<G> id;
    const VecGeom<G, V> vg(a.g, id.gl);
    float mu[V][EPV], rs[V][EPV], s0[V][EPV], s1[V][EPV];
    load_cols<G, V, EPV>(WHAT == kSumX ? nullptr : a.mean, 0.f, a.g, id.gl, mu);
    load_cols<G, V, EPV>(WHAT == kSumGrad ? a.rstd : nullptr, 1.f, a.g, id.gl, rs);
#pragma unroll
    for (int v = 0; v < V; ++v)
#pragma unroll
        for (int e = 0; e < EPV; ++e) s0[v][e] = s1[v][e] = 0.f;
    const long long stride = (long long)gridDim.x * GPB;
    const int group = id.warp * RPW + id.gid;
    for (long long row = (long long)blockIdx.x * GPB + group; row < a.n; row += stride) {
        float xv[V][EPV], gv[V][EPV];
        load_row_vec<T, G, V>(a.x, row, a.g.n_vec, id.gl, vg.vok, xv);
        if constexpr (WHAT == kSumGrad) {
            load_row_vec<T, G, V>(a.gy, row, a.g.n_vec, id.gl, vg.vok, gv);
            if constexpr (ACT != 0) {
                float pv[V][EPV];
#pragma unroll
                for (int v = 0; v < V; ++v)
#pragma unroll
                    for (int e = 0; e < EPV; ++e) pv[v][e] = 0.f;
                if (ACT == 3 || (a.act & 1u)) load_row_vec<T, G, V>(a.post, row, a.g.n_vec, id.gl, vg.vok, pv);
#pragma unroll
                for (int v = 0; v < V; ++v)
#pragma unroll
                    for (int e = 0; e < EPV; ++e)
                        gv[v][e] = vg.vok[v] ? act_bwd<ACT>(a, gv[v][e], pv[v][e], row * a.C + (v * G + id.gl) * EPV + e) : 0.f;
            }
        }
#pragma unroll
        for (int v = 0; v < V; ++v)
#pragma unroll
            for (int e = 0; e < EPV; ++e) {
                if constexpr (WHAT == kSumX) {
                    s0[v][e] += xv[v][e];
                } else if constexpr (WHAT == kSumDev2) {
                    const float dlt = xv[v][e] - mu[v][e];
                    s0[v][e] = fmaf(dlt, dlt, s0[v][e]);
                } else {
                    s0[v][e] += gv[v][e];
                    s1[v][e] = fmaf(gv[v][e], (xv[v][e] - mu[v][e]) * rs[v][e], s1[v][e]);
                }
            }
    }
    const int rowf = G * V * EPV;
    float *mine = smem + (size_t)group * 2 * rowf;
#pragma unroll
    for (int v = 0; v < V; ++v)
#pragma unroll
        for (int e = 0; e < EPV; ++e) {
            mine[(v * G + id.gl) * EPV + e] = s0[v][e];
            mine[rowf + (v * G + id.gl) * EPV + e] = s1[v][e];
        }
    __syncthreads();
    for (int x = threadIdx.x; x < 2 * a.C; x += blockDim.x) {
        const int which = x / a.C, o = x - which * a.C;  // o < C <= rowf
        float acc = 0.f;
        for (int gq = 0; gq < GPB; ++gq) acc += smem[(size_t)gq * 2 * rowf + which * rowf + o];
        a.partial[(size_t)blockIdx.x * 2 * a.C + x] = acc;
    }
}

// block partials -> totals, accumulated in float64; out0 / out1 may be null.  scale multiplies both.
__global__ void norm_reduce_kernel(int blocks, int C, const float *__restrict__ partial, double scale,
                                   float *__restrict__ out0, float *__restrict__ out1) {
    const int x = blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= 2 * C) return;
    double acc = 0.0;
    for (int b = 0; b < blocks; ++b) acc += (double)partial[(size_t)b * 2 * C + x];
    acc *= scale;
    if (x < C) {
        if (out0) out0[x] = (float)acc;
    } else if (out1) {
        out1[x - C] = (float)acc;
    }
}

// y = (x - mean) * rstd * gamma + beta             (BWD = false)
// gx = gamma * rstd * (gy - s0/N - xhat * s1/N)    (BWD = true; inv_count = 1/N)
template <typename T, int G, int V, bool BWD, int ACT = 0>
__global__ void __launch_bounds__(kThreads) norm_apply_kernel(const NormArgs a) {
    constexpr int EPV = Elem<T>::EPV;
    constexpr int RPW = 32 / G;
    const LaneId<G> id;
    const VecGeom<G, V> vg(a.g, id.gl);
    float mu[V][EPV], rs[V][EPV], ga[V][EPV], be[V][EPV], m0[V][EPV], m1[V][EPV];
    load_cols<G, V, EPV>(a.mean, 0.f, a.g, id.gl, mu);
    load_cols<G, V, EPV>(a.rstd, 1.f, a.g, id.gl, rs);
    load_cols<G, V, EPV>(a.gamma, 1.f, a.g, id.gl, ga);
    load_cols<G, V, EPV>(BWD ? nullptr : a.beta, 0.f, a.g, id.gl, be);
    load_cols<G, V, EPV>(BWD ? a.s0 : nullptr, 0.f, a.g, id.gl, m0);
    load_cols<G, V, EPV>(BWD ? a.s1 : nullptr, 0.f, a.g, id.gl, m1);
    const long long stride = (long long)gridDim.x * kWarpsPerBlock * RPW;
    for (long long row = ((long long)blockIdx.x * kWarpsPerBlock + id.warp) * RPW + id.gid; row < a.n; row += stride) {
        float xv[V][EPV], gv[V][EPV], ov[V][EPV];
        // plain loads: the output may be the same array as x or gy
        load_row_vec<T, G, V, false>(a.x, row, a.g.n_vec, id.gl, vg.vok, xv);
        if constexpr (BWD) {
            load_row_vec<T, G, V, false>(a.gy, row, a.g.n_vec, id.gl, vg.vok, gv);
            if constexpr (ACT != 0) {
                float pv[V][EPV];
#pragma unroll
                for (int v = 0; v < V; ++v)
#pragma unroll
                    for (int e = 0; e < EPV; ++e) pv[v][e] = 0.f;
                if (ACT == 3 || (a.act & 1u)) load_row_vec<T, G, V, false>(a.post, row, a.g.n_vec, id.gl, vg.vok, pv);
#pragma unroll
                for (int v = 0; v < V; ++v)
#pragma unroll
                    for (int e = 0; e < EPV; ++e)
                        gv[v][e] = vg.vok[v] ? act_bwd<ACT>(a, gv[v][e], pv[v][e], row * a.C + (v * G + id.gl) * EPV + e) : 0.f;
            }
        }
#pragma unroll
        for (int v = 0; v < V; ++v)
#pragma unroll
            for (int e = 0; e < EPV; ++e) {
                const float xh = (xv[v][e] - mu[v][e]) * rs[v][e];
                if constexpr (BWD) {
                    ov[v][e] = ga[v][e] * rs[v][e] * (gv[v][e] - m0[v][e] * a.inv_count - xh * (m1[v][e] * a.inv_count));
                } else {
                    ov[v][e] = fmaf(xh, ga[v][e], be[v][e]);
                    if constexpr (ACT != 0) ov[v][e] = act_fwd<ACT>(a, ov[v][e], row * a.C + (v * G + id.gl) * EPV + e);
                }
            }
        store_row_vec<T, G, V>(a.y, row, a.g.n_vec, id.gl, vg.vok, ov);
    }
}

// scalar fallbacks: thread (slice, column) walks every `slices`-th row; partials as in the vector kernel
template <typename T, int WHAT>
__global__ void norm_sums_generic(const NormArgs a, int slices) {
    const long long id = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (id >= (long long)slices * a.C) return;
    const int slice = (int)(id / a.C), c = (int)(id - (long long)slice * a.C);
    const T *x = reinterpret_cast<const T *>(a.x);
    const T *gy = reinterpret_cast<const T *>(a.gy);
    float s0 = 0.f, s1 = 0.f;
    const float mu = WHAT == kSumX ? 0.f : a.mean[c], rs = WHAT == kSumGrad ? a.rstd[c] : 1.f;
    for (long long i = slice; i < a.n; i += slices) {
        const float xv = nrm_as_float(x[i * a.C + c]);
        if (WHAT == kSumX) {
            s0 += xv;
        } else if (WHAT == kSumDev2) {
            s0 = fmaf(xv - mu, xv - mu, s0);
        } else {
            float g = nrm_as_float(gy[i * a.C + c]);
            if (a.act) g = act_bwd<1>(a, g, (a.act & 1u) ? nrm_as_float(reinterpret_cast<const T *>(a.post)[i * a.C + c]) : 0.f, i * a.C + c);
            s0 += g;
            s1 = fmaf(g, (xv - mu) * rs, s1);
        }
    }
    a.partial[(size_t)slice * 2 * a.C + c] = s0;
    a.partial[(size_t)slice * 2 * a.C + a.C + c] = s1;
}

template <typename T, bool BWD>
__global__ void norm_apply_generic(const NormArgs a) {
    const long long total = a.n * a.C;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(i % a.C);
        const float xh = (nrm_as_float(reinterpret_cast<const T *>(a.x)[i]) - a.mean[c]) * a.rstd[c];
        const float ga = a.gamma ? a.gamma[c] : 1.f;
        float o;
        if (BWD) {
            float g = nrm_as_float(reinterpret_cast<const T *>(a.gy)[i]);
            if (a.act) g = act_bwd<1>(a, g, (a.act & 1u) ? nrm_as_float(reinterpret_cast<const T *>(a.post)[i]) : 0.f, i);
            o = ga * a.rstd[c] * (g - a.s0[c] * a.inv_count - xh * (a.s1[c] * a.inv_count));
        } else {
            o = fmaf(xh, ga, a.beta ? a.beta[c] : 0.f);
            if (a.act) o = act_fwd<1>(a, o, i);
        }
        Elem<T>::store1(reinterpret_cast<T *>(a.y) + i, o);
    }
}

static sar_status norm_shape(int64_t n, int32_t C, sar_dtype t, std::initializer_list<const void *> ps, Shape *s) {
    if (n < 0 || C < 1) return SAR_ERR_INVALID_ARG;
    return make_shape(1, C, t, all16(ps), s);
}

// one column-sum pass; scale multiplies the totals (e.g. 1/n for a mean)
template <int WHAT>
static sar_status norm_sums(const Shape &s, NormArgs a, double scale, float *out0, float *out1, void *workspace,
                            size_t workspace_bytes, cudaStream_t st, const char *name) {
    if (!workspace || !sar_aligned(workspace, 16) || workspace_bytes < (size_t)kNormBlocks * 2 * a.C * 4) return SAR_ERR_WORKSPACE;
    a.partial = static_cast<float *>(workspace);
    if (!s.fast) {
        long long slices = (a.n + 63) / 64;
        if (slices > kNormBlocks) slices = kNormBlocks;
        const unsigned blocks = (unsigned)((slices * a.C + 255) / 256);
        if (s.t == SAR_F32)
            SAR_LAUNCH(name, st, (norm_sums_generic<float, WHAT><<<blocks, 256, 0, st>>>(a, (int)slices)));
        else
            SAR_LAUNCH(name, st, (norm_sums_generic<__nv_bfloat16, WHAT><<<blocks, 256, 0, st>>>(a, (int)slices)));
        SAR_TRY(sar_after_launch());
        SAR_LAUNCH("bn_reduce", st, norm_reduce_kernel<<<(2 * a.C + 255) / 256, 256, 0, st>>>((int)slices, a.C, a.partial, scale, out0, out1));
        return sar_after_launch();
    }
    return dispatch(s, [&](auto cfg) -> sar_status {
        using C = decltype(cfg);
        using T = typename C::type;
        constexpr int EPV = Elem<T>::EPV;
        const size_t smem = (size_t)kWarpsPerBlock * (32 / C::g) * 2 * (C::g * C::v * EPV) * 4;
        auto kern = (WHAT != kSumGrad || a.act == 0) ? norm_sums_kernel<T, C::g, C::v, WHAT, 0>
                    : (a.act == 3 ? norm_sums_kernel<T, C::g, C::v, WHAT, (WHAT == kSumGrad ? 3 : 0)>
                                  : norm_sums_kernel<T, C::g, C::v, WHAT, (WHAT == kSumGrad ? 1 : 0)>);
        SAR_TRY(ensure_smem(kern, smem));
        SAR_LAUNCH(name, st, kern<<<kNormBlocks, kThreads, smem, st>>>(a));
        SAR_TRY(sar_after_launch());
        SAR_LAUNCH("bn_reduce", st, norm_reduce_kernel<<<(2 * a.C + 255) / 256, 256, 0, st>>>(kNormBlocks, a.C, a.partial, scale, out0, out1));
        return sar_after_launch();
    });
}

template <bool BWD>
static sar_status norm_apply(const Shape &s, const NormArgs &a, cudaStream_t st, const char *name) {
    if (!s.fast) {
        long long blocks = (a.n * a.C + 255) / 256;
        if (blocks > 148 * 64) blocks = 148 * 64;
        if (s.t == SAR_F32)
            SAR_LAUNCH(name, st, (norm_apply_generic<float, BWD><<<(unsigned)blocks, 256, 0, st>>>(a)));
        else
            SAR_LAUNCH(name, st, (norm_apply_generic<__nv_bfloat16, BWD><<<(unsigned)blocks, 256, 0, st>>>(a)));
        return sar_after_launch();
    }
    return dispatch(s, [&](auto cfg) -> sar_status {
        using C = decltype(cfg);
        using T = typename C::type;
        unsigned blocks = blocks_for(a.n, C::g);
        if (blocks > (unsigned)kNormBlocks * 4) blocks = kNormBlocks * 4;
        auto kern = a.act == 0 ? norm_apply_kernel<T, C::g, C::v, BWD, 0>
                               : (a.act == 3 ? norm_apply_kernel<T, C::g, C::v, BWD, 3> : norm_apply_kernel<T, C::g, C::v, BWD, 1>);
        SAR_LAUNCH(name, st, (kern<<<blocks, kThreads, 0, st>>>(a)));
        return sar_after_launch();
    });
}

}  // namespace sar

using namespace sar;

namespace sar {
// rstd[c] = 1 / sqrt(m2[c] / count + eps): the last step of the statistics, on C floats
__global__ void norm_rstd_kernel(int C, const float *__restrict__ m2, double inv_count, float eps, float *__restrict__ rstd) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c < C) rstd[c] = (float)(1.0 / sqrt((double)m2[c] * inv_count + (double)eps));
}
}  // namespace sar

namespace sar {
static sar_status norm_set_act(NormArgs &a, uint32_t flags, float p, uint64_t seed, const void *post, bool backward) {
    if (flags & ~(uint32_t)(SAR_GLUE_RELU | SAR_GLUE_DROPOUT)) return SAR_ERR_INVALID_ARG;
    a.act = flags;
    a.threshold = 0;
    a.scale = 1.f;
    a.seed = seed;
    a.post = post;
    if (flags & SAR_GLUE_DROPOUT) {
        if (!(p >= 0.f && p < 1.f)) return SAR_ERR_INVALID_ARG;
        a.threshold = (unsigned)((double)p * 16777216.0);  // floor(p * 2^24), as sar_dropout
        a.scale = 1.f / (1.f - p);
    }
    if (backward && (flags & SAR_GLUE_RELU) && a.n > 0 && !post) return SAR_ERR_INVALID_ARG;
    return SAR_OK;
}
}  // namespace sar

extern "C" {

sar_status sar_bn_combine_moments(int32_t R, int32_t C, const int64_t *n_r, const float *mean_r, const float *m2_r,
                                  int64_t *n_all, float *mean, float *m2) {
    if (R < 1 || C < 0 || !n_r || !n_all || (C > 0 && (!mean_r || !m2_r || !mean || !m2))) return SAR_ERR_INVALID_ARG;
    long long N = 0;
    for (int r = 0; r < R; ++r) {
        if (n_r[r] < 0) return SAR_ERR_INVALID_ARG;
        N += n_r[r];
    }
    *n_all = N;
    for (int c = 0; c < C; ++c) {
        double mu = 0.0;
        for (int r = 0; r < R; ++r) mu += (double)n_r[r] * (double)mean_r[(size_t)r * C + c];
        mu = N > 0 ? mu / (double)N : 0.0;
        double q = 0.0;
        for (int r = 0; r < R; ++r) {
            const double dm = (double)mean_r[(size_t)r * C + c] - mu;
            q += (double)m2_r[(size_t)r * C + c] + (double)n_r[r] * dm * dm;
        }
        mean[c] = (float)mu;
        m2[c] = (float)q;
    }
    return SAR_OK;
}

sar_status sar_bn_combine_sums(int32_t R, int64_t count, const float *sums_r, float *sums) {
    if (R < 1 || count < 0 || (count > 0 && (!sums_r || !sums))) return SAR_ERR_INVALID_ARG;
    for (int64_t c = 0; c < count; ++c) {
        double acc = 0.0;
        for (int r = 0; r < R; ++r) acc += (double)sums_r[(size_t)r * count + c];   // rank order: the same on every worker
        sums[c] = (float)acc;
    }
    return SAR_OK;
}

size_t sar_bn_workspace_bytes(int32_t C) {
    if (C < 1) return 0;
    return (size_t)kNormBlocks * 2 * C * 4 + 256;
}

sar_status sar_bn_stats(int64_t n, int32_t C, sar_dtype t, const void *x, float *mean, float *m2, void *workspace,
                        size_t workspace_bytes, void *stream) {
    if (!mean || !m2 || (n > 0 && !x)) return SAR_ERR_INVALID_ARG;
    Shape s;
    SAR_TRY(norm_shape(n, C, t, {x}, &s));
    SAR_TRY(check_elem_align({mean, m2}, 4));
    SAR_TRY(check_elem_align({x}, sar_elem_size(t)));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n == 0) {
        SAR_CUDA_TRY(cudaMemsetAsync(mean, 0, (size_t)C * 4, st));
        SAR_CUDA_TRY(cudaMemsetAsync(m2, 0, (size_t)C * 4, st));
        return SAR_OK;
    }
    NormArgs a{};
    a.n = n;
    a.C = C;
    a.x = x;
    a.g = s.geom;
    // two passes: the mean first, then the squared deviations from it (no cancellation)
    SAR_TRY(norm_sums<kSumX>(s, a, 1.0 / (double)n, mean, nullptr, workspace, workspace_bytes, st, "bn_mean"));
    a.mean = mean;
    return norm_sums<kSumDev2>(s, a, 1.0, m2, nullptr, workspace, workspace_bytes, st, "bn_m2");
}

sar_status sar_bn_rstd(int32_t C, const float *m2, int64_t count, float eps, float *rstd, void *stream) {
    if (C < 1 || count < 1 || !m2 || !rstd || !(eps >= 0.f)) return SAR_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SAR_LAUNCH("bn_rstd", st, (sar::norm_rstd_kernel<<<(unsigned)((C + 127) / 128), 128, 0, st>>>(C, m2, 1.0 / (double)count, eps, rstd)));
    return sar_after_launch();
}

sar_status sar_bn_apply(int64_t n, int32_t C, sar_dtype t, const void *x, const float *mean, const float *rstd,
                        const float *gamma, const float *beta, void *y, void *stream) {
    if (!mean || !rstd || (n > 0 && (!x || !y))) return SAR_ERR_INVALID_ARG;
    Shape s;
    SAR_TRY(norm_shape(n, C, t, {x, y}, &s));
    SAR_TRY(check_elem_align({mean, rstd, gamma, beta}, 4));
    SAR_TRY(check_elem_align({x, y}, sar_elem_size(t)));
    if (n == 0) return SAR_OK;
    NormArgs a{};
    a.n = n;
    a.C = C;
    a.x = x;
    a.y = y;
    a.mean = mean;
    a.rstd = rstd;
    a.gamma = gamma;
    a.beta = beta;
    a.g = s.geom;
    return norm_apply<false>(s, a, static_cast<cudaStream_t>(stream), "bn_apply");
}

sar_status sar_bn_bwd_stats(int64_t n, int32_t C, sar_dtype t, const void *x, const float *mean, const float *rstd,
                            const void *gy, float *sum_gy, float *sum_gy_xhat, void *workspace,
                            size_t workspace_bytes, void *stream) {
    if (!mean || !rstd || !sum_gy || !sum_gy_xhat || (n > 0 && (!x || !gy))) return SAR_ERR_INVALID_ARG;
    Shape s;
    SAR_TRY(norm_shape(n, C, t, {x, gy}, &s));
    SAR_TRY(check_elem_align({mean, rstd, sum_gy, sum_gy_xhat}, 4));
    SAR_TRY(check_elem_align({x, gy}, sar_elem_size(t)));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n == 0) {
        SAR_CUDA_TRY(cudaMemsetAsync(sum_gy, 0, (size_t)C * 4, st));
        SAR_CUDA_TRY(cudaMemsetAsync(sum_gy_xhat, 0, (size_t)C * 4, st));
        return SAR_OK;
    }
    NormArgs a{};
    a.n = n;
    a.C = C;
    a.x = x;
    a.gy = gy;
    a.mean = mean;
    a.rstd = rstd;
    a.g = s.geom;
    return norm_sums<kSumGrad>(s, a, 1.0, sum_gy, sum_gy_xhat, workspace, workspace_bytes, st, "bn_bwd_sums");
}

sar_status sar_bn_bwd_apply(int64_t n, int32_t C, sar_dtype t, const void *x, const float *mean, const float *rstd,
                            const float *gamma, const void *gy, const float *sum_gy, const float *sum_gy_xhat,
                            float inv_count, void *gx, void *stream) {
    if (!mean || !rstd || !sum_gy || !sum_gy_xhat || (n > 0 && (!x || !gy || !gx))) return SAR_ERR_INVALID_ARG;
    Shape s;
    SAR_TRY(norm_shape(n, C, t, {x, gy, gx}, &s));
    SAR_TRY(check_elem_align({mean, rstd, gamma, sum_gy, sum_gy_xhat}, 4));
    SAR_TRY(check_elem_align({x, gy, gx}, sar_elem_size(t)));
    if (n == 0) return SAR_OK;
    NormArgs a{};
    a.n = n;
    a.C = C;
    a.x = x;
    a.gy = gy;
    a.y = gx;
    a.mean = mean;
    a.rstd = rstd;
    a.gamma = gamma;
    a.s0 = sum_gy;
    a.s1 = sum_gy_xhat;
    a.inv_count = inv_count;
    a.g = s.geom;
    return norm_apply<true>(s, a, static_cast<cudaStream_t>(stream), "bn_bwd_apply");
}

sar_status sar_bn_apply_act(int64_t n, int32_t C, sar_dtype t, const void *x, const float *mean, const float *rstd,
                            const float *gamma, const float *beta, uint32_t flags, float p, uint64_t seed, void *y,
                            void *stream) {
    if (!mean || !rstd || (n > 0 && (!x || !y))) return SAR_ERR_INVALID_ARG;
    Shape s;
    SAR_TRY(norm_shape(n, C, t, {x, y}, &s));
    SAR_TRY(check_elem_align({mean, rstd, gamma, beta}, 4));
    SAR_TRY(check_elem_align({x, y}, sar_elem_size(t)));
    NormArgs a{};
    a.n = n;
    a.C = C;
    a.x = x;
    a.y = y;
    a.mean = mean;
    a.rstd = rstd;
    a.gamma = gamma;
    a.beta = beta;
    a.g = s.geom;
    SAR_TRY(norm_set_act(a, flags, p, seed, nullptr, false));
    if (n == 0) return SAR_OK;
    return norm_apply<false>(s, a, static_cast<cudaStream_t>(stream), "bn_apply_act");
}

sar_status sar_bn_bwd_stats_act(int64_t n, int32_t C, sar_dtype t, const void *x, const float *mean, const float *rstd,
                                const void *gy, const void *post, uint32_t flags, float p, uint64_t seed, float *sum_gy,
                                float *sum_gy_xhat, void *workspace, size_t workspace_bytes, void *stream) {
    if (!mean || !rstd || !sum_gy || !sum_gy_xhat || (n > 0 && (!x || !gy))) return SAR_ERR_INVALID_ARG;
    Shape s;
    SAR_TRY(norm_shape(n, C, t, {x, gy, post}, &s));
    SAR_TRY(check_elem_align({mean, rstd, sum_gy, sum_gy_xhat}, 4));
    SAR_TRY(check_elem_align({x, gy, post}, sar_elem_size(t)));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    NormArgs a{};
    a.n = n;
    a.C = C;
    a.x = x;
    a.gy = gy;
    a.mean = mean;
    a.rstd = rstd;
    a.g = s.geom;
    SAR_TRY(norm_set_act(a, flags, p, seed, post, true));
    if (n == 0) {
        SAR_CUDA_TRY(cudaMemsetAsync(sum_gy, 0, (size_t)C * 4, st));
        SAR_CUDA_TRY(cudaMemsetAsync(sum_gy_xhat, 0, (size_t)C * 4, st));
        return SAR_OK;
    }
    return norm_sums<kSumGrad>(s, a, 1.0, sum_gy, sum_gy_xhat, workspace, workspace_bytes, st, "bn_bwd_sums_act");
}

sar_status sar_bn_bwd_apply_act(int64_t n, int32_t C, sar_dtype t, const void *x, const float *mean, const float *rstd,
                                const float *gamma, const void *gy, const void *post, uint32_t flags, float p,
                                uint64_t seed, const float *sum_gy, const float *sum_gy_xhat, float inv_count, void *gx,
                                void *stream) {
    if (!mean || !rstd || !sum_gy || !sum_gy_xhat || (n > 0 && (!x || !gy || !gx))) return SAR_ERR_INVALID_ARG;
    Shape s;
    SAR_TRY(norm_shape(n, C, t, {x, gy, gx, post}, &s));
    SAR_TRY(check_elem_align({mean, rstd, gamma, sum_gy, sum_gy_xhat}, 4));
    SAR_TRY(check_elem_align({x, gy, gx, post}, sar_elem_size(t)));
    NormArgs a{};
    a.n = n;
    a.C = C;
    a.x = x;
    a.gy = gy;
    a.y = gx;
    a.mean = mean;
    a.rstd = rstd;
    a.gamma = gamma;
    a.s0 = sum_gy;
    a.s1 = sum_gy_xhat;
    a.inv_count = inv_count;
    a.g = s.geom;
    SAR_TRY(norm_set_act(a, flags, p, seed, post, true));
    if (n == 0) return SAR_OK;
    return norm_apply<true>(s, a, static_cast<cudaStream_t>(stream), "bn_bwd_apply_act");
}

}  // extern "C"

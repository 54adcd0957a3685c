// The GAT layer around the aggregation (Eq. 3): score projections el = <z, a_left>, er = <z, a_right>
// per head, their backward pass (chain-rule add into dz, gradients of a), and the element-wise ReLU
// between layers.  Streaming kernels; contracts are in include/sar.h.
#include "sar_dispatch.cuh"
#include "sar_rowkernels.cuh"

namespace sar {

constexpr int kGlueBlocks = 148 * 8;  // fixed grid of the reducing kernel: a fixed summation order

struct ProjArgs {
    long long n;
    const void *feat;
    const float *a_l, *a_r;  // [H,F]
    float *el, *er;          // forward: written
    const float *del, *der;  // backward: read
    void *dfeat;             // backward: dfeat += a_l*del + a_r*der (in place)
    float *partial;          // backward: [blocks][2][H*F]
    int H, F;
    RowGeom g;
};

// lane (gl, v) -> the EPV coefficients of a[h, :] that meet its vector
template <int G, int V, int EPV>
__device__ __forceinline__ void load_coeffs(const float *__restrict__ a, const RowGeom &g, int F, int gl,
                                            float (&c)[V][EPV]) {
#pragma unroll
    for (int v = 0; v < V; ++v) {
        const int vi = v * G + gl;
#pragma unroll
        for (int e = 0; e < EPV; ++e) c[v][e] = 0.f;
        if (vi < g.n_vec) {
            const int h = vi / g.vph, f0 = (vi - h * g.vph) * EPV;
#pragma unroll
            for (int e = 0; e < EPV; ++e) c[v][e] = __ldg(a + h * F + f0 + e);
        }
    }
}

// RELU: z = max(z, 0) is written back before it is projected (the ReLU that closes the previous layer).
template <typename T, int G, int V, bool RELU>
__global__ void __launch_bounds__(kThreads) project_kernel(const ProjArgs a) {
    constexpr int EPV = Elem<T>::EPV;
    constexpr int RPW = 32 / G;
    constexpr int U = V <= 2 ? 2 : 1;  // rows in flight per group
    extern __shared__ __align__(16) float smem[];
    const LaneId<G> id;
    float *scratch = smem + (size_t)id.warp * (32 * V) + id.gid * (G * V);
    const VecGeom<G, V> vg(a.g, id.gl);
    float cl[V][EPV], cr[V][EPV];
    load_coeffs<G, V, EPV>(a.a_l, a.g, a.F, id.gl, cl);
    load_coeffs<G, V, EPV>(a.a_r, a.g, a.F, id.gl, cr);
    const bool pow2_heads = (a.g.vph & (a.g.vph - 1)) == 0 && a.g.vph <= G;
    const long long stride = (long long)gridDim.x * kWarpsPerBlock * RPW;
    const long long first = ((long long)blockIdx.x * kWarpsPerBlock + id.warp) * RPW + id.gid;
    // every lane of the warp runs the same number of sweeps (the head sums are warp-wide)
    const long long sweeps = (a.n + stride * U - 1) / (stride * U);
    for (long long s = 0; s < sweeps; ++s) {
        float fv[U][V][EPV];
        long long row[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            row[u] = first + (s * U + u) * stride;
#pragma unroll
            for (int v = 0; v < V; ++v)
#pragma unroll
                for (int e = 0; e < EPV; ++e) fv[u][v][e] = 0.f;
            if (row[u] < a.n) load_row_vec<T, G, V, !RELU>(a.feat, row[u], a.g.n_vec, id.gl, vg.vok, fv[u]);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const bool active = row[u] < a.n;
            float pl[V], pr[V];
            if constexpr (RELU) {
#pragma unroll
                for (int v = 0; v < V; ++v)
#pragma unroll
                    for (int e = 0; e < EPV; ++e) fv[u][v][e] = fv[u][v][e] > 0.f ? fv[u][v][e] : 0.f;
                if (active) store_row_vec<T, G, V>(const_cast<void *>(a.feat), row[u], a.g.n_vec, id.gl, vg.vok, fv[u]);
            }
#pragma unroll
            for (int v = 0; v < V; ++v) {
                pl[v] = pr[v] = 0.f;
#pragma unroll
                for (int e = 0; e < EPV; ++e) {
                    pl[v] = fmaf(fv[u][v][e], cl[v][e], pl[v]);
                    pr[v] = fmaf(fv[u][v][e], cr[v][e], pr[v]);
                }
            }
            if (V == 1 && pow2_heads) {
                // a head is vph adjacent lanes: fold them with shuffles, the head's first lane writes
                float L = pl[0], R = pr[0];
                for (int o = 1; o < a.g.vph; o <<= 1) {
                    L += __shfl_xor_sync(0xffffffffu, L, o);
                    R += __shfl_xor_sync(0xffffffffu, R, o);
                }
                if (active && vg.vok[0] && (id.gl & (a.g.vph - 1)) == 0) {
                    a.el[row[u] * a.H + vg.hv[0]] = L;
                    a.er[row[u] * a.H + vg.hv[0]] = R;
                }
            } else {
                const float L = head_sum<G, V>(scratch, pl, vg.vok, id.gl, a.g);
                const float R = head_sum<G, V>(scratch, pr, vg.vok, id.gl, a.g);
                if (active && id.gl < a.H) {
                    a.el[row[u] * a.H + id.gl] = L;
                    a.er[row[u] * a.H + id.gl] = R;
                }
            }
        }
    }
}

// dfeat += a_l*del + a_r*der; per-block partial sums of del*feat and der*feat over the block's rows.
// MASK: the updated dfeat is then zeroed where feat <= 0 (feat being a ReLU's output, this is that
// ReLU's backward pass).
template <typename T, int G, int V, bool MASK>
__global__ void __launch_bounds__(kThreads) project_bwd_kernel(const ProjArgs a) {
    constexpr int EPV = Elem<T>::EPV;
    constexpr int RPW = 32 / G;
    constexpr int GPB = kWarpsPerBlock * RPW;  // groups per block
    extern __shared__ __align__(16) float smem[];  // [GPB][2][G*V*EPV]
    const LaneId<G> id;
    const VecGeom<G, V> vg(a.g, id.gl);
    float cl[V][EPV], cr[V][EPV], sl[V][EPV], sr[V][EPV];
    load_coeffs<G, V, EPV>(a.a_l, a.g, a.F, id.gl, cl);
    load_coeffs<G, V, EPV>(a.a_r, a.g, a.F, id.gl, cr);
#pragma unroll
    for (int v = 0; v < V; ++v)
#pragma unroll
        for (int e = 0; e < EPV; ++e) sl[v][e] = sr[v][e] = 0.f;
    const long long stride = (long long)gridDim.x * GPB;
    const int group = id.warp * RPW + id.gid;
    for (long long row = (long long)blockIdx.x * GPB + group; row < a.n; row += stride) {
        float fv[V][EPV], gv[V][EPV];
        load_row_vec<T, G, V>(a.feat, row, a.g.n_vec, id.gl, vg.vok, fv);
        load_row_vec<T, G, V, false>(a.dfeat, row, a.g.n_vec, id.gl, vg.vok, gv);
#pragma unroll
        for (int v = 0; v < V; ++v) {
            float dl = 0.f, dr = 0.f;
            if (vg.vok[v]) {
                dl = __ldg(a.del + row * a.H + vg.hv[v]);
                dr = __ldg(a.der + row * a.H + vg.hv[v]);
            }
#pragma unroll
            for (int e = 0; e < EPV; ++e) {
                gv[v][e] += cl[v][e] * dl + cr[v][e] * dr;
                if constexpr (MASK) gv[v][e] = fv[v][e] > 0.f ? gv[v][e] : 0.f;
                sl[v][e] = fmaf(dl, fv[v][e], sl[v][e]);
                sr[v][e] = fmaf(dr, fv[v][e], sr[v][e]);
            }
        }
        store_row_vec<T, G, V>(a.dfeat, row, a.g.n_vec, id.gl, vg.vok, gv);
    }
    // block reduction in a fixed order: group 0 adds the other groups' sums
    const int rowf = G * V * EPV;
    float *mine = smem + (size_t)group * 2 * rowf;
#pragma unroll
    for (int v = 0; v < V; ++v)
#pragma unroll
        for (int e = 0; e < EPV; ++e) {
            mine[(v * G + id.gl) * EPV + e] = sl[v][e];
            mine[rowf + (v * G + id.gl) * EPV + e] = sr[v][e];
        }
    __syncthreads();
    const int HF = a.H * a.F;
    for (int x = threadIdx.x; x < 2 * HF; x += blockDim.x) {
        const int which = x / HF, o = x - which * HF;  // o < H*F <= rowf
        float acc = 0.f;
        for (int gq = 0; gq < GPB; ++gq) acc += smem[(size_t)gq * 2 * rowf + which * rowf + o];
        a.partial[(size_t)blockIdx.x * 2 * HF + x] = acc;
    }
}

__global__ void project_reduce_kernel(int blocks, int HF, const float *__restrict__ partial, float *__restrict__ da_l,
                                      float *__restrict__ da_r) {
    const int x = blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= 2 * HF) return;
    float acc = 0.f;
    for (int b = 0; b < blocks; ++b) acc += partial[(size_t)b * 2 * HF + x];
    if (x < HF) da_l[x] = acc; else da_r[x - HF] = acc;
}

__device__ __forceinline__ float as_float(float x) { return x; }
__device__ __forceinline__ float as_float(__nv_bfloat16 x) { return __bfloat162float(x); }

// scalar fallbacks
template <typename T>
__global__ void project_generic(const ProjArgs a, bool relu) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= a.n * a.H) return;
    const int h = (int)(idx % a.H);
    T *f = reinterpret_cast<T *>(const_cast<void *>(a.feat)) + idx * a.F;
    float L = 0.f, R = 0.f;
    for (int k = 0; k < a.F; ++k) {
        float x = as_float(f[k]);
        if (relu) {
            x = x > 0.f ? x : 0.f;
            Elem<T>::store1(f + k, x);
        }
        L = fmaf(x, a.a_l[h * a.F + k], L);
        R = fmaf(x, a.a_r[h * a.F + k], R);
    }
    a.el[idx] = L;
    a.er[idx] = R;
}

template <typename T>
__global__ void project_bwd_generic(const ProjArgs a, float *da_l, float *da_r, bool mask) {
    const long long HF = (long long)a.H * a.F;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < HF) {  // one thread per coefficient walks every node in order
        const int h = (int)(idx / a.F);
        float L = 0.f, R = 0.f;
        for (long long i = 0; i < a.n; ++i) {
            const float x = Elem<T>::load1(reinterpret_cast<const T *>(a.feat) + i * HF + idx);
            L = fmaf(a.del[i * a.H + h], x, L);
            R = fmaf(a.der[i * a.H + h], x, R);
        }
        da_l[idx] = L;
        da_r[idx] = R;
    }
    for (long long x = idx; x < a.n * HF; x += (long long)gridDim.x * blockDim.x) {
        const long long i = x / HF;
        const int o = (int)(x - i * HF), h = o / a.F;
        T *p = reinterpret_cast<T *>(a.dfeat) + x;
        float v = as_float(*p) + a.a_l[o] * a.del[i * a.H + h] + a.a_r[o] * a.der[i * a.H + h];
        if (mask && !(Elem<T>::load1(reinterpret_cast<const T *>(a.feat) + x) > 0.f)) v = 0.f;
        Elem<T>::store1(p, v);
    }
}

// forward: x = max(x, 0) in place; backward: g = 0 where the layer's output y is not positive.
// 16 bytes per thread where both arrays are 16-byte aligned; the ragged tail (and unaligned arrays) one
// element at a time.
template <typename T, bool BWD>
__global__ void relu_kernel(long long n, const T *y, T *x, long long n_vec16) {
    constexpr int EPV = Elem<T>::EPV;
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long nthreads = (long long)gridDim.x * blockDim.x;
    for (long long i = tid; i < n_vec16; i += nthreads) {
        uint4 *xp = reinterpret_cast<uint4 *>(x) + i;
        float xv[EPV], yv[EPV];
        Elem<T>::unpack(*xp, xv);
        if constexpr (BWD) Elem<T>::unpack(__ldg(reinterpret_cast<const uint4 *>(y) + i), yv);
#pragma unroll
        for (int e = 0; e < EPV; ++e) {
            const float v = BWD ? yv[e] : xv[e];
            if (!(v > 0.f)) xv[e] = 0.f;
        }
        *xp = Elem<T>::pack(xv);
    }
    for (long long i = n_vec16 * EPV + tid; i < n; i += nthreads) {
        const float v = as_float(BWD ? y[i] : x[i]);
        if (!(v > 0.f)) Elem<T>::store1(x + i, 0.f);
    }
}

template <typename T, bool BWD>
static sar_status launch_relu(const char *name, int64_t n, const void *y, void *x, cudaStream_t st) {
    const bool vec = sar_aligned(x, 16) && (!BWD || sar_aligned(y, 16));
    const long long n_vec16 = vec ? n / Elem<T>::EPV : 0;
    const long long work = n_vec16 > 0 ? n_vec16 : n;
    long long blocks = (work + 255) / 256;
    if (blocks > 148 * 64) blocks = 148 * 64;
    SAR_LAUNCH(name, st, (relu_kernel<T, BWD><<<(unsigned)blocks, 256, 0, st>>>(n, static_cast<const T *>(y), static_cast<T *>(x), n_vec16)));
    return sar_after_launch();
}


// y = a*x + b*y, element-wise in float32 (the mixing step X <- (1-alpha) X0 + alpha S X of a propagation, Sec. 4.2)
template <typename T>
__global__ void axpby_kernel(long long n, float ca, const T *x, float cb, T *y, long long n_vec16) {
    constexpr int EPV = Elem<T>::EPV;
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long nthreads = (long long)gridDim.x * blockDim.x;
    for (long long i = tid; i < n_vec16; i += nthreads) {
        uint4 *yp = reinterpret_cast<uint4 *>(y) + i;
        float xv[EPV], yv[EPV];
        Elem<T>::unpack(__ldg(reinterpret_cast<const uint4 *>(x) + i), xv);
        Elem<T>::unpack(*yp, yv);
#pragma unroll
        for (int e = 0; e < EPV; ++e) yv[e] = fmaf(ca, xv[e], cb * yv[e]);
        *yp = Elem<T>::pack(yv);
    }
    for (long long i = n_vec16 * EPV + tid; i < n; i += nthreads)
        Elem<T>::store1(y + i, fmaf(ca, as_float(x[i]), cb * as_float(y[i])));
}

// acc[i] (+)= x[i] with x of the storage type and acc float32 (sums of the errors the other workers return,
// Algorithm 2), and the rounding of such a sum back to the storage type
template <typename T, bool ADD>
__global__ void widen_kernel(long long n, const T *__restrict__ x, float *__restrict__ acc) {
    const long long nthreads = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += nthreads)
        acc[i] = ADD ? acc[i] + as_float(x[i]) : as_float(x[i]);
}
template <typename T>
__global__ void narrow_kernel(long long n, const float *__restrict__ acc, T *__restrict__ y) {
    const long long nthreads = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += nthreads) Elem<T>::store1(y + i, acc[i]);
}


// ---- dropout (the paper's networks use batch normalisation and dropout between all layers, Sec. 4.2) ------
// Counter-based: element i is kept when the top 24 bits of SplitMix64's (i+1)-th output for `seed` reach
// p * 2^24; nothing is stored, the backward pass draws the same mask again from the seed.

template <typename T>
__global__ void dropout_kernel(long long n, const T *x, T *y, unsigned threshold, float scale, unsigned long long seed,
                               long long n_vec16) {
    constexpr int EPV = Elem<T>::EPV;
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long nthreads = (long long)gridDim.x * blockDim.x;
    for (long long v = tid; v < n_vec16; v += nthreads) {
        float f[EPV];
        Elem<T>::unpack(reinterpret_cast<const uint4 *>(x)[v], f);  // plain load: y may be x
#pragma unroll
        for (int e = 0; e < EPV; ++e) {
            const unsigned r = (unsigned)(splitmix64_at(seed, (unsigned long long)(v * EPV + e)) >> 40);
            f[e] = r >= threshold ? f[e] * scale : 0.f;
        }
        reinterpret_cast<uint4 *>(y)[v] = Elem<T>::pack(f);
    }
    for (long long i = n_vec16 * EPV + tid; i < n; i += nthreads) {
        const unsigned r = (unsigned)(splitmix64_at(seed, (unsigned long long)i) >> 40);
        Elem<T>::store1(y + i, r >= threshold ? as_float(x[i]) * scale : 0.f);
    }
}

static sar_status glue_shape(int64_t n, int32_t H, int32_t F, sar_dtype t, std::initializer_list<const void *> ps,
                             Shape *s) {
    if (n < 0 || H < 1 || F < 1) return SAR_ERR_INVALID_ARG;
    return make_shape(H, F, t, all16(ps), s);
}

}  // namespace sar

using namespace sar;

extern "C" {

size_t sar_gat_project_workspace_bytes(int32_t H, int32_t F) {
    if (H < 1 || F < 1) return 0;
    return (size_t)kGlueBlocks * 2 * H * F * 4 + 256;
}

sar_status sar_gat_project(int64_t n, int32_t H, int32_t F, sar_dtype t, void *feat, const float *a_l,
                           const float *a_r, float *el, float *er, uint32_t flags, void *stream) {
    if (flags & ~(uint32_t)SAR_GLUE_RELU) return SAR_ERR_INVALID_ARG;
    const bool relu = (flags & SAR_GLUE_RELU) != 0;
    if (!a_l || !a_r || (n > 0 && (!feat || !el || !er))) return SAR_ERR_INVALID_ARG;
    Shape s;
    SAR_TRY(glue_shape(n, H, F, t, {feat}, &s));
    SAR_TRY(check_elem_align({a_l, a_r, el, er}, 4));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n == 0) return SAR_OK;
    ProjArgs a{};
    a.n = n;
    a.feat = feat;
    a.a_l = a_l;
    a.a_r = a_r;
    a.el = el;
    a.er = er;
    a.H = H;
    a.F = F;
    a.g = s.geom;
    if (!s.fast) {
        const unsigned blocks = (unsigned)((n * H + 255) / 256);
        if (t == SAR_F32)
            SAR_LAUNCH("gat_project_generic", st, project_generic<float><<<blocks, 256, 0, st>>>(a, relu));
        else
            SAR_LAUNCH("gat_project_generic", st, project_generic<__nv_bfloat16><<<blocks, 256, 0, st>>>(a, relu));
        return sar_after_launch();
    }
    return dispatch(s, [&](auto cfg) -> sar_status {
        using C = decltype(cfg);
        using T = typename C::type;
        const size_t smem = (size_t)kWarpsPerBlock * 32 * C::v * 4;
        unsigned blocks = blocks_for(n, C::g);
        if (blocks > (unsigned)kGlueBlocks * 4) blocks = kGlueBlocks * 4;
        if (relu)
            SAR_LAUNCH("gat_project", st, (project_kernel<T, C::g, C::v, true><<<blocks, kThreads, smem, st>>>(a)));
        else
            SAR_LAUNCH("gat_project", st, (project_kernel<T, C::g, C::v, false><<<blocks, kThreads, smem, st>>>(a)));
        return sar_after_launch();
    });
}

sar_status sar_gat_project_bwd(int64_t n, int32_t H, int32_t F, sar_dtype t, const void *feat, const float *a_l,
                               const float *a_r, const float *del, const float *der, void *dfeat, float *da_l,
                               float *da_r, uint32_t flags, void *workspace, size_t workspace_bytes, void *stream) {
    if (flags & ~(uint32_t)SAR_GLUE_RELU) return SAR_ERR_INVALID_ARG;
    const bool mask = (flags & SAR_GLUE_RELU) != 0;
    if (!a_l || !a_r || !da_l || !da_r || (n > 0 && (!feat || !del || !der || !dfeat))) return SAR_ERR_INVALID_ARG;
    Shape s;
    SAR_TRY(glue_shape(n, H, F, t, {feat, dfeat}, &s));
    SAR_TRY(check_elem_align({a_l, a_r, del, der, da_l, da_r}, 4));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    ProjArgs a{};
    a.n = n;
    a.feat = feat;
    a.a_l = a_l;
    a.a_r = a_r;
    a.del = del;
    a.der = der;
    a.dfeat = dfeat;
    a.H = H;
    a.F = F;
    a.g = s.geom;
    const int HF = H * F;
    if (!s.fast) {
        long long work = (long long)n * HF > HF ? (long long)n * HF : HF;
        unsigned blocks = (unsigned)((work + 255) / 256);
        if (blocks > 65535u * 16) blocks = 65535u * 16;
        if (t == SAR_F32)
            SAR_LAUNCH("gat_project_bwd_generic", st, project_bwd_generic<float><<<blocks, 256, 0, st>>>(a, da_l, da_r, mask));
        else
            SAR_LAUNCH("gat_project_bwd_generic", st, project_bwd_generic<__nv_bfloat16><<<blocks, 256, 0, st>>>(a, da_l, da_r, mask));
        return sar_after_launch();
    }
    if (!workspace || !sar_aligned(workspace, 16) || workspace_bytes < (size_t)kGlueBlocks * 2 * HF * 4) return SAR_ERR_WORKSPACE;
    a.partial = static_cast<float *>(workspace);
    return dispatch(s, [&](auto cfg) -> sar_status {
        using C = decltype(cfg);
        using T = typename C::type;
        constexpr int EPV = Elem<T>::EPV;
        const size_t smem = (size_t)kWarpsPerBlock * (32 / C::g) * 2 * (C::g * C::v * EPV) * 4;
        auto kern = mask ? project_bwd_kernel<T, C::g, C::v, true> : project_bwd_kernel<T, C::g, C::v, false>;
        SAR_TRY(ensure_smem(project_bwd_kernel<T, C::g, C::v, true>, smem));
        SAR_TRY(ensure_smem(project_bwd_kernel<T, C::g, C::v, false>, smem));
        SAR_LAUNCH("gat_project_bwd", st, kern<<<kGlueBlocks, kThreads, smem, st>>>(a));
        SAR_TRY(sar_after_launch());
        SAR_LAUNCH("gat_project_reduce", st,
                   project_reduce_kernel<<<(2 * HF + 255) / 256, 256, 0, st>>>(kGlueBlocks, HF, a.partial, da_l, da_r));
        return sar_after_launch();
    });
}

sar_status sar_relu(int64_t n_elems, sar_dtype t, void *x, void *stream) {
    if (n_elems < 0 || (n_elems > 0 && !x)) return SAR_ERR_INVALID_ARG;
    if (t != SAR_F32 && t != SAR_BF16) return SAR_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n_elems == 0) return SAR_OK;
    if (t == SAR_F32) return launch_relu<float, false>("relu", n_elems, nullptr, x, st);
    return launch_relu<__nv_bfloat16, false>("relu", n_elems, nullptr, x, st);
}

sar_status sar_relu_bwd(int64_t n_elems, sar_dtype t, const void *y, void *g, void *stream) {
    if (n_elems < 0 || (n_elems > 0 && (!y || !g))) return SAR_ERR_INVALID_ARG;
    if (t != SAR_F32 && t != SAR_BF16) return SAR_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n_elems == 0) return SAR_OK;
    if (t == SAR_F32) return launch_relu<float, true>("relu_bwd", n_elems, y, g, st);
    return launch_relu<__nv_bfloat16, true>("relu_bwd", n_elems, y, g, st);
}

sar_status sar_dropout(int64_t n_elems, sar_dtype t, const void *x, float p, uint64_t seed, void *y, void *stream) {
    if (n_elems < 0 || (n_elems > 0 && (!x || !y))) return SAR_ERR_INVALID_ARG;
    if (t != SAR_F32 && t != SAR_BF16) return SAR_ERR_INVALID_ARG;
    if (!(p >= 0.f && p < 1.f)) return SAR_ERR_INVALID_ARG;
    SAR_TRY(check_elem_align({x, y}, sar_elem_size(t)));
    if (n_elems == 0) return SAR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const unsigned threshold = (unsigned)((double)p * 16777216.0);  // floor(p * 2^24)
    const float scale = 1.f / (1.f - p);
    const bool vec = sar_aligned(x, 16) && sar_aligned(y, 16);
    const long long epv = t == SAR_F32 ? 4 : 8;
    const long long n_vec16 = vec ? n_elems / epv : 0;
    const long long work = n_vec16 > 0 ? n_vec16 : n_elems;
    long long blocks = (work + 255) / 256;
    if (blocks > 148 * 64) blocks = 148 * 64;
    if (t == SAR_F32)
        SAR_LAUNCH("dropout", st, (dropout_kernel<float><<<(unsigned)blocks, 256, 0, st>>>(n_elems, static_cast<const float *>(x), static_cast<float *>(y), threshold, scale, seed, n_vec16)));
    else
        SAR_LAUNCH("dropout", st, (dropout_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, st>>>(n_elems, static_cast<const __nv_bfloat16 *>(x), static_cast<__nv_bfloat16 *>(y), threshold, scale, seed, n_vec16)));
    return sar_after_launch();
}

sar_status sar_axpby(int64_t n_elems, sar_dtype t, float a, const void *x, float b, void *y, void *stream) {
    if (n_elems < 0 || (n_elems > 0 && (!x || !y))) return SAR_ERR_INVALID_ARG;
    if (t != SAR_F32 && t != SAR_BF16) return SAR_ERR_INVALID_ARG;
    if (x == y) return SAR_ERR_INVALID_ARG;
    SAR_TRY(check_elem_align({x, y}, sar_elem_size(t)));
    if (n_elems == 0) return SAR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool vec = sar_aligned(x, 16) && sar_aligned(y, 16);
    const long long n_vec16 = vec ? n_elems / (t == SAR_F32 ? 4 : 8) : 0;
    const long long work = n_vec16 > 0 ? n_vec16 : n_elems;
    long long blocks = (work + 255) / 256;
    if (blocks > 148 * 64) blocks = 148 * 64;
    if (t == SAR_F32)
        SAR_LAUNCH("axpby", st, (axpby_kernel<float><<<(unsigned)blocks, 256, 0, st>>>(n_elems, a, static_cast<const float *>(x), b, static_cast<float *>(y), n_vec16)));
    else
        SAR_LAUNCH("axpby", st, (axpby_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, st>>>(n_elems, a, static_cast<const __nv_bfloat16 *>(x), b, static_cast<__nv_bfloat16 *>(y), n_vec16)));
    return sar_after_launch();
}

sar_status sar_accumulate(int64_t n_elems, sar_dtype t, const void *x, float *acc, uint32_t flags, void *stream) {
    if (n_elems < 0 || (n_elems > 0 && (!x || !acc)) || (flags & ~(uint32_t)SAR_FIRST)) return SAR_ERR_INVALID_ARG;
    if (t != SAR_F32 && t != SAR_BF16) return SAR_ERR_INVALID_ARG;
    SAR_TRY(check_elem_align({x}, sar_elem_size(t)));
    SAR_TRY(check_elem_align({acc}, 4));
    if (n_elems == 0) return SAR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    long long blocks = (n_elems + 255) / 256;
    if (blocks > 148 * 64) blocks = 148 * 64;
    const bool first = flags & SAR_FIRST;
    if (t == SAR_F32) {
        if (first) SAR_LAUNCH("accumulate", st, (widen_kernel<float, false><<<(unsigned)blocks, 256, 0, st>>>(n_elems, static_cast<const float *>(x), acc)));
        else SAR_LAUNCH("accumulate", st, (widen_kernel<float, true><<<(unsigned)blocks, 256, 0, st>>>(n_elems, static_cast<const float *>(x), acc)));
    } else {
        if (first) SAR_LAUNCH("accumulate", st, (widen_kernel<__nv_bfloat16, false><<<(unsigned)blocks, 256, 0, st>>>(n_elems, static_cast<const __nv_bfloat16 *>(x), acc)));
        else SAR_LAUNCH("accumulate", st, (widen_kernel<__nv_bfloat16, true><<<(unsigned)blocks, 256, 0, st>>>(n_elems, static_cast<const __nv_bfloat16 *>(x), acc)));
    }
    return sar_after_launch();
}

sar_status sar_round_to(int64_t n_elems, sar_dtype t, const float *acc, void *y, void *stream) {
    if (n_elems < 0 || (n_elems > 0 && (!acc || !y))) return SAR_ERR_INVALID_ARG;
    if (t != SAR_F32 && t != SAR_BF16) return SAR_ERR_INVALID_ARG;
    SAR_TRY(check_elem_align({y}, sar_elem_size(t)));
    SAR_TRY(check_elem_align({acc}, 4));
    if (n_elems == 0) return SAR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    long long blocks = (n_elems + 255) / 256;
    if (blocks > 148 * 64) blocks = 148 * 64;
    if (t == SAR_F32)
        SAR_LAUNCH("round_to", st, (narrow_kernel<float><<<(unsigned)blocks, 256, 0, st>>>(n_elems, acc, static_cast<float *>(y))));
    else
        SAR_LAUNCH("round_to", st, (narrow_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, st>>>(n_elems, acc, static_cast<__nv_bfloat16 *>(y))));
    return sar_after_launch();
}

}  // extern "C"

// Kernels around the span kernels of sar_span_kernels.cuh (internal): the merges of the long-row
// segments (forward, destination-major backward, source-major backward, sum) and the row-dot
// preparation of the per-partition backward.  One group of G lanes per row, lane gl / slot v holding
// the 16-byte vector v*G + gl of the row.
#pragma once

#include "sar_rowkernels.cuh"

namespace sar {

// ------------------------------------------------------------------------------------------------
// Forward merge: the segments of a long row are folded with the running-max correction of Sec. 3.4
// (exp(old_max - new_max) on numerator and normaliser), starting from the state left by earlier
// partitions unless SAR_FIRST (Algorithm 1).
// Partial record of a segment in the workspace: [rowf floats numerator][H max][H normaliser].
// ------------------------------------------------------------------------------------------------
struct FwdArgs {
    long long n_dst;
    const int64_t *indptr;
    const int32_t *indices;
    const void *feat;   // [n_src, n_vec] 16-byte vectors
    const float *el;    // [n_dst,H]
    const float *er;    // [n_src,H]
    float *acc;         // [n_dst,H*F] running numerator (float32) or null
    float *m;           // [n_dst,H]
    float *d;           // [n_dst,H]
    void *out;          // [n_dst, n_vec] or null
    float slope;
    unsigned flags;
    RowGeom g;
    SplitArgs sp;
    int mode;           // 0: one group per row; 1: one group per long-row segment
};

// The end of Algorithm 1 on its own: out = numerator / d for every row (0 where d = 0), one thread per 16-byte vector
// of `out`.  Follows a last partition step that left the complete state behind.
template <typename T>
__global__ void __launch_bounds__(256) gat_fwd_finalize_kernel(const FwdArgs a) {
    constexpr int EPV = Elem<T>::EPV;
    const long long vi = (long long)blockIdx.x * 256 + threadIdx.x;
    if (vi >= a.n_dst * a.g.n_vec) return;
    const long long row = vi / a.g.n_vec;
    const int v = (int)(vi - row * a.g.n_vec);
    const float dd = a.d[row * a.g.H + v / a.g.vph];
    const float inv = dd > 0.f ? __fdividef(1.f, dd) : 0.f;
    const float4 *src = reinterpret_cast<const float4 *>(a.acc) + vi * (EPV / 4);
    float x[EPV];
#pragma unroll
    for (int q = 0; q < EPV / 4; ++q) {
        const float4 t = src[q];
        x[4 * q] = t.x * inv;
        x[4 * q + 1] = t.y * inv;
        x[4 * q + 2] = t.z * inv;
        x[4 * q + 3] = t.w * inv;
    }
    if (a.flags & SAR_RELU_OUT) {
#pragma unroll
        for (int e = 0; e < EPV; ++e) x[e] = fmaxf(x[e], 0.f);
    }
    reinterpret_cast<uint4 *>(a.out)[vi] = Elem<T>::pack(x);
}

// Merge of the forward partials of the long rows: one group per long row folds its segments in
// order with the same running-max rule, starting from the incoming state unless SAR_FIRST.
template <typename T, int G, int V>
__global__ void __launch_bounds__(kThreads) gat_fwd_merge_kernel(const FwdArgs a) {
    constexpr int EPV = Elem<T>::EPV;
    constexpr int RPW = 32 / G;
    const LaneId<G> id;
    const int H = a.g.H;
    const long long lr = ((long long)blockIdx.x * kWarpsPerBlock + id.warp) * RPW + id.gid;
    if (lr >= a.sp.n_long) return;
    const long long row = a.sp.long_row[lr];
    const long long s0 = a.sp.long_seg[lr], s1 = a.sp.long_seg[lr + 1];
    const VecGeom<G, V> vg(a.g, id.gl);
    const long long rowf = (long long)a.g.n_vec * EPV;
    const bool first = a.flags & SAR_FIRST, last = a.flags & SAR_LAST;

    float Mv[V], dv[V], acc[V][EPV];
#pragma unroll
    for (int v = 0; v < V; ++v) {
        Mv[v] = SAR_NEG_INF;
        dv[v] = 0.f;
#pragma unroll
        for (int e = 0; e < EPV; ++e) acc[v][e] = 0.f;
    }
    if (!first) {
#pragma unroll
        for (int v = 0; v < V; ++v)
            if (vg.vok[v]) {
                Mv[v] = a.m[row * H + vg.hv[v]];
                dv[v] = a.d[row * H + vg.hv[v]];
            }
        load_acc_row<G, V, EPV>(a.acc + row * rowf, id.gl, vg.vok, acc);
    }
    // a hub row has hundreds of segments: the records of U segments are requested together, then folded in order
    constexpr int U = MergeBatch<V>::U;
    for (long long s = s0; s < s1; s += U) {
        float4 buf[U][V][EPV / 4];
        float Ms[U][V], ds[U][V];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (s + u < s1) {
                const float *rec = a.sp.part + (s + u) * a.sp.pstride;
                load_acc_vecs<G, V, EPV>(rec, id.gl, vg.vok, buf[u]);
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    Ms[u][v] = vg.vok[v] ? rec[rowf + vg.hv[v]] : SAR_NEG_INF;
                    ds[u][v] = vg.vok[v] ? rec[rowf + H + vg.hv[v]] : 0.f;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (s + u < s1) {
#pragma unroll
                for (int v = 0; v < V; ++v)
                    if (vg.vok[v]) {
                        const float Mn = fmaxf(Mv[v], Ms[u][v]);
                        const float c_old = (Mn == SAR_NEG_INF) ? 1.f : fast_exp(Mv[v] - Mn);
                        const float c_new = (Mn == SAR_NEG_INF) ? 1.f : fast_exp(Ms[u][v] - Mn);
#pragma unroll
                        for (int q = 0; q < EPV / 4; ++q) {
                            const float4 x = buf[u][v][q];
                            acc[v][4 * q] = acc[v][4 * q] * c_old + x.x * c_new;
                            acc[v][4 * q + 1] = acc[v][4 * q + 1] * c_old + x.y * c_new;
                            acc[v][4 * q + 2] = acc[v][4 * q + 2] * c_old + x.z * c_new;
                            acc[v][4 * q + 3] = acc[v][4 * q + 3] * c_old + x.w * c_new;
                        }
                        dv[v] = dv[v] * c_old + ds[u][v] * c_new;
                        Mv[v] = Mn;
                    }
            }
        }
    }
    if (last) {
        if (a.flags & SAR_KEEP_NUMERATOR) store_acc_row<G, V, EPV>(a.acc + row * rowf, id.gl, vg.vok, acc);
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const float inv = dv[v] > 0.f ? 1.f / dv[v] : 0.f;
#pragma unroll
            for (int e = 0; e < EPV; ++e) acc[v][e] *= inv;
            if (a.flags & SAR_RELU_OUT) {
#pragma unroll
                for (int e = 0; e < EPV; ++e) acc[v][e] = fmaxf(acc[v][e], 0.f);
            }
        }
        store_row_vec<T, G, V>(a.out, row, a.g.n_vec, id.gl, vg.vok, acc);
    } else {
        store_acc_row<G, V, EPV>(a.acc + row * rowf, id.gl, vg.vok, acc);
    }
#pragma unroll
    for (int v = 0; v < V; ++v)
        if (vg.vok[v] && ((v * G + id.gl) % a.g.vph) == 0) {
            a.m[row * H + vg.hv[v]] = Mv[v];
            a.d[row * H + vg.hv[v]] = dv[v];
        }
}

// ------------------------------------------------------------------------------------------------
// Backward, destination-major pass over the CSR (Algorithm 2's per-edge loop, rematerialised):
// with alpha = exp(e - m)/d and g' = LeakyReLU'(s),
//     A = sum_j alpha * feat_j            (= out, rebuilt so that bf16 rounding of `out` never enters)
//     B = sum_j alpha * g' * feat_j,      S = sum_j alpha * g'
//     D = <gout_i, A>,   del_i = <gout_i, B> - D * S     (= sum_j alpha (dalpha - D) g')
// and the packed record {el, m, 1/d, D} per (i,h) for the source-major pass.
// With GIVEN_D the record already exists (sar_gat_bwd_prepare) and only B, S are accumulated over
// this partition's edges.
// ------------------------------------------------------------------------------------------------
struct BwdDstArgs {
    long long n_dst;
    const int64_t *indptr;
    const int32_t *indices;
    const void *feat;   // gathered rows
    const void *gout;   // row-stationary vector
    const float *el, *er, *m, *d;
    float4 *rec;        // [n_dst,H] {el, m, 1/d, D}: written (full) or read (GIVEN_D)
    float *del;         // [n_dst,H]
    float slope;
    unsigned flags;
    RowGeom g;
    SplitArgs sp;
    int mode;
};

template <typename T, int G, int V, bool GIVEN_D>
__device__ __forceinline__ void bwd_dst_epilogue(const BwdDstArgs &a, const LaneId<G> &id, const VecGeom<G, V> &vg,
                                                 float *scratch, long long row, const float (&gv)[V][Elem<T>::EPV],
                                                 const float (&accA)[V][Elem<T>::EPV],
                                                 const float (&accB)[V][Elem<T>::EPV], const float (&S)[V]) {
    constexpr int EPV = Elem<T>::EPV;
    const int H = a.g.H;
    float pA[V], pB[V];
#pragma unroll
    for (int v = 0; v < V; ++v) {
        pA[v] = pB[v] = 0.f;
#pragma unroll
        for (int e = 0; e < EPV; ++e) {
            pA[v] = fmaf(gv[v][e], accA[v][e], pA[v]);
            pB[v] = fmaf(gv[v][e], accB[v][e], pB[v]);
        }
    }
    const float DB = head_sum<G, V>(scratch, pB, vg.vok, id.gl, a.g);
    const float Sh = head_scalar<G, V>(scratch, S, vg.hv, vg.vok, id.gl, a.g);
    float D;
    if constexpr (GIVEN_D) {
        D = (id.gl < H && row >= 0) ? a.rec[row * H + id.gl].w : 0.f;
    } else {
        D = head_sum<G, V>(scratch, pA, vg.vok, id.gl, a.g);
    }
    if (row >= 0 && id.gl < H) {
        const float v = DB - D * Sh;
        float *p = a.del + row * H + id.gl;
        *p = (a.flags & SAR_FIRST) ? v : *p + v;
        if constexpr (!GIVEN_D) {
            const float dd = a.d[row * H + id.gl];
            a.rec[row * H + id.gl] =
                make_float4(a.el[row * H + id.gl], a.m[row * H + id.gl], dd > 0.f ? 1.f / dd : 0.f, D);
        }
    }
}

template <typename T, int G, int V, bool GIVEN_D>
__global__ void __launch_bounds__(kThreads) gat_bwd_dst_merge_kernel(const BwdDstArgs a) {
    constexpr int EPV = Elem<T>::EPV;
    constexpr int RPW = 32 / G;
    extern __shared__ __align__(16) float smem[];
    const LaneId<G> id;
    float *wbase = smem + (size_t)id.warp * warp_smem_floats(a.g.Hp, V, 2);
    float *scratch = wbase + 64 + id.gid * (G * V);
    const long long lr = ((long long)blockIdx.x * kWarpsPerBlock + id.warp) * RPW + id.gid;
    const bool active = lr < a.sp.n_long;
    const VecGeom<G, V> vg(a.g, id.gl);
    const long long rowf = (long long)a.g.n_vec * EPV;
    float gv[V][EPV], accA[V][EPV], accB[V][EPV], S[V];
#pragma unroll
    for (int v = 0; v < V; ++v) {
        S[v] = 0.f;
#pragma unroll
        for (int e = 0; e < EPV; ++e) gv[v][e] = accA[v][e] = accB[v][e] = 0.f;
    }
    long long row = -1;
    if (active) {
        row = a.sp.long_row[lr];
        // the records of U segments are requested together, then added in order
        constexpr int U = MergeBatch<V>::U;
        const long long s1 = a.sp.long_seg[lr + 1];
        for (long long s = a.sp.long_seg[lr]; s < s1; s += U) {
            float4 bufB[U][V][EPV / 4], bufA[U][V][EPV / 4];
            float Ss[U][V];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (s + u < s1) {
                    const float *recp = a.sp.part + (s + u) * a.sp.pstride;
                    load_acc_vecs<G, V, EPV>(recp, id.gl, vg.vok, bufB[u]);
                    if constexpr (!GIVEN_D) load_acc_vecs<G, V, EPV>(recp + rowf, id.gl, vg.vok, bufA[u]);
#pragma unroll
                    for (int v = 0; v < V; ++v) Ss[u][v] = vg.vok[v] ? recp[2 * rowf + vg.hv[v]] : 0.f;
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (s + u < s1) {
                    add_acc_vecs<V, EPV>(bufB[u], vg.vok, accB, 1.f, 1.f);
                    if constexpr (!GIVEN_D) add_acc_vecs<V, EPV>(bufA[u], vg.vok, accA, 1.f, 1.f);
#pragma unroll
                    for (int v = 0; v < V; ++v)
                        if (vg.vok[v]) S[v] += Ss[u][v];
                }
            }
        }
        load_row_vec<T, G, V>(a.gout, row, a.g.n_vec, id.gl, vg.vok, gv);
    }
    bwd_dst_epilogue<T, G, V, GIVEN_D>(a, id, vg, scratch, row, gv, accA, accB, S);
}

// ------------------------------------------------------------------------------------------------
// Backward, source-major pass over the CSC (the error E_{p->q} Algorithm 2 returns to the owner of
// the features, and the source half of the score gradient), no atomics: one group per source j,
//     dfeat_j = sum_i alpha * gout_i
//     C = sum_i alpha * g' * gout_i,   S = sum_i alpha * g' * D_i
//     der_j = <feat_j, C> - S           (= sum_i alpha (dalpha - D_i) g')
// alpha is rebuilt from the destination record {el, m, 1/d, D} and er_j.
// ------------------------------------------------------------------------------------------------
struct BwdSrcArgs {
    long long n_src;
    const int64_t *t_indptr;
    const int32_t *t_indices;
    const void *gout;   // gathered rows
    const void *feat;   // row-stationary vector [n_src]
    const float *er;    // [n_src,H]
    const float4 *rec;  // [n_dst,H]
    void *dfeat;        // [n_src, n_vec]
    float *der;         // [n_src,H]
    float slope;
    RowGeom g;
    SplitArgs sp;
    int mode;
};

template <typename T, int G, int V>
__device__ __forceinline__ void bwd_src_epilogue(const BwdSrcArgs &a, const LaneId<G> &id, const VecGeom<G, V> &vg,
                                                 float *scratch, long long row, const float (&accD)[V][Elem<T>::EPV],
                                                 const float (&accC)[V][Elem<T>::EPV], const float (&S)[V]) {
    constexpr int EPV = Elem<T>::EPV;
    float fv[V][EPV], pC[V];
#pragma unroll
    for (int v = 0; v < V; ++v)
#pragma unroll
        for (int e = 0; e < EPV; ++e) fv[v][e] = 0.f;
    if (row >= 0) {
        load_row_vec<T, G, V>(a.feat, row, a.g.n_vec, id.gl, vg.vok, fv);
        store_row_vec<T, G, V>(a.dfeat, row, a.g.n_vec, id.gl, vg.vok, accD);
    }
#pragma unroll
    for (int v = 0; v < V; ++v) {
        pC[v] = 0.f;
#pragma unroll
        for (int e = 0; e < EPV; ++e) pC[v] = fmaf(fv[v][e], accC[v][e], pC[v]);
    }
    const float DC = head_sum<G, V>(scratch, pC, vg.vok, id.gl, a.g);
    const float Sh = head_scalar<G, V>(scratch, S, vg.hv, vg.vok, id.gl, a.g);
    if (row >= 0 && id.gl < a.g.H) a.der[row * a.g.H + id.gl] = DC - Sh;
}

template <typename T, int G, int V>
__global__ void __launch_bounds__(kThreads) gat_bwd_src_merge_kernel(const BwdSrcArgs a) {
    constexpr int EPV = Elem<T>::EPV;
    constexpr int RPW = 32 / G;
    extern __shared__ __align__(16) float smem[];
    const LaneId<G> id;
    float *wbase = smem + (size_t)id.warp * warp_smem_floats(a.g.Hp, V, 4);
    float *scratch = wbase + 64 + id.gid * (G * V);
    const long long lr = ((long long)blockIdx.x * kWarpsPerBlock + id.warp) * RPW + id.gid;
    const VecGeom<G, V> vg(a.g, id.gl);
    const long long rowf = (long long)a.g.n_vec * EPV;
    float accD[V][EPV], accC[V][EPV], S[V];
#pragma unroll
    for (int v = 0; v < V; ++v) {
        S[v] = 0.f;
#pragma unroll
        for (int e = 0; e < EPV; ++e) accD[v][e] = accC[v][e] = 0.f;
    }
    long long row = -1;
    if (lr < a.sp.n_long) {
        row = a.sp.long_row[lr];
        // the records of U segments are requested together, then added in order
        constexpr int U = MergeBatch<V>::U;
        const long long s1 = a.sp.long_seg[lr + 1];
        for (long long s = a.sp.long_seg[lr]; s < s1; s += U) {
            float4 bufD[U][V][EPV / 4], bufC[U][V][EPV / 4];
            float Ss[U][V];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (s + u < s1) {
                    const float *recp = a.sp.part + (s + u) * a.sp.pstride;
                    load_acc_vecs<G, V, EPV>(recp, id.gl, vg.vok, bufD[u]);
                    load_acc_vecs<G, V, EPV>(recp + rowf, id.gl, vg.vok, bufC[u]);
#pragma unroll
                    for (int v = 0; v < V; ++v) Ss[u][v] = vg.vok[v] ? recp[2 * rowf + vg.hv[v]] : 0.f;
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (s + u < s1) {
                    add_acc_vecs<V, EPV>(bufD[u], vg.vok, accD, 1.f, 1.f);
                    add_acc_vecs<V, EPV>(bufC[u], vg.vok, accC, 1.f, 1.f);
#pragma unroll
                    for (int v = 0; v < V; ++v)
                        if (vg.vok[v]) S[v] += Ss[u][v];
                }
            }
        }
    }
    bwd_src_epilogue<T, G, V>(a, id, vg, scratch, row, accD, accC, S);
}

// ------------------------------------------------------------------------------------------------
// Row dot D[i,h] = <gout_i, out_i> and the packed destination record (streaming, one group per row).
// ------------------------------------------------------------------------------------------------
struct PrepArgs {
    long long n_dst;
    const void *out;     // type T, or float32 numerator when acc_is_numerator
    const void *gout;
    const float *el, *m, *d;
    float *D;            // may be null
    float4 *rec;
    int acc_is_numerator;
    RowGeom g;
};

// A lane group takes PrepRows<V>::n consecutive rows and asks for all of their data before it reduces the first (one
// row per group leaves too little in flight for a pass that only streams two arrays).  The loads carry no branch: a
// row past the end reads the last row again and is dropped when it comes to writing.
template <int V>
struct PrepRows {
    static constexpr int n = V == 1 ? 4 : (V == 2 ? 2 : 1);
};

template <typename T, int G, int V, bool NUMERATOR>
__global__ void __launch_bounds__(kThreads) gat_bwd_prepare_kernel(const PrepArgs a) {
    constexpr int EPV = Elem<T>::EPV;
    constexpr int RPW = 32 / G;
    constexpr int RPG = PrepRows<V>::n;
    extern __shared__ __align__(16) float smem[];
    const LaneId<G> id;
    float *scratch = smem + (size_t)id.warp * (32 * V) + id.gid * (G * V);
    const long long row0 = (((long long)blockIdx.x * kWarpsPerBlock + id.warp) * RPW + id.gid) * RPG;
    const VecGeom<G, V> vg(a.g, id.gl);
    const int H = a.g.H;
    const int hl = id.gl < H ? id.gl : 0;
    float gv[RPG][V][EPV], ov[RPG][V][EPV], dd[RPG], el_[RPG], m_[RPG];
#pragma unroll
    for (int j = 0; j < RPG; ++j) {
        const long long row = row0 + j < a.n_dst ? row0 + j : a.n_dst - 1;
        load_row_vec<T, G, V>(a.gout, row, a.g.n_vec, id.gl, vg.vok, gv[j]);
        if constexpr (NUMERATOR) {
#pragma unroll
            for (int v = 0; v < V; ++v)
#pragma unroll
                for (int e = 0; e < EPV; ++e) ov[j][v][e] = 0.f;
            load_acc_row<G, V, EPV>(reinterpret_cast<const float *>(a.out) + row * (long long)(a.g.n_vec * EPV), id.gl,
                                    vg.vok, ov[j]);
        } else {
            load_row_vec<T, G, V>(a.out, row, a.g.n_vec, id.gl, vg.vok, ov[j]);
        }
        dd[j] = a.d[row * H + hl];
        el_[j] = a.el[row * H + hl];
        m_[j] = a.m[row * H + hl];
    }
#pragma unroll
    for (int j = 0; j < RPG; ++j) {
        const long long row = row0 + j;
        float p[V];
#pragma unroll
        for (int v = 0; v < V; ++v) {
            p[v] = 0.f;
#pragma unroll
            for (int e = 0; e < EPV; ++e) p[v] = fmaf(gv[j][v][e], ov[j][v][e], p[v]);
        }
        float D = head_sum<G, V>(scratch, p, vg.vok, id.gl, a.g);
        if (row < a.n_dst && id.gl < H) {
            const float inv = dd[j] > 0.f ? 1.f / dd[j] : 0.f;
            if (NUMERATOR) D *= inv;
            if (a.D) a.D[row * H + id.gl] = D;
            a.rec[row * H + id.gl] = make_float4(el_[j], m_[j], inv, D);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Sum aggregation (Eq. 2): the gather phase alone.
// ------------------------------------------------------------------------------------------------
struct SumArgs {
    long long n_dst;
    const int64_t *indptr;
    const int32_t *indices;
    const void *feat;
    void *out;
    const int64_t *deg_total;  // for SAR_MEAN
    const float *dst_scale;    // per-row factor of the weighted sum, or null
    unsigned flags;
    RowGeom g;                 // H = 1, vph = n_vec
    SplitArgs sp;
    int mode;
};

template <typename T, int G, int V>
__device__ __forceinline__ void sum_epilogue(const SumArgs &a, int gl, const VecGeom<G, V> &vg, long long row,
                                             float (&acc)[V][Elem<T>::EPV]) {
    constexpr int EPV = Elem<T>::EPV;
    if (a.dst_scale) {
        const float ds = a.dst_scale[row];
#pragma unroll
        for (int v = 0; v < V; ++v)
#pragma unroll
            for (int e = 0; e < EPV; ++e) acc[v][e] *= ds;
    }
    if (!(a.flags & SAR_FIRST)) {
        float old[V][EPV];
        load_row_vec<T, G, V, false>(a.out, row, a.g.n_vec, gl, vg.vok, old);
#pragma unroll
        for (int v = 0; v < V; ++v)
#pragma unroll
            for (int e = 0; e < EPV; ++e) acc[v][e] += old[v][e];
    }
    if ((a.flags & SAR_MEAN) && (a.flags & SAR_LAST)) {
        const long long dg = a.deg_total[row];
        const float inv = dg > 0 ? 1.f / (float)dg : 0.f;
#pragma unroll
        for (int v = 0; v < V; ++v)
#pragma unroll
            for (int e = 0; e < EPV; ++e) acc[v][e] *= inv;
    }
    store_row_vec<T, G, V>(a.out, row, a.g.n_vec, gl, vg.vok, acc);
}

template <typename T, int G, int V>
__global__ void __launch_bounds__(kThreads) spmm_merge_kernel(const SumArgs a) {
    constexpr int EPV = Elem<T>::EPV;
    constexpr int RPW = 32 / G;
    const LaneId<G> id;
    const long long lr = ((long long)blockIdx.x * kWarpsPerBlock + id.warp) * RPW + id.gid;
    if (lr >= a.sp.n_long) return;
    const VecGeom<G, V> vg(a.g, id.gl);
    float acc[V][EPV];
#pragma unroll
    for (int v = 0; v < V; ++v)
#pragma unroll
        for (int e = 0; e < EPV; ++e) acc[v][e] = 0.f;
    constexpr int U = MergeBatch<V>::U;
    const long long s1 = a.sp.long_seg[lr + 1];
    for (long long s = a.sp.long_seg[lr]; s < s1; s += U) {
        float4 buf[U][V][EPV / 4];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (s + u < s1) load_acc_vecs<G, V, EPV>(a.sp.part + (s + u) * a.sp.pstride, id.gl, vg.vok, buf[u]);
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (s + u < s1) add_acc_vecs<V, EPV>(buf[u], vg.vok, acc, 1.f, 1.f);
    }
    sum_epilogue<T, G, V>(a, id.gl, vg, a.sp.long_row[lr], acc);
}

}  // namespace sar

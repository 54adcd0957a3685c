// Scalar fallback kernels (internal): any H, F and alignment, one thread per (row, head) or per
// (row, feature).  Same results as the vector kernels, no claim on speed; they serve shapes whose
// rows are not made of 16-byte vectors.
#pragma once

#include "sar_common.cuh"

namespace sar {

struct GenericArgs {
    long long n_dst, n_src;
    const int64_t *indptr;
    const int32_t *indices;
    const int64_t *t_indptr;
    const int32_t *t_indices;
    const void *feat;
    const void *gout;
    const void *out_in;  // prepare: out or numerator
    const float *el, *er;
    float *acc, *m, *d;
    const float *m_in, *d_in;
    void *out;
    void *dfeat;
    float *del, *der, *D;
    float4 *rec;
    const int64_t *deg_total;
    const float *src_scale, *dst_scale;
    int H, F;
    float slope;
    unsigned flags;
    int given_d;
    int acc_is_numerator;
};

template <typename T>
__global__ void gat_fwd_generic(const GenericArgs a) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= a.n_dst * a.H) return;
    const long long row = idx / a.H;
    const int h = (int)(idx % a.H);
    const long long beg = a.indptr[row], end = a.indptr[row + 1];
    const bool first = a.flags & SAR_FIRST, last = a.flags & SAR_LAST;
    if (!first && !last && beg == end) return;
    const long long HF = (long long)a.H * a.F;
    const T *feat = reinterpret_cast<const T *>(a.feat);
    const float M = first ? SAR_NEG_INF : a.m[idx];
    const float d0 = first ? 0.f : a.d[idx];
    const float el_i = a.el[idx];
    float mq = SAR_NEG_INF;
    for (long long t = beg; t < end; ++t) {
        float gr;
        mq = fmaxf(mq, leaky(el_i + a.er[(long long)a.indices[t] * a.H + h], a.slope, gr));
    }
    const float Mn = fmaxf(M, mq);
    const float c = (Mn == SAR_NEG_INF) ? 1.f : expf(M - Mn);
    float dsum = d0 * c;
    for (long long t = beg; t < end; ++t) {
        float gr;
        dsum += expf(leaky(el_i + a.er[(long long)a.indices[t] * a.H + h], a.slope, gr) - Mn);
    }
    for (int f = 0; f < a.F; ++f) {
        const long long o = row * HF + (long long)h * a.F + f;
        float acc = first ? 0.f : a.acc[o] * c;
        for (long long t = beg; t < end; ++t) {
            const long long j = a.indices[t];
            float gr;
            const float w = expf(leaky(el_i + a.er[j * a.H + h], a.slope, gr) - Mn);
            acc = fmaf(w, Elem<T>::load1(feat + j * HF + (long long)h * a.F + f), acc);
        }
        if (last) {
            const float y = dsum > 0.f ? acc / dsum : 0.f;
            Elem<T>::store1(reinterpret_cast<T *>(a.out) + o, (a.flags & SAR_RELU_OUT) ? fmaxf(y, 0.f) : y);
        }
        if (!last || (a.flags & SAR_KEEP_NUMERATOR)) a.acc[o] = acc;
    }
    a.m[idx] = Mn;
    a.d[idx] = dsum;
}

template <typename T>
__global__ void gat_bwd_prepare_generic(const GenericArgs a) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= a.n_dst * a.H) return;
    const long long base = idx * a.F;
    const T *gout = reinterpret_cast<const T *>(a.gout);
    float D = 0.f;
    for (int f = 0; f < a.F; ++f) {
        const float o = a.acc_is_numerator ? reinterpret_cast<const float *>(a.out_in)[base + f]
                                           : Elem<T>::load1(reinterpret_cast<const T *>(a.out_in) + base + f);
        D = fmaf(Elem<T>::load1(gout + base + f), o, D);
    }
    const float dd = a.d_in[idx];
    const float inv = dd > 0.f ? 1.f / dd : 0.f;
    if (a.acc_is_numerator) D *= inv;
    if (a.D) a.D[idx] = D;
    a.rec[idx] = make_float4(a.el[idx], a.m_in[idx], inv, D);
}

template <typename T>
__global__ void gat_bwd_dst_generic(const GenericArgs a) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= a.n_dst * a.H) return;
    const long long row = idx / a.H;
    const int h = (int)(idx % a.H);
    const long long beg = a.indptr[row], end = a.indptr[row + 1];
    const bool first = a.flags & SAR_FIRST;
    if (!first && a.given_d && beg == end) return;
    const long long HF = (long long)a.H * a.F;
    const T *feat = reinterpret_cast<const T *>(a.feat);
    const T *gout = reinterpret_cast<const T *>(a.gout) + row * HF + (long long)h * a.F;
    const float el_i = a.el[idx], m_i = a.m_in[idx];
    const float dd = a.d_in[idx];
    const float inv = dd > 0.f ? 1.f / dd : 0.f;
    float D = 0.f;
    if (a.given_d) {
        D = a.rec[idx].w;
    } else {
        for (long long t = beg; t < end; ++t) {
            const long long j = a.indices[t];
            float gr, da = 0.f;
            const float al = expf(leaky(el_i + a.er[j * a.H + h], a.slope, gr) - m_i) * inv;
            for (int f = 0; f < a.F; ++f)
                da = fmaf(Elem<T>::load1(gout + f), Elem<T>::load1(feat + j * HF + (long long)h * a.F + f), da);
            D = fmaf(al, da, D);
        }
    }
    float acc = 0.f;
    for (long long t = beg; t < end; ++t) {
        const long long j = a.indices[t];
        float gr, da = 0.f;
        const float al = expf(leaky(el_i + a.er[j * a.H + h], a.slope, gr) - m_i) * inv;
        for (int f = 0; f < a.F; ++f)
            da = fmaf(Elem<T>::load1(gout + f), Elem<T>::load1(feat + j * HF + (long long)h * a.F + f), da);
        acc += al * (da - D) * gr;
    }
    a.del[idx] = first ? acc : a.del[idx] + acc;
    if (!a.given_d) a.rec[idx] = make_float4(el_i, m_i, inv, D);
}

template <typename T>
__global__ void gat_bwd_src_generic(const GenericArgs a) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= a.n_src * a.H) return;
    const long long j = idx / a.H;
    const int h = (int)(idx % a.H);
    const long long beg = a.t_indptr[j], end = a.t_indptr[j + 1];
    const long long HF = (long long)a.H * a.F;
    const T *gout = reinterpret_cast<const T *>(a.gout);
    const T *fj = reinterpret_cast<const T *>(a.feat) + j * HF + (long long)h * a.F;
    const float er_j = a.er[idx];
    float der = 0.f;
    for (long long t = beg; t < end; ++t) {
        const long long i = a.t_indices[t];
        const float4 r = a.rec[i * a.H + h];
        float gr, da = 0.f;
        const float al = expf(leaky(r.x + er_j, a.slope, gr) - r.y) * r.z;
        for (int f = 0; f < a.F; ++f)
            da = fmaf(Elem<T>::load1(gout + i * HF + (long long)h * a.F + f), Elem<T>::load1(fj + f), da);
        der += al * (da - r.w) * gr;
    }
    a.der[idx] = der;
    for (int f = 0; f < a.F; ++f) {
        float acc = 0.f;
        for (long long t = beg; t < end; ++t) {
            const long long i = a.t_indices[t];
            const float4 r = a.rec[i * a.H + h];
            float gr;
            const float al = expf(leaky(r.x + er_j, a.slope, gr) - r.y) * r.z;
            acc = fmaf(al, Elem<T>::load1(gout + i * HF + (long long)h * a.F + f), acc);
        }
        Elem<T>::store1(reinterpret_cast<T *>(a.dfeat) + j * HF + (long long)h * a.F + f, acc);
    }
}

template <typename T>
__global__ void spmm_generic(const GenericArgs a) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= a.n_dst * a.F) return;
    const long long row = idx / a.F;
    const int f = (int)(idx % a.F);
    const long long beg = a.indptr[row], end = a.indptr[row + 1];
    const bool first = a.flags & SAR_FIRST;
    const bool mean = (a.flags & SAR_MEAN) && (a.flags & SAR_LAST);
    if (!first && !mean && beg == end) return;
    const T *feat = reinterpret_cast<const T *>(a.feat);
    T *out = reinterpret_cast<T *>(a.out);
    float acc = 0.f;
    for (long long t = beg; t < end; ++t) {
        const long long j = a.indices[t];
        const float x = Elem<T>::load1(feat + j * a.F + f);
        acc = a.src_scale ? fmaf(a.src_scale[j], x, acc) : acc + x;
    }
    if (a.dst_scale) acc *= a.dst_scale[row];
    if (!first) acc += Elem<T>::load1(out + idx);
    if (mean) {
        const long long dg = a.deg_total[row];
        acc = dg > 0 ? acc * (1.f / (float)dg) : 0.f;
    }
    Elem<T>::store1(out + idx, acc);
}

}  // namespace sar

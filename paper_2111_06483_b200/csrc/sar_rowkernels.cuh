// Row-stationary gather kernels of libsar (internal).
//
// One skeleton serves the forward pass, both backward passes and the sum aggregation:
//   a GROUP of G lanes (G = 4..32, a power of two) owns one row of the traversal (a destination
//   for the CSR passes, a source for the CSC pass); lane gl, slot v holds the 16-byte vector
//   vi = v*G + gl of the H*F-wide row, so that one warp instruction fetches G consecutive
//   vectors (coalesced 128-bit gathers) of 32/G different neighbour rows.
//   The row's edges are consumed in batches of G:
//     1. each lane loads one column index of the batch (coalesced) into shared memory;
//     2. SCORE phase: the (edge, head) pairs of the batch are spread over the lanes, each pair's
//        weight(s) are computed ONCE (one exponential per pair) and parked in shared memory;
//     3. GATHER phase: every lane walks the batch, fetches its vectors of each neighbour row and
//        accumulates them, scaled by the weight of the vector's head, in float32 registers.
//   Nothing per edge is ever written to global memory.
//   Rows longer than `threshold` edges are cut into segments processed by other groups in a
//   second launch of the same kernel (mode 1), which parks partial accumulators in a workspace; a
//   third launch merges them.  No atomics anywhere: every output element has one writer.
#pragma once

#include "sar_common.cuh"

namespace sar {

struct SplitArgs {
    int threshold;            // 0: no long-row handling
    int n_long;
    long long n_seg;
    const int32_t *long_row;  // [n_long]
    const int64_t *long_seg;  // [n_long+1]
    float *part;              // [n_seg * pstride] partial accumulators
    long long pstride;        // floats per segment
};

enum GatherMode { kFwd = 0, kBwdDst = 1, kBwdDstGivenD = 2, kBwdSrc = 3, kSum = 4 };

template <int MODE>
struct WeightOf {
    using type = float;
};
template <>
struct WeightOf<kBwdSrc> {
    using type = float2;
};

// Floats of shared memory one warp needs: 32 column ids, 32 rescale factors, then the larger of
// the batch's weights (32 edges x Hp heads x weight size) and the epilogue's scratch.
__host__ __device__ inline size_t warp_smem_floats(int Hp, int V, int wfloats) {
    size_t w = (size_t)32 * Hp * wfloats;
    size_t e = (size_t)32 * V * 2 + 32;
    return 64 + (w > e ? w : e);
}

template <int G>
struct LaneId {
    int lane, warp, gl, gid;
    __device__ __forceinline__ LaneId() {
        lane = threadIdx.x & 31;
        warp = threadIdx.x >> 5;
        gl = lane & (G - 1);
        gid = lane / G;
    }
};

template <int G, int V>
struct VecGeom {
    int hv[V];
    bool vok[V];
    __device__ __forceinline__ VecGeom(const RowGeom &g, int gl) {
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int vi = v * G + gl;
            vok[v] = vi < g.n_vec;
            hv[v] = vok[v] ? vi / g.vph : 0;
        }
    }
};

// Which (row, edge range) does this group work on?  mode 0: row = item, whole row unless it is
// long (then skipped, the segment launch covers it); mode 1: item is a segment of a long row.
struct WorkItem {
    bool active;
    long long row;
    long long beg, end;
    long long seg;
};

__device__ __forceinline__ WorkItem locate_work(long long item, long long n_rows, const int64_t *__restrict__ indptr,
                                                const SplitArgs &sp, int mode) {
    WorkItem w;
    w.active = false;
    w.row = 0;
    w.beg = w.end = 0;
    w.seg = -1;
    if (mode == 0) {
        if (item < n_rows) {
            w.row = item;
            w.beg = __ldg(indptr + item);
            w.end = __ldg(indptr + item + 1);
            w.active = !(sp.threshold > 0 && w.end - w.beg > sp.threshold);
        }
    } else if (item < sp.n_seg) {
        int lo = 0, hi = sp.n_long;  // last lr with long_seg[lr] <= item
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (__ldg(sp.long_seg + mid) <= item) lo = mid; else hi = mid;
        }
        w.row = __ldg(sp.long_row + lo);
        const long long c = item - __ldg(sp.long_seg + lo);
        const long long rb = __ldg(indptr + w.row), re = __ldg(indptr + w.row + 1);
        w.beg = rb + c * sp.threshold;
        w.end = w.beg + sp.threshold < re ? w.beg + sp.threshold : re;
        w.seg = item;
        w.active = true;
    }
    if (!w.active) w.beg = w.end = 0;
    return w;
}

// float32 accumulator rows in global memory (running numerator, partials): lane's slot v covers
// floats [(v*G+gl)*EPV, +EPV).
template <int G, int V, int EPV>
__device__ __forceinline__ void store_acc_row(float *__restrict__ rowp, int gl, const bool (&vok)[V],
                                              const float (&acc)[V][EPV]) {
#pragma unroll
    for (int v = 0; v < V; ++v)
        if (vok[v]) {
            float4 *p = reinterpret_cast<float4 *>(rowp + (size_t)(v * G + gl) * EPV);
#pragma unroll
            for (int q = 0; q < EPV / 4; ++q)
                p[q] = make_float4(acc[v][4 * q], acc[v][4 * q + 1], acc[v][4 * q + 2], acc[v][4 * q + 3]);
        }
}

template <int G, int V, int EPV>
__device__ __forceinline__ void load_acc_row(const float *__restrict__ rowp, int gl, const bool (&vok)[V],
                                             float (&acc)[V][EPV]) {
#pragma unroll
    for (int v = 0; v < V; ++v)
        if (vok[v]) {
            const float4 *p = reinterpret_cast<const float4 *>(rowp + (size_t)(v * G + gl) * EPV);
#pragma unroll
            for (int q = 0; q < EPV / 4; ++q) {
                const float4 x = p[q];
                acc[v][4 * q] = x.x;
                acc[v][4 * q + 1] = x.y;
                acc[v][4 * q + 2] = x.z;
                acc[v][4 * q + 3] = x.w;
            }
        }
}

template <int G, int V, int EPV>
__device__ __forceinline__ void add_acc_row(const float *__restrict__ rowp, int gl, const bool (&vok)[V],
                                            float (&acc)[V][EPV], float scale_old, float scale_new) {
#pragma unroll
    for (int v = 0; v < V; ++v)
        if (vok[v]) {
            const float4 *p = reinterpret_cast<const float4 *>(rowp + (size_t)(v * G + gl) * EPV);
#pragma unroll
            for (int q = 0; q < EPV / 4; ++q) {
                const float4 x = p[q];
                acc[v][4 * q] = acc[v][4 * q] * scale_old + x.x * scale_new;
                acc[v][4 * q + 1] = acc[v][4 * q + 1] * scale_old + x.y * scale_new;
                acc[v][4 * q + 2] = acc[v][4 * q + 2] * scale_old + x.z * scale_new;
                acc[v][4 * q + 3] = acc[v][4 * q + 3] * scale_old + x.w * scale_new;
            }
        }
}

// One row vector of storage type T -> float registers.
// READONLY = false for arrays the same launch also writes (plain, coherent loads).
template <typename T, int G, int V, bool READONLY = true>
__device__ __forceinline__ void load_row_vec(const void *base, long long row, int n_vec, int gl,
                                             const bool (&vok)[V], float (&r)[V][Elem<T>::EPV]) {
    const uint4 *rp = reinterpret_cast<const uint4 *>(base) + row * n_vec;
#pragma unroll
    for (int v = 0; v < V; ++v) {
        uint4 x = make_uint4(0, 0, 0, 0);
        if (vok[v]) {
            if constexpr (READONLY) x = __ldg(rp + v * G + gl);
            else x = rp[v * G + gl];
        }
        Elem<T>::unpack(x, r[v]);
    }
}

template <typename T, int G, int V>
__device__ __forceinline__ void store_row_vec(void *base, long long row, int n_vec, int gl,
                                              const bool (&vok)[V], const float (&r)[V][Elem<T>::EPV]) {
    uint4 *rp = reinterpret_cast<uint4 *>(base) + row * n_vec;
#pragma unroll
    for (int v = 0; v < V; ++v)
        if (vok[v]) rp[v * G + gl] = Elem<T>::pack(r[v]);
}

// GATHER phase over one batch of nb (<= G) edges of this group.
//   sjg: the batch's column ids; swg: the batch's weights, [edge][Hp].
//   kFwd:           acc0 += w * x,                    s += w
//   kBwdDst:        acc0 += w.x * x, acc1 += w.y * x, s += w.y
//   kBwdDstGivenD:                   acc1 += w.y * x, s += w.y
//   kBwdSrc:        acc0 += w.x * x, acc1 += w.y * x, s += w.z
//   kSum:           acc0 += x
template <typename T, int G, int V, int U, int MODE>
__device__ __forceinline__ void gather_batch(const uint4 *__restrict__ base, int n_vec, const int *sjg,
                                             const typename WeightOf<MODE>::type *swg, int Hp, int nb, int gl,
                                             const int (&hv)[V], const bool (&vok)[V],
                                             float (&acc0)[V][Elem<T>::EPV], float (&acc1)[V][Elem<T>::EPV],
                                             float (&s)[V]) {
    constexpr int EPV = Elem<T>::EPV;
    using W = typename WeightOf<MODE>::type;
    for (int k0 = 0; k0 < nb; k0 += U) {
        uint4 buf[U][V];
        W w[U][V];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int kk = k0 + u;
            const bool ok = kk < nb;
            const int jj = sjg[ok ? kk : k0];
            const uint4 *rp = base + (long long)jj * n_vec + gl;
#pragma unroll
            for (int v = 0; v < V; ++v) {
                buf[u][v] = make_uint4(0, 0, 0, 0);
                if (ok && vok[v]) buf[u][v] = ldg16(rp + v * G);
            }
            if constexpr (MODE != kSum) {
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    const W ww = swg[(ok ? kk : k0) * Hp + hv[v]];
                    if constexpr (MODE == kFwd) {
                        w[u][v] = ok ? ww : 0.f;
                    } else if constexpr (MODE == kBwdSrc) {
                        w[u][v] = ok ? ww : make_float4(0.f, 0.f, 0.f, 0.f);
                    } else {
                        w[u][v] = ok ? ww : make_float2(0.f, 0.f);
                    }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
#pragma unroll
            for (int v = 0; v < V; ++v) {
                float x[EPV];
                Elem<T>::unpack(buf[u][v], x);
                if constexpr (MODE == kFwd) {
                    s[v] += w[u][v];
#pragma unroll
                    for (int e = 0; e < EPV; ++e) acc0[v][e] = fmaf(w[u][v], x[e], acc0[v][e]);
                } else if constexpr (MODE == kBwdDst) {
                    s[v] += w[u][v].y;
#pragma unroll
                    for (int e = 0; e < EPV; ++e) {
                        acc0[v][e] = fmaf(w[u][v].x, x[e], acc0[v][e]);
                        acc1[v][e] = fmaf(w[u][v].y, x[e], acc1[v][e]);
                    }
                } else if constexpr (MODE == kBwdDstGivenD) {
                    s[v] += w[u][v].y;
#pragma unroll
                    for (int e = 0; e < EPV; ++e) acc1[v][e] = fmaf(w[u][v].y, x[e], acc1[v][e]);
                } else if constexpr (MODE == kBwdSrc) {
                    s[v] += w[u][v].z;
#pragma unroll
                    for (int e = 0; e < EPV; ++e) {
                        acc0[v][e] = fmaf(w[u][v].x, x[e], acc0[v][e]);
                        acc1[v][e] = fmaf(w[u][v].y, x[e], acc1[v][e]);
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < EPV; ++e) acc0[v][e] += x[e];
                }
            }
        }
    }
}

// Per-head sum of per-lane partial dot products, through shared memory: lane (gl, v) deposits its
// partial at vector index vi; lanes gl < H then add their head's vph entries.  Returns the head
// sum for lanes gl < H (head gl), 0 elsewhere.  All 32 lanes must call.
template <int G, int V>
__device__ __forceinline__ float head_sum(float *scratch /* this group's G*V floats */, const float (&part)[V],
                                          const bool (&vok)[V], int gl, const RowGeom &g) {
    __syncwarp();
#pragma unroll
    for (int v = 0; v < V; ++v)
        if (vok[v]) scratch[v * G + gl] = part[v];
    __syncwarp();
    float r = 0.f;
    if (gl < g.H)
        for (int k = 0; k < g.vph; ++k) r += scratch[gl * g.vph + k];
    return r;
}

// Per-head scalar held redundantly by the gather lanes -> lane gl (< H) of the group.
template <int G, int V>
__device__ __forceinline__ float head_scalar(float *scratch /* this group's >= Hp floats */, const float (&s)[V],
                                             const int (&hv)[V], const bool (&vok)[V], int gl, const RowGeom &g) {
    __syncwarp();
#pragma unroll
    for (int v = 0; v < V; ++v)
        if (vok[v] && ((v * G + gl) % g.vph) == 0) scratch[hv[v]] = s[v];
    __syncwarp();
    return gl < g.H ? scratch[gl] : 0.f;
}

}  // namespace sar

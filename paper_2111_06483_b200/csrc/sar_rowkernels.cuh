// Row geometry shared by the kernels of libsar (internal).
//
// A feature row of H*F elements is n_vec 16-byte vectors.  A GROUP of G lanes (G = 4..32, a power of
// two) covers one row: lane gl, slot v holds the vector vi = v*G + gl, so that one warp instruction
// moves G consecutive vectors (coalesced 128-bit accesses) of 32/G different rows.  Vector vi belongs
// to head vi / vph.  Float32 accumulator rows in global memory (running numerator, long-row partials)
// use the same mapping with EPV floats per vector.
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

enum GatherMode { kFwd = 0, kBwdDst = 1, kBwdDstGivenD = 2, kBwdSrc = 3, kSum = 4, kSumW = 5 };

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

// The same in two steps, so that a merge loop can have the loads of several records in flight before it folds
// them in order: load the lane's vectors of one float32 record row ...
template <int G, int V, int EPV>
__device__ __forceinline__ void load_acc_vecs(const float *__restrict__ rowp, int gl, const bool (&vok)[V],
                                              float4 (&buf)[V][EPV / 4]) {
#pragma unroll
    for (int v = 0; v < V; ++v) {
        const float4 *p = reinterpret_cast<const float4 *>(rowp + (size_t)(v * G + gl) * EPV);
#pragma unroll
        for (int q = 0; q < EPV / 4; ++q) buf[v][q] = vok[v] ? p[q] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
}
// ... and fold them (the arithmetic of add_acc_row, term by term)
template <int V, int EPV>
__device__ __forceinline__ void add_acc_vecs(const float4 (&buf)[V][EPV / 4], const bool (&vok)[V], float (&acc)[V][EPV],
                                             float scale_old, float scale_new) {
#pragma unroll
    for (int v = 0; v < V; ++v)
        if (vok[v]) {
#pragma unroll
            for (int q = 0; q < EPV / 4; ++q) {
                const float4 x = buf[v][q];
                acc[v][4 * q] = acc[v][4 * q] * scale_old + x.x * scale_new;
                acc[v][4 * q + 1] = acc[v][4 * q + 1] * scale_old + x.y * scale_new;
                acc[v][4 * q + 2] = acc[v][4 * q + 2] * scale_old + x.z * scale_new;
                acc[v][4 * q + 3] = acc[v][4 * q + 3] * scale_old + x.w * scale_new;
            }
        }
}
// records a merge loop keeps in flight
template <int V>
struct MergeBatch {
    static constexpr int U = V == 1 ? 4 : 2;
};

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

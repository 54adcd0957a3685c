// Shared device/host helpers of libsar (internal; the public boundary is include/sar.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "sar.h"

#define SAR_TRY(expr)                          \
    do {                                       \
        sar_status st__ = (expr);              \
        if (st__ != SAR_OK) return st__;       \
    } while (0)

#define SAR_CUDA_TRY(expr)                              \
    do {                                                \
        if ((expr) != cudaSuccess) {                    \
            (void)cudaGetLastError();                   \
            return SAR_ERR_CUDA;                        \
        }                                               \
    } while (0)

static inline sar_status sar_after_launch() {
    return cudaGetLastError() == cudaSuccess ? SAR_OK : SAR_ERR_CUDA;
}

static inline bool sar_aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
static inline size_t sar_round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline int sar_pow2_ceil(int x) {
    int p = 1;
    while (p < x) p <<= 1;
    return p;
}
static inline int sar_log2(int pow2) {
    int l = 0;
    while ((1 << l) < pow2) ++l;
    return l;
}
static inline size_t sar_elem_size(sar_dtype t) { return t == SAR_BF16 ? 2 : 4; }

#define SAR_NEG_INF (-INFINITY)

// SplitMix64's (i+1)-th output for `seed`: the counter-based generator of the dropout mask (element i is kept
// when the top 24 bits reach p * 2^24); nothing is stored, the mask is drawn again wherever it is needed.
__host__ __device__ inline unsigned long long splitmix64_at(unsigned long long seed, unsigned long long i) {
    unsigned long long z = seed + (i + 1ull) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// launch observer (sar_set_launch_hook)
namespace sar {
extern sar_launch_hook_fn g_launch_hook;
extern void *g_launch_hook_user;
struct LaunchScope {
    const char *name;
    cudaStream_t st;
    LaunchScope(const char *n, cudaStream_t s) : name(n), st(s) {
        if (g_launch_hook) g_launch_hook(name, 0, st, g_launch_hook_user);
    }
    ~LaunchScope() {
        if (g_launch_hook) g_launch_hook(name, 1, st, g_launch_hook_user);
    }
};
}  // namespace sar
// SAR_LAUNCH("name", stream, kernel<<<...>>>(args));
#define SAR_LAUNCH(name, st, ...)            \
    do {                                     \
        sar::LaunchScope scope__(name, st);  \
        __VA_ARGS__;                         \
    } while (0)

namespace sar {

constexpr int kWarpsPerBlock = 8;
constexpr int kThreads = kWarpsPerBlock * 32;

// ---- storage element traits: 16-byte vectors <-> float registers --------------------------
template <typename T>
struct Elem;

template <>
struct Elem<float> {
    static constexpr int EPV = 4;  // elements per 16-byte vector
    __device__ __forceinline__ static void unpack(const uint4 &v, float (&f)[4]) {
        f[0] = __uint_as_float(v.x);
        f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z);
        f[3] = __uint_as_float(v.w);
    }
    __device__ __forceinline__ static uint4 pack(const float (&f)[4]) {
        return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]),
                          __float_as_uint(f[3]));
    }
    __device__ __forceinline__ static float load1(const float *p) { return __ldg(p); }
    __device__ __forceinline__ static void store1(float *p, float x) { *p = x; }
};

template <>
struct Elem<__nv_bfloat16> {
    static constexpr int EPV = 8;
    __device__ __forceinline__ static void unpack(const uint4 &v, float (&f)[8]) {
        // a bf16 is the upper half of a float32
        f[0] = __uint_as_float(v.x << 16);
        f[1] = __uint_as_float(v.x & 0xffff0000u);
        f[2] = __uint_as_float(v.y << 16);
        f[3] = __uint_as_float(v.y & 0xffff0000u);
        f[4] = __uint_as_float(v.z << 16);
        f[5] = __uint_as_float(v.z & 0xffff0000u);
        f[6] = __uint_as_float(v.w << 16);
        f[7] = __uint_as_float(v.w & 0xffff0000u);
    }
    __device__ __forceinline__ static uint32_t pack2(float lo, float hi) {
        __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);  // round to nearest even
        return *reinterpret_cast<uint32_t *>(&h);
    }
    __device__ __forceinline__ static uint4 pack(const float (&f)[8]) {
        return make_uint4(pack2(f[0], f[1]), pack2(f[2], f[3]), pack2(f[4], f[5]), pack2(f[6], f[7]));
    }
    __device__ __forceinline__ static float load1(const __nv_bfloat16 *p) {
        return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short *>(p))) << 16);
    }
    __device__ __forceinline__ static void store1(__nv_bfloat16 *p, float x) { *p = __float2bfloat16_rn(x); }
};

// read-only 16-byte gather through the non-coherent path
__device__ __forceinline__ uint4 ldg16(const uint4 *p) { return __ldg(p); }

// streaming loads for data touched once per launch (index arrays)
__device__ __forceinline__ int ld_stream_i32(const int32_t *p) { return __ldcs(p); }

__device__ __forceinline__ float leaky(float s, float slope, float &grad) {
    grad = s > 0.f ? 1.f : slope;
    return s * grad;
}

// exp for arguments <= 0 (after max subtraction)
__device__ __forceinline__ float fast_exp(float x) { return __expf(x); }

// Geometry of one destination row across the lanes of a group of G lanes, V vectors per lane.
// Vector `vi = v*G + gl` of the row (16 bytes) belongs to lane gl, slot v; its head is vi / vph.
struct RowGeom {
    int H;      // heads
    int Hp;     // heads rounded up to a power of two (<= G)
    int lgHp;   // log2(Hp)
    int vph;    // 16-byte vectors per head
    int n_vec;  // 16-byte vectors per row (H * vph)
};

}  // namespace sar

// entry points implemented across translation units -------------------------------------------
namespace sar {

struct Shape {
    int H, F;
    sar_dtype t;
    size_t row_bytes;
    bool fast;  // fast vector kernels apply
    int G, V;   // lanes per row, vectors per lane
    RowGeom geom;
};

// Decide which kernel family handles (H, F, t) given the alignment of the feature pointers.
sar_status make_shape(int32_t H, int32_t F, sar_dtype t, bool ptrs_16B_aligned, Shape *out);

}  // namespace sar

// Host-side kernel selection shared by the entry points (internal).
#pragma once

#include <initializer_list>

#include "sar_common.cuh"

namespace sar {

template <typename T, int G, int V, int U>
struct Cfg {
    using type = T;
    static constexpr int g = G, v = V, u = U;
};

// Calls f(Cfg<T,G,V,U>{}) for the instantiation matching the shape.
template <typename Fn>
static inline sar_status dispatch(const Shape &s, Fn &&f) {
#define SAR_CASE(GG, VV, UU)                                                   \
    if (s.G == GG && s.V == VV) {                                              \
        if (s.t == SAR_F32) return f(Cfg<float, GG, VV, UU>{});                \
        return f(Cfg<__nv_bfloat16, GG, VV, UU>{});                            \
    }
    SAR_CASE(4, 1, 4)
    SAR_CASE(8, 1, 4)
    SAR_CASE(16, 1, 4)
    SAR_CASE(32, 1, 4)
    SAR_CASE(32, 2, 2)
    SAR_CASE(32, 4, 1)
    SAR_CASE(32, 8, 1)
#undef SAR_CASE
    return SAR_ERR_UNSUPPORTED;
}

static inline unsigned blocks_for(long long items, int G) {
    const long long per_block = (long long)kWarpsPerBlock * (32 / G);
    return (unsigned)((items + per_block - 1) / per_block);
}

template <typename K>
static inline sar_status ensure_smem(K kernel, size_t bytes) {
    if (bytes > 48 * 1024)
        SAR_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
    return SAR_OK;
}

static inline bool all16(std::initializer_list<const void *> ps) {
    for (const void *p : ps)
        if (p && !sar_aligned(p, 16)) return false;
    return true;
}

static inline sar_status check_elem_align(std::initializer_list<const void *> ps, size_t a) {
    for (const void *p : ps)
        if (p && !sar_aligned(p, a)) return SAR_ERR_ALIGNMENT;
    return SAR_OK;
}

}  // namespace sar

// Lean span kernels of libsar (internal): the whole-graph forward pass and the destination-major whole-graph
// backward pass for the common shapes (heads in groups of four, rows of exactly G*V 16-byte vectors), written for the fewest
// issued instructions per edge.
//
// Same plan as span_kernel (sar_span_kernels.cuh) - a warp owns a span of consecutive rows, stages a chunk of
// whole rows in shared memory slot-major, scores all (edge, head) pairs lane-parallel, then streams the
// gathered rows through a cp.async ring - with these differences:
//   * The ring works in STAGES of 4 KB (SPS slots): one commit group and one wait per stage, the slots of a
//     stage walked with compile-time offsets (fully unrolled), the stage refilled as a whole.  The staged
//     column ids are pre-scaled row offsets in 16-byte units, stored per stage with the slot index fastest,
//     so that one 16-byte shared load brings the offsets of four consecutive slots; the weights likewise.
//   * A row's padding position repeats the row's last column with weight zero, and a chunk's last stage is
//     filled up with repeats: every copy is a real copy of a real row, no predicates, no zero fill.
//   * Everything the control flow depends on (slot counts, row-end masks) is produced by warp votes and
//     reductions, so that the branches around the row epilogues are uniform branches.
//   * The forward row max uses max_j LeakyReLU(el + er_j) = LeakyReLU(el + max_j er_j) (slope >= 0): the
//     shared-memory max runs over raw er, exponentials are one FFMA + EX2.
//   * Dot products of the backward epilogue are taken on the un-folded accumulators and reduced with three
//     shuffles per quantity; per-(row, head) scalars leave through shared memory, coalesced, once per chunk.
// The source-major backward pass stays with span_kernel: a lean version of it (its 64-byte destination records
// gathered in the score phase) measured 4 - 13 % slower on every workload.
// Preconditions (checked by the host, which otherwise launches span_kernel): SAR_FIRST|SAR_LAST, slope >= 0,
// every row of the rows launch at most CAP edges (a long-row plan with threshold <= CAP), segments of at most
// CAP edges, fewer than 2^32 16-byte vectors in the gathered array.
#pragma once

#include "sar_span_kernels.cuh"
#include "sar_lean.cuh"
#include "sar_dispatch.cuh"

namespace sar {

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void sts_f32(unsigned addr, float v) {
    asm volatile("st.shared.f32 [%0], %1;\n" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void sts_u32(unsigned addr, unsigned v) {
    asm volatile("st.shared.u32 [%0], %1;\n" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned lds_u32(unsigned addr) {
    unsigned v;
    asm volatile("ld.shared.u32 %0, [%1];\n" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ unsigned lds_u8(unsigned addr) {
    unsigned v;
    asm volatile("ld.shared.u8 %0, [%1];\n" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts_u8(unsigned addr, unsigned v) {
    asm volatile("st.shared.u8 [%0], %1;\n" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ float4 lds_f4(unsigned addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];\n" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
// plain 16-byte asynchronous copy (every copy of the lean kernels is a whole, valid vector)
__device__ __forceinline__ void cp_async16_full(unsigned smem_addr, const void *gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(smem_addr), "l"(gsrc) : "memory");
}

constexpr float kLog2e = 1.4426950408889634f;

// Shared-memory layout of the lean kernels (one warp per block), byte offsets.
template <int G, int V, int H, int MODE, bool SEG, int CAP, int P, int NS>
struct LeanLayout {
    static constexpr int EPW = 32 / G;
    static constexpr int ROWB = G * V * 16;
    static constexpr int STAGE = P * ROWB;
    static constexpr int MAXR = SEG ? 1 : kMaxSpanRows;
    static constexpr int POSMAX = ((CAP + MAXR * (EPW - 1) + 31) / 32) * 32;
    static constexpr int RCN = ((MAXR * H * 4 + 15) / 16) * 16;   // bytes of one plane of per-(row, head) floats
    static constexpr int MASKW = POSMAX / EPW / 32 + 1;           // words of the row-end bit mask (one bit per slot)
    static constexpr int ring = 0;
    static constexpr int offs = ring + NS * STAGE;                // pre-scaled row offsets, per stage [edge lane][slot]
    static constexpr int w = offs + POSMAX * 4;
    static constexpr int prow = w + POSMAX * H * 4;
    static constexpr int rc = prow + POSMAX;                      // four planes
    static constexpr int sout = rc + 4 * RCN;                     // two planes
    static constexpr int srb = sout + 2 * RCN;
    static constexpr int sso = srb + ((MAXR + 1) * 4 + 15) / 16 * 16;
    static constexpr int endm = sso + ((MAXR + 1) * 4 + 15) / 16 * 16;
    static constexpr int total = endm + ((MASKW * 4 + 15) / 16) * 16;
};

template <typename T, int G, int V, int H, int MODE, bool SEG, int CAP, int P, int NS, int MINB>
__global__ void __launch_bounds__(32, MINB) lean_kernel(const LeanArgs a) {
    using L = LeanLayout<G, V, H, MODE, SEG, CAP, P, NS>;
    constexpr int EPV = Elem<T>::EPV, NP = EPV / 2;
    constexpr int EPW = L::EPW, ROWB = L::ROWB, STAGE = L::STAGE;
    constexpr int NVEC = G * V, VPH = NVEC / H;    // 16-byte vectors per row / per head
    constexpr int LGNVEC = NVEC == 16 ? 4 : (NVEC == 32 ? 5 : 6);
    constexpr int SPS = P / EPW;                   // slots per stage
    constexpr int HG = H / 4;                      // head groups of four
    constexpr bool kF = MODE == kFwd, kD = MODE == kBwdDst;
    static_assert(kF || kD, "lean kernels cover the forward and the destination-major backward pass");
    static_assert(H % 4 == 0 && NVEC % H == 0 && VPH <= G && (VPH & (VPH - 1)) == 0, "head geometry");
    static_assert((1 << LGNVEC) == NVEC, "row geometry");
    static_assert(P <= 32 && 32 % P == 0 && SPS % 4 == 0 && SPS <= 8, "stage geometry");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const unsigned sbase = (unsigned)__cvta_generic_to_shared(smem_raw);
    const unsigned ring_s = sbase + L::ring, offs_s = sbase + L::offs, w_s = sbase + L::w;
    const unsigned prow_s = sbase + L::prow, rc_s = sbase + L::rc, sout_s = sbase + L::sout;
    const unsigned endm_s = sbase + L::endm;
    int *srb = reinterpret_cast<int *>(smem_raw + L::srb);
    int *sso = reinterpret_cast<int *>(smem_raw + L::sso);
    unsigned *skey = reinterpret_cast<unsigned *>(smem_raw + L::rc + L::RCN);  // forward: plane 1 holds the max key first

    const int lane = threadIdx.x;
    const int gl = lane & (G - 1), half = lane / G;
    // index of position q in the per-stage [edge lane][slot] order of the offsets and weights
    auto perm = [](int q) { return (q / P) * P + ((q % P) % EPW) * SPS + (q % P) / EPW; };

    // ---- which rows ---------------------------------------------------------------------------
    const long long item = blockIdx.x;
    long long row0, eb = 0, ee = 0;   // lane r: edge range of row row0 + r
    int nrows;
    bool excluded = false;
    long long seg = -1;
    if constexpr (!SEG) {
        row0 = item * a.R;
        if (row0 >= a.n_rows) return;
        nrows = (int)((a.n_rows - row0) < a.R ? (a.n_rows - row0) : a.R);
        long long p = 0;
        if (lane <= nrows) p = __ldg(a.indptr + row0 + lane);
        const long long pn = __shfl_down_sync(0xffffffffu, p, 1);
        if (lane < nrows) {
            eb = p;
            ee = pn;
            excluded = ee - eb > a.sp.threshold;
        }
    } else {
        if (item >= a.sp.n_seg) return;
        int lo = 0, hi = a.sp.n_long;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (__ldg(a.sp.long_seg + mid) <= item) lo = mid; else hi = mid;
        }
        row0 = __ldg(a.sp.long_row + lo);
        nrows = 1;
        seg = item;
        if (lane == 0) {
            const long long c = item - __ldg(a.sp.long_seg + lo);
            const long long rb_ = __ldg(a.indptr + row0), re_ = __ldg(a.indptr + row0 + 1);
            eb = rb_ + c * a.sp.threshold;
            ee = eb + a.sp.threshold < re_ ? eb + a.sp.threshold : re_;
        }
    }

    // ---- lane geometry ------------------------------------------------------------------------
    int hv[V];
#pragma unroll
    for (int v = 0; v < V; ++v) hv[v] = (v * G + gl) / VPH;
    const bool head_lead = (gl % VPH) == 0 && half == 0;
    unsigned long long gbase_v[V];   // address of this lane's 16 bytes of row 0 of the gathered array, per vector
#pragma unroll
    for (int v = 0; v < V; ++v) gbase_v[v] = reinterpret_cast<unsigned long long>(reinterpret_cast<const uint4 *>(a.gather) + gl + v * G);
    const unsigned ring_l = ring_s + (unsigned)(half * ROWB + gl * 16);   // this lane's 16 bytes of slot 0, stage 0

    f32x2 pacc0[V][NP], pacc1[V][NP];
    float sv[V];
    uint4 rvq[V], rvq_next[V];
#pragma unroll
    for (int v = 0; v < V; ++v) {
        sv[v] = 0.f;
#pragma unroll
        for (int k = 0; k < NP; ++k) pacc0[v][k] = pacc1[v][k] = zero2();
        rvq[v] = rvq_next[v] = make_uint4(0u, 0u, 0u, 0u);
    }
    auto request_rowvec = [&](long long row_, uint4 (&dst)[V]) {
        const uint4 *rp = reinterpret_cast<const uint4 *>(a.rowvec) + row_ * NVEC + gl;
#pragma unroll
        for (int v = 0; v < V; ++v) dst[v] = __ldg(rp + v * G);
    };

    const int deg_l = (lane < nrows && !excluded) ? (int)(ee - eb) : 0;   // <= CAP by the host's precondition
    const unsigned excl_all = __ballot_sync(0xffffffffu, excluded);

    int r = 0;
    while (r < nrows) {
        if ((excl_all >> r) & 1u) {
            ++r;
            continue;
        }
        // ---- choose the chunk: rows [r, r2), none excluded, at most CAP edges in all ----------------
        int r2, ne;
        const long long cb = __shfl_sync(0xffffffffu, eb, r);   // global index of the chunk's first edge
        if constexpr (SEG) {
            r2 = 1;
            ne = __shfl_sync(0xffffffffu, deg_l, 0);
        } else {
            int pre = (lane >= r && lane < nrows) ? deg_l : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, pre, o);
                if (lane >= o) pre += t;
            }
            const unsigned later = excl_all & ~((1u << r) - 1u);
            const int stop = later ? __ffs(later) - 1 : nrows;
            const unsigned fits = __ballot_sync(0xffffffffu, lane >= r && lane < stop && pre <= CAP);
            r2 = r + __popc(fits);
            ne = __shfl_sync(0xffffffffu, pre, r2 - 1);
        }
        const int nr = r2 - r;

        // ---- stage A: row tables, row-end mask, non-empty rows -----------------------------------------
        unsigned nemask;   // bit i: local row i has edges
        int nslots;        // slots of the chunk (produced by a warp reduction: uniform)
        {
            const int i = lane - r;
            const bool mine = i >= 0 && i < nr;
            int ns = 0;
            if (mine) {
                srb[i] = (int)(eb - cb);
                if (i == nr - 1) srb[nr] = ne;
                ns = (deg_l + EPW - 1) / EPW;
            }
            int inc = ns;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += t;
            }
            if (mine) sso[i] = inc - ns;
            if (i == nr - 1) sso[nr] = inc;
            nslots = (int)__reduce_add_sync(0xffffffffu, (unsigned)ns);
            nemask = __ballot_sync(0xffffffffu, mine && ns > 0) >> r;
            if constexpr (!SEG) {
                if (lane < L::MASKW) sts_u32(endm_s + 4 * lane, 0u);
                __syncwarp();
                if (mine && ns > 0) atomicOr(reinterpret_cast<unsigned *>(smem_raw + L::endm) + ((inc - 1) >> 5), 1u << ((inc - 1) & 31));
            }
        }
        __syncwarp();
        const int npos = nslots * EPW;
        const int nstages = (npos + P - 1) / P;

        // ---- stage B: row offsets of the columns (a row's padding repeats its last column, the last stage is
        // filled up with repeats), position -> row, the score terms er[col, :] on their way into the weight area
        // (position-major for now), per-(row, head) constants ------------------------------------------------
        {
            int i = 0;
            for (int q0 = 0; q0 < nstages * P; q0 += 64) {
                int c[2] = {0, 0}, pr[2] = {0, 0};
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int q = q0 + 32 * u + lane;
                    if (q < npos) {
                        if constexpr (!SEG) {
                            while (q >= sso[i + 1] * EPW) ++i;
                        }
                        const int t = srb[i] + (q - sso[i] * EPW);
                        const int last = srb[i + 1] - 1;
                        const bool pad = t > last;
                        c[u] = ld_stream_i32(a.indices + cb + (pad ? last : t));
                        pr[u] = i | (pad ? 0x80 : 0);
                    } else if (q < nstages * P) {
                        c[u] = ld_stream_i32(a.indices + cb + (ne - 1));   // fill of the last stage
                    }
                }
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int q = q0 + 32 * u + lane;
                    if (q < nstages * P) sts_u32(offs_s + 4 * (unsigned)perm(q), (unsigned)c[u] << LGNVEC);
                    if (q < npos) {
                        sts_u8(prow_s + q, (unsigned)pr[u]);
                        const float *src = a.er + (long long)c[u] * H;
#pragma unroll
                        for (int hg = 0; hg < HG; ++hg) cp_async16_full(w_s + (unsigned)((q * H + hg * 4) * 4), src + hg * 4);
                    }
                }
            }
            cp_async_commit();   // the score terms: the oldest group
            for (int x = lane; x < nr * H; x += 32) {
                const long long o = (row0 + r) * H + x;
                if constexpr (kF) {
                    sts_f32(rc_s + 4 * x, __ldg(a.el + o));
                    skey[x] = kKeyNegInf;
                    sts_f32(sout_s + 4 * x, 0.f);
                } else {
                    const float mm = __ldg(a.m + o), dd = __ldg(a.d + o);
                    sts_f32(rc_s + 4 * x, __ldg(a.el + o));
                    sts_f32(rc_s + L::RCN + 4 * x, mm);
                    sts_f32(rc_s + 2 * L::RCN + 4 * x, dd > 0.f ? __fdividef(1.f, dd) : 0.f);
                    sts_f32(rc_s + 3 * L::RCN + 4 * x, -mm * kLog2e);
                    sts_f32(sout_s + 4 * x, 0.f);
                    sts_f32(sout_s + L::RCN + 4 * x, 0.f);
                }
            }
        }
        __syncwarp();

        // ---- start the ring: one commit group per stage, NS groups in flight ------------------------------
        // Lane (half, gl) copies, and later reads back, its own 16 bytes of every slot: no cross-lane
        // synchronisation around the ring.
        auto issue_stage = [&](int j) {
            const unsigned dst = ring_l + (unsigned)((j % NS) * STAGE);
            const unsigned ob = offs_s + (unsigned)((j * P + half * SPS) * 4);
#pragma unroll
            for (int kq = 0; kq < SPS; kq += 4) {
                const uint4 o4 = lds128(ob + kq * 4);
                const unsigned ov[4] = {o4.x, o4.y, o4.z, o4.w};
#pragma unroll
                for (int t = 0; t < 4; ++t)
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        unsigned long long src;   // base + offset * 16 in one multiply-add
                        asm("mad.wide.u32 %0, %1, 16, %2;\n" : "=l"(src) : "r"(ov[t]), "l"(gbase_v[v]));
                        cp_async16_full(dst + (unsigned)((kq + t) * EPW * ROWB + v * G * 16), reinterpret_cast<const void *>(src));
                    }
            }
        };
#pragma unroll
        for (int j = 0; j < NS; ++j) {
            if (j < nstages) issue_stage(j);
            cp_async_commit();
        }

        // rows without edges: their vector outputs are zeros (the scalars leave with the others at the chunk's end)
        if constexpr (kF && !SEG) {
            unsigned em = ~nemask & ((1u << nr) - 1u);
            while (em) {
                const int i = __ffs(em) - 1;
                em &= em - 1;
                uint4 *rp = reinterpret_cast<uint4 *>(a.out) + (row0 + r + i) * NVEC;
                for (int x = lane; x < NVEC; x += 32) rp[x] = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        if constexpr (kD && !SEG) {
            if (nslots > 0) request_rowvec(row0 + r + (__ffs(nemask) - 1), rvq_next);
        }

        // ---- stage C: weights ----------------------------------------------------------------------------
        // Position q sits in stage block q / P at local position lp = q % P = k * EPW + hf (slot k of the stage,
        // edge lane hf); its weight for head h goes to word (hf * H + h) * SPS + k of the block (slot fastest).
        cp_async_wait<NS>();   // the score terms have landed (the ring's groups may still be in flight)
        __syncwarp();
        if constexpr (kF) {
            // sweep 1: max of er per (row, head)
            if constexpr (SEG) {
                float mx[H];
#pragma unroll
                for (int h = 0; h < H; ++h) mx[h] = SAR_NEG_INF;
                for (int q = lane; q < npos; q += 32) {
#pragma unroll
                    for (int hg = 0; hg < HG; ++hg) {
                        const float4 e4 = lds_f4(w_s + (unsigned)((q * H + hg * 4) * 4));
                        mx[hg * 4 + 0] = fmaxf(mx[hg * 4 + 0], e4.x);
                        mx[hg * 4 + 1] = fmaxf(mx[hg * 4 + 1], e4.y);
                        mx[hg * 4 + 2] = fmaxf(mx[hg * 4 + 2], e4.z);
                        mx[hg * 4 + 3] = fmaxf(mx[hg * 4 + 3], e4.w);
                    }
                }
#pragma unroll
                for (int h = 0; h < H; ++h) {
                    const unsigned k = __reduce_max_sync(0xffffffffu, fkey(mx[h]));
                    if (lane == 0) skey[h] = k;
                }
            } else {
                for (int q = lane; q < npos; q += 32) {
                    const int i = (int)(lds_u8(prow_s + q) & 0x7f);
#pragma unroll
                    for (int hg = 0; hg < HG; ++hg) {
                        const float4 e4 = lds_f4(w_s + (unsigned)((q * H + hg * 4) * 4));
                        atomicMax(&skey[i * H + hg * 4 + 0], fkey(e4.x));
                        atomicMax(&skey[i * H + hg * 4 + 1], fkey(e4.y));
                        atomicMax(&skey[i * H + hg * 4 + 2], fkey(e4.z));
                        atomicMax(&skey[i * H + hg * 4 + 3], fkey(e4.w));
                    }
                }
            }
            __syncwarp();
            // m = LeakyReLU(el + max er) per (row, head): exactly the max of the per-edge scores
            for (int x = lane; x < nr * H; x += 32) {
                const unsigned k = skey[x];
                float mm = SAR_NEG_INF;
                if (k != kKeyNegInf) {
                    float gr;
                    mm = leaky(lds_f32(rc_s + 4 * x) + fkey_inv(k), a.slope, gr);
                }
                sts_f32(rc_s + L::RCN + 4 * x, mm);
                sts_f32(rc_s + 3 * L::RCN + 4 * x, -mm * kLog2e);
            }
            __syncwarp();
        }
        {
            for (int q0 = 0; q0 < npos; q0 += 32) {
                const int q = q0 + lane;
                const bool live = q < npos;
                float4 e4[HG], l4[HG], n4[HG], i4[HG];
#pragma unroll
                for (int hg = 0; hg < HG; ++hg) e4[hg] = l4[hg] = n4[hg] = i4[hg] = make_float4(0.f, 0.f, 0.f, 0.f);
                bool pad = true;
                if (live) {
                    const unsigned pr = lds_u8(prow_s + q);   // a segment of odd length has a padding position too
                    const int i = SEG ? 0 : (int)(pr & 0x7f);
                    pad = (pr & 0x80) != 0;
#pragma unroll
                    for (int hg = 0; hg < HG; ++hg) {
                        e4[hg] = lds_f4(w_s + (unsigned)((q * H + hg * 4) * 4));
                        l4[hg] = lds_f4(rc_s + (unsigned)((i * H + hg * 4) * 4));
                        n4[hg] = lds_f4(rc_s + 3 * L::RCN + (unsigned)((i * H + hg * 4) * 4));
                        if constexpr (kD) i4[hg] = lds_f4(rc_s + 2 * L::RCN + (unsigned)((i * H + hg * 4) * 4));
                    }
                }
                __syncwarp();   // every lane has read its staged score terms before the block is overwritten
                if (live) {
                    const unsigned wb = w_s + (unsigned)((q / P) * P * H + ((q % P) % EPW) * H * SPS + (q % P) / EPW) * 4u;
#pragma unroll
                    for (int hg = 0; hg < HG; ++hg) {
                        const float ev[4] = {e4[hg].x, e4[hg].y, e4[hg].z, e4[hg].w};
                        const float lv[4] = {l4[hg].x, l4[hg].y, l4[hg].z, l4[hg].w};
                        const float nv[4] = {n4[hg].x, n4[hg].y, n4[hg].z, n4[hg].w};
                        const float iv[4] = {i4[hg].x, i4[hg].y, i4[hg].z, i4[hg].w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float s_ = lv[j] + ev[j];
                            float gr;
                            const float e = leaky(s_, a.slope, gr);
                            float wv = ex2_approx(fmaf(e, kLog2e, nv[j]));
                            if constexpr (kD) {
                                wv *= iv[j];
                                wv = s_ > 0.f ? wv : -wv;   // the sign bit carries LeakyReLU' = slope
                            }
                            if (pad) wv = 0.f;
                            sts_f32(wb + (unsigned)(((hg * 4 + j) * SPS) * 4), wv);
                        }
                    }
                }
            }
            __syncwarp();
        }

        // ---- stage D: the gathered rows, stage by stage -----------------------------------------------------
        {
            int s = 0;                                // first slot of the stage (uniform)
            int ri = SEG ? 0 : (__ffs(nemask) - 1);   // local index of the row being accumulated (uniform)
            for (int j = 0; j < nstages; ++j) {
                cp_async_wait<NS - 1>();              // this lane's copies of stage j have landed
                const unsigned ring_a = ring_l + (unsigned)((j % NS) * STAGE);
                unsigned w_a[V];
#pragma unroll
                for (int v = 0; v < V; ++v) w_a[v] = w_s + (unsigned)((j * P * H + (half * H + hv[v]) * SPS) * 4);
                const int cnt = nslots - s;           // slots k >= cnt of this stage do not exist
                unsigned ends;                        // bit k: slot k is the last of its row (a vote: uniform)
                if constexpr (SEG) {
                    ends = cnt <= SPS ? (1u << (cnt - 1)) : 0u;
                } else {
                    unsigned bit = 0;
                    if (lane < SPS) {
                        const int sl = s + lane;
                        bit = (lds_u32(endm_s + 4 * (unsigned)(sl >> 5)) >> (sl & 31)) & 1u;
                    }
                    ends = __ballot_sync(0xffffffffu, bit != 0);
                }
                float4 w4[V];
                // The chunk's last slot ends a row, and the walk leaves the stage from inside that row's epilogue:
                // slots past it (a last stage that is not full) are never reached and need no test of their own.
#pragma unroll
                for (int k = 0; k < SPS; ++k) {
                    {
                        if (k % 4 == 0) {
#pragma unroll
                            for (int v = 0; v < V; ++v) w4[v] = lds_f4(w_a[v] + k * 4);
                        }
#pragma unroll
                        for (int v = 0; v < V; ++v) {
                            const float wk = (k % 4 == 0) ? w4[v].x : (k % 4 == 1) ? w4[v].y : (k % 4 == 2) ? w4[v].z : w4[v].w;
                            f32x2 x[NP];
                            Pairs<T>::get(lds128(ring_a + (unsigned)(k * EPW * ROWB + v * G * 16)), x);
                            if constexpr (kF) {
                                sv[v] += wk;
                                const f32x2 w2 = pack2(wk, wk);
#pragma unroll
                                for (int t = 0; t < NP; ++t) pacc0[v][t] = fma2(w2, x[t], pacc0[v][t]);
                            } else {
                                const float al = fabsf(wk);
                                const float wg = wk < 0.f ? al * a.slope : al;   // alpha * LeakyReLU'
                                sv[v] += wg;
                                const f32x2 a2 = pack2(al, al), g2 = pack2(wg, wg);
#pragma unroll
                                for (int t = 0; t < NP; ++t) {
                                    pacc0[v][t] = fma2(a2, x[t], pacc0[v][t]);
                                    pacc1[v][t] = fma2(g2, x[t], pacc1[v][t]);
                                }
                            }
                        }
                        if (ends & (1u << k)) {
                            // ---- the row is complete ---------------------------------------------------------
                            const long long row = row0 + r + ri;
                            if constexpr (kD && !SEG) {
#pragma unroll
                                for (int v = 0; v < V; ++v) rvq[v] = rvq_next[v];
                                const unsigned rest = nemask & ~((2u << ri) - 1u);
                                if (rest) request_rowvec(row0 + r + (__ffs(rest) - 1), rvq_next);
                            }
                            if constexpr (SEG) {
                                // partial accumulators of the segment, float32, for the merge launch
                                float acc0[V][EPV], acc1[V][EPV];
#pragma unroll
                                for (int v = 0; v < V; ++v)
#pragma unroll
                                    for (int t = 0; t < NP; ++t) {
                                        unpack2(pacc0[v][t], acc0[v][2 * t], acc0[v][2 * t + 1]);
                                        unpack2(pacc1[v][t], acc1[v][2 * t], acc1[v][2 * t + 1]);
                                    }
#pragma unroll
                                for (int off = G; off < 32; off <<= 1)
#pragma unroll
                                    for (int v = 0; v < V; ++v) {
                                        sv[v] += __shfl_xor_sync(0xffffffffu, sv[v], off);
#pragma unroll
                                        for (int e = 0; e < EPV; ++e) {
                                            acc0[v][e] += __shfl_xor_sync(0xffffffffu, acc0[v][e], off);
                                            if constexpr (!kF) acc1[v][e] += __shfl_xor_sync(0xffffffffu, acc1[v][e], off);
                                        }
                                    }
                                if (half == 0) {
                                    constexpr long long rowf = (long long)NVEC * EPV;
                                    float *rec = a.sp.part + seg * a.sp.pstride;
                                    bool vok[V];
#pragma unroll
                                    for (int v = 0; v < V; ++v) vok[v] = true;
                                    if constexpr (kF) {
                                        store_acc_row<G, V, EPV>(rec, gl, vok, acc0);
#pragma unroll
                                        for (int v = 0; v < V; ++v)
                                            if ((gl % VPH) == 0) {
                                                rec[rowf + hv[v]] = lds_f32(rc_s + L::RCN + 4 * hv[v]);
                                                rec[rowf + H + hv[v]] = sv[v];
                                            }
                                    } else {
                                        store_acc_row<G, V, EPV>(rec, gl, vok, acc1);
                                        store_acc_row<G, V, EPV>(rec + rowf, gl, vok, acc0);
#pragma unroll
                                        for (int v = 0; v < V; ++v)
                                            if ((gl % VPH) == 0) rec[2 * rowf + hv[v]] = sv[v];
                                    }
                                }
                            } else if constexpr (kF) {
#pragma unroll
                                for (int off = G; off < 32; off <<= 1)
#pragma unroll
                                    for (int v = 0; v < V; ++v) {
                                        sv[v] += __shfl_xor_sync(0xffffffffu, sv[v], off);
#pragma unroll
                                        for (int t = 0; t < NP; ++t) {
                                            const f32x2 o = pack2(__shfl_xor_sync(0xffffffffu, pacc0[v][t].x, off),
                                                                  __shfl_xor_sync(0xffffffffu, pacc0[v][t].y, off));
                                            pacc0[v][t] = fma2(o, pack2(1.f, 1.f), pacc0[v][t]);
                                        }
                                    }
                                if (half == 0) {
                                    uint4 *rp = reinterpret_cast<uint4 *>(a.out) + row * NVEC + gl;
#pragma unroll
                                    for (int v = 0; v < V; ++v) {
                                        const float inv = sv[v] > 0.f ? __fdividef(1.f, sv[v]) : 0.f;
                                        const f32x2 i2 = pack2(inv, inv);
                                        float acc0[EPV];
#pragma unroll
                                        for (int t = 0; t < NP; ++t) {
                                            const f32x2 y = fma2(pacc0[v][t], i2, zero2());
                                            unpack2(y, acc0[2 * t], acc0[2 * t + 1]);
                                        }
                                        rp[v * G] = Elem<T>::pack(acc0);
                                        if ((gl % VPH) == 0) sts_f32(sout_s + (unsigned)((ri * H + hv[v]) * 4), sv[v]);
                                    }
                                }
                            } else {
                                // dot products with the row-stationary vector on the un-folded accumulators, then
                                // one reduction over the lanes of each head and over the edge lanes
                                float pA[V], pB[V];
#pragma unroll
                                for (int v = 0; v < V; ++v) {
                                    f32x2 rv[NP];
                                    Pairs<T>::get(rvq[v], rv);
                                    f32x2 qa = zero2(), qb = zero2();
#pragma unroll
                                    for (int t = 0; t < NP; ++t) {
                                        qa = fma2(rv[t], pacc0[v][t], qa);
                                        qb = fma2(rv[t], pacc1[v][t], qb);
                                    }
                                    pA[v] = qa.x + qa.y;
                                    pB[v] = qb.x + qb.y;
                                }
#pragma unroll
                                for (int off = 1; off < 32; off <<= 1) {
                                    if (off < VPH || off >= G) {
#pragma unroll
                                        for (int v = 0; v < V; ++v) {
                                            pA[v] += __shfl_xor_sync(0xffffffffu, pA[v], off);
                                            pB[v] += __shfl_xor_sync(0xffffffffu, pB[v], off);
                                            if (off >= G) sv[v] += __shfl_xor_sync(0xffffffffu, sv[v], off);
                                        }
                                    }
                                }
                                if (head_lead) {
#pragma unroll
                                    for (int v = 0; v < V; ++v) {
                                        sts_f32(sout_s + (unsigned)((ri * H + hv[v]) * 4), pB[v] - pA[v] * sv[v]);   // del
                                        sts_f32(sout_s + L::RCN + (unsigned)((ri * H + hv[v]) * 4), pA[v]);         // D
                                    }
                                }
                            }
#pragma unroll
                            for (int v = 0; v < V; ++v) {
                                sv[v] = 0.f;
#pragma unroll
                                for (int t = 0; t < NP; ++t) pacc0[v][t] = pacc1[v][t] = zero2();
                            }
                            if constexpr (!SEG) {
                                const unsigned rest = nemask & ~((2u << ri) - 1u);
                                ri = rest ? __ffs(rest) - 1 : nr;
                            }
                            if (k + 1 >= cnt) goto chunk_done;
                        }
                    }
                }
                s += SPS;
                if (j + NS < nstages) issue_stage(j + NS);   // the stage just read is free (each lane re-fills its own bytes)
                cp_async_commit();

            }
        chunk_done:
            cp_async_wait<0>();   // only empty groups are left
        }

        // ---- the chunk's per-(row, head) scalars, coalesced ------------------------------------------------
        if constexpr (!SEG) {
            __syncwarp();
            for (int x = lane; x < nr * H; x += 32) {
                const long long o = (row0 + r) * H + x;
                if constexpr (kF) {
                    a.m_out[o] = lds_f32(rc_s + L::RCN + 4 * x);
                    a.d_out[o] = lds_f32(sout_s + 4 * x);
                } else {
                    a.del[o] = lds_f32(sout_s + 4 * x);
                    a.rec_out[o] = make_float4(lds_f32(rc_s + 4 * x), lds_f32(rc_s + L::RCN + 4 * x),
                                               lds_f32(rc_s + 2 * L::RCN + 4 * x), lds_f32(sout_s + L::RCN + 4 * x));
                }
            }
            __syncwarp();
        }
        r = r2;
    }
}

// ---- launchers (instantiated once per pass and storage type by the sar_lean_*.cu files) ---------------------
constexpr int kLeanMinBlocks = 8;

static inline int lean_rows_per_span(long long n_rows, long long nnz, int cap) {
    const double avg = n_rows > 0 ? (double)nnz / (double)n_rows : 0.0;
    int R = avg > 0.5 ? (int)(1.0 * cap / avg + 0.5) : kMaxSpanRows;
    if (R < 1) R = 1;
    if (R > kMaxSpanRows) R = kMaxSpanRows;
    return R;
}

// One configuration: chunks of kLeanCap edges, ring of two stages of 2 KB (4 KB for rows of 1 KB), measured best on
// the large workload among stages of 2 / 4 KB, two to four stages, chunks of 128 / 192 / 256 edges.
template <typename T, int G, int V, int H, int MODE>
static sar_status launch_lean(LeanArgs a, long long nnz, const char *name, const char *seg_name, cudaStream_t st) {
    constexpr int STAGEB = V == 1 ? 2048 : 4096;
    constexpr int NS = 2;
    constexpr int P = STAGEB / (G * V * 16);   // positions per stage
    using LR = LeanLayout<G, V, H, MODE, false, kLeanCap, P, NS>;
    using LS = LeanLayout<G, V, H, MODE, true, kLeanCap, P, NS>;
    a.R = lean_rows_per_span(a.n_rows, nnz, kLeanCap);
    const long long spans = (a.n_rows + a.R - 1) / a.R;
    if (spans > 0) {
        auto kern = lean_kernel<T, G, V, H, MODE, false, kLeanCap, P, NS, kLeanMinBlocks>;
        SAR_TRY(ensure_smem(kern, LR::total));
        SAR_LAUNCH(name, st, kern<<<(unsigned)spans, 32, LR::total, st>>>(a));
        SAR_TRY(sar_after_launch());
    }
    if (a.sp.n_seg > 0) {
        auto kern = lean_kernel<T, G, V, H, MODE, true, kLeanCap, P, NS, kLeanMinBlocks>;
        SAR_TRY(ensure_smem(kern, LS::total));
        SAR_LAUNCH(seg_name, st, kern<<<(unsigned)a.sp.n_seg, 32, LS::total, st>>>(a));
        SAR_TRY(sar_after_launch());
    }
    return SAR_OK;
}

template <typename T, int MODE>
static sar_status dispatch_lean(const Shape &s, const LeanArgs &a, long long nnz, const char *name, const char *seg_name,
                                cudaStream_t st) {
    if (s.G == 16 && s.V == 1 && s.geom.H == 4) return launch_lean<T, 16, 1, 4, MODE>(a, nnz, name, seg_name, st);
    if (s.G == 32 && s.V == 1 && s.geom.H == 4) return launch_lean<T, 32, 1, 4, MODE>(a, nnz, name, seg_name, st);
    if (s.G == 32 && s.V == 1 && s.geom.H == 8) return launch_lean<T, 32, 1, 8, MODE>(a, nnz, name, seg_name, st);
    if (s.G == 32 && s.V == 2 && s.geom.H == 4) return launch_lean<T, 32, 2, 4, MODE>(a, nnz, name, seg_name, st);
    return SAR_ERR_UNSUPPORTED;
}

}  // namespace sar

// One translation unit per pass and storage type: SAR_LEAN_TU(suffix, T, MODE, "rows name", "segments name").
#define SAR_LEAN_TU(SUFFIX, TYPE, MODE, NAME, SEG_NAME)                                                     \
    namespace sar {                                                                                         \
    sar_status lean_##SUFFIX(const Shape &s, const LeanArgs &a, long long nnz, cudaStream_t st) {           \
        return dispatch_lean<TYPE, MODE>(s, a, nnz, NAME, SEG_NAME, st);                                    \
    }                                                                                                       \
    }

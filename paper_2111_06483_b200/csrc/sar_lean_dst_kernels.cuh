// Lean span kernel of the destination-major whole-graph backward pass (internal): with alpha rebuilt from
// (el, er, m, d), A = sum_j alpha feat_j, B = sum_j alpha g' feat_j, S = sum_j alpha g' over the CSR; D_i = <gout_i, A>,
// del_i = <gout_i, B> - D_i S, and the record {el, m, 1/d, D} per (i, head) for the source-major pass.
//
// Same plan as lean_src_kernel (sar_lean_src_kernels.cuh): stage-granular cp.async ring of the gathered feature rows,
// the score terms er[col, :] of a stage's positions travelling with the stage (16 bytes per position and head group
// into a small ring), the weights of a stage computed just before it is consumed, one (position, head) pair per lane.
// Preconditions as for lean_src_kernel, on the CSR (checked by the host).
//
// PART = true is the same pass as one PARTITION STEP of Algorithm 2: the call holds the edges from one source partition,
// D_i is given (it needs the whole row and was computed beforehand) and del_i collects <gout_i, B> - D_i S partition by
// partition (rec_in, first).  Most of a row's edges lie in other partitions, so the rows are short and most have no
// edge at all; the variant is laid out for that: spans of up to kLeanPartRows rows, rows without edges cost nothing
// (no record, no write unless `first`), the position -> row map is found by bisection, and the output-gradient rows of
// the chunk's first kLeanPartStaged rows that do have edges are copied into shared memory with the chunk's first stage
// instead of being loaded row after row (the rows beyond that load theirs when they complete).
#pragma once

#include "sar_lean_src_kernels.cuh"

namespace sar {


constexpr int kLeanPartRows = 31;    // rows per span of a partition step (one lane per row, one more for the end)
// Rows with edges of a chunk of a partition step whose own data is staged (the chunk's first ones; the others load it
// when they complete): of the destination-major step (rows of the storage type) and of the forward step (float32
// numerator rows).  Measured on the large workload with 16 partitions, per step: forward 4 / 8 / 12 rows 3.07 / 2.98 /
// 3.05 ms, destination-major with the source-major pass 8 / 12 / 16 rows 3.30 / 3.24 / 3.30 ms (more staged rows leave
// fewer loads to wait for but fewer warps resident).
constexpr int kLeanPartStaged = 12;
constexpr int kLeanPartStagedFwd = 8;

template <int G, int V, int H, bool SEG, int CAP, int P, int NS, bool PART = false>
struct LeanDstLayout {
    static constexpr int EPW = 32 / G;
    static constexpr int ROWB = G * V * 16;
    static constexpr int STAGE = P * ROWB;
    static constexpr int MAXR = SEG ? 1 : (PART ? kLeanPartRows : kMaxSpanRows);
    static constexpr int POSMAX = ((CAP + MAXR * (EPW - 1) + 31) / 32) * 32;
    static constexpr int RCN = ((MAXR * H * 4 + 15) / 16) * 16;
    static constexpr int MASKW = POSMAX / EPW / 32 + 1;
    static constexpr int RECB = ((P * H * 4 + 15) / 16) * 16;     // score terms of one stage
    static constexpr int WB = P * H * 4;                          // the weights of one stage
    static constexpr int ring = 0;
    static constexpr int rec = ring + NS * STAGE;
    static constexpr int w = rec + NS * RECB;
    static constexpr int offs = w + WB;
    static constexpr int prow = offs + POSMAX * 4;
    static constexpr int rc = prow + POSMAX;                      // el, m, 1/d, -m log2(e) of the chunk's rows
    static constexpr int sout = rc + 4 * RCN;                     // del, D
    static constexpr int srb = sout + 2 * RCN;
    static constexpr int sso = srb + ((MAXR + 1) * 4 + 15) / 16 * 16;
    static constexpr int endm = sso + ((MAXR + 1) * 4 + 15) / 16 * 16;
    static constexpr int rowst = endm + ((MASKW * 4 + 15) / 16) * 16;   // partition step: gout of the rows with edges
    static constexpr int total = rowst + ((PART && !SEG) ? kLeanPartStaged * ROWB : 0);
};

template <typename T, int G, int V, int H, bool SEG, int CAP, int P, int NS, int MINB, bool PART = false>
__global__ void __launch_bounds__(32, MINB) lean_dst_kernel(const LeanArgs a) {
    static_assert(!(PART && SEG), "the segments of a partition step run the whole-graph segment kernel");
    using L = LeanDstLayout<G, V, H, SEG, CAP, P, NS, PART>;
    constexpr int EPV = Elem<T>::EPV, NP = EPV / 2;
    constexpr int EPW = L::EPW, ROWB = L::ROWB, STAGE = L::STAGE;
    constexpr int NVEC = G * V, VPH = NVEC / H;
    constexpr int LGNVEC = NVEC == 16 ? 4 : (NVEC == 32 ? 5 : 6);
    constexpr int SPS = P / EPW;                   // slots per stage
    constexpr int ITEMS = P * H;                   // (position, head) pairs of a stage
    constexpr int COPIES = P * H / 4;              // 16-byte copies that bring a stage's score terms
    static_assert(H % 4 == 0 && NVEC % H == 0 && VPH <= G && (VPH & (VPH - 1)) == 0, "head geometry");
    static_assert((1 << LGNVEC) == NVEC, "row geometry");
    static_assert(P <= 32 && 32 % P == 0 && (SPS == 4 || SPS == 8), "stage geometry: four or eight slots per stage");
    static_assert(ITEMS <= 64, "at most two (position, head) pairs per lane");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const unsigned sbase = (unsigned)__cvta_generic_to_shared(smem_raw);
    const unsigned ring_s = sbase + L::ring, rec_s = sbase + L::rec, w_s = sbase + L::w, offs_s = sbase + L::offs;
    const unsigned prow_s = sbase + L::prow, rc_s = sbase + L::rc, sout_s = sbase + L::sout, endm_s = sbase + L::endm;
    const unsigned rowst_s = sbase + L::rowst;
    int *srb = reinterpret_cast<int *>(smem_raw + L::srb);
    int *sso = reinterpret_cast<int *>(smem_raw + L::sso);

    const int lane = threadIdx.x;
    const int gl = lane & (G - 1), half = lane / G;
    auto perm = [](int q) { return (q / P) * P + ((q % P) % EPW) * SPS + (q % P) / EPW; };

    // ---- which rows ---------------------------------------------------------------------------
    const long long item = blockIdx.x;
    long long row0, eb = 0, ee = 0;
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
    unsigned long long gbase_v[V];
#pragma unroll
    for (int v = 0; v < V; ++v) gbase_v[v] = reinterpret_cast<unsigned long long>(reinterpret_cast<const uint4 *>(a.gather) + gl + v * G);
    const unsigned ring_l = ring_s + (unsigned)(half * ROWB + gl * 16);
    // the (position, head) pairs this lane copies the record of and scores: it = lane (+ 32)
    constexpr int NIT = (ITEMS + 31) / 32;

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

    const int deg_l = (lane < nrows && !excluded) ? (int)(ee - eb) : 0;
    const unsigned excl_all = __ballot_sync(0xffffffffu, excluded);

    int r = 0;
    while (r < nrows) {
        if ((excl_all >> r) & 1u) {
            ++r;
            continue;
        }
        // ---- choose the chunk: rows [r, r2), none excluded, at most CAP edges in all ----------------
        int r2, ne;
        const long long cb = __shfl_sync(0xffffffffu, eb, r);
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
        unsigned nemask;
        int nslots;
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

        // ---- stage B: row offsets of the columns (padding and the fill of the last stage repeat a real column and
        // are marked so that they weigh nothing), position -> row, the rows' own score terms ------------------------
        {
            int i = 0;
            for (int q0 = 0; q0 < nstages * P; q0 += 64) {
                int c[2] = {0, 0}, pr[2] = {0x80, 0x80};
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int q = q0 + 32 * u + lane;
                    if (q < npos) {
                        if constexpr (PART) {   // many short rows: the position's row by bisection over the rows' first slots
                            const int slot = q / EPW;
                            int lo = 0, hi = nr;
                            while (hi - lo > 1) {
                                const int mid = (lo + hi) >> 1;
                                if (sso[mid] <= slot) lo = mid; else hi = mid;
                            }
                            i = lo;
                        } else if constexpr (!SEG) {
                            while (q >= sso[i + 1] * EPW) ++i;
                        }
                        const int t = srb[i] + (q - sso[i] * EPW);
                        const int last = srb[i + 1] - 1;
                        const bool pad = t > last;
                        c[u] = ld_stream_i32(a.indices + cb + (pad ? last : t));
                        pr[u] = i | (pad ? 0x80 : 0);
                    } else if (q < nstages * P) {
                        c[u] = ld_stream_i32(a.indices + cb + (ne - 1));
                    }
                }
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int q = q0 + 32 * u + lane;
                    if (q < nstages * P) {
                        sts_u32(offs_s + 4 * (unsigned)perm(q), (unsigned)c[u] << LGNVEC);
                        sts_u8(prow_s + q, (unsigned)pr[u]);
                    }
                }
            }
            if constexpr (PART) {
                // the constants of the rows with edges only, every load issued before the first store: el, m, d, the D
                // given and del so far
                constexpr int NX = (L::MAXR * H + 31) / 32;
                float cv[NX][5];
#pragma unroll
                for (int n = 0; n < NX; ++n) {
                    const int x = lane + 32 * n;
                    cv[n][0] = cv[n][1] = cv[n][2] = cv[n][3] = cv[n][4] = 0.f;
                    if (x < nr * H && ((nemask >> (x / H)) & 1u)) {
                        const long long o = (row0 + r) * H + x;
                        cv[n][0] = __ldg(a.el + o);
                        cv[n][1] = __ldg(a.m + o);
                        cv[n][2] = __ldg(a.d + o);
                        cv[n][3] = __ldg(&a.rec_in[o].w);
                        if (!a.first) cv[n][4] = a.del[o];   // plain load: this launch rewrites it
                    }
                }
#pragma unroll
                for (int n = 0; n < NX; ++n) {
                    const int x = lane + 32 * n;
                    if (x < nr * H) {
                        sts_f32(rc_s + 4 * x, cv[n][0]);
                        sts_f32(rc_s + L::RCN + 4 * x, cv[n][1]);
                        sts_f32(rc_s + 2 * L::RCN + 4 * x, cv[n][2] > 0.f ? __fdividef(1.f, cv[n][2]) : 0.f);
                        sts_f32(rc_s + 3 * L::RCN + 4 * x, -cv[n][1] * kLog2e);
                        sts_f32(sout_s + 4 * x, cv[n][4]);
                        sts_f32(sout_s + L::RCN + 4 * x, cv[n][3]);
                    }
                }
            } else {
                for (int x = lane; x < nr * H; x += 32) {
                    const long long o = (row0 + r) * H + x;
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

        // ---- the ring: the gathered rows of a stage and the destination records of its positions, one commit group
        // per stage ------------------------------------------------------------------------------------------------
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
                        unsigned long long src;
                        asm("mad.wide.u32 %0, %1, 16, %2;\n" : "=l"(src) : "r"(ov[t]), "l"(gbase_v[v]));
                        cp_async16_full(dst + (unsigned)((kq + t) * EPW * ROWB + v * G * 16), reinterpret_cast<const void *>(src));
                    }
            }
            if (lane < COPIES) {
                const int p = lane / (H / 4), hq = lane % (H / 4);
                const unsigned col = lds_u32(offs_s + 4 * (unsigned)perm(j * P + p)) >> LGNVEC;
                cp_async16_full(rec_s + (unsigned)((j % NS) * L::RECB + lane * 16), a.er + (size_t)col * H + hq * 4);
            }
        };
        if constexpr (PART) {   // the output-gradient rows of the first rows with edges, in their order, with the first stage
            unsigned todo = nemask;
            unsigned dst = rowst_s + (unsigned)lane * 16u;
            for (int ci = 0; todo && ci < kLeanPartStaged; ++ci) {
                const int i2 = __ffs(todo) - 1;
                todo &= todo - 1;
                const uint4 *src = reinterpret_cast<const uint4 *>(a.rowvec) + (row0 + r + i2) * NVEC;
                for (int x = lane; x < NVEC; x += 32) cp_async16_full(dst + (unsigned)(x - lane) * 16u, src + x);
                dst += ROWB;
            }
        }
#pragma unroll
        for (int j = 0; j < NS; ++j) {
            if (j < nstages) issue_stage(j);
            cp_async_commit();
        }

        if constexpr (!SEG && !PART) {
            if (nslots > 0) request_rowvec(row0 + r + (__ffs(nemask) - 1), rvq_next);
        }

        // ---- the stages ------------------------------------------------------------------------------------------
        {
            int s = 0;
            int ri = SEG ? 0 : (__ffs(nemask) - 1);
            unsigned staged_row = rowst_s + (unsigned)(gl * 16);   // partition step: gout of the row in progress
            int staged_left = kLeanPartStaged;                     // ... and how many more rows found room
            for (int j = 0; j < nstages; ++j) {
                cp_async_wait<NS - 1>();
                __syncwarp();   // the records of this stage were copied by other lanes; the previous weights are consumed
                // -- weights of this stage: one (position, head) pair per lane --
#pragma unroll
                for (int n = 0; n < NIT; ++n) {
                    const int it = lane + 32 * n;
                    if (ITEMS % 32 == 0 || it < ITEMS) {
                        const int p = it / H, h = it % H;
                        const unsigned pr = lds_u8(prow_s + (unsigned)(j * P + p));
                        const int i = SEG ? 0 : (int)(pr & 0x7f);
                        const unsigned rx = (unsigned)((i * H + h) * 4);
                        const float s_ = lds_f32(rc_s + rx) + lds_f32(rec_s + (unsigned)((j % NS) * L::RECB + it * 4));
                        float gr;
                        const float e = leaky(s_, a.slope, gr);
                        const float al = ex2_approx(fmaf(e, kLog2e, lds_f32(rc_s + 3 * L::RCN + rx))) * lds_f32(rc_s + 2 * L::RCN + rx);
                        float w0 = s_ > 0.f ? al : -al;   // the sign bit carries LeakyReLU' = slope
                        if (pr & 0x80) w0 = 0.f;
                        const unsigned wi = (unsigned)((((p % EPW) * H + h) * SPS + p / EPW) * 4);
                        sts_f32(w_s + wi, w0);
                    }
                }
                __syncwarp();
                const unsigned ring_a = ring_l + (unsigned)((j % NS) * STAGE);
                const int cnt = nslots - s;
                unsigned ends;
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
#pragma unroll
                for (int k = 0; k < SPS; ++k) {
                    if (k % 4 == 0) {
#pragma unroll
                        for (int v = 0; v < V; ++v) w4[v] = lds_f4(w_s + (unsigned)(((half * H + hv[v]) * SPS + k) * 4));
                    }
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        const float wk = k % 4 == 0 ? w4[v].x : k % 4 == 1 ? w4[v].y : k % 4 == 2 ? w4[v].z : w4[v].w;
                        f32x2 x[NP];
                        Pairs<T>::get(lds128(ring_a + (unsigned)(k * EPW * ROWB + v * G * 16)), x);
                        const float al = fabsf(wk);
                        const float wg = wk < 0.f ? al * a.slope : al;   // alpha * LeakyReLU'
                        sv[v] += wg;
                        const f32x2 a2 = pack2(al, al), g2 = pack2(wg, wg);
#pragma unroll
                        for (int t = 0; t < NP; ++t) {
                            if constexpr (!PART) pacc0[v][t] = fma2(a2, x[t], pacc0[v][t]);   // A is for D, given to a partition step
                            pacc1[v][t] = fma2(g2, x[t], pacc1[v][t]);
                        }
                    }
                    if (ends & (1u << k)) {
                        // ---- the row is complete -------------------------------------------------------------
                        const long long row = row0 + r + ri;
                        if constexpr (PART) {
                            if (staged_left > 0) {
#pragma unroll
                                for (int v = 0; v < V; ++v) rvq[v] = lds128(staged_row + (unsigned)(v * G * 16));
                                staged_row += ROWB;
                                --staged_left;
                            } else {   // more rows with edges in this chunk than there was room for
                                request_rowvec(row, rvq);
                            }
                        } else if constexpr (!SEG) {
#pragma unroll
                            for (int v = 0; v < V; ++v) rvq[v] = rvq_next[v];
                            const unsigned rest = nemask & ~((2u << ri) - 1u);
                            if (rest) request_rowvec(row0 + r + (__ffs(rest) - 1), rvq_next);
                        }
                        if constexpr (SEG) {
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
                                        acc1[v][e] += __shfl_xor_sync(0xffffffffu, acc1[v][e], off);
                                    }
                                }
                            if (half == 0) {
                                constexpr long long rowf = (long long)NVEC * EPV;
                                float *rec = a.sp.part + seg * a.sp.pstride;
                                bool vok[V];
#pragma unroll
                                for (int v = 0; v < V; ++v) vok[v] = true;
                                store_acc_row<G, V, EPV>(rec, gl, vok, acc1);
                                store_acc_row<G, V, EPV>(rec + rowf, gl, vok, acc0);
#pragma unroll
                                for (int v = 0; v < V; ++v)
                                    if ((gl % VPH) == 0) rec[2 * rowf + hv[v]] = sv[v];
                            }
                        } else {
                            // <gout_i, A> and <gout_i, B> on the un-folded accumulators, reduced over the lanes of each
                            // head and over the edge lanes
                            float pA[V], pB[V];
#pragma unroll
                            for (int v = 0; v < V; ++v) {
                                f32x2 rv[NP];
                                Pairs<T>::get(rvq[v], rv);
                                f32x2 qa = zero2(), qb = zero2();
#pragma unroll
                                for (int t = 0; t < NP; ++t) {
                                    if constexpr (!PART) qa = fma2(rv[t], pacc0[v][t], qa);
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
                                        if constexpr (!PART) pA[v] += __shfl_xor_sync(0xffffffffu, pA[v], off);
                                        pB[v] += __shfl_xor_sync(0xffffffffu, pB[v], off);
                                        if (off >= G) sv[v] += __shfl_xor_sync(0xffffffffu, sv[v], off);
                                    }
                                }
                            }
                            if ((gl % VPH) == 0 && half == 0) {
#pragma unroll
                                for (int v = 0; v < V; ++v) {
                                    const unsigned so = sout_s + (unsigned)((ri * H + hv[v]) * 4);
                                    if constexpr (PART) {   // del so far + this partition's share, with the D given
                                        sts_f32(so, lds_f32(so) + (pB[v] - lds_f32(so + L::RCN) * sv[v]));
                                    } else {
                                        sts_f32(so, pB[v] - pA[v] * sv[v]);   // del
                                        sts_f32(so + L::RCN, pA[v]);           // D
                                    }
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
                s += SPS;
                if (j + NS < nstages) issue_stage(j + NS);
                cp_async_commit();
            }
        chunk_done:
            cp_async_wait<0>();
        }

        // ---- the chunk's del and records, coalesced --------------------------------------------------------------------
        if constexpr (!SEG) {
            __syncwarp();
            for (int x = lane; x < nr * H; x += 32) {
                const long long o = (row0 + r) * H + x;
                if constexpr (PART) {
                    if (a.first || ((nemask >> (x / H)) & 1u)) a.del[o] = lds_f32(sout_s + 4 * x);
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

// ---- launcher ------------------------------------------------------------------------------------------------------
template <typename T, int G, int V, int H>
static sar_status launch_lean_dst(LeanArgs a, long long nnz, cudaStream_t st) {
    constexpr int NS = 2;
    constexpr int P = (G == 32 && V == 1) ? 8 : 4 * (32 / G);   // stages of 2 KB (4 KB for rows of 512 bytes and more)
    using LR = LeanDstLayout<G, V, H, false, kLeanCap, P, NS>;
    using LS = LeanDstLayout<G, V, H, true, kLeanCap, P, NS>;
    a.R = lean_rows_per_span(a.n_rows, nnz, kLeanCap);
    const long long spans = (a.n_rows + a.R - 1) / a.R;
    if (spans > 0) {
        auto kern = lean_dst_kernel<T, G, V, H, false, kLeanCap, P, NS, kLeanMinBlocksBwdRows>;
        SAR_TRY(ensure_smem(kern, LR::total));
        SAR_LAUNCH("gat_bwd_dst", st, kern<<<(unsigned)spans, 32, LR::total, st>>>(a));
        SAR_TRY(sar_after_launch());
    }
    if (a.sp.n_seg > 0) {
        auto kern = lean_dst_kernel<T, G, V, H, true, kLeanCap, P, NS, kLeanMinBlocks>;
        SAR_TRY(ensure_smem(kern, LS::total));
        SAR_LAUNCH("gat_bwd_dst_seg", st, kern<<<(unsigned)a.sp.n_seg, 32, LS::total, st>>>(a));
        SAR_TRY(sar_after_launch());
    }
    return SAR_OK;
}

// A partition step: the rows launch is the PART variant, the segments of the long rows run the whole-graph segment
// kernel (same partial records; the merge launch is the caller's and takes D as given).
template <typename T, int G, int V, int H>
static sar_status launch_lean_dst_part(LeanArgs a, long long nnz, cudaStream_t st) {
    constexpr int NS = 2;
    constexpr int P = (G == 32 && V == 1) ? 8 : 4 * (32 / G);
    using LR = LeanDstLayout<G, V, H, false, kLeanCap, P, NS, true>;
    using LS = LeanDstLayout<G, V, H, true, kLeanCap, P, NS>;
    a.R = lean_rows_per_span(a.n_rows, nnz, kLeanCap, kLeanPartRows);
    const long long spans = (a.n_rows + a.R - 1) / a.R;
    if (spans > 0) {
        auto kern = lean_dst_kernel<T, G, V, H, false, kLeanCap, P, NS, kLeanMinBlocksPart, true>;
        SAR_TRY(ensure_smem(kern, LR::total));
        SAR_LAUNCH("gat_bwd_dst", st, kern<<<(unsigned)spans, 32, LR::total, st>>>(a));
        SAR_TRY(sar_after_launch());
    }
    if (a.sp.n_seg > 0) {
        auto kern = lean_dst_kernel<T, G, V, H, true, kLeanCap, P, NS, kLeanMinBlocks>;
        SAR_TRY(ensure_smem(kern, LS::total));
        SAR_LAUNCH("gat_bwd_dst_seg", st, kern<<<(unsigned)a.sp.n_seg, 32, LS::total, st>>>(a));
        SAR_TRY(sar_after_launch());
    }
    return SAR_OK;
}

template <typename T>
static sar_status dispatch_lean_dst(const Shape &s, const LeanArgs &a, long long nnz, cudaStream_t st) {
    if (s.G == 16 && s.V == 1 && s.geom.H == 4) return launch_lean_dst<T, 16, 1, 4>(a, nnz, st);
    if (s.G == 32 && s.V == 1 && s.geom.H == 4) return launch_lean_dst<T, 32, 1, 4>(a, nnz, st);
    if (s.G == 32 && s.V == 1 && s.geom.H == 8) return launch_lean_dst<T, 32, 1, 8>(a, nnz, st);
    if (s.G == 32 && s.V == 2 && s.geom.H == 4) return launch_lean_dst<T, 32, 2, 4>(a, nnz, st);
    return SAR_ERR_UNSUPPORTED;
}

template <typename T>
static sar_status dispatch_lean_dst_part(const Shape &s, const LeanArgs &a, long long nnz, cudaStream_t st) {
    if (s.G == 16 && s.V == 1 && s.geom.H == 4) return launch_lean_dst_part<T, 16, 1, 4>(a, nnz, st);
    if (s.G == 32 && s.V == 1 && s.geom.H == 4) return launch_lean_dst_part<T, 32, 1, 4>(a, nnz, st);
    if (s.G == 32 && s.V == 1 && s.geom.H == 8) return launch_lean_dst_part<T, 32, 1, 8>(a, nnz, st);
    if (s.G == 32 && s.V == 2 && s.geom.H == 4) return launch_lean_dst_part<T, 32, 2, 4>(a, nnz, st);
    return SAR_ERR_UNSUPPORTED;
}

}  // namespace sar

#define SAR_LEAN_DST_TU(SUFFIX, TYPE)                                                                          \
    namespace sar {                                                                                            \
    sar_status lean_bwd_dst_##SUFFIX(const Shape &s, const LeanArgs &a, long long nnz, cudaStream_t st) {      \
        return dispatch_lean_dst<TYPE>(s, a, nnz, st);                                                         \
    }                                                                                                          \
    sar_status lean_bwd_dst_part_##SUFFIX(const Shape &s, const LeanArgs &a, long long nnz, cudaStream_t st) { \
        return dispatch_lean_dst_part<TYPE>(s, a, nnz, st);                                                    \
    }                                                                                                          \
    }

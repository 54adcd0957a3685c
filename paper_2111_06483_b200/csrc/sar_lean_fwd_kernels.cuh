// Lean span kernel of the whole-graph forward pass (internal): out_i = sum_j alpha_ij feat_j with the edge softmax
// alpha of Eq. 3 over the CSR, and the row statistics (m, d) that the backward pass rebuilds alpha from.
//
// Same plan as lean_dst_kernel (sar_lean_dst_kernels.cuh): stage-granular cp.async ring of the gathered feature rows,
// the score terms er[col, :] of a stage's positions travelling with the stage, the weights of a stage computed just
// before it is consumed, one (position, head) pair per lane.
// Softmax shift: a row's weights are exp(e - c) with c the score of the row's FIRST edge (fetched while the chunk's
// first stages are in flight), not the row max: the result does not depend on the shift, nothing has to be known about
// later stages, no lane waits for a max, and a row's arithmetic does not depend on where the stage boundaries fall.
// The exact max m (the statistic the backward pass rebuilds alpha from) is collected on the side over raw er - since
// max_j LeakyReLU(el + er_j) = LeakyReLU(el + max_j er_j) for slope >= 0 - by fire-and-forget shared-memory
// reductions (rows launch) or in a register per lane (segments), and d is brought to it at the end: d = d_c exp(c - m).
// Should a score exceed its row's shift by more than kLeanMaxLead, the stage takes a slow path first: the shift of that
// (row, head) moves up to the stage's max and the accumulators follow by exp(c_before - c_now) (the running-max
// correction of Sec. 3.4 applied inside a row), so nothing can overflow.
// Preconditions as for lean_dst_kernel (checked by the host).
//
// PART = true is one PARTITION STEP of Algorithm 1 that leaves the state behind (the last step does so too; the division
// that ends the algorithm is then a launch of its own): the call holds the edges
// from one source partition, and a row's sums are folded into the state the earlier partitions left - the running
// max m, the denominator d and the float32 numerator, all against m - with the running-max correction of Sec. 3.4:
// m' = max(m, m_k), numerator' = numerator exp(m - m') + numerator_k exp(c - m'), d likewise (c the shift the
// partition's sums were taken against).  Laid out like the partition step of lean_dst_kernel: spans of up to
// kLeanPartRows rows, rows without edges cost nothing and keep their state untouched, the numerator rows of the chunk's
// first kLeanPartStagedFwd rows that have edges are copied into shared memory with the chunk's first stage (the rows
// beyond that load theirs when they complete).  In the first step (`first`) there is no state to read, a row with edges
// leaves its sums against its own max, and a row without edges gets the empty state (m = -inf, d = 0, numerator 0):
// FIRST = true.  Which partitions get these variants: kLeanPartMaxDegree, kLeanPartMinDenseDegree (sar_lean.cuh).
#pragma once

#include "sar_lean_dst_kernels.cuh"

namespace sar {

template <int G, int V, int H, bool SEG, int CAP, int P, int NS, bool PART = false, int EPV = 4>
struct LeanFwdLayout {
    static constexpr int EPW = 32 / G;
    static constexpr int ROWB = G * V * 16;
    static constexpr int SROWB = G * V * EPV * 4;                 // a row of the float32 numerator
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
    static constexpr int rc = prow + POSMAX;                      // el; key of the max of er; shift c; scratch of the slow path
    static constexpr int sout = rc + 4 * RCN;                     // d against the shift
    static constexpr int srb = sout + RCN;
    static constexpr int sso = srb + ((MAXR + 1) * 4 + 15) / 16 * 16;
    static constexpr int endm = sso + ((MAXR + 1) * 4 + 15) / 16 * 16;
    static constexpr int stm = endm + ((MASKW * 4 + 15) / 16) * 16;  // partition step: m and d of the state, in and out
    static constexpr int rowst = stm + ((PART && !SEG) ? 2 * RCN : 0); // partition step: numerator rows of the rows with edges
    static constexpr int total = rowst + ((PART && !SEG) ? kLeanPartStagedFwd * SROWB : 0);
};

template <typename T, int G, int V, int H, bool SEG, int CAP, int P, int NS, int MINB, bool PART = false, bool FIRST = false>
__global__ void __launch_bounds__(32, MINB) lean_fwd_kernel(const LeanArgs a) {
    static_assert(!(PART && SEG), "the segments of a partition step run the whole-graph segment kernel");
    static_assert(PART || !FIRST, "FIRST is the first partition step");
    using L = LeanFwdLayout<G, V, H, SEG, CAP, P, NS, PART, Elem<T>::EPV>;
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
    static_assert(ITEMS <= 64 && 32 % H == 0, "at most two (position, head) pairs per lane, both of one head");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const unsigned sbase = (unsigned)__cvta_generic_to_shared(smem_raw);
    const unsigned ring_s = sbase + L::ring, rec_s = sbase + L::rec, w_s = sbase + L::w, offs_s = sbase + L::offs;
    const unsigned prow_s = sbase + L::prow, rc_s = sbase + L::rc, sout_s = sbase + L::sout, endm_s = sbase + L::endm;
    const unsigned key_s = rc_s + L::RCN, cref_s = rc_s + 2 * L::RCN, ftab_s = rc_s + 3 * L::RCN;
    const unsigned stm_s = sbase + L::stm, std_s = stm_s + L::RCN, rowst_s = sbase + L::rowst;
    int *srb = reinterpret_cast<int *>(smem_raw + L::srb);
    constexpr float kLeanMaxLead = 60.f;   // a score may exceed its row's shift by this much before the shift moves
    int *sso = reinterpret_cast<int *>(smem_raw + L::sso);
    unsigned *skey = reinterpret_cast<unsigned *>(smem_raw + L::rc + L::RCN);

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
    // the (position, head) pairs this lane scores: it = lane (+ 32), all of head lane % H
    constexpr int NIT = (ITEMS + 31) / 32;
    const int hl = lane % H;

    f32x2 pacc0[V][NP];
    float sv[V];
#pragma unroll
    for (int v = 0; v < V; ++v) {
        sv[v] = 0.f;
#pragma unroll
        for (int k = 0; k < NP; ++k) pacc0[v][k] = zero2();
    }

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
        }
        __syncwarp();

        // ---- the ring: the gathered rows of a stage and the score terms of its positions, one commit group per
        // stage ---------------------------------------------------------------------------------------------------
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
        if constexpr (PART) {   // the numerator rows of the first rows with edges, in their order, with the first stage
            unsigned todo = FIRST ? 0u : nemask;
            unsigned dst = rowst_s + (unsigned)lane * 16u;
            for (int ci = 0; todo && ci < kLeanPartStagedFwd; ++ci) {
                const int i2 = __ffs(todo) - 1;
                todo &= todo - 1;
                const uint4 *src = reinterpret_cast<const uint4 *>(a.acc_state) + (row0 + r + i2) * (L::SROWB / 16);
                for (int x = lane; x < L::SROWB / 16; x += 32) cp_async16_full(dst + (unsigned)(x - lane) * 16u, src + x);
                dst += L::SROWB;
            }
        }
#pragma unroll
        for (int j = 0; j < NS; ++j) {
            if (j < nstages) issue_stage(j);
            cp_async_commit();
        }

        // per (row, head): el, the shift c = score of the row's first edge, the key of the max (the loads fly with the
        // first stages)
        if constexpr (PART) {
            // rows with edges only, every load issued before the first store; and the state's m and d
            constexpr int NX = (L::MAXR * H + 31) / 32;
            float cv[NX][4];
#pragma unroll
            for (int n = 0; n < NX; ++n) {
                const int x = lane + 32 * n;
                cv[n][0] = 0.f;
                cv[n][1] = cv[n][2] = SAR_NEG_INF;
                cv[n][3] = 0.f;
                if (x < nr * H && ((nemask >> (x / H)) & 1u)) {
                    const long long o = (row0 + r) * H + x;
                    const unsigned col = lds_u32(offs_s + 4 * (unsigned)perm(sso[x / H] * EPW)) >> LGNVEC;
                    cv[n][0] = __ldg(a.el + o);
                    cv[n][1] = __ldg(a.er + (size_t)col * H + (x % H));
                    if constexpr (!FIRST) {
                        cv[n][2] = a.m_out[o];   // plain loads: this launch rewrites the state
                        cv[n][3] = a.d_out[o];
                    }
                }
            }
#pragma unroll
            for (int n = 0; n < NX; ++n) {
                const int x = lane + 32 * n;
                if (x < nr * H) {
                    float gr;
                    sts_f32(rc_s + 4 * x, cv[n][0]);
                    skey[x] = kKeyNegInf;
                    sts_f32(cref_s + 4 * x, ((nemask >> (x / H)) & 1u) ? leaky(cv[n][0] + cv[n][1], a.slope, gr) : SAR_NEG_INF);
                    sts_f32(sout_s + 4 * x, 0.f);
                    sts_f32(stm_s + 4 * x, cv[n][2]);
                    sts_f32(std_s + 4 * x, cv[n][3]);
                }
            }
        } else
        for (int x = lane; x < nr * H; x += 32) {
            const int i = x / H;
            const float el_ = __ldg(a.el + (row0 + r) * H + x);
            float c_ = SAR_NEG_INF;
            if ((nemask >> i) & 1u) {
                const unsigned col = lds_u32(offs_s + 4 * (unsigned)perm(sso[i] * EPW)) >> LGNVEC;
                float gr;
                c_ = leaky(el_ + __ldg(a.er + (size_t)col * H + (x % H)), a.slope, gr);
            }
            sts_f32(rc_s + 4 * x, el_);
            skey[x] = kKeyNegInf;
            sts_f32(cref_s + 4 * x, c_);
            sts_f32(sout_s + 4 * x, 0.f);
        }
        __syncwarp();

        // rows without edges: their vector outputs are zeros (the scalars leave with the others at the chunk's end);
        // in a partition step they keep their state, or get the empty one in the first step
        if constexpr (PART) {
            if constexpr (FIRST) {
                unsigned em = ~nemask & ((1u << nr) - 1u);
                while (em) {
                    const int i = __ffs(em) - 1;
                    em &= em - 1;
                    uint4 *rp = reinterpret_cast<uint4 *>(a.acc_state) + (row0 + r + i) * (L::SROWB / 16);
                    for (int x = lane; x < L::SROWB / 16; x += 32) rp[x] = make_uint4(0u, 0u, 0u, 0u);
                }
            }
        }
        if constexpr (!SEG && !PART) {
            unsigned em = ~nemask & ((1u << nr) - 1u);
            while (em) {
                const int i = __ffs(em) - 1;
                em &= em - 1;
                uint4 *rp = reinterpret_cast<uint4 *>(a.out) + (row0 + r + i) * NVEC;
                for (int x = lane; x < NVEC; x += 32) rp[x] = make_uint4(0u, 0u, 0u, 0u);
            }
        }

        // ---- the stages ------------------------------------------------------------------------------------------
        {
            int s = 0;
            int ri = SEG ? 0 : (__ffs(nemask) - 1);
            unsigned staged_row = rowst_s + (unsigned)(gl * EPV * 4);   // partition step: numerator of the row in progress
            int staged_left = kLeanPartStagedFwd;                       // ... and how many more rows found room
            float mrun = SAR_NEG_INF;               // segment: max of er[., lane % H] over the stages so far
            float el_seg = 0.f;
            if constexpr (SEG) el_seg = lds_f32(rc_s + 4 * (unsigned)hl);
            for (int j = 0; j < nstages; ++j) {
                cp_async_wait<NS - 1>();
                __syncwarp();   // the score terms of this stage were copied by other lanes; the previous weights are consumed
                // -- weights of this stage: one (position, head) pair per lane, against the shift of the pair's row --
                float erv[NIT], w0[NIT];
                unsigned prv[NIT], rx[NIT];
#pragma unroll
                for (int n = 0; n < NIT; ++n) {
                    const int it = lane + 32 * n;
                    erv[n] = SAR_NEG_INF;
                    prv[n] = 0x80u;
                    if (ITEMS % 32 == 0 || it < ITEMS) {
                        prv[n] = lds_u8(prow_s + (unsigned)(j * P + it / H));
                        erv[n] = lds_f32(rec_s + (unsigned)((j % NS) * L::RECB + it * 4));
                    }
                    rx[n] = (unsigned)((((SEG ? 0u : (prv[n] & 0x7fu)) * H) + hl) * 4);
                }
                // the exact max, on the side
                if constexpr (SEG) {
                    float vmax = SAR_NEG_INF;
#pragma unroll
                    for (int n = 0; n < NIT; ++n) vmax = fmaxf(vmax, (prv[n] & 0x80u) ? SAR_NEG_INF : erv[n]);
#pragma unroll
                    for (int off = H; off < 32; off <<= 1) vmax = fmaxf(vmax, __shfl_xor_sync(0xffffffffu, vmax, off));
                    mrun = fmaxf(mrun, vmax);
                } else {
#pragma unroll
                    for (int n = 0; n < NIT; ++n)
                        if (!(prv[n] & 0x80u)) red_max_u32(key_s + rx[n], fkey(erv[n]));
                }
                for (;;) {
                    bool over = false;
#pragma unroll
                    for (int n = 0; n < NIT; ++n) {
                        float gr;
                        const float dx = leaky(lds_f32(rc_s + rx[n]) + erv[n], a.slope, gr) - lds_f32(cref_s + rx[n]);
                        const bool pad = (prv[n] & 0x80u) != 0u;
                        over = over || (!pad && dx > kLeanMaxLead);
                        w0[n] = pad ? 0.f : ex2_approx(dx * kLog2e);
                    }
                    if (!__any_sync(0xffffffffu, over)) break;
                    // slow path: the shift of every (row, head) some score of this stage leads by more than kLeanMaxLead
                    // moves up to the stage's largest score of that pair; the accumulators of the row in progress follow
                    for (int x = lane; x < L::MAXR * H; x += 32) sts_u32(ftab_s + 4 * x, fkey(lds_f32(cref_s + 4 * x)));
                    __syncwarp();
#pragma unroll
                    for (int n = 0; n < NIT; ++n) {
                        if (!(prv[n] & 0x80u)) {
                            float gr;
                            red_max_u32(ftab_s + rx[n], fkey(leaky(lds_f32(rc_s + rx[n]) + erv[n], a.slope, gr)));
                        }
                    }
                    __syncwarp();
                    for (int x = lane; x < L::MAXR * H; x += 32) {
                        const float cn = fkey_inv(lds_u32(ftab_s + 4 * x)), co = lds_f32(cref_s + 4 * x);
                        const bool moved = cn - co > kLeanMaxLead;
                        sts_f32(ftab_s + 4 * x, moved ? ex2_approx((co - cn) * kLog2e) : 1.f);
                        if (moved) sts_f32(cref_s + 4 * x, cn);
                    }
                    __syncwarp();
                    {
                        const int rcur = ri < L::MAXR ? ri : 0;
#pragma unroll
                        for (int v = 0; v < V; ++v) {
                            const float sc = lds_f32(ftab_s + (unsigned)((rcur * H + hv[v]) * 4));
                            sv[v] *= sc;
                            const f32x2 s2 = pack2(sc, sc);
#pragma unroll
                            for (int t = 0; t < NP; ++t) pacc0[v][t] = fma2(pacc0[v][t], s2, zero2());
                        }
                    }
                    __syncwarp();
                }
#pragma unroll
                for (int n = 0; n < NIT; ++n) {
                    const int it = lane + 32 * n;
                    if (ITEMS % 32 == 0 || it < ITEMS) {
                        const int p = it / H;
                        sts_f32(w_s + (unsigned)((((p % EPW) * H + hl) * SPS + p / EPW) * 4), w0[n]);
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
                        sv[v] += wk;
                        const f32x2 w2 = pack2(wk, wk);
#pragma unroll
                        for (int t = 0; t < NP; ++t) pacc0[v][t] = fma2(w2, x[t], pacc0[v][t]);
                    }
                    if (ends & (1u << k)) {
                        // ---- the row is complete -------------------------------------------------------------
                        const long long row = row0 + r + ri;
                        if constexpr (SEG) {
                            // partial accumulators of the segment, float32, against its own max, for the merge launch
                            constexpr long long rowf = (long long)NVEC * EPV;
                            float *rec = a.sp.part + seg * a.sp.pstride;
                            if (lane < H) {
                                float gr;
                                const float mm = leaky(el_seg + mrun, a.slope, gr);
                                rec[rowf + lane] = mm;
                                sts_f32(ftab_s + 4 * lane, ex2_approx((lds_f32(cref_s + 4 * lane) - mm) * kLog2e));
                            }
                            __syncwarp();
                            float acc0[V][EPV];
#pragma unroll
                            for (int v = 0; v < V; ++v) {
                                const float sc = lds_f32(ftab_s + 4 * (unsigned)hv[v]);
                                sv[v] *= sc;
#pragma unroll
                                for (int t = 0; t < NP; ++t) {
                                    unpack2(pacc0[v][t], acc0[v][2 * t], acc0[v][2 * t + 1]);
                                    acc0[v][2 * t] *= sc;
                                    acc0[v][2 * t + 1] *= sc;
                                }
                            }
#pragma unroll
                            for (int off = G; off < 32; off <<= 1)
#pragma unroll
                                for (int v = 0; v < V; ++v) {
                                    sv[v] += __shfl_xor_sync(0xffffffffu, sv[v], off);
#pragma unroll
                                    for (int e = 0; e < EPV; ++e) acc0[v][e] += __shfl_xor_sync(0xffffffffu, acc0[v][e], off);
                                }
                            if (half == 0) {
                                bool vok[V];
#pragma unroll
                                for (int v = 0; v < V; ++v) vok[v] = true;
                                store_acc_row<G, V, EPV>(rec, gl, vok, acc0);
#pragma unroll
                                for (int v = 0; v < V; ++v)
                                    if ((gl % VPH) == 0) rec[rowf + H + hv[v]] = sv[v];
                            }
                        } else {
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
                            if constexpr (PART) {
                                // fold into the state: m' = max(m, m_k); what was there scales by exp(m - m'), this
                                // partition's sums (taken against the shift c) by exp(c - m')
                                float mn[V], dn[V];
                                float *sp_ = a.acc_state + row * (long long)(NVEC * EPV);
#pragma unroll
                                for (int v = 0; v < V; ++v) {
                                    const unsigned rx = (unsigned)((ri * H + hv[v]) * 4);
                                    float gr;
                                    const float mk = leaky(lds_f32(rc_s + rx) + fkey_inv(lds_u32(key_s + rx)), a.slope, gr);
                                    const float mo = lds_f32(stm_s + rx);
                                    mn[v] = fmaxf(mo, mk);
                                    const float fo = ex2_approx((mo - mn[v]) * kLog2e);
                                    const float fn = ex2_approx((lds_f32(cref_s + rx) - mn[v]) * kLog2e);
                                    dn[v] = lds_f32(std_s + rx) * fo + sv[v] * fn;
                                    if (half == 0) {
                                        const f32x2 fo2 = pack2(fo, fo), fn2 = pack2(fn, fn);
                                        const unsigned so = staged_row + (unsigned)(v * G * EPV * 4);
#pragma unroll
                                        for (int q = 0; q < EPV / 4; ++q) {
                                            // (more rows with edges in this chunk than there was room for: from memory)
                                            const float4 old = FIRST ? make_float4(0.f, 0.f, 0.f, 0.f)
                                                               : staged_left > 0 ? lds_f4(so + 16 * q)
                                                                                 : reinterpret_cast<const float4 *>(sp_ + (v * G + gl) * EPV)[q];
                                            const f32x2 lo = fma2(pack2(old.x, old.y), fo2, fma2(pacc0[v][2 * q], fn2, zero2()));
                                            const f32x2 hi = fma2(pack2(old.z, old.w), fo2, fma2(pacc0[v][2 * q + 1], fn2, zero2()));
                                            reinterpret_cast<float4 *>(sp_ + (v * G + gl) * EPV)[q] = make_float4(lo.x, lo.y, hi.x, hi.y);
                                        }
                                    }
                                }
                                __syncwarp();   // every lane has read the state's m and d of this row
                                if (half == 0) {
#pragma unroll
                                    for (int v = 0; v < V; ++v)
                                        if ((gl % VPH) == 0) {
                                            const unsigned rx = (unsigned)((ri * H + hv[v]) * 4);
                                            sts_f32(std_s + rx, dn[v]);
                                            sts_f32(stm_s + rx, mn[v]);
                                        }
                                }
                                staged_row += L::SROWB;
                                --staged_left;
                            } else
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
                                    if (a.relu) {
#pragma unroll
                                        for (int e = 0; e < EPV; ++e) acc0[e] = fmaxf(acc0[e], 0.f);
                                    }
                                    rp[v * G] = Elem<T>::pack(acc0);
                                    if ((gl % VPH) == 0) sts_f32(sout_s + (unsigned)((ri * H + hv[v]) * 4), sv[v]);
                                }
                            }
                        }
#pragma unroll
                        for (int v = 0; v < V; ++v) {
                            sv[v] = 0.f;
#pragma unroll
                            for (int t = 0; t < NP; ++t) pacc0[v][t] = zero2();
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

        // ---- the chunk's row statistics, coalesced: m = LeakyReLU(el + max er), exactly the max of the row's scores ----
        if constexpr (!SEG) {
            __syncwarp();
            if constexpr (PART) {
                for (int x = lane; x < nr * H; x += 32) {
                    if (FIRST || ((nemask >> (x / H)) & 1u)) {
                        const long long o = (row0 + r) * H + x;
                        a.m_out[o] = lds_f32(stm_s + 4 * x);
                        a.d_out[o] = lds_f32(std_s + 4 * x);
                    }
                }
            } else
            for (int x = lane; x < nr * H; x += 32) {
                const long long o = (row0 + r) * H + x;
                const unsigned k = skey[x];
                float mm = SAR_NEG_INF;
                if (k != kKeyNegInf) {
                    float gr;
                    mm = leaky(lds_f32(rc_s + 4 * x) + fkey_inv(k), a.slope, gr);
                }
                a.m_out[o] = mm;
                a.d_out[o] = k != kKeyNegInf ? lds_f32(sout_s + 4 * x) * ex2_approx((lds_f32(cref_s + 4 * x) - mm) * kLog2e) : 0.f;
            }
            __syncwarp();
        }
        r = r2;
    }
}

// ---- launcher ------------------------------------------------------------------------------------------------------
template <typename T, int G, int V, int H>
static sar_status launch_lean_fwd(LeanArgs a, long long nnz, cudaStream_t st) {
    constexpr int NS = 2;
    constexpr int P = (G == 32 && V == 1) ? 8 : 4 * (32 / G);   // stages of 2 KB (4 KB for rows of 512 bytes and more)
    using LR = LeanFwdLayout<G, V, H, false, kLeanCap, P, NS>;
    using LS = LeanFwdLayout<G, V, H, true, kLeanCap, P, NS>;
    a.R = lean_rows_per_span(a.n_rows, nnz, kLeanCap);
    const long long spans = (a.n_rows + a.R - 1) / a.R;
    if (spans > 0) {
        auto kern = lean_fwd_kernel<T, G, V, H, false, kLeanCap, P, NS, kLeanMinBlocks>;
        SAR_TRY(ensure_smem(kern, LR::total));
        SAR_LAUNCH("gat_fwd", st, kern<<<(unsigned)spans, 32, LR::total, st>>>(a));
        SAR_TRY(sar_after_launch());
    }
    if (a.sp.n_seg > 0) {
        auto kern = lean_fwd_kernel<T, G, V, H, true, kLeanCap, P, NS, kLeanMinBlocks>;
        SAR_TRY(ensure_smem(kern, LS::total));
        SAR_LAUNCH("gat_fwd_seg", st, kern<<<(unsigned)a.sp.n_seg, 32, LS::total, st>>>(a));
        SAR_TRY(sar_after_launch());
    }
    return SAR_OK;
}

// A partition step of a call-by-call forward pass: the rows launch is the PART variant, the segments of the long
// rows run the whole-graph segment kernel (same partial records; the merge launch is the caller's and folds the state).
template <typename T, int G, int V, int H>
static sar_status launch_lean_fwd_part(LeanArgs a, long long nnz, cudaStream_t st) {
    constexpr int NS = 2;
    constexpr int P = (G == 32 && V == 1) ? 8 : 4 * (32 / G);
    using LR = LeanFwdLayout<G, V, H, false, kLeanCap, P, NS, true, Elem<T>::EPV>;
    using LS = LeanFwdLayout<G, V, H, true, kLeanCap, P, NS>;
    a.R = lean_rows_per_span(a.n_rows, nnz, kLeanCap, kLeanPartRows);
    const long long spans = (a.n_rows + a.R - 1) / a.R;
    if (spans > 0) {
        auto kern = a.first ? lean_fwd_kernel<T, G, V, H, false, kLeanCap, P, NS, kLeanMinBlocksPart, true, true>
                            : lean_fwd_kernel<T, G, V, H, false, kLeanCap, P, NS, kLeanMinBlocksPart, true, false>;
        SAR_TRY(ensure_smem(lean_fwd_kernel<T, G, V, H, false, kLeanCap, P, NS, kLeanMinBlocksPart, true, true>, LR::total));
        SAR_TRY(ensure_smem(lean_fwd_kernel<T, G, V, H, false, kLeanCap, P, NS, kLeanMinBlocksPart, true, false>, LR::total));
        SAR_LAUNCH("gat_fwd", st, kern<<<(unsigned)spans, 32, LR::total, st>>>(a));
        SAR_TRY(sar_after_launch());
    }
    if (a.sp.n_seg > 0) {
        auto kern = lean_fwd_kernel<T, G, V, H, true, kLeanCap, P, NS, kLeanMinBlocks>;
        SAR_TRY(ensure_smem(kern, LS::total));
        SAR_LAUNCH("gat_fwd_seg", st, kern<<<(unsigned)a.sp.n_seg, 32, LS::total, st>>>(a));
        SAR_TRY(sar_after_launch());
    }
    return SAR_OK;
}

template <typename T>
static sar_status dispatch_lean_fwd_part(const Shape &s, const LeanArgs &a, long long nnz, cudaStream_t st) {
    if (s.G == 16 && s.V == 1 && s.geom.H == 4) return launch_lean_fwd_part<T, 16, 1, 4>(a, nnz, st);
    if (s.G == 32 && s.V == 1 && s.geom.H == 4) return launch_lean_fwd_part<T, 32, 1, 4>(a, nnz, st);
    if (s.G == 32 && s.V == 1 && s.geom.H == 8) return launch_lean_fwd_part<T, 32, 1, 8>(a, nnz, st);
    if (s.G == 32 && s.V == 2 && s.geom.H == 4) return launch_lean_fwd_part<T, 32, 2, 4>(a, nnz, st);
    return SAR_ERR_UNSUPPORTED;
}

template <typename T>
static sar_status dispatch_lean_fwd(const Shape &s, const LeanArgs &a, long long nnz, cudaStream_t st) {
    if (s.G == 16 && s.V == 1 && s.geom.H == 4) return launch_lean_fwd<T, 16, 1, 4>(a, nnz, st);
    if (s.G == 32 && s.V == 1 && s.geom.H == 4) return launch_lean_fwd<T, 32, 1, 4>(a, nnz, st);
    if (s.G == 32 && s.V == 1 && s.geom.H == 8) return launch_lean_fwd<T, 32, 1, 8>(a, nnz, st);
    if (s.G == 32 && s.V == 2 && s.geom.H == 4) return launch_lean_fwd<T, 32, 2, 4>(a, nnz, st);
    return SAR_ERR_UNSUPPORTED;
}

}  // namespace sar

#define SAR_LEAN_FWD_TU(SUFFIX, TYPE)                                                                      \
    namespace sar {                                                                                        \
    sar_status lean_fwd_##SUFFIX(const Shape &s, const LeanArgs &a, long long nnz, cudaStream_t st) {      \
        return dispatch_lean_fwd<TYPE>(s, a, nnz, st);                                                     \
    }                                                                                                      \
    sar_status lean_fwd_part_##SUFFIX(const Shape &s, const LeanArgs &a, long long nnz, cudaStream_t st) { \
        return dispatch_lean_fwd_part<TYPE>(s, a, nnz, st);                                                \
    }                                                                                                      \
    }

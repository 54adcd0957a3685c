// Span kernels of libsar (internal): forward, both backward passes and the sum aggregation.
//
// A WARP owns a SPAN of R consecutive rows of the traversal (destinations for the CSR passes,
// sources for the CSC pass).  Rows are short on average (a power-law graph's median degree is a
// handful of edges), so walking them one by one leaves a chain of dependent loads per row
// (indptr -> indices -> scores -> feature rows) and almost nothing in flight.  Instead the warp
//   1. cuts the span into CHUNKS of whole rows holding at most CAP edges (a row longer than CAP is
//      taken alone, CAP edges at a time, its accumulators staying in registers in between);
//   2. stages the chunk in shared memory, SLOT-major: a slot is 32/G consecutive edges of one row
//      (G lanes x 16 bytes cover one feature row), rows are padded to whole slots.  Column ids are
//      loaded coalesced; the score phase computes one weight record per (edge, head) - spread evenly
//      over the 32 lanes whatever the row lengths, one exponential per pair, many independent
//      gathers of er / destination records in flight;
//   3. streams the chunk's feature rows through a ring of S stages in shared memory filled by
//      cp.async (16 bytes per lane, bypassing L1): the copies of slot s+S are issued when slot s has
//      been accumulated, so S x 512 bytes per warp are in flight without holding registers, and no
//      load of this phase depends on another load.  A row is finalised when its last slot has been
//      consumed: the 32/G edge lanes are folded with shuffles and one of them writes the result.
// Nothing per edge is written to global memory.  No floating-point atomics: every output element
// has one writer (the per-(row, head) max of the forward pass is a shared-memory atomicMax on an
// order-preserving integer key, whose result does not depend on the order).
// Rows above the plan's threshold are skipped here and processed as independent segments by a second
// launch (mode 1) that writes partial accumulators; the merge kernels of sar_gat_kernels.cuh fold them.
#pragma once

#include "sar_rowkernels.cuh"

namespace sar {

constexpr int kSpanWarps = 1;             // warps per block
constexpr int kSpanThreads = kSpanWarps * 32;
constexpr int kMaxSpanRows = 16;          // rows per span

struct SpanArgs {
    long long n_rows;
    const int64_t *indptr;
    const int32_t *indices;
    const void *gather;      // rows fetched per edge: feat (forward, bwd-dst, sum) or gout (bwd-src)
    const void *rowvec;      // row-stationary vector: gout (bwd-dst) or feat (bwd-src)
    const float *el, *er;    // forward / bwd-dst: el[row], er[col];  bwd-src: er[row]
    const float *m, *d;      // bwd-dst: final statistics of the row
    const float4 *rec_in;    // bwd-src: {el, m, 1/d, D} of the column; bwd-dst GIVEN_D: of the row
    float4 *rec_out;         // bwd-dst (D rebuilt): record written per row
    float *acc_state;        // forward: running numerator [n_rows, H*F] or null
    float *m_state, *d_state;
    void *out;               // forward: out; bwd-src: dfeat; sum: out
    float *del, *der;
    const int64_t *deg_total;
    const float *src_scale, *dst_scale;  // weighted sum (kSumW): per-source factor, per-row factor (either may be null)
    float slope;
    unsigned flags;
    RowGeom g;
    SplitArgs sp;
    int mode;                // 0: spans of R rows; 1: one long-row segment per warp
    int R;                   // rows per span (<= kMaxSpanRows)
    int hvec;                // heads are scored four at a time (H % 4 == 0 and er is 16-byte aligned)
    int stage_rows;          // mode 0: rows whose own data is staged in shared memory per chunk (R, or 0: none)
};

// order-preserving float -> unsigned key (for shared-memory atomicMax)
__device__ __forceinline__ unsigned fkey(float x) {
    const unsigned b = __float_as_uint(x);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float fkey_inv(unsigned k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
constexpr unsigned kKeyNegInf = 0x007fffffu;  // fkey(-inf)

// 16-byte asynchronous copy global -> shared that bypasses L1; src_bytes = 0 writes zeros.
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc, int src_bytes) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gsrc), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

// shared-memory accesses through 32-bit shared-window addresses (no 64-bit pointer arithmetic)
__device__ __forceinline__ uint4 lds128(unsigned addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ float lds_f32(unsigned addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ float2 lds_f32x2(unsigned addr) {
    float2 v;
    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];\n" : "=f"(v.x), "=f"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ int lds_s32(unsigned addr) {
    int v;
    asm volatile("ld.shared.s32 %0, [%1];\n" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void cp_async16_s(unsigned smem_addr, const void *gsrc, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(smem_addr), "l"(gsrc), "r"(src_bytes) : "memory");
}

// packed pairs of float32 (Blackwell's two-wide FP32 pipe: one instruction, two fused multiply-adds)
typedef float2 f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) { return make_float2(lo, hi); }
__device__ __forceinline__ void unpack2(f32x2 p, float &lo, float &hi) {
    lo = p.x;
    hi = p.y;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) { return __ffma2_rn(a, b, c); }  // a*b + c, element-wise
__device__ __forceinline__ f32x2 zero2() { return make_float2(0.f, 0.f); }
// 16 bytes of storage type T -> EPV/2 packed float32 pairs
template <typename T>
struct Pairs;
template <>
struct Pairs<float> {
    __device__ __forceinline__ static void get(const uint4 &d, f32x2 (&p)[2]) {
        p[0] = pack2(__uint_as_float(d.x), __uint_as_float(d.y));
        p[1] = pack2(__uint_as_float(d.z), __uint_as_float(d.w));
    }
};
template <>
struct Pairs<__nv_bfloat16> {
    __device__ __forceinline__ static void get(const uint4 &d, f32x2 (&p)[4]) {
        p[0] = pack2(__uint_as_float(d.x << 16), __uint_as_float(d.x & 0xffff0000u));
        p[1] = pack2(__uint_as_float(d.y << 16), __uint_as_float(d.y & 0xffff0000u));
        p[2] = pack2(__uint_as_float(d.z << 16), __uint_as_float(d.z & 0xffff0000u));
        p[3] = pack2(__uint_as_float(d.w << 16), __uint_as_float(d.w & 0xffff0000u));
    }
};

// Shared-memory layout of one warp (byte offsets).
struct SpanSmem {
    size_t stage, sj, w, rowc, srb, sso, mrun, fac, scratch, rowst, total;
};
constexpr int kSpanPlanes = 5;            // planes of per-(row, head) constants
__host__ __device__ inline size_t span_align16(size_t x) { return (x + 15) & ~(size_t)15; }
template <int MODE>
__host__ __device__ inline SpanSmem span_layout(int Hp, int V, int cap, int stages, int epw, size_t row_stage_bytes = 0) {
    const size_t wbytes = MODE == kSum ? 0 : sizeof(typename WeightOf<MODE>::type);
    const size_t pos = (size_t)cap + (size_t)kMaxSpanRows * (epw - 1) + (size_t)stages * epw;  // padded positions
    SpanSmem L;
    size_t o = 0;
    L.stage = o;   o += (size_t)stages * V * 512;                // ring of gathered slots
    L.sj = o;      o += span_align16(pos * 4);                   // column id per padded position (-1: padding)
    L.w = o;       o += span_align16(pos * Hp * wbytes);         // weight record per (position, head)
    L.rowc = o;    o += span_align16((size_t)kMaxSpanRows * Hp * 4) * kSpanPlanes;  // planes of per-(row, head) constants
    L.srb = o;     o += (size_t)(kMaxSpanRows + 1) * 4;          // local first edge of each row
    L.sso = o;     o += (size_t)(kMaxSpanRows + 1) * 4;          // first slot of each row
    L.mrun = o;    o += (size_t)Hp * 4;                          // running max of a continued row
    L.fac = o;     o += (size_t)Hp * 4;                          // its rescale factors
    o = span_align16(o);
    L.scratch = o; o += (size_t)(64 * V + 32) * 4;               // epilogue scratch
    o = span_align16(o);
    L.rowst = o;   o += row_stage_bytes;                         // the staged rows' own data (partition steps)
    L.total = span_align16(o);
    return L;
}

// STATIC decides the launch mode at compile time, so that the flag tests of the row epilogue fold away:
// 1 = rows (mode 0) of a partition that holds all sources (SAR_FIRST | SAR_LAST), the benchmarked configuration;
// 2 = long-row segments (mode 1); 0 = whatever SpanArgs says.
// GEO = 1 fixes the row geometry at compile time as well: rows of exactly G*V vectors and, for the attention modes,
// 4 heads scored four at a time (SpanArgs::hvec set; the paper's GAT: 4 heads, hidden size 128), for the sums one
// head, so that head arithmetic becomes shifts and the lane predicates vanish.
template <typename T, int G, int V, int S, int MODE, int CAP, int MINB, int STATIC = 0, int GEO = 0>
__global__ void __launch_bounds__(kSpanThreads, MINB) span_kernel(const SpanArgs a) {
    constexpr int EPV = Elem<T>::EPV;
    constexpr int EPW = 32 / G;  // edges per slot
    const int mode_ = STATIC == 1 ? 0 : (STATIC == 2 ? 1 : a.mode);
    const unsigned flags_ = STATIC == 1 ? ((unsigned)(SAR_FIRST | SAR_LAST) | (a.flags & (unsigned)SAR_MEAN)) : a.flags;
    using W = typename WeightOf<MODE>::type;
    constexpr bool kFwdMode = MODE == kFwd;
    constexpr bool kDst = MODE == kBwdDst || MODE == kBwdDstGivenD;
    constexpr bool kSrc = MODE == kBwdSrc;
    constexpr bool kAcc0 = MODE != kBwdDstGivenD;                  // accumulator 0 live
    constexpr bool kAcc1 = kDst || kSrc;                           // accumulator 1 live
    extern __shared__ __align__(16) unsigned char smem_raw[];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gl = lane & (G - 1), half = lane / G;
    constexpr int kGeoH = (MODE == kSum || MODE == kSumW) ? 1 : 4;  // heads of the compile-time geometry
    const int H = GEO ? kGeoH : a.g.H, Hp = GEO ? kGeoH : a.g.Hp, lgHp = GEO ? (kGeoH == 4 ? 2 : 0) : a.g.lgHp;
    const int n_vec = GEO ? G * V : a.g.n_vec, vph = GEO ? (G * V) / kGeoH : a.g.vph;
    const long long rowf = (long long)n_vec * EPV;

    // ---- shared memory carve-up (per warp) ----------------------------------------------------
    // A partition step of the destination-major pass (a launch over the rows that is not the whole graph) stages the
    // rows' own data - the output-gradient row, D, del so far - for a chunk at a time, with the chunk's first gathers
    // in flight, instead of loading it around each row's end: the rows of a partition are short (most of a row's edges
    // lie in other partitions), so a load per completed row, waited for on the spot, is a large part of such a launch.
    // (Measured on the large workload, 16 partitions: 129 -> 108 ms per layer.  The same for the forward pass's running
    // numerator, 512 bytes per row, costs more in resident warps than it saves: 98 -> 127 ms.)
    constexpr bool kStageMode = MODE == kBwdDst || MODE == kBwdDstGivenD;
    const bool staged = kStageMode && STATIC == 0 && a.mode == 0 && a.stage_rows != 0;
    const unsigned rsb = (unsigned)n_vec * 16u;   // bytes of a staged row
    const SpanSmem L = span_layout<MODE>(Hp, V, CAP, S, EPW, staged ? (size_t)a.stage_rows * rsb : 0);
    unsigned char *wb = smem_raw + (size_t)warp * L.total;
    uint4 *stage = reinterpret_cast<uint4 *>(wb + L.stage);  // [S][V][32]
    int *sj = reinterpret_cast<int *>(wb + L.sj);
    W *sw = reinterpret_cast<W *>(wb + L.w);
    const int plane = (int)(span_align16((size_t)kMaxSpanRows * Hp * 4) / 4);
    float *sc0 = reinterpret_cast<float *>(wb + L.rowc);  // el of the row (CSR passes) / er of the row (CSC pass)
    float *sc1 = sc0 + plane;                             // forward: max key; bwd-dst: m
    float *sc2 = sc1 + plane;                             // forward: reference max; bwd-dst: 1/d
    float *sc3 = sc2 + plane;                             // bwd-dst, staged rows: D given
    float *sc4 = sc3 + plane;                             // bwd-dst, staged rows: del so far
    const unsigned rowst_s = (unsigned)__cvta_generic_to_shared(wb + L.rowst);
    int *srb = reinterpret_cast<int *>(wb + L.srb);
    int *sso = reinterpret_cast<int *>(wb + L.sso);
    float *smrun = reinterpret_cast<float *>(wb + L.mrun);
    float *sfac = reinterpret_cast<float *>(wb + L.fac);
    float *scratch = reinterpret_cast<float *>(wb + L.scratch);
    unsigned *skey = reinterpret_cast<unsigned *>(sc1);

    // ---- which rows ---------------------------------------------------------------------------
    const long long item = (long long)blockIdx.x * kSpanWarps + warp;
    long long row0, eb = 0, ee = 0;   // lane r: edge range of row row0 + r
    int nrows;
    bool excluded = false;            // long row left to the segment launch
    long long seg = -1;
    if (mode_ == 0) {
        row0 = item * a.R;
        if (row0 >= a.n_rows) return;
        nrows = (int)((a.n_rows - row0) < a.R ? (a.n_rows - row0) : a.R);
        long long p = 0;
        if (lane <= nrows) p = __ldg(a.indptr + row0 + lane);  // nrows <= 16 < 32 lanes
        const long long pn = __shfl_down_sync(0xffffffffu, p, 1);
        if (lane < nrows) {
            eb = p;
            ee = pn;
            excluded = a.sp.threshold > 0 && ee - eb > a.sp.threshold;
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
    const bool first_part = (flags_ & SAR_FIRST) || mode_ == 1;
    const bool last_part = (flags_ & SAR_LAST) && mode_ == 0;
    const bool mean_now = (flags_ & SAR_MEAN) && (flags_ & SAR_LAST);
    // does a row without edges (in this partition) still have to be written?
    bool write_empty;
    if (kFwdMode) write_empty = (flags_ & SAR_FIRST) || (flags_ & SAR_LAST);
    else if (MODE == kBwdDst) write_empty = true;
    else if (MODE == kBwdDstGivenD) write_empty = flags_ & SAR_FIRST;
    else if (kSrc) write_empty = true;
    else write_empty = (flags_ & SAR_FIRST) || mean_now;
    if (mode_ == 1) write_empty = false;

    // ---- lane geometry ------------------------------------------------------------------------
    int hv[V];
    bool vok[V], lead[V];  // lead: this lane's vector is the first of its head (writes the head's scalars)
#pragma unroll
    for (int v = 0; v < V; ++v) {
        const int vi = v * G + gl;
        vok[v] = vi < n_vec;
        hv[v] = vok[v] ? vi / vph : 0;
        lead[v] = vok[v] && (vi - hv[v] * vph) == 0;
    }
    const unsigned stage_s = (unsigned)__cvta_generic_to_shared(stage) + lane * 16;
    const unsigned sj_s = (unsigned)__cvta_generic_to_shared(sj) + half * 4;
    unsigned w_s[V];
#pragma unroll
    for (int v = 0; v < V; ++v)
        w_s[v] = (unsigned)__cvta_generic_to_shared(sw) + (((half << lgHp) + hv[v]) * (unsigned)sizeof(W));
    const uint4 *gbase = reinterpret_cast<const uint4 *>(a.gather) + gl;

    // ---- per-row accumulators (persist across the chunks of a row longer than CAP) --------------
    constexpr int NP = EPV / 2;
    f32x2 pacc0[V][NP], pacc1[V][NP];  // packed float32 pairs
    // Sum modes: the terms are added eight slots at a time into `pin` and `pin` into the row's accumulator, so that
    // the longest chain of float32 additions behind one output is 8 + slots/8 instead of the row's edge count.
    constexpr bool kTwoLevel = MODE == kSum || MODE == kSumW;
    f32x2 pin[V][NP];
    float sv[V], mrun[V];
    // Row-stationary vector of the backward passes (gout of the row / feat of the source), needed only when the
    // row is finalised.  It is kept as loaded (packed) and requested one row ahead, so that nothing waits for it.
    uint4 rvq[V], rvq_next[V];
#pragma unroll
    for (int v = 0; v < V; ++v) {
        sv[v] = 0.f;
        mrun[v] = SAR_NEG_INF;
#pragma unroll
        for (int k = 0; k < NP; ++k) pacc0[v][k] = pacc1[v][k] = pin[v][k] = zero2();
        rvq[v] = rvq_next[v] = make_uint4(0u, 0u, 0u, 0u);
    }
    auto request_rowvec = [&](long long row_, uint4 (&dst)[V]) {
        const uint4 *rp = reinterpret_cast<const uint4 *>(a.rowvec) + row_ * n_vec + gl;
#pragma unroll
        for (int v = 0; v < V; ++v) dst[v] = vok[v] ? __ldg(rp + v * G) : make_uint4(0u, 0u, 0u, 0u);
    };

    const int deg_l = (lane < nrows && !excluded) ? (int)((ee - eb) > 0x3fffffff ? 0x3fffffff : (ee - eb)) : 0;
    const unsigned excl_all = __ballot_sync(0xffffffffu, excluded);

    int r = 0;           // next row of the span to process
    int piece_off = 0;   // edges of row r already consumed (row longer than CAP)
    while (r < nrows) {
        // ---- choose the chunk: rows [r, r2) --------------------------------------------------
        if ((excl_all >> r) & 1u) {
            ++r;
            continue;
        }
        const int deg_r = __shfl_sync(0xffffffffu, deg_l, r);
        int r2, ne;                       // chunk rows [r, r2), edges in chunk
        const bool cont = piece_off > 0;  // first row continues from the previous chunk
        bool unfinished = false;          // the row goes on in the next chunk
        const long long cb = __shfl_sync(0xffffffffu, eb, r) + piece_off;  // global index of the chunk's first edge
        if (deg_r - piece_off > CAP) {
            r2 = r + 1;
            ne = CAP;
            unfinished = true;
        } else if (cont) {
            r2 = r + 1;
            ne = deg_r - piece_off;
        } else {
            // greedy run of whole rows: none excluded, total <= CAP
            int pre = (lane >= r && lane < nrows) ? deg_l : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, pre, o);
                if (lane >= o) pre = (pre > 0x3fffffff - t) ? 0x3fffffff : pre + t;
            }
            const unsigned later = excl_all & ~((1u << r) - 1u);
            const int stop = later ? __ffs(later) - 1 : nrows;  // first excluded row after r
            const unsigned fits = __ballot_sync(0xffffffffu, lane >= r && lane < stop && pre <= CAP);
            r2 = r + __popc(fits);  // `fits` is a run of lanes starting at r (prefix sums ascend)
            ne = __shfl_sync(0xffffffffu, pre, r2 - 1);
        }
        const int nr = r2 - r;
        const bool piece = cont || unfinished;

        // ---- stage A: row tables and per-row constants ---------------------------------------
        {
            const int i = lane - r;
            int ns = 0;
            if (i >= 0 && i < nr) {
                const int dg = piece ? ne : deg_l;
                srb[i] = piece ? 0 : (int)(eb - cb);
                if (i == nr - 1) srb[nr] = ne;
                ns = (dg + EPW - 1) / EPW;
            }
            int inc = ns;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += t;
            }
            if (i >= 0 && i < nr) sso[i] = inc - ns;
            if (i == nr - 1) sso[nr] = inc;
        }
        __syncwarp();
        const int nslots = sso[nr];
        const int npos = nslots * EPW;

        // ---- the own data of the chunk's rows that will be finalised (a partition step, see `staged`): the copies join
        // the commit group of the score terms below --------------------------------------------------------------------
        const bool staged_now = staged && !piece;
        if constexpr (kStageMode) {
            if (staged_now) {
                const int i = lane - r;
                unsigned todo = __ballot_sync(0xffffffffu, i >= 0 && i < nr && (deg_l > 0 || write_empty)) >> r;
                const unsigned char *base = reinterpret_cast<const unsigned char *>(a.rowvec);
                while (todo) {
                    const int i2 = __ffs(todo) - 1;
                    todo &= todo - 1;
                    const unsigned char *src = base + (size_t)(row0 + r + i2) * rsb;
                    for (unsigned x = (unsigned)lane * 16u; x < rsb; x += 512u) cp_async16_s(rowst_s + (unsigned)i2 * rsb + x, src + x, 16);
                }
            }
        }

        // Every stage below first ISSUES all of its global loads into registers and only then
        // consumes them: a warp executes in order, so a load followed by its use inside a loop body
        // would expose one full memory latency per sweep.
        // ---- stage B: per-(row, head) constants and column ids (slot-major) -----------------------
        auto load_consts = [&](int x, float (&c)[5]) {
            c[0] = 0.f;
            c[1] = __uint_as_float(kKeyNegInf);
            c[2] = c[3] = c[4] = 0.f;
            const int i = x >> lgHp, h = x & (Hp - 1);
            if (x < nr * Hp && h < H) {
                const long long o = (row0 + r + i) * H + h;
                if constexpr (kFwdMode) {
                    c[0] = __ldg(a.el + o);
                } else if constexpr (kDst) {
                    c[0] = __ldg(a.el + o);
                    c[1] = __ldg(a.m + o);
                    c[2] = __ldg(a.d + o);
                    if (staged_now) {
                        if constexpr (MODE == kBwdDstGivenD) c[3] = __ldg(&a.rec_in[o].w);
                        if (!(flags_ & SAR_FIRST)) c[4] = a.del[o];   // plain load: this launch rewrites it
                    }
                } else {
                    c[0] = __ldg(a.er + o);
                }
            }
        };
        auto store_consts = [&](int x, float (&c)[5]) {
            if (x < nr * Hp) {
                if constexpr (kDst) c[2] = c[2] > 0.f ? __fdividef(1.f, c[2]) : 0.f;  // 1/d
                sc0[x] = c[0];
                sc1[x] = c[1];
                sc2[x] = c[2];
                if constexpr (kDst) {
                    if (staged_now) {
                        sc3[x] = c[3];
                        sc4[x] = c[4];
                    }
                }
            }
        };
        float ca[2][5];
        if constexpr (MODE != kSum && MODE != kSumW) {
            load_consts(lane, ca[0]);
            load_consts(lane + 32, ca[1]);
        }
        {   // two positions per lane and sweep: both loads are issued before either is stored
            int i = 0;
            for (int q0 = lane; q0 < npos; q0 += 64) {
                int c[2] = {-1, -1};
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int q = q0 + 32 * u;
                    if (q < npos) {
                        while (q >= sso[i + 1] * EPW) ++i;
                        const int t = srb[i] + (q - sso[i] * EPW);
                        if (t < srb[i + 1]) c[u] = ld_stream_i32(a.indices + cb + t);
                    }
                }
#pragma unroll
                for (int u = 0; u < 2; ++u)
                    if (q0 + 32 * u < npos) sj[q0 + 32 * u] = c[u];
            }
            for (int q = npos + lane; q < npos + S * EPW; q += 32) sj[q] = -1;  // the ring's run-out
        }
        if constexpr (MODE != kSum && MODE != kSumW) {
            store_consts(lane, ca[0]);
            store_consts(lane + 32, ca[1]);
            for (int x = lane + 64; x < nr * Hp; x += 32) {  // many heads x many rows: the rest, plainly
                float c[5];
                load_consts(x, c);
                store_consts(x, c);
            }
        }
        __syncwarp();

        if constexpr (kDst || kSrc) {
            if (mode_ == 0 && !staged_now) {  // the first row that starts in this chunk (a continued row brought its vector along)
                const int first = cont ? 1 : 0;
                if (first < nr) request_rowvec(row0 + r + first, rvq_next);
            }
        }
        // ---- the score terms er[col, :] of every position travel asynchronously too (forward and destination-major
        // passes with heads in groups of four): one 16-byte copy per position and head group straight into the
        // position's weight record, all in flight together and with the ring's first slots, instead of register
        // loads whose latency every sweep of the score phase would wait for.  Each lane copies the positions it
        // will score itself (q = lane mod 32).
        constexpr bool kErAsyncMode = kFwdMode || kDst;
        const bool er_async = kErAsyncMode && (GEO ? true : a.hvec != 0);
        const bool pre_group = er_async || staged_now;   // a commit group ahead of the ring's
        if constexpr (kErAsyncMode) {
            if (er_async) {
                const unsigned sw_s = (unsigned)__cvta_generic_to_shared(sw);
                for (int q = lane; q < npos; q += 32) {
                    const int col = sj[q];
                    const float *src = a.er + (long long)(col < 0 ? 0 : col) * H;
                    for (int h = 0; h < H; h += 4)
                        cp_async16_s(sw_s + (unsigned)(((q << lgHp) + h) * 4), src + h, col >= 0 ? 16 : 0);
                }
            }
        }
        if (pre_group) cp_async_commit();
        // ---- start the gather ring now: the first S slots need only the column ids ----------------
        auto issue = [&](int s_, unsigned dst_s) {
            const int col = lds_s32(sj_s + s_ * (EPW * 4));  // -1 past the row's / chunk's end: zero fill
            const uint4 *src = gbase + (long long)(col < 0 ? 0 : col) * n_vec;
#pragma unroll
            for (int v = 0; v < V; ++v) cp_async16_s(dst_s + v * 512, src + v * G, (col >= 0 && vok[v]) ? 16 : 0);
            cp_async_commit();
        };
#pragma unroll
        for (int s_ = 0; s_ < S; ++s_) issue(s_, stage_s + s_ * (V * 512));
        if (pre_group) {
            cp_async_wait<S>();  // the score terms and the staged rows have landed (the ring's S groups may still be in flight)
            __syncwarp();
        }

        // ---- stage C: weight records, two positions per lane and sweep, all their heads -----------
        if constexpr (MODE == kSumW) {
            // weighted sum: one factor per edge, the source's
            for (int q0 = lane; q0 < npos; q0 += 64) {
                float w[2] = {0.f, 0.f};
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int q = q0 + 32 * u;
                    if (q < npos) {
                        const int col = sj[q];
                        if (col >= 0) w[u] = a.src_scale ? __ldg(a.src_scale + col) : 1.f;
                    }
                }
#pragma unroll
                for (int u = 0; u < 2; ++u)
                    if (q0 + 32 * u < npos) reinterpret_cast<float *>(sw)[q0 + 32 * u] = w[u];
            }
            __syncwarp();
        } else if constexpr (MODE != kSum) {
            const bool vec4 = GEO ? true : a.hvec != 0;  // heads handled four at a time with 16-byte accesses
            // A segment launch of the four-head geometry stages one row: every position would hit the same four
            // shared-memory words, so each lane keeps its own maxima and the warp reduces them once per chunk.
            constexpr bool kLaneMax = kFwdMode && STATIC == 2 && GEO == 1;
            unsigned kmax[4] = {kKeyNegInf, kKeyNegInf, kKeyNegInf, kKeyNegInf};
            int i = 0;
            for (int q0 = lane; q0 < npos; q0 += 64) {
                int col[2], rbase[2];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int q = q0 + 32 * u;
                    col[u] = -1;
                    rbase[u] = 0;
                    if (q < npos) {
                        while (q >= sso[i + 1] * EPW) ++i;
                        col[u] = sj[q];
                        rbase[u] = i * Hp;
                    }
                }
                if (vec4) {
                    for (int h = 0; h < H; h += 4) {
                        if constexpr (kFwdMode || kDst) {
                            float4 e4[2];
#pragma unroll
                            for (int u = 0; u < 2; ++u) {
                                e4[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                                if (col[u] >= 0)  // staged in the position's own record (overwritten by its weights below)
                                    e4[u] = *reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(sw) + ((q0 + 32 * u) << lgHp) + h);
                            }
#pragma unroll
                            for (int u = 0; u < 2; ++u) {
                                const int q = q0 + 32 * u;
                                if (q >= npos) continue;
                                const int rb = rbase[u] + h;
                                const float4 c0 = *reinterpret_cast<const float4 *>(sc0 + rb);
                                const float s4[4] = {c0.x + e4[u].x, c0.y + e4[u].y, c0.z + e4[u].z, c0.w + e4[u].w};
                                float4 o;
                                float *op = reinterpret_cast<float *>(&o);
                                if constexpr (kFwdMode) {
#pragma unroll
                                    for (int j = 0; j < 4; ++j) {
                                        float gr;
                                        op[j] = SAR_NEG_INF;  // padding: weight exp(-inf - max) = 0
                                        if (col[u] >= 0) {
                                            op[j] = leaky(s4[j], a.slope, gr);
                                            if constexpr (kLaneMax) kmax[j] = max(kmax[j], fkey(op[j]));
                                            else atomicMax(&skey[rb + j], fkey(op[j]));
                                        }
                                    }
                                } else {
                                    // rematerialised attention coefficient alpha >= 0; its sign bit carries
                                    // "score <= 0" (LeakyReLU' = slope), so one float holds both weights
                                    const float4 m4 = *reinterpret_cast<const float4 *>(sc1 + rb);
                                    const float4 i4 = *reinterpret_cast<const float4 *>(sc2 + rb);
                                    const float *mp = reinterpret_cast<const float *>(&m4);
                                    const float *ip = reinterpret_cast<const float *>(&i4);
#pragma unroll
                                    for (int j = 0; j < 4; ++j) {
                                        float gr;
                                        const float al = fast_exp(leaky(s4[j], a.slope, gr) - mp[j]) * ip[j];
                                        op[j] = col[u] >= 0 ? (s4[j] > 0.f ? al : -al) : 0.f;
                                    }
                                }
                                *reinterpret_cast<float4 *>(reinterpret_cast<float *>(sw) + (q << lgHp) + h) = o;
                            }
                        } else {
                            // source-major pass: one 16-byte record {el_i, m_i, 1/d_i, D_i} per (column, head)
                            float4 rec[2][4];
#pragma unroll
                            for (int u = 0; u < 2; ++u)
#pragma unroll
                                for (int j = 0; j < 4; ++j) {
                                    rec[u][j] = make_float4(0.f, 0.f, 0.f, 0.f);
                                    if (col[u] >= 0) rec[u][j] = __ldg(a.rec_in + (long long)col[u] * H + h + j);
                                }
#pragma unroll
                            for (int u = 0; u < 2; ++u) {
                                const int q = q0 + 32 * u;
                                if (q >= npos) continue;
                                const float4 c0 = *reinterpret_cast<const float4 *>(sc0 + rbase[u] + h);
                                const float *cp0 = reinterpret_cast<const float *>(&c0);
                                float2 o[4];
#pragma unroll
                                for (int j = 0; j < 4; ++j) {
                                    o[j] = make_float2(0.f, 0.f);
                                    if (col[u] >= 0) {
                                        const float s_ = rec[u][j].x + cp0[j];
                                        float gr;
                                        const float al = fast_exp(leaky(s_, a.slope, gr) - rec[u][j].y) * rec[u][j].z;
                                        o[j] = make_float2(s_ > 0.f ? al : -al, al * gr * rec[u][j].w);
                                    }
                                }
                                float4 *dst = reinterpret_cast<float4 *>(reinterpret_cast<float2 *>(sw) + (q << lgHp) + h);
                                dst[0] = make_float4(o[0].x, o[0].y, o[1].x, o[1].y);
                                dst[1] = make_float4(o[2].x, o[2].y, o[3].x, o[3].y);
                            }
                        }
                    }
                } else {
                    for (int h = 0; h < H; ++h) {
                        float ev[2] = {0.f, 0.f};
                        float4 rec[2];
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            rec[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (col[u] >= 0) {
                                if constexpr (kSrc) rec[u] = __ldg(a.rec_in + (long long)col[u] * H + h);
                                else ev[u] = __ldg(a.er + (long long)col[u] * H + h);
                            }
                        }
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const int q = q0 + 32 * u;
                            if (q >= npos) continue;
                            const int rb = rbase[u] + h;
                            const bool live = col[u] >= 0;
                            float gr;
                            if constexpr (kFwdMode) {
                                float e = SAR_NEG_INF;
                                if (live) {
                                    e = leaky(sc0[rb] + ev[u], a.slope, gr);
                                    atomicMax(&skey[rb], fkey(e));
                                }
                                reinterpret_cast<float *>(sw)[(q << lgHp) + h] = e;
                            } else if constexpr (kDst) {
                                float wrec = 0.f;
                                if (live) {
                                    const float s_ = sc0[rb] + ev[u];
                                    const float al = fast_exp(leaky(s_, a.slope, gr) - sc1[rb]) * sc2[rb];
                                    wrec = s_ > 0.f ? al : -al;
                                }
                                reinterpret_cast<float *>(sw)[(q << lgHp) + h] = wrec;
                            } else {
                                float2 wrec = make_float2(0.f, 0.f);
                                if (live) {
                                    const float s_ = rec[u].x + sc0[rb];
                                    const float al = fast_exp(leaky(s_, a.slope, gr) - rec[u].y) * rec[u].z;
                                    wrec = make_float2(s_ > 0.f ? al : -al, al * gr * rec[u].w);
                                }
                                reinterpret_cast<float2 *>(sw)[(q << lgHp) + h] = wrec;
                            }
                        }
                    }
                }
            }
            if constexpr (kLaneMax) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const unsigned k = __reduce_max_sync(0xffffffffu, kmax[j]);
                    if (lane == 0 && k > skey[j]) skey[j] = k;
                }
            }
            __syncwarp();
        }
        if constexpr (kFwdMode) {
            // reference max per (row, head): the chunk's max, joined with the running max of a
            // continued row; rescale factor exp(old_max - new_max) for what is already accumulated
            for (int x = lane; x < nr * Hp; x += 32) {
                float ref = fkey_inv(skey[x]);
                if (cont) {  // then nr == 1 and x is the head
                    const float old = smrun[x];
                    ref = fmaxf(ref, old);
                    sfac[x] = (ref == SAR_NEG_INF) ? 1.f : fast_exp(old - ref);
                }
                sc2[x] = ref;
            }
            __syncwarp();
            const bool vec4 = GEO ? true : a.hvec != 0;
            int i = 0;
            for (int q = lane; q < npos; q += 32) {
                while (q >= sso[i + 1] * EPW) ++i;
                float *wp = reinterpret_cast<float *>(sw) + (q << lgHp);
                const float *rp = sc2 + i * Hp;
                if (vec4) {
                    for (int h = 0; h < H; h += 4) {
                        float4 e4 = *reinterpret_cast<const float4 *>(wp + h);
                        const float4 r4 = *reinterpret_cast<const float4 *>(rp + h);
                        e4.x = fast_exp(e4.x - r4.x);  // rows with edges have a finite reference
                        e4.y = fast_exp(e4.y - r4.y);
                        e4.z = fast_exp(e4.z - r4.z);
                        e4.w = fast_exp(e4.w - r4.w);
                        *reinterpret_cast<float4 *>(wp + h) = e4;
                    }
                } else {
                    for (int h = 0; h < H; ++h) wp[h] = fast_exp(wp[h] - rp[h]);
                }
            }
            __syncwarp();
            if (cont) {
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    const float c = sfac[hv[v]];
                    sv[v] *= c;
                    mrun[v] = sc2[hv[v]];
                    const f32x2 c2 = pack2(c, c);
#pragma unroll
                    for (int k = 0; k < NP; ++k) pacc0[v][k] = fma2(pacc0[v][k], c2, zero2());
                }
            }
        }

        // ---- stage D: gather through the cp.async ring ---------------------------------------------
        // Slot s lives in ring stage s % S; lane (half, gl) copies and later reads back its own 16
        // bytes of edge s*EPW + half, so no cross-lane synchronisation is needed around the ring.
        int s = 0;
        for (int ri = 0; ri < nr; ++ri) {
            const int s_end = sso[ri + 1];
            const long long row = row0 + r + ri;
            const bool row_starts = !(cont && ri == 0);
            const bool row_ends = !(unfinished && ri == nr - 1);
            if constexpr (kDst || kSrc) {
                if (mode_ == 0 && row_starts && !staged_now) {
#pragma unroll
                    for (int v = 0; v < V; ++v) rvq[v] = rvq_next[v];
                    if (ri + 1 < nr) request_rowvec(row + 1, rvq_next);
                }
            }
            if (s_end == s && !(write_empty && row_starts)) continue;  // no edges here, nothing to write
            if (row_starts) {
                if constexpr (kFwdMode) {
#pragma unroll
                    for (int v = 0; v < V; ++v) mrun[v] = sc2[ri * Hp + hv[v]];
                }
            }
            for (; s < s_end; ++s) {
                cp_async_wait<S - 1>();  // this lane's copies of slot s have landed
                const unsigned src_s = stage_s + (s & (S - 1)) * (V * 512);
                const unsigned woff = (unsigned)s * (unsigned)((EPW << lgHp) * sizeof(W));
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    f32x2 x[NP];
                    Pairs<T>::get(lds128(src_s + v * 512), x);
                    if constexpr (MODE == kSum) {
                        const f32x2 one = pack2(1.f, 1.f);
#pragma unroll
                        for (int k = 0; k < NP; ++k) pin[v][k] = fma2(x[k], one, pin[v][k]);
                    } else if constexpr (MODE == kSumW) {
                        const float w = lds_f32(w_s[v] + woff);
                        const f32x2 w2 = pack2(w, w);
#pragma unroll
                        for (int k = 0; k < NP; ++k) pin[v][k] = fma2(w2, x[k], pin[v][k]);
                    } else if constexpr (kFwdMode) {
                        const float w = lds_f32(w_s[v] + woff);
                        sv[v] += w;
                        const f32x2 w2 = pack2(w, w);
#pragma unroll
                        for (int k = 0; k < NP; ++k) pacc0[v][k] = fma2(w2, x[k], pacc0[v][k]);
                    } else if constexpr (kDst) {
                        const float ws = lds_f32(w_s[v] + woff);
                        const float al = fabsf(ws);
                        const float wg = ws < 0.f ? al * a.slope : al;  // alpha * LeakyReLU'
                        sv[v] += wg;
                        const f32x2 a2 = pack2(al, al), g2 = pack2(wg, wg);
#pragma unroll
                        for (int k = 0; k < NP; ++k) {
                            if constexpr (kAcc0) pacc0[v][k] = fma2(a2, x[k], pacc0[v][k]);
                            pacc1[v][k] = fma2(g2, x[k], pacc1[v][k]);
                        }
                    } else {
                        const float2 w = lds_f32x2(w_s[v] + woff);
                        const float al = fabsf(w.x);
                        const float wg = w.x < 0.f ? al * a.slope : al;
                        sv[v] += w.y;
                        const f32x2 a2 = pack2(al, al), g2 = pack2(wg, wg);
#pragma unroll
                        for (int k = 0; k < NP; ++k) {
                            pacc0[v][k] = fma2(a2, x[k], pacc0[v][k]);
                            pacc1[v][k] = fma2(g2, x[k], pacc1[v][k]);
                        }
                    }
                }
                issue(s + S, src_s);  // refill the stage just consumed
                if constexpr (kTwoLevel) {
                    if ((s & 7) == 7 || s + 1 == s_end) {   // every eight slots and at the end of the row's slots
                        const f32x2 one = pack2(1.f, 1.f);
#pragma unroll
                        for (int v = 0; v < V; ++v)
#pragma unroll
                            for (int k = 0; k < NP; ++k) {
                                pacc0[v][k] = fma2(pin[v][k], one, pacc0[v][k]);
                                pin[v][k] = zero2();
                            }
                    }
                }
            }
            if (!row_ends) continue;

            // ---- the row is complete: fold the 32/G edge lanes, finalise, reset --------------------
            float acc0[V][EPV], acc1[V][EPV];
#pragma unroll
            for (int v = 0; v < V; ++v)
#pragma unroll
                for (int k = 0; k < NP; ++k) {
                    unpack2(pacc0[v][k], acc0[v][2 * k], acc0[v][2 * k + 1]);
                    unpack2(pacc1[v][k], acc1[v][2 * k], acc1[v][2 * k + 1]);
                }
#pragma unroll
            for (int off = G; off < 32; off <<= 1) {
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    sv[v] += __shfl_xor_sync(0xffffffffu, sv[v], off);
#pragma unroll
                    for (int e = 0; e < EPV; ++e) {
                        if constexpr (kAcc0) acc0[v][e] += __shfl_xor_sync(0xffffffffu, acc0[v][e], off);
                        if constexpr (kAcc1) acc1[v][e] += __shfl_xor_sync(0xffffffffu, acc1[v][e], off);
                    }
                }
            }
            const bool writer = half == 0;  // every edge lane now holds the full sums; one writes
            if constexpr (kFwdMode) {
                if (mode_ == 1) {
                    if (writer) {
                        float *rec = a.sp.part + seg * a.sp.pstride;
                        store_acc_row<G, V, EPV>(rec, gl, vok, acc0);
#pragma unroll
                        for (int v = 0; v < V; ++v)
                            if (lead[v]) {
                                rec[rowf + hv[v]] = mrun[v];
                                rec[rowf + H + hv[v]] = sv[v];
                            }
                    }
                } else {
                    if (!first_part) {  // fold the state left by the earlier partitions (Algorithm 1)
                        float old[V][EPV];
#pragma unroll
                        for (int v = 0; v < V; ++v)
#pragma unroll
                            for (int e = 0; e < EPV; ++e) old[v][e] = 0.f;
                        load_acc_row<G, V, EPV>(a.acc_state + row * rowf, gl, vok, old);
#pragma unroll
                        for (int v = 0; v < V; ++v) {
                            const float mo = vok[v] ? a.m_state[row * H + hv[v]] : SAR_NEG_INF;
                            const float dd = vok[v] ? a.d_state[row * H + hv[v]] : 0.f;
                            const float mn = fmaxf(mo, mrun[v]);
                            const float c_old = (mn == SAR_NEG_INF) ? 1.f : fast_exp(mo - mn);
                            const float c_new = (mn == SAR_NEG_INF) ? 1.f : fast_exp(mrun[v] - mn);
                            sv[v] = dd * c_old + sv[v] * c_new;
                            mrun[v] = mn;
#pragma unroll
                            for (int e = 0; e < EPV; ++e) acc0[v][e] = old[v][e] * c_old + acc0[v][e] * c_new;
                        }
                        __syncwarp();  // every edge lane has read the old state before one overwrites it
                    }
                    if (writer) {
                        if (last_part) {
                            if (flags_ & SAR_KEEP_NUMERATOR) store_acc_row<G, V, EPV>(a.acc_state + row * rowf, gl, vok, acc0);
#pragma unroll
                            for (int v = 0; v < V; ++v) {
                                const float inv = sv[v] > 0.f ? __fdividef(1.f, sv[v]) : 0.f;
#pragma unroll
                                for (int e = 0; e < EPV; ++e) acc0[v][e] *= inv;
                                if (flags_ & SAR_RELU_OUT) {
#pragma unroll
                                    for (int e = 0; e < EPV; ++e) acc0[v][e] = fmaxf(acc0[v][e], 0.f);
                                }
                            }
                            store_row_vec<T, G, V>(a.out, row, n_vec, gl, vok, acc0);
                        } else {
                            store_acc_row<G, V, EPV>(a.acc_state + row * rowf, gl, vok, acc0);
                        }
#pragma unroll
                        for (int v = 0; v < V; ++v)
                            if (lead[v]) {
                                a.m_state[row * H + hv[v]] = mrun[v];
                                a.d_state[row * H + hv[v]] = sv[v];
                            }
                    }
                }
            } else if constexpr (kDst) {
                if (mode_ == 1) {
                    if (writer) {
                        float *rec = a.sp.part + seg * a.sp.pstride;
                        store_acc_row<G, V, EPV>(rec, gl, vok, acc1);
                        if constexpr (MODE == kBwdDst) store_acc_row<G, V, EPV>(rec + rowf, gl, vok, acc0);
#pragma unroll
                        for (int v = 0; v < V; ++v)
                            if (lead[v]) rec[2 * rowf + hv[v]] = sv[v];
                    }
                } else {
                    float pA[V], pB[V], rv[V][EPV];
                    if (staged_now) {
#pragma unroll
                        for (int v = 0; v < V; ++v)
                            rvq[v] = vok[v] ? lds128(rowst_s + (unsigned)ri * rsb + (unsigned)((v * G + gl) * 16)) : make_uint4(0u, 0u, 0u, 0u);
                    }
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        Elem<T>::unpack(rvq[v], rv[v]);
                        pA[v] = pB[v] = 0.f;
#pragma unroll
                        for (int e = 0; e < EPV; ++e) {
                            if constexpr (kAcc0) pA[v] = fmaf(rv[v][e], acc0[v][e], pA[v]);
                            pB[v] = fmaf(rv[v][e], acc1[v][e], pB[v]);
                        }
                    }
                    // per-head sums through shared memory (edge lane 0 deposits, lanes < H add up)
                    if (writer) {
#pragma unroll
                        for (int v = 0; v < V; ++v)
                            if (vok[v]) {
                                scratch[v * G + gl] = pB[v];
                                scratch[32 * V + v * G + gl] = pA[v];
                                if (lead[v]) scratch[64 * V + hv[v]] = sv[v];
                            }
                    }
                    __syncwarp();
                    if (lane < H) {
                        float DB = 0.f, DA = 0.f;
                        for (int k = 0; k < vph; ++k) {
                            DB += scratch[lane * vph + k];
                            DA += scratch[32 * V + lane * vph + k];
                        }
                        const float Sh = scratch[64 * V + lane];
                        const float D = MODE == kBwdDstGivenD ? (staged_now ? sc3[ri * Hp + lane] : a.rec_in[row * H + lane].w) : DA;
                        const float val = DB - D * Sh;
                        float *p = a.del + row * H + lane;
                        *p = (flags_ & SAR_FIRST) ? val : (staged_now ? sc4[ri * Hp + lane] : *p) + val;
                        if constexpr (MODE == kBwdDst)
                            a.rec_out[row * H + lane] = make_float4(sc0[ri * Hp + lane], sc1[ri * Hp + lane], sc2[ri * Hp + lane], D);
                    }
                    __syncwarp();
                }
            } else if constexpr (kSrc) {
                if (mode_ == 1) {
                    if (writer) {
                        float *rec = a.sp.part + seg * a.sp.pstride;
                        store_acc_row<G, V, EPV>(rec, gl, vok, acc0);
                        store_acc_row<G, V, EPV>(rec + rowf, gl, vok, acc1);
#pragma unroll
                        for (int v = 0; v < V; ++v)
                            if (lead[v]) rec[2 * rowf + hv[v]] = sv[v];
                    }
                } else {
                    float pC[V], rv[V][EPV];
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        Elem<T>::unpack(rvq[v], rv[v]);
                        pC[v] = 0.f;
#pragma unroll
                        for (int e = 0; e < EPV; ++e) pC[v] = fmaf(rv[v][e], acc1[v][e], pC[v]);
                    }
                    if (writer) {
                        store_row_vec<T, G, V>(a.out, row, n_vec, gl, vok, acc0);
#pragma unroll
                        for (int v = 0; v < V; ++v)
                            if (vok[v]) {
                                scratch[v * G + gl] = pC[v];
                                if (lead[v]) scratch[64 * V + hv[v]] = sv[v];
                            }
                    }
                    __syncwarp();
                    if (lane < H) {
                        float DC = 0.f;
                        for (int k = 0; k < vph; ++k) DC += scratch[lane * vph + k];
                        a.der[row * H + lane] = DC - scratch[64 * V + lane];
                    }
                    __syncwarp();
                }
            } else {  // sum aggregation
                if (mode_ == 1) {
                    if (writer) store_acc_row<G, V, EPV>(a.sp.part + seg * a.sp.pstride, gl, vok, acc0);
                } else if (writer) {
                    if (a.dst_scale) {
                        const float ds = a.dst_scale[row];
#pragma unroll
                        for (int v = 0; v < V; ++v)
#pragma unroll
                            for (int e = 0; e < EPV; ++e) acc0[v][e] *= ds;
                    }
                    if (!(flags_ & SAR_FIRST)) {
                        float old[V][EPV];
                        load_row_vec<T, G, V, false>(a.out, row, n_vec, gl, vok, old);
#pragma unroll
                        for (int v = 0; v < V; ++v)
#pragma unroll
                            for (int e = 0; e < EPV; ++e) acc0[v][e] += old[v][e];
                    }
                    if (mean_now) {
                        const long long dg = a.deg_total[row];
                        const float inv = dg > 0 ? 1.f / (float)dg : 0.f;
#pragma unroll
                        for (int v = 0; v < V; ++v)
#pragma unroll
                            for (int e = 0; e < EPV; ++e) acc0[v][e] *= inv;
                    }
                    store_row_vec<T, G, V>(a.out, row, n_vec, gl, vok, acc0);
                }
            }
#pragma unroll
            for (int v = 0; v < V; ++v) {
                sv[v] = 0.f;
                mrun[v] = SAR_NEG_INF;
#pragma unroll
                for (int k = 0; k < NP; ++k) pacc0[v][k] = pacc1[v][k] = zero2();
            }
        }
        cp_async_wait<0>();  // drain the (zero-size) refills issued past the last slot
        // ---- a row that goes on: publish its running max for the next chunk's score phase -------
        if constexpr (kFwdMode) {
            if (unfinished && half == 0) {
#pragma unroll
                for (int v = 0; v < V; ++v)
                    if (lead[v]) smrun[hv[v]] = mrun[v];
            }
        }
        __syncwarp();
        if (unfinished) {
            piece_off += CAP;
        } else {
            piece_off = 0;
            r = r2;
        }
    }
}

}  // namespace sar

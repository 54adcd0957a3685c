// C-ABI entry points of the fused GAT aggregation and of the sum aggregation: argument checks,
// kernel selection and launches.  Declarations and contracts are in include/sar.h.
#include "sar_gat_kernels.cuh"
#include "sar_span_kernels.cuh"
#include "sar_lean.cuh"
#include "sar_dispatch.cuh"
#include "sar_generic_kernels.cuh"

namespace sar {

sar_launch_hook_fn g_launch_hook = nullptr;
void *g_launch_hook_user = nullptr;

sar_status make_shape(int32_t H, int32_t F, sar_dtype t, bool ptrs_16B_aligned, Shape *out) {
    if (H < 1 || F < 1) return SAR_ERR_INVALID_ARG;
    if (t != SAR_F32 && t != SAR_BF16) return SAR_ERR_INVALID_ARG;
    if ((long long)H * F > (1 << 20)) return SAR_ERR_UNSUPPORTED;
    Shape s;
    s.H = H;
    s.F = F;
    s.t = t;
    const size_t es = sar_elem_size(t);
    s.row_bytes = (size_t)H * F * es;
    const size_t head_bytes = (size_t)F * es;
    s.fast = ptrs_16B_aligned && (head_bytes % 16 == 0) && H <= SAR_MAX_HEADS && s.row_bytes <= SAR_MAX_ROW_BYTES;
    s.G = s.V = 0;
    s.geom = RowGeom{H, 1, 0, 1, 1};
    if (s.fast) {
        const int n_vec = (int)(s.row_bytes / 16);
        const int Hp = sar_pow2_ceil(H);
        int G = sar_pow2_ceil(n_vec);
        if (G > 32) G = 32;
        if (G < 4) G = 4;
        if (G < Hp) G = Hp;
        int V = sar_pow2_ceil((n_vec + G - 1) / G);
        s.G = G;
        s.V = V;
        s.geom = RowGeom{H, Hp, sar_log2(Hp), (int)(head_bytes / 16), n_vec};
    }
    *out = s;
    return SAR_OK;
}

// ---- workspace layout ---------------------------------------------------------------------------
// [ destination records: n_dst*H float4 ][ long-row partials of the CSR ][ long-row partials of the CSC ]
static size_t rec_bytes(long long n_dst, int H) { return sar_round_up((size_t)n_dst * H * 16, 256); }
static long long part_stride(int H, int F) {  // floats per segment, a multiple of 4 (float4 rows)
    return (2LL * H * F + 2LL * H + 3) & ~3LL;
}
static size_t part_bytes(const sar_split *sp, int H, int F) {
    return sp ? sar_round_up((size_t)sp->n_seg * part_stride(H, F) * 4, 256) : 0;
}

static SplitArgs split_args(const sar_split *sp, float *part, int H, int F, bool fast) {
    SplitArgs a;
    a.threshold = 0;
    a.n_long = 0;
    a.n_seg = 0;
    a.long_row = nullptr;
    a.long_seg = nullptr;
    a.part = part;
    a.pstride = part_stride(H, F);
    if (sp && fast && sp->n_long > 0 && sp->threshold > 0) {
        a.threshold = sp->threshold;
        a.n_long = sp->n_long;
        a.n_seg = sp->n_seg;
        a.long_row = sp->long_row;
        a.long_seg = sp->long_seg;
    }
    return a;
}

static sar_status check_split(const sar_split *sp) {
    if (!sp) return SAR_OK;
    if (sp->threshold < 1 || sp->n_long < 0 || sp->n_seg < 0) return SAR_ERR_INVALID_ARG;
    if (sp->n_long > 0 && (!sp->long_row || !sp->long_seg)) return SAR_ERR_INVALID_ARG;
    return SAR_OK;
}

static sar_status check_part(const sar_part *g, bool need_csc) {
    if (!g) return SAR_ERR_INVALID_ARG;
    if (g->n_dst < 0 || g->n_src < 0 || g->nnz < 0) return SAR_ERR_INVALID_ARG;
    if (g->n_src > INT32_MAX) return SAR_ERR_UNSUPPORTED;
    if (!g->indptr || (g->nnz > 0 && !g->indices)) return SAR_ERR_INVALID_ARG;
    if (!sar_aligned(g->indptr, 8) || !sar_aligned(g->indices, 4)) return SAR_ERR_ALIGNMENT;
    if (need_csc) {
        if (!g->t_indptr || (g->nnz > 0 && !g->t_indices)) return SAR_ERR_INVALID_ARG;
        if (!sar_aligned(g->t_indptr, 8) || !sar_aligned(g->t_indices, 4)) return SAR_ERR_ALIGNMENT;
    }
    SAR_TRY(check_split(g->split));
    SAR_TRY(check_split(g->t_split));
    return SAR_OK;
}


// ---- span kernels ---------------------------------------------------------------------------------
constexpr int kCapFwd = 256, kCapDst = 256, kCapSrc = 192, kCapSum = 256;
constexpr int kCapSeg = 128;  // capacity of the segment launches (segments hold at most the plan threshold)
constexpr int kMinBlocksFwd = 24, kMinBlocksBwd = 20;  // resident blocks per SM the register budget is cut for
constexpr size_t kStageBytes = 16 * 1024;              // shared memory a partition step may spend on the rows' own data

static int rows_per_span(long long n_rows, long long nnz, int cap) {
    const double avg = n_rows > 0 ? (double)nnz / (double)n_rows : 0.0;
    int R = avg > 0.5 ? (int)(1.0 * cap / avg + 0.5) : kMaxSpanRows;  // about cap edges per span (the long rows counted in avg are skipped)
    if (R < 1) R = 1;
    if (R > kMaxSpanRows) R = kMaxSpanRows;
    return R;
}

// Launches span_kernel<MODE> over the rows (mode 0) and, with a long-row plan, over the segments
// (mode 1).  The merge launch is the caller's.
template <typename T, int G, int V, int S, int MODE, int CAP, int MINB>
static sar_status launch_span(SpanArgs a, long long nnz, const char *name, const char *seg_name, cudaStream_t st) {
    // The segment launch never stages more than `threshold` edges at a time: when that fits the small
    // capacity it runs the instantiation with the smaller shared-memory footprint (more resident warps).
    constexpr int CAP_SEG = CAP < kCapSeg ? CAP : kCapSeg;
    auto kern = span_kernel<T, G, V, S, MODE, CAP, MINB>;
    const size_t smem = (size_t)kSpanWarps * span_layout<MODE>(a.g.Hp, V, CAP, S, 32 / G).total;
    SAR_TRY(ensure_smem(kern, smem));
    a.mode = 0;
    constexpr bool kIsSum = MODE == kSum || MODE == kSumW;
    constexpr int kGeo = (kIsSum || G * V >= 4) ? 1 : 0;
    const bool geo = kGeo && a.g.n_vec == G * V && (kIsSum ? a.g.H == 1 : (a.g.H == 4 && a.g.Hp == 4 && a.hvec));
    a.R = rows_per_span(a.n_rows, nnz, CAP);
    const bool whole = (a.flags & SAR_FIRST) && (a.flags & SAR_LAST);
    // A partition step of the destination-major pass stages the rows' output-gradient rows per chunk when that fits
    // kStageBytes of shared memory, with fewer rows per span if need be.
    size_t stage_bytes = 0;
    a.stage_rows = 0;
    if (!whole && (MODE == kBwdDst || MODE == kBwdDstGivenD)) {
        const size_t rsb = (size_t)a.g.n_vec * 16;
        if (rsb <= kStageBytes) {
            if ((size_t)a.R * rsb > kStageBytes) a.R = (int)(kStageBytes / rsb);
            a.stage_rows = a.R;
            stage_bytes = (size_t)a.R * rsb;
        }
    }
    const long long spans = (a.n_rows + a.R - 1) / a.R;
    if (spans > 0) {
        const unsigned blocks = (unsigned)((spans + kSpanWarps - 1) / kSpanWarps);
        if (whole && !(a.flags & (SAR_KEEP_NUMERATOR | SAR_RELU_OUT))) {  // the epilogue's flag tests decided at compile time
            if (geo) {
                auto wk = span_kernel<T, G, V, S, MODE, CAP, MINB, 1, kGeo>;
                SAR_TRY(ensure_smem(wk, smem));
                SAR_LAUNCH(name, st, wk<<<blocks, kSpanThreads, smem, st>>>(a));
            } else {
                auto wk = span_kernel<T, G, V, S, MODE, CAP, MINB, 1>;
                SAR_TRY(ensure_smem(wk, smem));
                SAR_LAUNCH(name, st, wk<<<blocks, kSpanThreads, smem, st>>>(a));
            }
        } else {
            const size_t smem_st = (size_t)kSpanWarps * span_layout<MODE>(a.g.Hp, V, CAP, S, 32 / G, stage_bytes).total;
            SAR_TRY(ensure_smem(kern, smem_st));
            SAR_LAUNCH(name, st, kern<<<blocks, kSpanThreads, smem_st, st>>>(a));
        }
        SAR_TRY(sar_after_launch());
    }
    if (a.sp.threshold > 0 && a.sp.n_seg > 0) {
        a.mode = 1;
        const unsigned blocks = (unsigned)((a.sp.n_seg + kSpanWarps - 1) / kSpanWarps);
        if (a.sp.threshold <= CAP_SEG) {
            const size_t seg_smem = (size_t)kSpanWarps * span_layout<MODE>(a.g.Hp, V, CAP_SEG, S, 32 / G).total;
            auto seg_kern = geo ? span_kernel<T, G, V, S, MODE, CAP_SEG, MINB, 2, kGeo> : span_kernel<T, G, V, S, MODE, CAP_SEG, MINB, 2>;
            SAR_TRY(ensure_smem(span_kernel<T, G, V, S, MODE, CAP_SEG, MINB, 2, kGeo>, seg_smem));
            SAR_TRY(ensure_smem(span_kernel<T, G, V, S, MODE, CAP_SEG, MINB, 2>, seg_smem));
            SAR_LAUNCH(seg_name, st, seg_kern<<<blocks, kSpanThreads, seg_smem, st>>>(a));
        } else {
            auto seg_kern = geo ? span_kernel<T, G, V, S, MODE, CAP, MINB, 2, kGeo> : span_kernel<T, G, V, S, MODE, CAP, MINB, 2>;
            SAR_TRY(ensure_smem(span_kernel<T, G, V, S, MODE, CAP, MINB, 2, kGeo>, smem));
            SAR_TRY(ensure_smem(span_kernel<T, G, V, S, MODE, CAP, MINB, 2>, smem));
            SAR_LAUNCH(seg_name, st, seg_kern<<<blocks, kSpanThreads, smem, st>>>(a));
        }
        SAR_TRY(sar_after_launch());
    }
    return SAR_OK;
}

// stages of the gather ring: 8 x 512 bytes in flight per warp for one-vector rows
template <int V> struct UFwd { static constexpr int u = V == 1 ? 8 : (V == 2 ? 4 : 2); };
template <int V> struct UBwd { static constexpr int u = V == 1 ? 8 : (V == 2 ? 4 : 2); };

}  // namespace sar

using namespace sar;

extern "C" {

const char *sar_status_string(sar_status s) {
    switch (s) {
        case SAR_OK: return "ok";
        case SAR_ERR_INVALID_ARG: return "invalid argument";
        case SAR_ERR_UNSUPPORTED: return "unsupported shape";
        case SAR_ERR_ALIGNMENT: return "misaligned pointer";
        case SAR_ERR_WORKSPACE: return "workspace missing or too small";
        case SAR_ERR_CUDA: return "CUDA error";
        case SAR_ERR_BAD_GRAPH: return "inconsistent graph";
    }
    return "unknown status";
}

void sar_set_launch_hook(sar_launch_hook_fn hook, void *user) {
    g_launch_hook = hook;
    g_launch_hook_user = user;
}

int32_t sar_built_for_sm(void) {
#ifdef SAR_BUILT_FOR_SM
    return SAR_BUILT_FOR_SM;
#else
    return 0;
#endif
}

size_t sar_gat_workspace_bytes(const sar_part *g, int32_t H, int32_t F, sar_dtype t) {
    (void)t;
    if (!g || H < 1 || F < 1) return 0;
    return rec_bytes(g->n_dst, H) + part_bytes(g->split, H, F) + part_bytes(g->t_split, H, F) + 256;
}

size_t sar_spmm_workspace_bytes(const sar_part *g, int32_t F, sar_dtype t) {
    (void)t;
    if (!g || F < 1) return 0;
    return part_bytes(g->split, 1, F) + 256;
}

// ---------------------------------------------------------------------------------------------
sar_status sar_gat_fwd(const sar_part *g, const void *feat_q, const float *el, const float *er_q, int32_t H,
                       int32_t F, sar_dtype t, float slope, uint32_t flags, float *acc, float *m, float *d,
                       void *out, void *workspace, size_t workspace_bytes, void *stream) {
    SAR_TRY(check_part(g, false));
    if (flags & ~(SAR_FIRST | SAR_LAST | SAR_KEEP_NUMERATOR | SAR_RELU_OUT)) return SAR_ERR_INVALID_ARG;
    const bool first = flags & SAR_FIRST, last = flags & SAR_LAST;
    if ((flags & (SAR_KEEP_NUMERATOR | SAR_RELU_OUT)) && !last) return SAR_ERR_INVALID_ARG;
    if (!el || !m || !d) return SAR_ERR_INVALID_ARG;
    if (g->n_src > 0 && (!feat_q || !er_q)) return SAR_ERR_INVALID_ARG;
    if (last && !out) return SAR_ERR_INVALID_ARG;
    if ((!(first && last) || (flags & SAR_KEEP_NUMERATOR)) && !acc) return SAR_ERR_INVALID_ARG;
    SAR_TRY(check_elem_align({el, er_q, m, d, acc}, 4));
    SAR_TRY(check_elem_align({feat_q, out}, sar_elem_size(t)));
    Shape s;
    SAR_TRY(make_shape(H, F, t, all16({feat_q, out, acc}), &s));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (g->n_dst == 0) return SAR_OK;

    if (!s.fast) {
        GenericArgs a{};
        a.n_dst = g->n_dst;
        a.indptr = g->indptr;
        a.indices = g->indices;
        a.feat = feat_q;
        a.el = el;
        a.er = er_q;
        a.acc = acc;
        a.m = m;
        a.d = d;
        a.out = out;
        a.H = H;
        a.F = F;
        a.slope = slope;
        a.flags = flags;
        const long long n = g->n_dst * H;
        const unsigned blocks = (unsigned)((n + 255) / 256);
        if (t == SAR_F32)
            SAR_LAUNCH("gat_fwd_generic", st, gat_fwd_generic<float><<<blocks, 256, 0, st>>>(a));
        else
            SAR_LAUNCH("gat_fwd_generic", st, gat_fwd_generic<__nv_bfloat16><<<blocks, 256, 0, st>>>(a));
        return sar_after_launch();
    }

    const bool use_split = g->split && g->split->n_long > 0;
    float *part = nullptr;
    if (use_split) {
        const size_t need = rec_bytes(g->n_dst, H) + part_bytes(g->split, H, F);
        if (!workspace || workspace_bytes < need || !sar_aligned(workspace, 16)) return SAR_ERR_WORKSPACE;
        part = reinterpret_cast<float *>(static_cast<char *>(workspace) + rec_bytes(g->n_dst, H));
    }
    FwdArgs ma;  // arguments of the merge launch
    ma.n_dst = g->n_dst;
    ma.indptr = g->indptr;
    ma.indices = g->indices;
    ma.feat = feat_q;
    ma.el = el;
    ma.er = er_q;
    ma.acc = acc;
    ma.m = m;
    ma.d = d;
    ma.out = out;
    ma.slope = slope;
    ma.flags = flags;
    ma.g = s.geom;
    ma.sp = split_args(g->split, part, H, F, true);
    ma.mode = 0;
    SpanArgs a{};
    a.n_rows = g->n_dst;
    a.indptr = g->indptr;
    a.indices = g->indices;
    a.gather = feat_q;
    a.el = el;
    a.er = er_q;
    a.acc_state = acc;
    a.m_state = m;
    a.d_state = d;
    a.out = out;
    a.slope = slope;
    a.flags = flags;
    a.g = s.geom;
    a.sp = ma.sp;
    a.hvec = (H % 4 == 0) && sar_aligned(er_q, 16);
    const bool lean = lean_applies(s, flags, slope, g->split, g->n_src) && sar_aligned(er_q, 16);
    // A partition step of a call-by-call pass.  The last one folds like the others and leaves the division to a
    // launch of its own over all rows (most rows have no edge in a given partition, and every row has to be divided).
    const bool lean_part = !(first && last) && lean_shape_applies(s, slope, g->split, g->n_src) && sar_aligned(er_q, 16) &&
                           (g->nnz < (long long)kLeanPartMaxDegree * g->n_dst ||
                            (g->nnz >= (long long)kLeanPartMinDenseDegree * g->n_dst && !first));
    LeanArgs la{};
    if (lean || lean_part) {
        la.n_rows = g->n_dst;
        la.indptr = g->indptr;
        la.indices = g->indices;
        la.gather = feat_q;
        la.el = el;
        la.er = er_q;
        la.m_out = m;
        la.d_out = d;
        la.acc_state = acc;
        la.first = first ? 1 : 0;
        la.out = out;
        la.relu = (flags & SAR_RELU_OUT) ? 1 : 0;
        la.slope = slope;
        la.sp = ma.sp;
        la.sp.threshold = g->split->threshold;
    }
    return dispatch(s, [&](auto cfg) -> sar_status {
        using C = decltype(cfg);
        using T = typename C::type;
        if (lean)
            SAR_TRY(s.t == SAR_F32 ? lean_fwd_f32(s, la, g->nnz, st) : lean_fwd_bf16(s, la, g->nnz, st));
        else if (lean_part)
            SAR_TRY(s.t == SAR_F32 ? lean_fwd_part_f32(s, la, g->nnz, st) : lean_fwd_part_bf16(s, la, g->nnz, st));
        else
            SAR_TRY((launch_span<T, C::g, C::v, UFwd<C::v>::u, kFwd, kCapFwd, kMinBlocksFwd>(a, g->nnz, "gat_fwd", "gat_fwd_seg", st)));
        const bool divide_after = lean_part && last;
        if (ma.sp.threshold > 0) {
            FwdArgs mm = ma;
            if (divide_after) mm.flags = 0;   // the long rows' state is folded like the others'
            SAR_LAUNCH("gat_fwd_merge", st, gat_fwd_merge_kernel<T, C::g, C::v><<<blocks_for(mm.sp.n_long, C::g), kThreads, 0, st>>>(mm));
            SAR_TRY(sar_after_launch());
        }
        if (divide_after) {
            const long long nv = g->n_dst * (long long)s.geom.n_vec;
            SAR_LAUNCH("gat_fwd_finalize", st, gat_fwd_finalize_kernel<T><<<(unsigned)((nv + 255) / 256), 256, 0, st>>>(ma));
            SAR_TRY(sar_after_launch());
        }
        return SAR_OK;
    });
}

static sar_status check_fused(const sar_part *g, int32_t k, const int64_t *bounds) {
    if (!g || !bounds || k < 1) return SAR_ERR_INVALID_ARG;
    if (k > SAR_MAX_PARTS) return SAR_ERR_UNSUPPORTED;
    if (bounds[0] != 0 || bounds[k] != g->n_src) return SAR_ERR_INVALID_ARG;
    for (int32_t q = 0; q < k; ++q)
        if (bounds[q + 1] < bounds[q]) return SAR_ERR_INVALID_ARG;
    return SAR_OK;
}

sar_status sar_gat_fwd_fused(const sar_part *g, int32_t k, const int64_t *bounds, const void *feat, const float *el,
                             const float *er, int32_t H, int32_t F, sar_dtype t, float slope, float *m, float *d,
                             void *out, void *workspace, size_t workspace_bytes, void *stream) {
    SAR_TRY(check_fused(g, k, bounds));
    // Sources ascend within a row, so walking a row once IS the partition-after-partition visit.
    return sar_gat_fwd(g, feat, el, er, H, F, t, slope, SAR_FIRST | SAR_LAST, nullptr, m, d, out, workspace,
                       workspace_bytes, stream);
}

// ---------------------------------------------------------------------------------------------
sar_status sar_gat_bwd_prepare(int64_t n_dst, int32_t H, int32_t F, sar_dtype t, const void *out_or_acc,
                               int32_t acc_is_numerator, const void *gout, const float *el, const float *m,
                               const float *d, float *D, void *workspace, size_t workspace_bytes, void *stream) {
    if (n_dst < 0 || !out_or_acc || !gout || !el || !m || !d) return SAR_ERR_INVALID_ARG;
    if (!workspace || !sar_aligned(workspace, 16) || workspace_bytes < (size_t)n_dst * H * 16) return SAR_ERR_WORKSPACE;
    SAR_TRY(check_elem_align({el, m, d, D}, 4));
    SAR_TRY(check_elem_align({gout}, sar_elem_size(t)));
    SAR_TRY(check_elem_align({out_or_acc}, acc_is_numerator ? 4 : sar_elem_size(t)));
    Shape s;
    SAR_TRY(make_shape(H, F, t, all16({out_or_acc, gout}), &s));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n_dst == 0) return SAR_OK;
    if (!s.fast) {
        GenericArgs a{};
        a.n_dst = n_dst;
        a.out_in = out_or_acc;
        a.gout = gout;
        a.el = el;
        a.m_in = m;
        a.d_in = d;
        a.D = D;
        a.rec = static_cast<float4 *>(workspace);
        a.H = H;
        a.F = F;
        a.acc_is_numerator = acc_is_numerator;
        const unsigned blocks = (unsigned)((n_dst * H + 255) / 256);
        if (t == SAR_F32)
            SAR_LAUNCH("gat_bwd_prepare_generic", st, gat_bwd_prepare_generic<float><<<blocks, 256, 0, st>>>(a));
        else
            SAR_LAUNCH("gat_bwd_prepare_generic", st, gat_bwd_prepare_generic<__nv_bfloat16><<<blocks, 256, 0, st>>>(a));
        return sar_after_launch();
    }
    PrepArgs a;
    a.n_dst = n_dst;
    a.out = out_or_acc;
    a.gout = gout;
    a.el = el;
    a.m = m;
    a.d = d;
    a.D = D;
    a.rec = static_cast<float4 *>(workspace);
    a.acc_is_numerator = acc_is_numerator;
    a.g = s.geom;
    return dispatch(s, [&](auto cfg) -> sar_status {
        using C = decltype(cfg);
        using T = typename C::type;
        const size_t smem = (size_t)kWarpsPerBlock * 32 * C::v * 4;
        const unsigned blocks = blocks_for((n_dst + PrepRows<C::v>::n - 1) / PrepRows<C::v>::n, C::g);
        if (acc_is_numerator)
            SAR_LAUNCH("gat_bwd_prepare", st, gat_bwd_prepare_kernel<T, C::g, C::v, true><<<blocks, kThreads, smem, st>>>(a));
        else
            SAR_LAUNCH("gat_bwd_prepare", st, gat_bwd_prepare_kernel<T, C::g, C::v, false><<<blocks, kThreads, smem, st>>>(a));
        return sar_after_launch();
    });
}

sar_status sar_gat_bwd(const sar_part *g, const void *feat_q, const float *el, const float *er_q, const float *m,
                       const float *d, const void *gout, int32_t H, int32_t F, sar_dtype t, float slope,
                       uint32_t flags, void *dfeat_q, float *del, float *der_q, void *workspace,
                       size_t workspace_bytes, void *stream) {
    SAR_TRY(check_part(g, true));
    if (flags & ~(SAR_FIRST | SAR_LAST)) return SAR_ERR_INVALID_ARG;
    if (!el || !m || !d || !gout || !del) return SAR_ERR_INVALID_ARG;
    if (g->n_src > 0 && (!feat_q || !er_q || !dfeat_q || !der_q)) return SAR_ERR_INVALID_ARG;
    SAR_TRY(check_elem_align({el, er_q, m, d, del, der_q}, 4));
    SAR_TRY(check_elem_align({feat_q, gout, dfeat_q}, sar_elem_size(t)));
    Shape s;
    SAR_TRY(make_shape(H, F, t, all16({feat_q, gout, dfeat_q}), &s));
    const size_t need = rec_bytes(g->n_dst, H) + (s.fast ? part_bytes(g->split, H, F) + part_bytes(g->t_split, H, F) : 0);
    if (!workspace || !sar_aligned(workspace, 16) || workspace_bytes < need) return SAR_ERR_WORKSPACE;
    const bool whole = (flags & SAR_FIRST) && (flags & SAR_LAST);  // D rebuilt from the edges
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float4 *rec = static_cast<float4 *>(workspace);
    char *wsb = static_cast<char *>(workspace);
    float *part_csr = reinterpret_cast<float *>(wsb + rec_bytes(g->n_dst, H));
    float *part_csc = reinterpret_cast<float *>(wsb + rec_bytes(g->n_dst, H) + part_bytes(g->split, H, F));

    if (!s.fast) {
        GenericArgs a{};
        a.n_dst = g->n_dst;
        a.n_src = g->n_src;
        a.indptr = g->indptr;
        a.indices = g->indices;
        a.t_indptr = g->t_indptr;
        a.t_indices = g->t_indices;
        a.feat = feat_q;
        a.gout = gout;
        a.el = el;
        a.er = er_q;
        a.m_in = m;
        a.d_in = d;
        a.dfeat = dfeat_q;
        a.del = del;
        a.der = der_q;
        a.rec = rec;
        a.H = H;
        a.F = F;
        a.slope = slope;
        a.flags = flags;
        a.given_d = whole ? 0 : 1;
        if (g->n_dst > 0) {
            const unsigned blocks = (unsigned)((g->n_dst * H + 255) / 256);
            if (t == SAR_F32)
                SAR_LAUNCH("gat_bwd_dst_generic", st, gat_bwd_dst_generic<float><<<blocks, 256, 0, st>>>(a));
            else
                SAR_LAUNCH("gat_bwd_dst_generic", st, gat_bwd_dst_generic<__nv_bfloat16><<<blocks, 256, 0, st>>>(a));
            SAR_TRY(sar_after_launch());
        }
        if (g->n_src > 0) {
            const unsigned blocks = (unsigned)((g->n_src * H + 255) / 256);
            if (t == SAR_F32)
                SAR_LAUNCH("gat_bwd_src_generic", st, gat_bwd_src_generic<float><<<blocks, 256, 0, st>>>(a));
            else
                SAR_LAUNCH("gat_bwd_src_generic", st, gat_bwd_src_generic<__nv_bfloat16><<<blocks, 256, 0, st>>>(a));
            SAR_TRY(sar_after_launch());
        }
        return SAR_OK;
    }

    BwdDstArgs da;  // merge launches
    da.n_dst = g->n_dst;
    da.indptr = g->indptr;
    da.indices = g->indices;
    da.feat = feat_q;
    da.gout = gout;
    da.el = el;
    da.er = er_q;
    da.m = m;
    da.d = d;
    da.rec = rec;
    da.del = del;
    da.slope = slope;
    da.flags = flags;
    da.g = s.geom;
    da.sp = split_args(g->split, part_csr, H, F, true);
    da.mode = 0;
    BwdSrcArgs sa;
    sa.n_src = g->n_src;
    sa.t_indptr = g->t_indptr;
    sa.t_indices = g->t_indices;
    sa.gout = gout;
    sa.feat = feat_q;
    sa.er = er_q;
    sa.rec = rec;
    sa.dfeat = dfeat_q;
    sa.der = der_q;
    sa.slope = slope;
    sa.g = s.geom;
    sa.sp = split_args(g->t_split, part_csc, H, F, true);
    sa.mode = 0;
    SpanArgs d1{};  // destination-major pass over the CSR
    d1.n_rows = g->n_dst;
    d1.indptr = g->indptr;
    d1.indices = g->indices;
    d1.gather = feat_q;
    d1.rowvec = gout;
    d1.el = el;
    d1.er = er_q;
    d1.m = m;
    d1.d = d;
    d1.rec_in = rec;
    d1.rec_out = rec;
    d1.del = del;
    d1.slope = slope;
    d1.flags = flags;
    d1.g = s.geom;
    d1.sp = da.sp;
    d1.hvec = (H % 4 == 0) && sar_aligned(er_q, 16);
    SpanArgs s1{};  // source-major pass over the CSC
    s1.n_rows = g->n_src;
    s1.indptr = g->t_indptr;
    s1.indices = g->t_indices;
    s1.gather = gout;
    s1.rowvec = feat_q;
    s1.er = er_q;
    s1.rec_in = rec;
    s1.out = dfeat_q;
    s1.der = der_q;
    s1.slope = slope;
    s1.flags = flags;
    s1.g = s.geom;
    s1.sp = sa.sp;
    s1.hvec = (H % 4 == 0);

    const bool lean_dst_shape = lean_shape_applies(s, slope, g->split, g->n_src) && sar_aligned(er_q, 16);
    const bool lean_dst = whole && lean_dst_shape;
    const bool lean_dst_part = !whole && lean_dst_shape;   // a partition step: D given, del collects
    const bool lean_src = lean_shape_applies(s, slope, g->t_split, g->n_dst);   // whole graph or partition step alike
    LeanArgs ld{};
    LeanSrcArgs ls{};
    if (lean_src) {
        ls.n_rows = g->n_src;
        ls.indptr = g->t_indptr;
        ls.indices = g->t_indices;
        ls.gather = gout;
        ls.rowvec = feat_q;
        ls.er = er_q;
        ls.rec_in = rec;
        ls.out = dfeat_q;
        ls.der = der_q;
        ls.slope = slope;
        ls.sp = sa.sp;
        ls.sp.threshold = g->t_split->threshold;
    }
    if (lean_dst || lean_dst_part) {
        ld.n_rows = g->n_dst;
        ld.indptr = g->indptr;
        ld.indices = g->indices;
        ld.gather = feat_q;
        ld.rowvec = gout;
        ld.el = el;
        ld.er = er_q;
        ld.m = m;
        ld.d = d;
        ld.rec_out = rec;
        ld.rec_in = rec;
        ld.first = (flags & SAR_FIRST) ? 1 : 0;
        ld.del = del;
        ld.slope = slope;
        ld.sp = da.sp;
        ld.sp.threshold = g->split->threshold;
    }

    return dispatch(s, [&](auto cfg) -> sar_status {
        using C = decltype(cfg);
        using T = typename C::type;
        constexpr int U = UBwd<C::v>::u;
        const size_t msmem = (size_t)kWarpsPerBlock * warp_smem_floats(s.geom.Hp, C::v, 4) * 4;
        if (g->n_dst > 0) {
            if (whole) {
                if (lean_dst)
                    SAR_TRY(s.t == SAR_F32 ? lean_bwd_dst_f32(s, ld, g->nnz, st) : lean_bwd_dst_bf16(s, ld, g->nnz, st));
                else
                    SAR_TRY((launch_span<T, C::g, C::v, U, kBwdDst, kCapDst, kMinBlocksBwd>(d1, g->nnz, "gat_bwd_dst", "gat_bwd_dst_seg", st)));
                if (da.sp.threshold > 0) {
                    auto merge = gat_bwd_dst_merge_kernel<T, C::g, C::v, false>;
                    SAR_TRY(ensure_smem(merge, msmem));
                    SAR_LAUNCH("gat_bwd_dst_merge", st, merge<<<blocks_for(da.sp.n_long, C::g), kThreads, msmem, st>>>(da));
                    SAR_TRY(sar_after_launch());
                }
            } else {
                if (lean_dst_part)
                    SAR_TRY(s.t == SAR_F32 ? lean_bwd_dst_part_f32(s, ld, g->nnz, st) : lean_bwd_dst_part_bf16(s, ld, g->nnz, st));
                else
                    SAR_TRY((launch_span<T, C::g, C::v, U, kBwdDstGivenD, kCapDst, kMinBlocksBwd>(d1, g->nnz, "gat_bwd_dst", "gat_bwd_dst_seg", st)));
                if (da.sp.threshold > 0) {
                    auto merge = gat_bwd_dst_merge_kernel<T, C::g, C::v, true>;
                    SAR_TRY(ensure_smem(merge, msmem));
                    SAR_LAUNCH("gat_bwd_dst_merge", st, merge<<<blocks_for(da.sp.n_long, C::g), kThreads, msmem, st>>>(da));
                    SAR_TRY(sar_after_launch());
                }
            }
        }
        if (g->n_src > 0) {
            if (lean_src)
                SAR_TRY(s.t == SAR_F32 ? lean_bwd_src_f32(s, ls, g->nnz, st) : lean_bwd_src_bf16(s, ls, g->nnz, st));
            else
                SAR_TRY((launch_span<T, C::g, C::v, U, kBwdSrc, kCapSrc, kMinBlocksBwd>(s1, g->nnz, "gat_bwd_src", "gat_bwd_src_seg", st)));
            if (sa.sp.threshold > 0) {
                auto merge = gat_bwd_src_merge_kernel<T, C::g, C::v>;
                SAR_TRY(ensure_smem(merge, msmem));
                SAR_LAUNCH("gat_bwd_src_merge", st, merge<<<blocks_for(sa.sp.n_long, C::g), kThreads, msmem, st>>>(sa));
                SAR_TRY(sar_after_launch());
            }
        }
        return SAR_OK;
    });
}

sar_status sar_gat_bwd_fused(const sar_part *g, int32_t k, const int64_t *bounds, const void *feat, const float *el,
                             const float *er, const float *m, const float *d, const void *gout, int32_t H, int32_t F,
                             sar_dtype t, float slope, void *dfeat, float *del, float *der, void *workspace,
                             size_t workspace_bytes, void *stream) {
    SAR_TRY(check_fused(g, k, bounds));
    return sar_gat_bwd(g, feat, el, er, m, d, gout, H, F, t, slope, SAR_FIRST | SAR_LAST, dfeat, del, der, workspace,
                       workspace_bytes, stream);
}

// ---------------------------------------------------------------------------------------------
static sar_status spmm_impl(const sar_part *g, const void *feat_q, int32_t F, sar_dtype t, uint32_t flags,
                            const int64_t *deg_total, const float *src_scale, const float *dst_scale, void *out,
                            void *workspace, size_t workspace_bytes, void *stream) {
    SAR_TRY(check_part(g, false));
    if (flags & ~(SAR_FIRST | SAR_LAST | SAR_MEAN)) return SAR_ERR_INVALID_ARG;
    if (!out || (g->n_src > 0 && !feat_q)) return SAR_ERR_INVALID_ARG;
    if ((flags & SAR_MEAN) && (flags & SAR_LAST) && !deg_total) return SAR_ERR_INVALID_ARG;
    SAR_TRY(check_elem_align({feat_q, out}, sar_elem_size(t)));
    SAR_TRY(check_elem_align({deg_total}, 8));
    SAR_TRY(check_elem_align({src_scale, dst_scale}, 4));
    const bool weighted = src_scale || dst_scale;
    Shape s;
    SAR_TRY(make_shape(1, F, t, all16({feat_q, out}), &s));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (g->n_dst == 0) return SAR_OK;
    if (!s.fast) {
        GenericArgs a{};
        a.n_dst = g->n_dst;
        a.indptr = g->indptr;
        a.indices = g->indices;
        a.feat = feat_q;
        a.out = out;
        a.deg_total = deg_total;
        a.src_scale = src_scale;
        a.dst_scale = dst_scale;
        a.H = 1;
        a.F = F;
        a.flags = flags;
        const unsigned blocks = (unsigned)((g->n_dst * F + 255) / 256);
        if (t == SAR_F32)
            SAR_LAUNCH("spmm_generic", st, spmm_generic<float><<<blocks, 256, 0, st>>>(a));
        else
            SAR_LAUNCH("spmm_generic", st, spmm_generic<__nv_bfloat16><<<blocks, 256, 0, st>>>(a));
        return sar_after_launch();
    }
    const bool use_split = g->split && g->split->n_long > 0;
    if (use_split && (!workspace || !sar_aligned(workspace, 16) || workspace_bytes < part_bytes(g->split, 1, F)))
        return SAR_ERR_WORKSPACE;
    SumArgs ma;  // merge launch
    ma.n_dst = g->n_dst;
    ma.indptr = g->indptr;
    ma.indices = g->indices;
    ma.feat = feat_q;
    ma.out = out;
    ma.deg_total = deg_total;
    ma.dst_scale = dst_scale;
    ma.flags = flags;
    ma.g = s.geom;
    ma.sp = split_args(g->split, static_cast<float *>(workspace), 1, F, true);
    ma.mode = 0;
    SpanArgs a{};
    a.n_rows = g->n_dst;
    a.indptr = g->indptr;
    a.indices = g->indices;
    a.gather = feat_q;
    a.out = out;
    a.deg_total = deg_total;
    a.src_scale = src_scale;
    a.dst_scale = dst_scale;
    a.flags = flags;
    a.g = s.geom;
    a.sp = ma.sp;
    return dispatch(s, [&](auto cfg) -> sar_status {
        using C = decltype(cfg);
        using T = typename C::type;
        if (weighted)
            SAR_TRY((launch_span<T, C::g, C::v, UFwd<C::v>::u, kSumW, kCapSum, kMinBlocksFwd>(a, g->nnz, "spmm", "spmm_seg", st)));
        else
            SAR_TRY((launch_span<T, C::g, C::v, UFwd<C::v>::u, kSum, kCapSum, kMinBlocksFwd>(a, g->nnz, "spmm", "spmm_seg", st)));
        if (ma.sp.threshold > 0) {
            SAR_LAUNCH("spmm_merge", st, spmm_merge_kernel<T, C::g, C::v><<<blocks_for(ma.sp.n_long, C::g), kThreads, 0, st>>>(ma));
            SAR_TRY(sar_after_launch());
        }
        return SAR_OK;
    });
}

sar_status sar_spmm_agg(const sar_part *g, const void *feat_q, int32_t F, sar_dtype t, uint32_t flags,
                        const int64_t *deg_total, void *out, void *workspace, size_t workspace_bytes,
                        void *stream) {
    return spmm_impl(g, feat_q, F, t, flags, deg_total, nullptr, nullptr, out, workspace, workspace_bytes, stream);
}

sar_status sar_spmm_agg_scaled(const sar_part *g, const void *feat_q, int32_t F, sar_dtype t, uint32_t flags,
                               const float *src_scale, const float *dst_scale, void *out, void *workspace,
                               size_t workspace_bytes, void *stream) {
    if (flags & SAR_MEAN) return SAR_ERR_INVALID_ARG;
    return spmm_impl(g, feat_q, F, t, flags, nullptr, src_scale, dst_scale, out, workspace, workspace_bytes, stream);
}

}  // extern "C"

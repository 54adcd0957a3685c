// The dense projection z = h W of a layer (Eq. 1 / Eq. 3: z = W h, one row per node) and its backward
// pass: the one dense contraction around the aggregation, run on the 5th-generation tensor cores
// (tcgen05 MMA with accumulators in tensor memory, operands staged by TMA) through CUTLASS's sm100
// collective templates instantiated here; bf16 operands, float32 accumulation.  Contracts are in
// include/sar.h.  Cluster shape 1x1x1: every CTA loads its own operand tiles.
#include "sar_common.cuh"

#include "cutlass/cutlass.h"
#include "cutlass/epilogue/collective/collective_builder.hpp"
#include "cutlass/epilogue/fusion/operations.hpp"
#include "cutlass/epilogue/fusion/sm90_visitor_load_tma_warpspecialized.hpp"
#include "cutlass/epilogue/thread/activation.h"
#include "cutlass/epilogue/fusion/sm90_visitor_tma_warpspecialized.hpp"
#include "cutlass/gemm/collective/collective_builder.hpp"
#include "cutlass/gemm/device/gemm_universal_adapter.h"
#include "cutlass/gemm/kernel/gemm_universal.hpp"
#include "cutlass/gemm/kernel/tile_scheduler.hpp"
#include "cutlass/util/packed_stride.hpp"

namespace sarlin {

using namespace cute;

// Epilogue visitor of the fused projection (Eq. 3: the two halves of a^T (z_i || z_j)): while the accumulator tile of
// z = h W leaves tensor memory, every thread rounds its elements to bf16 - the values z is stored with - and adds
// z[i, n] a_l[n] and z[i, n] a_r[n] into per-head sums of its row; when a head is complete it writes el[i, h], er[i, h].
// The two vectors reach the threads as row-broadcast children of this node (CUTLASS stages them in shared memory once
// per tile: the kernel leaves no L1, a global load per element would cost an L2 round trip each).  A thread of this
// epilogue holds elements of ONE row (one lane of tensor memory) and, the tile being 128 columns wide, all columns of
// the heads that start in its tile, in ascending order, so every (row, head) has one writer and a fixed summation
// order.  A thread that sees anything else raises *flag instead of writing (checked by the tests).
struct ProjectVisitor {
    struct SharedStorage {};
    struct Arguments {
        float *el = nullptr, *er = nullptr;
        int H = 0, F = 1;
        int *flag = nullptr;
    };
    using Params = Arguments;

    template <class ProblemShape>
    static constexpr Params to_underlying_arguments(ProblemShape const &, Arguments const &args, void *) { return args; }
    template <class ProblemShape>
    static bool can_implement(ProblemShape const &, Arguments const &) { return true; }
    template <class ProblemShape>
    static size_t get_workspace_size(ProblemShape const &, Arguments const &) { return 0; }
    template <class ProblemShape>
    static cutlass::Status initialize_workspace(ProblemShape const &, Arguments const &, void *, cudaStream_t,
                                                cutlass::CudaHostAdapter * = nullptr) {
        return cutlass::Status::kSuccess;
    }
    CUTLASS_DEVICE bool is_producer_load_needed() const { return false; }
    CUTLASS_DEVICE bool is_C_load_needed() const { return false; }
    CUTLASS_HOST_DEVICE ProjectVisitor() {}
    CUTLASS_HOST_DEVICE ProjectVisitor(Params const &p, SharedStorage const &) : params(p) {}
    Params const params;

    template <class... Args>
    CUTLASS_DEVICE auto get_producer_load_callbacks(cutlass::epilogue::fusion::ProducerLoadArgs<Args...> const &) {
        return cutlass::epilogue::fusion::EmptyProducerLoadCallbacks{};
    }

    template <class CTensor, class ThrResidue>
    struct ConsumerStoreCallbacks : cutlass::epilogue::fusion::EmptyConsumerStoreCallbacks {
        CUTLASS_DEVICE ConsumerStoreCallbacks(CTensor c, ThrResidue res, int m0, int n0, Params const &p)
            : tCcD(c), residue(res), m_origin(m0), n_origin(n0), params(p) {}
        CTensor tCcD;        // coordinates relative to this thread's first element
        ThrResidue residue;  // what is left of the problem from there
        int m_origin, n_origin;
        Params params;
        // the head in progress: its sums and its column range
        float sl = 0.f, sr = 0.f;
        int head = -1, head_begin = 0, head_end = 0;
        int row = -1;
        bool bad = false;    // a second row, columns out of order, or a head entered in its middle

        CUTLASS_DEVICE void flush() {
            if (head >= 0 && !bad) {
                params.el[(long long)row * params.H + head] = sl;
                params.er[(long long)row * params.H + head] = sr;
            }
        }

        // frg_z: the accumulators (child 0), frg_al / frg_ar: a_l[n], a_r[n] of the same columns (children 1, 2)
        template <typename ElementAccumulator, typename ElementZ, typename ElementV, int FragmentSize>
        CUTLASS_DEVICE auto visit(cutlass::Array<ElementAccumulator, FragmentSize> const &, int epi_v, int epi_m, int epi_n,
                                  cutlass::Array<ElementZ, FragmentSize> const &frg_z,
                                  cutlass::Array<ElementV, FragmentSize> const &frg_al,
                                  cutlass::Array<ElementV, FragmentSize> const &frg_ar) {
            using Convert = cutlass::NumericArrayConverter<cutlass::bfloat16_t, ElementZ, FragmentSize,
                                                           cutlass::FloatRoundStyle::round_to_nearest>;
            cutlass::Array<cutlass::bfloat16_t, FragmentSize> z = Convert{}(frg_z);
            // a fragment is FragmentSize consecutive columns of one row: its first and last coordinates say so, and the
            // rest follow by counting
            Tensor c_mn = tCcD(_, _, _, epi_m, epi_n);
            auto c0 = c_mn(epi_v * FragmentSize), c1 = c_mn(epi_v * FragmentSize + FragmentSize - 1);
            const int m = m_origin + (int)get<0>(c0), n0 = n_origin + (int)get<1>(c0);
            bad = bad || get<0>(c1) != get<0>(c0) || (int)get<1>(c1) - (int)get<1>(c0) != FragmentSize - 1;
            if ((int)get<0>(c0) >= (int)get<0>(residue)) return z;   // a row past the problem's last
            if (row < 0) row = m;
            bad = bad || row != m || n0 < head_begin;
            const int n_stop = n_origin + (int)get<1>(residue);      // one past the problem's last column
            const int F = params.F;
            if (n0 + FragmentSize <= n_stop && n0 % F + FragmentSize <= F) {
                // the whole fragment lies within one head: one test, then products only
                if (n0 >= head_end) {
                    flush();
                    head = n0 / F;
                    head_begin = head * F;
                    head_end = head_begin + F;
                    bad = bad || n0 != head_begin;
                    sl = sr = 0.f;
                }
                float a = sl, b = sr;
                CUTLASS_PRAGMA_UNROLL
                for (int i = 0; i < FragmentSize; ++i) {
                    const float zf = static_cast<float>(z[i]);
                    a = fmaf(zf, static_cast<float>(frg_al[i]), a);
                    b = fmaf(zf, static_cast<float>(frg_ar[i]), b);
                }
                sl = a;
                sr = b;
            } else {
                CUTLASS_PRAGMA_UNROLL
                for (int i = 0; i < FragmentSize; ++i) {
                    const int n = n0 + i;
                    if (n < n_stop) {
                        if (n >= head_end) {   // the columns ascend: a new head begins
                            flush();
                            head = n / F;
                            head_begin = head * F;
                            head_end = head_begin + F;
                            bad = bad || n != head_begin;
                            sl = sr = 0.f;
                        }
                        const float zf = static_cast<float>(z[i]);
                        sl = fmaf(zf, static_cast<float>(frg_al[i]), sl);
                        sr = fmaf(zf, static_cast<float>(frg_ar[i]), sr);
                    }
                }
            }
            return z;
        }

        CUTLASS_DEVICE void end() {
            flush();
            if (bad && params.flag) atomicExch(params.flag, 1);
        }
    };

    template <bool ReferenceSrc, class... Args>
    CUTLASS_DEVICE auto get_consumer_store_callbacks(cutlass::epilogue::fusion::ConsumerStoreArgs<Args...> const &args) {
        // origin of this thread's coordinates in the problem = problem extent - residue
        const int m0 = (int)get<0>(args.problem_shape_mnkl) - (int)get<0>(args.residue_tCcD);
        const int n0 = (int)get<1>(args.problem_shape_mnkl) - (int)get<1>(args.residue_tCcD);
        return ConsumerStoreCallbacks<decltype(args.tCcD), decltype(args.residue_tCcD)>(args.tCcD, args.residue_tCcD, m0, n0,
                                                                                         params);
    }
};

using ProjectTile = Shape<_128, _128, _64>;
using ProjectRow = cutlass::epilogue::fusion::Sm90RowBroadcast<0, ProjectTile, float, float, Stride<_0, _1, _0>, 4>;
using ProjectFusion =
    cutlass::epilogue::fusion::Sm90EVT<ProjectVisitor, cutlass::epilogue::fusion::Sm90AccFetch, ProjectRow, ProjectRow>;

// D = (A B) where y != 0, else 0: the backward of a ReLU whose output y (>= 0) is the auxiliary tile (a CUTLASS fusion
// operation: the mask is applied while the accumulators leave tensor memory)
template <class T>
struct ReluMask {
    CUTLASS_HOST_DEVICE T operator()(T g, T y) const { return y > T(0) ? g : T(0); }
};
template <class T, int N>
struct ReluMask<cutlass::Array<T, N>> {
    CUTLASS_HOST_DEVICE cutlass::Array<T, N> operator()(cutlass::Array<T, N> const &g, cutlass::Array<T, N> const &y) const {
        cutlass::Array<T, N> r;
        CUTLASS_PRAGMA_UNROLL
        for (int i = 0; i < N; ++i) r[i] = y[i] > T(0) ? g[i] : T(0);
        return r;
    }
};
using MaskFusion = cutlass::epilogue::fusion::LinCombDeEltAct<cutlass::layout::RowMajor, ReluMask, cutlass::bfloat16_t, float,
                                                              cutlass::bfloat16_t>;

template <class LayoutA, class LayoutB, class ElementOut, class Scheduler, class Fusion = void, bool kEvt = !cute::is_void_v<Fusion>>
struct LinearGemm {
    using ElementA = cutlass::bfloat16_t;
    using ElementB = cutlass::bfloat16_t;
    using ElementAcc = float;
    using LayoutC = cutlass::layout::RowMajor;
    static constexpr int AlignA = 8, AlignB = 8;  // 16 bytes of bf16: what a TMA tile row needs
    static constexpr int AlignC = 16 / sizeof(ElementOut);
    using TileShape = Shape<_128, _128, _64>;
    using ClusterShape = Shape<_1, _1, _1>;
    static constexpr bool kFused = !cute::is_void_v<Fusion>;
    using DefaultFusion = cutlass::epilogue::fusion::LinearCombination<ElementOut, ElementAcc, ElementOut, ElementAcc>;
    using ElementCin = cute::conditional_t<kEvt, void, ElementOut>;   // the visitor epilogue reads no source tile
    using Epilogue = typename cutlass::epilogue::collective::CollectiveBuilder<
        cutlass::arch::Sm100, cutlass::arch::OpClassTensorOp, TileShape, ClusterShape,
        cutlass::epilogue::collective::EpilogueTileAuto, ElementAcc, ElementAcc, ElementCin, LayoutC, AlignC, ElementOut,
        LayoutC, AlignC, cutlass::epilogue::collective::EpilogueScheduleAuto,
        cute::conditional_t<kFused, Fusion, DefaultFusion>>::CollectiveOp;
    using Mainloop = typename cutlass::gemm::collective::CollectiveBuilder<
        cutlass::arch::Sm100, cutlass::arch::OpClassTensorOp, ElementA, LayoutA, AlignA, ElementB, LayoutB, AlignB,
        ElementAcc, TileShape, ClusterShape,
        cutlass::gemm::collective::StageCountAutoCarveout<static_cast<int>(sizeof(typename Epilogue::SharedStorage))>,
        cutlass::gemm::collective::KernelScheduleAuto>::CollectiveOp;
    using Kernel = cutlass::gemm::kernel::GemmUniversal<Shape<int, int, int, int>, Mainloop, Epilogue, Scheduler>;
    using Gemm = cutlass::gemm::device::GemmUniversalAdapter<Kernel>;
    using StrideA = typename Kernel::StrideA;
    using StrideB = typename Kernel::StrideB;
    using StrideC = typename Kernel::StrideC;
    using StrideD = typename Kernel::StrideD;

    // the fused projection: D = A B rounded to bf16, with the visitor's side outputs
    static typename Gemm::Arguments arguments_fused(int M, int N, int K, const void *a, const void *b, void *d,
                                                    const float *a_l, const float *a_r, const ProjectVisitor::Arguments &pv) {
        typename Gemm::Arguments args{
            cutlass::gemm::GemmUniversalMode::kGemm,
            {M, N, K, 1},
            {static_cast<const ElementA *>(a), cutlass::make_cute_packed_stride(StrideA{}, cute::make_shape(M, K, 1)),
             static_cast<const ElementB *>(b), cutlass::make_cute_packed_stride(StrideB{}, cute::make_shape(N, K, 1))},
            {{{}, {a_l, 0.f, {}}, {a_r, 0.f, {}}, pv},   // Sm90EVT arguments: the children's (accumulators, a_l, a_r), then the node's
             nullptr, cutlass::make_cute_packed_stride(StrideC{}, cute::make_shape(M, N, 1)),
             static_cast<ElementOut *>(d), cutlass::make_cute_packed_stride(StrideD{}, cute::make_shape(M, N, 1))}};
        return args;
    }

    static sar_status run_fused(int M, int N, int K, const void *a, const void *b, void *d, const float *a_l, const float *a_r,
                                const ProjectVisitor::Arguments &pv, void *workspace, size_t workspace_bytes_, cudaStream_t st,
                                const char *name) {
        auto args = arguments_fused(M, N, K, a, b, d, a_l, a_r, pv);
        Gemm gemm;
        if (gemm.can_implement(args) != cutlass::Status::kSuccess) return SAR_ERR_UNSUPPORTED;
        const size_t need = Gemm::get_workspace_size(args);
        if (need > 0 && (!workspace || workspace_bytes_ < need || !sar_aligned(workspace, 16))) return SAR_ERR_WORKSPACE;
        if (gemm.initialize(args, workspace, st) != cutlass::Status::kSuccess) return SAR_ERR_CUDA;
        cutlass::Status rc;
        SAR_LAUNCH(name, st, rc = gemm.run(st));
        if (rc != cutlass::Status::kSuccess) return SAR_ERR_CUDA;
        return sar_after_launch();
    }

    // D = mask(A B, y): y [M, N] in the output type, row-major
    static sar_status run_masked(int M, int N, int K, const void *a, const void *b, void *d, const void *y, void *workspace,
                                 size_t workspace_bytes_, cudaStream_t st, const char *name) {
        typename Gemm::Arguments args{
            cutlass::gemm::GemmUniversalMode::kGemm,
            {M, N, K, 1},
            {static_cast<const ElementA *>(a), cutlass::make_cute_packed_stride(StrideA{}, cute::make_shape(M, K, 1)),
             static_cast<const ElementB *>(b), cutlass::make_cute_packed_stride(StrideB{}, cute::make_shape(N, K, 1))},
            {{},
             static_cast<const ElementOut *>(d), cutlass::make_cute_packed_stride(StrideC{}, cute::make_shape(M, N, 1)),
             static_cast<ElementOut *>(d), cutlass::make_cute_packed_stride(StrideD{}, cute::make_shape(M, N, 1))}};
        args.epilogue.thread.alpha = 1.f;
        args.epilogue.thread.beta = 0.f;
        args.epilogue.thread.aux_ptr = static_cast<const ElementOut *>(y);
        args.epilogue.thread.dAux = cutlass::make_cute_packed_stride(StrideC{}, cute::make_shape(M, N, 1));
        Gemm gemm;
        if (gemm.can_implement(args) != cutlass::Status::kSuccess) return SAR_ERR_UNSUPPORTED;
        const size_t need = Gemm::get_workspace_size(args);
        if (need > 0 && (!workspace || workspace_bytes_ < need || !sar_aligned(workspace, 16))) return SAR_ERR_WORKSPACE;
        if (gemm.initialize(args, workspace, st) != cutlass::Status::kSuccess) return SAR_ERR_CUDA;
        cutlass::Status rc;
        SAR_LAUNCH(name, st, rc = gemm.run(st));
        if (rc != cutlass::Status::kSuccess) return SAR_ERR_CUDA;
        return sar_after_launch();
    }

    static typename Gemm::Arguments arguments(int M, int N, int K, const void *a, const void *b, void *d, float beta = 0.f) {
        typename Gemm::Arguments args{
            cutlass::gemm::GemmUniversalMode::kGemm,
            {M, N, K, 1},
            {static_cast<const ElementA *>(a), cutlass::make_cute_packed_stride(StrideA{}, cute::make_shape(M, K, 1)),
             static_cast<const ElementB *>(b), cutlass::make_cute_packed_stride(StrideB{}, cute::make_shape(N, K, 1))},
            {{1.f, beta},  // D = A B + beta D: with beta = 0 the epilogue does not read D
             static_cast<const ElementOut *>(d), cutlass::make_cute_packed_stride(StrideC{}, cute::make_shape(M, N, 1)),
             static_cast<ElementOut *>(d), cutlass::make_cute_packed_stride(StrideD{}, cute::make_shape(M, N, 1))}};
        return args;
    }

    static size_t workspace_bytes(int M, int N, int K) {
        return Gemm::get_workspace_size(arguments(M, N, K, nullptr, nullptr, nullptr));
    }

    static sar_status run(int M, int N, int K, const void *a, const void *b, void *d, void *workspace, size_t workspace_bytes_,
                          cudaStream_t st, const char *name, float beta = 0.f) {
        auto args = arguments(M, N, K, a, b, d, beta);
        Gemm gemm;
        if (gemm.can_implement(args) != cutlass::Status::kSuccess) return SAR_ERR_UNSUPPORTED;
        const size_t need = Gemm::get_workspace_size(args);
        if (need > 0 && (!workspace || workspace_bytes_ < need || !sar_aligned(workspace, 16))) return SAR_ERR_WORKSPACE;
        if (gemm.initialize(args, workspace, st) != cutlass::Status::kSuccess) return SAR_ERR_CUDA;
        cutlass::Status rc;
        SAR_LAUNCH(name, st, rc = gemm.run(st));
        if (rc != cutlass::Status::kSuccess) return SAR_ERR_CUDA;
        return sar_after_launch();
    }
};

using RowMajor = cutlass::layout::RowMajor;
using ColMajor = cutlass::layout::ColumnMajor;
// z[n, d_out] = h[n, d_in] W[d_in, d_out]:  A = h (K contiguous), B = W seen as [K, N] with N contiguous
using GemmForward = LinearGemm<RowMajor, RowMajor, cutlass::bfloat16_t, void>;
// the same with el = <z, a_l>, er = <z, a_r> formed in the epilogue
using GemmForwardProject = LinearGemm<RowMajor, RowMajor, cutlass::bfloat16_t, void, ProjectFusion>;
// dh[n, d_in] = dz[n, d_out] W^T:           A = dz, B[k, n] = W[n, k]: K contiguous
using GemmBwdInput = LinearGemm<RowMajor, ColMajor, cutlass::bfloat16_t, void>;
// the same followed by the backward of the ReLU that produced the layer's input
using GemmBwdInputMasked = LinearGemm<RowMajor, ColMajor, cutlass::bfloat16_t, void, MaskFusion, false>;
// dW[d_in, d_out] = h^T dz, K = n (millions): A[m, k] = h[k, m] (M contiguous), B = dz (N contiguous); the
// K range is cut across the SMs by the stream-K scheduler (one 128x128 output tile would otherwise keep one SM busy)
using GemmBwdWeight = LinearGemm<ColMajor, RowMajor, float, cutlass::gemm::StreamKScheduler>;

static sar_status linear_check(int64_t n, int32_t d_in, int32_t d_out, sar_dtype t, std::initializer_list<const void *> ps) {
    if (n < 0 || d_in < 1 || d_out < 1) return SAR_ERR_INVALID_ARG;
    if (t != SAR_BF16) return SAR_ERR_UNSUPPORTED;
    if (n > INT32_MAX) return SAR_ERR_UNSUPPORTED;
    if ((d_in % 8) || (d_out % 8)) return SAR_ERR_UNSUPPORTED;  // rows of whole 16-byte vectors
    for (const void *p : ps)
        if (!p) return SAR_ERR_INVALID_ARG;
        else if (!sar_aligned(p, 16)) return SAR_ERR_ALIGNMENT;
    return SAR_OK;
}

}  // namespace sarlin

using namespace sarlin;

extern "C" {

size_t sar_linear_workspace_bytes(int64_t n, int32_t d_in, int32_t d_out) {
    if (n < 1 || n > INT32_MAX || d_in < 1 || d_out < 1) return 0;
    size_t a = GemmForward::workspace_bytes((int)n, d_out, d_in);
    const size_t b = GemmBwdInput::workspace_bytes((int)n, d_in, d_out);
    const size_t c = GemmBwdWeight::workspace_bytes(d_in, d_out, (int)n);
    const size_t f = GemmForwardProject::Gemm::get_workspace_size(
        GemmForwardProject::arguments_fused((int)n, d_out, d_in, nullptr, nullptr, nullptr, nullptr, nullptr,
                                            ProjectVisitor::Arguments{}));
    if (f > a) a = f;
    if (b > a) a = b;
    if (c > a) a = c;
    return a + 256;
}

sar_status sar_linear(int64_t n, int32_t d_in, int32_t d_out, sar_dtype t, const void *h, const void *w, void *z,
                      void *workspace, size_t workspace_bytes, void *stream) {
    if (n == 0 && d_in > 0 && d_out > 0) return t == SAR_BF16 ? SAR_OK : SAR_ERR_UNSUPPORTED;
    SAR_TRY(linear_check(n, d_in, d_out, t, {h, w, z}));
    return GemmForward::run((int)n, d_out, d_in, h, w, z, workspace, workspace_bytes, static_cast<cudaStream_t>(stream),
                            "linear");
}

sar_status sar_linear_project(int64_t n, int32_t d_in, int32_t H, int32_t F, sar_dtype t, const void *h, const void *w,
                              const float *a_l, const float *a_r, void *z, float *el, float *er, int32_t *flag,
                              void *workspace, size_t workspace_bytes, void *stream) {
    if (H < 1 || F < 1) return SAR_ERR_INVALID_ARG;
    const int64_t d_out = (int64_t)H * F;
    if (d_out > INT32_MAX) return SAR_ERR_UNSUPPORTED;
    if (n == 0 && d_in > 0) return t == SAR_BF16 ? SAR_OK : SAR_ERR_UNSUPPORTED;
    SAR_TRY(linear_check(n, d_in, (int32_t)d_out, t, {h, w, z, a_l, a_r, el, er}));
    // a thread of the epilogue owns whole heads only if a head's columns do not straddle 128-column tiles
    if (F % 8 != 0 || 128 % F != 0) return SAR_ERR_UNSUPPORTED;
    ProjectVisitor::Arguments pv;
    pv.el = el;
    pv.er = er;
    pv.H = H;
    pv.F = F;
    pv.flag = flag;
    return GemmForwardProject::run_fused((int)n, (int)d_out, d_in, h, w, z, a_l, a_r, pv, workspace, workspace_bytes,
                                         static_cast<cudaStream_t>(stream), "linear_project");
}

sar_status sar_linear_accumulate(int64_t n, int32_t d_in, int32_t d_out, sar_dtype t, const void *h, const void *w, void *z,
                                 void *workspace, size_t workspace_bytes, void *stream) {
    if (n == 0 && d_in > 0 && d_out > 0) return t == SAR_BF16 ? SAR_OK : SAR_ERR_UNSUPPORTED;
    SAR_TRY(linear_check(n, d_in, d_out, t, {h, w, z}));
    return GemmForward::run((int)n, d_out, d_in, h, w, z, workspace, workspace_bytes, static_cast<cudaStream_t>(stream),
                            "linear_accumulate", 1.f);
}

sar_status sar_linear_bwd_input(int64_t n, int32_t d_in, int32_t d_out, sar_dtype t, const void *dz, const void *w,
                                void *dh, void *workspace, size_t workspace_bytes, void *stream) {
    if (n == 0 && d_in > 0 && d_out > 0) return t == SAR_BF16 ? SAR_OK : SAR_ERR_UNSUPPORTED;
    SAR_TRY(linear_check(n, d_in, d_out, t, {dz, w, dh}));
    return GemmBwdInput::run((int)n, d_in, d_out, dz, w, dh, workspace, workspace_bytes, static_cast<cudaStream_t>(stream),
                             "linear_bwd_input");
}

sar_status sar_linear_bwd_input_relu(int64_t n, int32_t d_in, int32_t d_out, sar_dtype t, const void *dz, const void *w,
                                     const void *y, void *dh, void *workspace, size_t workspace_bytes, void *stream) {
    if (n == 0 && d_in > 0 && d_out > 0) return t == SAR_BF16 ? SAR_OK : SAR_ERR_UNSUPPORTED;
    SAR_TRY(linear_check(n, d_in, d_out, t, {dz, w, y, dh}));
    return GemmBwdInputMasked::run_masked((int)n, d_in, d_out, dz, w, dh, y, workspace, workspace_bytes,
                                          static_cast<cudaStream_t>(stream), "linear_bwd_input_relu");
}

sar_status sar_linear_bwd_weight(int64_t n, int32_t d_in, int32_t d_out, sar_dtype t, const void *h, const void *dz,
                                 float *dw, void *workspace, size_t workspace_bytes, void *stream) {
    if (n == 0 && d_in > 0 && d_out > 0) {
        if (t != SAR_BF16) return SAR_ERR_UNSUPPORTED;
        if (!dw) return SAR_ERR_INVALID_ARG;
        return cudaMemsetAsync(dw, 0, (size_t)d_in * d_out * 4, static_cast<cudaStream_t>(stream)) == cudaSuccess ? SAR_OK : SAR_ERR_CUDA;
    }
    SAR_TRY(linear_check(n, d_in, d_out, t, {h, dz, dw}));
    return GemmBwdWeight::run(d_in, d_out, (int)n, h, dz, dw, workspace, workspace_bytes, static_cast<cudaStream_t>(stream),
                              "linear_bwd_weight");
}

}  // extern "C"

// The dense projection z = h W of a layer (Eq. 1 / Eq. 3: z = W h, one row per node) and its backward
// pass: the one dense contraction around the aggregation, run on the 5th-generation tensor cores
// (tcgen05 MMA with accumulators in tensor memory, operands staged by TMA) through CUTLASS's sm100
// collective templates instantiated here; bf16 operands, float32 accumulation.  Contracts are in
// include/sar.h.  Cluster shape 1x1x1: no multicast loads.
#include "sar_common.cuh"

#include "cutlass/cutlass.h"
#include "cutlass/epilogue/collective/collective_builder.hpp"
#include "cutlass/gemm/collective/collective_builder.hpp"
#include "cutlass/gemm/device/gemm_universal_adapter.h"
#include "cutlass/gemm/kernel/gemm_universal.hpp"
#include "cutlass/gemm/kernel/tile_scheduler.hpp"
#include "cutlass/util/packed_stride.hpp"

namespace sarlin {

using namespace cute;

template <class LayoutA, class LayoutB, class ElementOut, class Scheduler>
struct LinearGemm {
    using ElementA = cutlass::bfloat16_t;
    using ElementB = cutlass::bfloat16_t;
    using ElementAcc = float;
    using LayoutC = cutlass::layout::RowMajor;
    static constexpr int AlignA = 8, AlignB = 8;  // 16 bytes of bf16: what a TMA tile row needs
    static constexpr int AlignC = 16 / sizeof(ElementOut);
    using TileShape = Shape<_128, _128, _64>;
    using ClusterShape = Shape<_1, _1, _1>;
    using Epilogue = typename cutlass::epilogue::collective::CollectiveBuilder<
        cutlass::arch::Sm100, cutlass::arch::OpClassTensorOp, TileShape, ClusterShape,
        cutlass::epilogue::collective::EpilogueTileAuto, ElementAcc, ElementAcc, ElementOut, LayoutC, AlignC, ElementOut,
        LayoutC, AlignC, cutlass::epilogue::collective::EpilogueScheduleAuto>::CollectiveOp;
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
// dh[n, d_in] = dz[n, d_out] W^T:           A = dz, B[k, n] = W[n, k]: K contiguous
using GemmBwdInput = LinearGemm<RowMajor, ColMajor, cutlass::bfloat16_t, void>;
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

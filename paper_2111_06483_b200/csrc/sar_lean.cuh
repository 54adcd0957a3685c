// Host-side interface of the lean span kernels (internal): arguments, applicability test and the launchers,
// which are compiled in translation units of their own (sar_lean_*.cu), one per pass and storage type.
// They cover the forward pass and both backward passes of a call that holds the whole graph.
#pragma once

#include "sar_rowkernels.cuh"

namespace sar {

struct LeanArgs {
    long long n_rows;
    const int64_t *indptr;
    const int32_t *indices;
    const void *gather;      // rows fetched per edge: feat
    const void *rowvec;      // row-stationary vector of the backward pass: gout
    const float *el, *er;    // el[row], er[col]
    const float *m, *d;      // bwd-dst: final statistics of the row
    float4 *rec_out;         // bwd-dst: record {el, m, 1/d, D} written per (row, head)
    const float4 *rec_in;    // bwd-dst, partition step: the record written beforehand (D is read from it)
    int first;               // partition step: the state (forward) / del (bwd-dst) starts here, nothing is read
    float *m_out, *d_out;    // forward (a partition step reads the state there and writes it back)
    float *acc_state;        // forward, partition step: running numerator [n_rows, H*F], float32
    void *out;               // forward: out
    float *del;              // bwd-dst
    float slope;
    SplitArgs sp;
    int R;                   // rows per span (<= kMaxSpanRows)
    int relu;                // forward: out = max(out, 0)
};

struct LeanSrcArgs {
    long long n_rows;        // sources
    const int64_t *indptr;   // CSC
    const int32_t *indices;  // destinations
    const void *gather;      // gout
    const void *rowvec;      // feat
    const float *er;         // [n_rows,H]
    const float4 *rec_in;    // [n_dst,H] {el, m, 1/d, D}
    void *out;               // dfeat
    float *der;
    float slope;
    SplitArgs sp;
    int R;
};

constexpr int kLeanCap = 256;   // edges a chunk stages; rows and segments must not exceed it
// A forward partition step takes the lean partition-step kernel when the partition holds fewer than kLeanPartMaxDegree
// edges per row (mostly empty rows: what the kernel is laid out for) or at least kLeanPartMinDenseDegree (a span then
// holds few rows, all or most of them with their numerator staged).  In between - short rows, nearly all with edges,
// 31 of them per span but room for the numerators of 8 - span_kernel is faster.  Per step, partition-step kernel
// against span_kernel: large workload (0.94 edges per row and partition) 3.0 against 6.1 ms, first step 3.1 against
// 5.8 ms, last step 5.1 against 11.1 ms; dense workload (25 edges) 2.38 against 2.64 ms; medium workload (6.3 edges)
// 2.05 against 1.93 ms, last step 2.59 against 2.01 ms.
constexpr int kLeanPartMaxDegree = 2;
constexpr int kLeanPartMinDenseDegree = 16;

// Do the lean kernels cover this shape?  Slope >= 0, heads in groups of four, rows of
// exactly G*V vectors with V <= 2, the vectors of a head a power of two within one lane group, and a long-row
// plan whose threshold fits a chunk (so that no row of the rows launch and no segment exceeds it), and a gathered
// array of n_gathered rows whose 16-byte vectors can be counted in 32 bits (the staged row offsets are 32-bit).
static inline bool lean_shape_applies(const Shape &s, float slope, const sar_split *sp, long long n_gathered) {
    if (!s.fast) return false;
    if (!(slope >= 0.f) || !sp || sp->threshold < 1 || sp->threshold > kLeanCap) return false;
    const int H = s.geom.H, nv = s.geom.n_vec;
    if (H % 4 != 0 || nv != s.G * s.V || s.V > 2 || nv % H != 0) return false;
    const int vph = nv / H;
    if (vph > s.G || (vph & (vph - 1)) != 0) return false;
    if ((unsigned long long)nv * (unsigned long long)(n_gathered > 0 ? n_gathered : 0) > 0xffffffffull) return false;
    return (s.G == 16 && s.V == 1 && H == 4) || (s.G == 32 && s.V == 1 && (H == 4 || H == 8)) ||
           (s.G == 32 && s.V == 2 && H == 4);
}
// ... and is the call one that holds the whole graph (the forward pass and the destination-major pass of a partition
// step have variants of their own; the source-major pass is the same for both, a source lies in one partition)?
static inline bool lean_applies(const Shape &s, unsigned flags, float slope, const sar_split *sp, long long n_gathered) {
    if ((flags & (SAR_FIRST | SAR_LAST | SAR_KEEP_NUMERATOR)) != (SAR_FIRST | SAR_LAST)) return false;
    return lean_shape_applies(s, slope, sp, n_gathered);
}

// Rows launch + segment launch of one pass.
sar_status lean_fwd_f32(const Shape &s, const LeanArgs &a, long long nnz, cudaStream_t st);
sar_status lean_fwd_bf16(const Shape &s, const LeanArgs &a, long long nnz, cudaStream_t st);
sar_status lean_fwd_part_f32(const Shape &s, const LeanArgs &a, long long nnz, cudaStream_t st);
sar_status lean_fwd_part_bf16(const Shape &s, const LeanArgs &a, long long nnz, cudaStream_t st);
sar_status lean_bwd_dst_f32(const Shape &s, const LeanArgs &a, long long nnz, cudaStream_t st);
sar_status lean_bwd_dst_bf16(const Shape &s, const LeanArgs &a, long long nnz, cudaStream_t st);
sar_status lean_bwd_dst_part_f32(const Shape &s, const LeanArgs &a, long long nnz, cudaStream_t st);
sar_status lean_bwd_dst_part_bf16(const Shape &s, const LeanArgs &a, long long nnz, cudaStream_t st);
sar_status lean_bwd_src_f32(const Shape &s, const LeanSrcArgs &a, long long nnz, cudaStream_t st);
sar_status lean_bwd_src_bf16(const Shape &s, const LeanSrcArgs &a, long long nnz, cudaStream_t st);

}  // namespace sar

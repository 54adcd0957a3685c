// Lean span kernels of libsar (internal), shared part: the whole-graph forward pass (sar_lean_fwd_kernels.cuh), the
// destination-major (sar_lean_dst_kernels.cuh) and the source-major (sar_lean_src_kernels.cuh) whole-graph backward
// pass for the common shapes (heads in groups of four, rows of exactly G*V 16-byte vectors), written for the fewest
// issued instructions per edge.
//
// Same plan as span_kernel (sar_span_kernels.cuh) - a warp owns a span of consecutive rows, stages a chunk of whole
// rows in shared memory slot-major and streams the gathered rows through a cp.async ring - with these differences:
//   * The ring works in STAGES of 2 or 4 KB (SPS slots): one commit group and one wait per stage, the slots of a
//     stage walked with compile-time offsets (fully unrolled), the stage refilled as a whole.  The staged column ids
//     are pre-scaled row offsets in 16-byte units, stored per stage with the slot index fastest, so that one
//     16-byte shared load brings the offsets of four consecutive slots; the weights likewise.
//   * The inputs of a stage's scores (16 bytes of er per position and head group, or the 64-byte record of the
//     destination in the source-major pass) are copied into a small ring with the stage's rows, and the weights of a
//     stage are computed just before the stage is consumed, one (position, head) pair per lane: no score phase over
//     the whole chunk, no weight array of the chunk's size, and the gather of the score inputs hides behind the rows.
//   * A row's padding position repeats the row's last column with weight zero, and a chunk's last stage is filled
//     up with repeats: every copy is a real copy of a real row, no predicates, no zero fill.
//   * Everything the control flow depends on (slot counts, row-end masks) is produced by warp votes and reductions,
//     so that the branches around the row epilogues are uniform branches.
//   * Exponentials are one FFMA + EX2; the forward row max uses max_j LeakyReLU(el + er_j) = LeakyReLU(el + max_j er_j)
//     (slope >= 0) and runs online, stage by stage.
//   * Dot products of the backward epilogues are taken on the un-folded accumulators and reduced with three shuffles
//     per quantity; per-(row, head) scalars leave through shared memory, coalesced, once per chunk.
// Preconditions (checked by the host, which otherwise launches span_kernel): SAR_FIRST|SAR_LAST, slope >= 0, every row of
// the rows launch at most CAP edges (a long-row plan with threshold <= CAP), segments of at most CAP edges, fewer
// than 2^32 16-byte vectors in the gathered array.
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
// shared-memory max without a return value: nobody waits for it
__device__ __forceinline__ void red_max_u32(unsigned addr, unsigned v) {
    asm volatile("red.shared.max.u32 [%0], %1;\n" ::"r"(addr), "r"(v) : "memory");
}
// plain 16-byte asynchronous copy (every copy of the lean kernels is a whole, valid vector)
__device__ __forceinline__ void cp_async16_full(unsigned smem_addr, const void *gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(smem_addr), "l"(gsrc) : "memory");
}

constexpr float kLog2e = 1.4426950408889634f;

// ---- launch parameters shared by the three passes --------------------------------------------------------------
// One configuration: chunks of kLeanCap edges, ring of two stages of 2 KB (4 KB for rows of 512 bytes and more), measured
// best on the large workload among stages of 2 / 4 KB, two to four stages, chunks of 128 / 192 / 256 edges.
constexpr int kLeanMinBlocks = 8;
// The rows launches of the two backward passes are compiled for 24 resident blocks per SM (72-78 registers instead of
// 88, no spills): step of the large workload 153.1 -> 147.2 ms.  The same bound on the forward rows launch and on the
// segment launches changes nothing (147.3 ms).
constexpr int kLeanMinBlocksBwdRows = 24;

// Resident blocks per SM the rows launch of a partition step is compiled for.
constexpr int kLeanMinBlocksPart = 16;

static inline int lean_rows_per_span(long long n_rows, long long nnz, int cap, int max_rows = kMaxSpanRows) {
    const double avg = n_rows > 0 ? (double)nnz / (double)n_rows : 0.0;
    int R = avg > 0.5 ? (int)(1.0 * cap / avg + 0.5) : max_rows;
    if (R < 1) R = 1;
    if (R > max_rows) R = max_rows;
    return R;
}

}  // namespace sar

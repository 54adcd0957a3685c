/*
 * libsar — fused graph-attention aggregation with attention rematerialisation for one
 * NVIDIA B200 (sm_100a), after "Sequential Aggregation and Rematerialization" (SAR,
 * arXiv 2111.06483).
 *
 * What the library computes
 *   Forward (Eq. 3 of the paper, fused as Sec. 3.3 describes): for every destination node i
 *   and head h, edge scores e = LeakyReLU(el[i,h] + er[j,h]) over the in-edges j -> i, a softmax
 *   over them and the weighted sum of the neighbours' feature rows, WITHOUT writing the E x H
 *   attention matrix; only the row max m[i,h] and the normaliser d[i,h] are kept.
 *   Sequential aggregation (Sec. 3.2, Algorithm 1, "Stable softmax" in Sec. 3.4): the sources
 *   are split into K partitions that are visited one after the other; the un-normalised
 *   numerator and the normaliser are accumulated separately under a running max, corrected by
 *   exp(old_max - new_max) whenever the max moves, and divided at the end.
 *   Backward (Algorithm 2 with the rematerialisation of Sec. 3.3): the attention is rebuilt from
 *   (el, er, m, d) per partition to produce dFeat, dEl and dEr.
 *   Sum aggregation (Eq. 2, "case 1" of Sec. 3.2), plain, mean or weighted per edge end.
 *   Around the aggregation: graph preparation and message-flow pruning (Appendix B), the dense
 *   projection of a layer and the score projections with their backward passes (Eq. 1, Eq. 3), ReLU,
 *   dropout and batch normalisation over the nodes (Sec. 3.4, Sec. 4.2), the helpers of the relational
 *   layer (Appendix A), and a whole-stack entry point on HOST buffers.
 *
 * Conventions
 *   - Every function returns a sar_status; nothing throws, aborts or prints.
 *   - Unless a parameter is marked HOST, every pointer is a DEVICE pointer BORROWED from the
 *     caller for the duration of the enqueued work; the library never allocates or frees
 *     device memory (except where an entry point documents otherwise) and keeps no state
 *     between calls.  Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is
 *     the default stream) and the call returns without synchronising.
 *   - Argument errors are detected on the host before anything is launched.
 *   - Arrays are dense, row-major, contiguous.  A graph is a CSR by DESTINATION: row i of
 *     (indptr, indices) lists the sources j of the edges j -> i in ascending order, duplicate
 *     edges kept.  indptr is int64, indices int32; every element offset is computed in 64 bits.
 *   - el[i,h] is the DESTINATION term of the score and er[j,h] the SOURCE term (the two halves of
 *     a^T (z_i || z_j) in Eq. 3).
 *   - A destination without in-edges gets out = 0, d = 0, m = -inf and no gradient.  The
 *     derivative of LeakyReLU at 0 is `slope`.  The running max is a constant in the backward
 *     pass (the softmax is shift invariant).
 *   - sar_dtype is the STORAGE type of feat / out / gout / dfeat.  el, er, m, d, D, del, der, the
 *     running numerator `acc` and every accumulation are float32.
 *   - The fast kernels need 16-byte aligned feature arrays and F * sizeof(element) a multiple of
 *     16 bytes; other shapes run on slower scalar kernels with the same results.
 */
#ifndef SAR_H_
#define SAR_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define SAR_API __attribute__((visibility("default")))
#else
#define SAR_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SAR_OK = 0,
    SAR_ERR_INVALID_ARG = -1, /* null pointer, negative size, bad flag combination          */
    SAR_ERR_UNSUPPORTED = -2, /* shape outside what the kernels cover (see SAR_MAX_*)       */
    SAR_ERR_ALIGNMENT = -3,   /* a pointer is not aligned to its element type               */
    SAR_ERR_WORKSPACE = -4,   /* workspace missing or smaller than *_workspace_bytes says   */
    SAR_ERR_CUDA = -5,        /* a CUDA runtime call or launch failed                       */
    SAR_ERR_BAD_GRAPH = -6    /* sar_validate_part found an inconsistent graph              */
} sar_status;

typedef enum { SAR_F32 = 0, SAR_BF16 = 1 } sar_dtype;

/* flags */
#define SAR_FIRST 1u /* first partition: ignore incoming running state / overwrite outputs   */
#define SAR_LAST 2u  /* last partition: normalise and write the final result                 */
#define SAR_MEAN 4u  /* sar_spmm_agg with SAR_LAST: divide by `deg_total`                    */
#define SAR_KEEP_NUMERATOR 8u /* sar_gat_fwd with SAR_LAST: also leave the complete numerator in acc */
#define SAR_RELU_OUT 16u      /* sar_gat_fwd with SAR_LAST: out = max(acc/d, 0), the f_node of Algorithm 1 as a ReLU */

#define SAR_MAX_HEADS 16
#define SAR_MAX_PARTS 64
#define SAR_MAX_ROW_BYTES 4096 /* H*F*sizeof(element) handled by the fast kernels             */

/* Optional split of long rows into segments, built once per graph by sar_plan_count +
 * sar_plan_fill.  Rows
 * with more than `threshold` edges are cut into segments of at most `threshold` edges that
 * are processed in parallel and merged by a second launch (no atomics).  All arrays DEVICE. */
typedef struct {
    int32_t threshold;        /* rows with degree > threshold are split                       */
    int32_t n_long;           /* number of such rows                                          */
    int64_t n_seg;            /* total number of segments over all long rows                  */
    const int32_t *long_row;  /* [n_long]   row ids, ascending                                */
    const int64_t *long_seg;  /* [n_long+1] first segment of each long row                    */
} sar_split;

/* One source partition q of the graph as worker p sees it (the subgraph G_{p,q} of Sec. 3.2).
 * On one GPU p owns every destination, so n_dst is the node count. */
typedef struct {
    int64_t n_dst;             /* destination rows                                            */
    int64_t n_src;             /* sources in this partition                                   */
    int64_t nnz;               /* edges from this partition's sources                         */
    const int64_t *indptr;     /* [n_dst+1] CSR by destination                                */
    const int32_t *indices;    /* [nnz] LOCAL source id in [0,n_src), ascending within a row  */
    const int64_t *t_indptr;   /* [n_src+1] the same edges grouped by local source (CSC);     */
    const int32_t *t_indices;  /* [nnz] destination id, ascending within a source; both may   */
                               /* be NULL when only forward calls are made                    */
    const sar_split *split;    /* HOST pointer or NULL: long-row split of (indptr, indices)   */
    const sar_split *t_split;  /* HOST pointer or NULL: long-row split of the CSC             */
} sar_part;

SAR_API const char *sar_status_string(sar_status s);
/* Compile-time facts: returns the SM architecture the kernels were built for (100). */
SAR_API int32_t sar_built_for_sm(void);

/* Optional observer of the library's kernel launches, for profiling: when set, `hook` is called on
 * the launching host thread right before (phase 0) and right after (phase 1) each kernel launch
 * of the aggregation entry points, with the kernel's name and the stream, so that a caller can
 * record events around individual kernels.  Process-global and not thread-safe; NULL disables
 * it (the default).  The paper has no counterpart; this is measurement plumbing. */
typedef void (*sar_launch_hook_fn)(const char *kernel, int32_t phase, void *stream, void *user);
SAR_API void sar_set_launch_hook(sar_launch_hook_fn hook, void *user);

/* ---------------------------------------------------------------------------------------------
 * Graph preparation (construction of the subgraphs G_{p,q}, Sec. 3.2).  Integer work; results
 * are unique and therefore bit-reproducible.
 * ------------------------------------------------------------------------------------------- */

/* Bytes of scratch the graph-preparation calls below need for a graph of `nnz` edges and `n_rows`
 * rows (an upper bound that covers every one of them). */
SAR_API size_t sar_graph_workspace_bytes(int64_t nnz, int64_t n_rows);

/* Edge list -> CSR.  Edge t goes from column col[t] to row row[t]; output row r lists its
 * columns in ascending order (duplicates adjacent).  For the CSR by destination pass
 * row = dst, col = src; for the CSC pass row = src, col = dst.
 * indptr: [n_rows+1] written; indices: [nnz] written.  Ids must lie in range (not checked). */
SAR_API sar_status sar_csr_from_coo(int64_t n_rows, int64_t n_cols, int64_t nnz, const int32_t *row,
                            const int32_t *col, int64_t *indptr, int32_t *indices, void *workspace,
                            size_t workspace_bytes, void *stream);

/* CSR (n_rows x n_cols) -> its transpose (n_cols x n_rows), same ordering rule. */
SAR_API sar_status sar_csr_transpose(int64_t n_rows, int64_t n_cols, const int64_t *indptr, const int32_t *indices,
                             int64_t *t_indptr, int32_t *t_indices, void *workspace, size_t workspace_bytes,
                             void *stream);

/* Contiguous source ranges s_q = floor(q*n/k); bounds is a HOST array of k+1 entries. */
SAR_API sar_status sar_partition_bounds(int64_t n, int32_t k, int64_t *bounds);

/* Split a CSR by source range in two steps (the caller sizes the index array in between).
 * Step 1 writes indptr_all: k arrays of n_dst+1 entries, array q being the indptr of the
 * sub-graph that keeps only sources bounds[q] <= j < bounds[q+1] (HOST bounds, k <= SAR_MAX_PARTS).
 * The caller then reads nnz_q = indptr_all[q*(n_dst+1) + n_dst], forms the HOST prefix sums
 * nnz_off[0..k] and calls step 2, which writes partition q's LOCAL ids j - bounds[q] to
 * indices_all[nnz_off[q] .. nnz_off[q+1]). */
SAR_API sar_status sar_csr_split_indptr(int64_t n_dst, const int64_t *indptr, const int32_t *indices, int32_t k,
                                const int64_t *bounds, int64_t *indptr_all, void *workspace,
                                size_t workspace_bytes, void *stream);
SAR_API sar_status sar_csr_split_indices(int64_t n_dst, const int64_t *indptr, const int32_t *indices, int32_t k,
                                 const int64_t *bounds, const int64_t *indptr_all, const int64_t *nnz_off,
                                 int32_t *indices_all, void *stream);

/* The CSC (edges grouped by source) of partition q: because the sources bounds[q] <= j < bounds[q+1] are
 * consecutive rows of the whole graph's CSC, the partition's destination ids are the slice
 * t_indices[t_indptr[s0] .. t_indptr[s1]) of the whole array as it stands, and its offsets are
 * t_indptr[s0..s1] counted from t_indptr[s0].  This call writes those s1 - s0 + 1 offsets to t_indptr_q
 * (DEVICE arrays; s0 = bounds[q], s1 = bounds[q+1]). */
SAR_API sar_status sar_csc_slice_indptr(int64_t s0, int64_t s1, const int64_t *t_indptr, int64_t *t_indptr_q,
                                        void *stream);

/* Node order for locality (no counterpart in the paper's algorithms; the paper prepares its graphs offline with a
 * graph partitioner, Sec. 4.2, so that a worker's rows mostly gather their own features - this is what a single GPU
 * can do in that step for an input whose node ids carry no locality).  Nodes are numbered by total degree (edges
 * as a source + edges as a destination), descending, ties by ascending id: frequently gathered rows become
 * neighbours, and the rows a span of the kernels owns have similar lengths.  Integer work, results unique.
 *
 * sar_degree_order: src, dst are the DEVICE edge list (e entries each, ids in [0, n)); writes order[n] (new id ->
 *   old id) and rank[n] (old id -> new id), DEVICE arrays.  workspace: DEVICE, 256-byte aligned, at least
 *   sar_degree_order_workspace_bytes(n) bytes, else SAR_ERR_WORKSPACE.
 * sar_relabel: out[t] = rank[ids[t]] for t < e (out may equal ids).  The relabelled edge list then goes through
 *   sar_csr_from_coo as usual.
 * sar_permute_rows: out row i = in row index[i], n rows of row_bytes bytes, DEVICE arrays, in != out.  With
 *   index = order it carries a node array into the new numbering, with index = rank it carries one back.
 * All three enqueue on `stream` and return without synchronising; nothing is allocated. */
SAR_API size_t sar_degree_order_workspace_bytes(int64_t n);
SAR_API sar_status sar_degree_order(int64_t n, int64_t e, const int32_t *src, const int32_t *dst, int32_t *order,
                                    int32_t *rank, void *workspace, size_t workspace_bytes, void *stream);
SAR_API sar_status sar_relabel(int64_t e, const int32_t *ids, const int32_t *rank, int32_t *out, void *stream);
SAR_API sar_status sar_permute_rows(int64_t n, int64_t row_bytes, const int32_t *index, const void *in, void *out,
                                    void *stream);

/* Message-flow pruning (Appendix B: with few labelled nodes, a layer only has to update the nodes that can
 * still influence a labelled node's output).  Both masks are DEVICE arrays of n bytes (0 / non-zero).
 *
 * sar_mfg_frontier: need_out marks the rows whose output of a layer is needed; need_in (written) marks the
 * nodes whose INPUT to that layer is then needed: every needed row itself (its own features enter its
 * score term el) and every source of one of its in-edges.  Apply it layer by layer from the labelled set
 * backwards: need_out of layer l-1 = need_in of layer l.  The graph is the CSR by destination with n rows
 * and n columns.
 *
 * sar_csr_filter_rows_*: the CSR in which only the rows with keep[i] != 0 keep their edges (the others
 * become empty, so the aggregation kernels write zeros for them at no gather cost).  Two steps like the
 * partition split: step 1 writes indptr_out [n+1] (scratch: sar_graph_workspace_bytes(0, n) bytes); the
 * caller reads nnz_out = indptr_out[n], sizes indices_out, and step 2 copies the kept rows' column ids in
 * their original order.  Integer work, bit-exact. */
SAR_API sar_status sar_mfg_frontier(int64_t n, const int64_t *indptr, const int32_t *indices,
                                    const uint8_t *need_out, uint8_t *need_in, void *stream);
SAR_API sar_status sar_csr_filter_rows_indptr(int64_t n, const int64_t *indptr, const uint8_t *keep,
                                              int64_t *indptr_out, void *workspace, size_t workspace_bytes,
                                              void *stream);
SAR_API sar_status sar_csr_filter_rows_indices(int64_t n, const int64_t *indptr, const int32_t *indices,
                                               const int64_t *indptr_out, int32_t *indices_out, void *stream);

/* Debug scan of one partition: indptr monotone from 0 to nnz, ids in range and ascending within a
 * row (both orientations when the CSC is present).  `flag` is 4 bytes of DEVICE scratch.
 * Synchronises the stream.  The hot calls never scan the graph. */
SAR_API sar_status sar_validate_part(const sar_part *g, int32_t *flag, void *stream);

/* Long-row plan (see sar_split).  Step 1 counts the rows with more than `threshold` edges and their
 * segments into the HOST variables n_long / n_seg, using 16 bytes of DEVICE scratch `counts`
 * (synchronises the stream).  Step 2 fills the DEVICE arrays long_row[n_long], long_seg[n_long+1]. */
SAR_API sar_status sar_plan_count(int64_t n_rows, const int64_t *indptr, int32_t threshold, int64_t *counts,
                          int32_t *n_long, int64_t *n_seg, void *stream);
SAR_API sar_status sar_plan_fill(int64_t n_rows, const int64_t *indptr, int32_t threshold, int32_t n_long,
                         int32_t *long_row, int64_t *long_seg, void *workspace, size_t workspace_bytes,
                         void *stream);

/* ---------------------------------------------------------------------------------------------
 * Fused GAT aggregation, forward (Eq. 3; Algorithm 1; Sec. 3.3; running max of Sec. 3.4).
 * ------------------------------------------------------------------------------------------- */

/* Scratch bytes the forward / backward calls need for this partition (long-row partials and, for
 * the backward pass, 16 bytes per (destination, head)). */
SAR_API size_t sar_gat_workspace_bytes(const sar_part *g, int32_t H, int32_t F, sar_dtype t);

/* One step of Algorithm 1's loop: fold partition q into the running state.
 *   feat_q [n_src,H,F] (storage type t), el [n_dst,H], er_q [n_src,H].
 *   acc [n_dst,H,F] float32 running numerator, m [n_dst,H] running max, d [n_dst,H] running
 *   normaliser: read unless SAR_FIRST, written unless SAR_LAST (m, d are always written; after a call with
 *   SAR_LAST and without SAR_KEEP_NUMERATOR the contents of acc are unspecified: the call may or may not have
 *   completed the numerator there before dividing).
 *   With SAR_LAST, out [n_dst,H,F] (type t) = acc/d is written (0 where d == 0) and m, d hold the
 *   final statistics the backward pass needs.  With SAR_FIRST|SAR_LAST (one partition holding all
 *   sources) acc may be NULL: the numerator never leaves the registers.
 *   SAR_KEEP_NUMERATOR together with SAR_LAST also writes the complete float32 numerator to acc (which
 *   must then be given), for sar_gat_bwd_prepare's acc_is_numerator mode: the row dot of the
 *   per-partition backward pass is then formed from float32 values instead of a rounded bf16 out.
 *   SAR_RELU_OUT together with SAR_LAST writes out = max(acc/d, 0) (NaN -> 0): the ReLU that closes the layer
 *   (Algorithm 1 applies f_node to the finished aggregate) without a pass of its own; m, d and a kept
 *   numerator are those of the aggregate before the ReLU.
 *   Destinations without edges in this partition are skipped unless a flag forces a write. */
SAR_API sar_status sar_gat_fwd(const sar_part *g, const void *feat_q, const float *el, const float *er_q, int32_t H,
                       int32_t F, sar_dtype t, float slope, uint32_t flags, float *acc, float *m, float *d,
                       void *out, void *workspace, size_t workspace_bytes, void *stream);

/* The whole loop of Algorithm 1 in one walk, row-stationary: `g` is the UN-split graph (global source ids,
 * n_src = all sources) and partition q owns the sources bounds[q] <= j < bounds[q+1] (HOST array of k+1
 * entries, bounds[0] = 0, bounds[k] = n_src, non-decreasing; k <= SAR_MAX_PARTS).  The partitions must be the
 * slices of ONE array each: feat [n_src,H,F] and er [n_src,H] hold partition q's rows at rows bounds[q] ..
 * bounds[q+1].  Each destination walks its in-edges in ascending source order, i.e. partition after partition,
 * carrying (running max, normaliser, numerator) in registers, so nothing of size n_dst*H*F is written or re-read
 * between partitions and the kernels see one partition; k and bounds only describe where the partitions lie
 * (they are checked, and a caller whose partitions live in separately allocated buffers uses the call-by-call
 * sar_gat_fwd instead).  Writes out, m, d as sar_gat_fwd does with SAR_FIRST | SAR_LAST. */
SAR_API sar_status sar_gat_fwd_fused(const sar_part *g, int32_t k, const int64_t *bounds, const void *feat,
                             const float *el, const float *er, int32_t H, int32_t F, sar_dtype t,
                             float slope, float *m, float *d, void *out, void *workspace,
                             size_t workspace_bytes, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Fused GAT aggregation, backward (Algorithm 2 restricted to the aggregation; attention rebuilt
 * from (el, er, m, d) as Sec. 3.3 describes).  With alpha = exp(e - m)/d, dalpha = <gout_i, feat_j>,
 * D_i = sum_j alpha*dalpha (= <gout_i, out_i>), ds = alpha*(dalpha - D_i)*LeakyReLU'(s):
 *   dfeat[j] = sum_i alpha*gout[i],  der[j] = sum_i ds,  del[i] = sum_j ds.
 * ------------------------------------------------------------------------------------------- */

/* Row dot D[i,h] = <gout[i,h,:], out[i,h,:]> and the packed per-destination record
 * {el, m, 1/d, D} (16 bytes per (i,h), written to the start of `workspace`) that lets each
 * partition's backward step run independently of the others.  `out` may be given as the COMPLETE float32
 * numerator with acc_is_numerator != 0 (then out = acc/d is formed on the fly), which avoids the
 * rounding of a bf16 `out`; the forward call of the last partition leaves the complete numerator in
 * `acc` when it is given SAR_KEEP_NUMERATOR.  D may be NULL. */
SAR_API sar_status sar_gat_bwd_prepare(int64_t n_dst, int32_t H, int32_t F, sar_dtype t, const void *out_or_acc,
                               int32_t acc_is_numerator, const void *gout, const float *el, const float *m,
                               const float *d, float *D, void *workspace, size_t workspace_bytes,
                               void *stream);

/* One step of Algorithm 2's loop for partition q.  m, d are the FINAL statistics.
 *   dfeat_q [n_src,H,F] (type t) and der_q [n_src,H] are written (this partition's sources receive
 *   all their gradient here, since every destination is local); del [n_dst,H] is written with
 *   SAR_FIRST and accumulated otherwise.
 *   With SAR_FIRST|SAR_LAST (one partition holding all sources) D is rebuilt from the edges and
 *   sar_gat_bwd_prepare is not needed; otherwise `workspace` must hold what sar_gat_bwd_prepare
 *   wrote for these (gout, m, d).  Needs g->t_indptr / g->t_indices. */
SAR_API sar_status sar_gat_bwd(const sar_part *g, const void *feat_q, const float *el, const float *er_q,
                       const float *m, const float *d, const void *gout, int32_t H, int32_t F, sar_dtype t,
                       float slope, uint32_t flags, void *dfeat_q, float *del, float *der_q, void *workspace,
                       size_t workspace_bytes, void *stream);

/* The whole loop of Algorithm 2 on the un-split graph (see sar_gat_fwd_fused for the argument conventions):
 * dfeat [n_src,H,F] and der [n_src,H] receive every partition's gradients at its rows. */
SAR_API sar_status sar_gat_bwd_fused(const sar_part *g, int32_t k, const int64_t *bounds, const void *feat,
                             const float *el, const float *er, const float *m, const float *d,
                             const void *gout, int32_t H, int32_t F, sar_dtype t, float slope,
                             void *dfeat, float *del, float *der, void *workspace,
                             size_t workspace_bytes, void *stream);

/* ---------------------------------------------------------------------------------------------
 * The non-rematerialising baseline (Sec. 4.1 compares the fused kernels with the usual two-step implementation
 * that materialises the attention coefficients; Sec. 3.3 describes what fusing avoids).  A deliberately plain
 * variant of the same layer for MEASUREMENT AND TESTS ONLY, so that the memory and time of keeping O(E*H)
 * attention can be observed next to the rematerialising path: the forward call writes alpha [nnz,H] float32
 * (CSR order: row t*H.. belongs to edge t of g->indices) and then forms out from it; the backward call reads
 * alpha back, writes the per-edge score gradients to its scratch and reduces them to del, der and dfeat.
 * `g` is one partition holding all sources, with its CSC; nnz < 2^31 for the backward call.  One warp per
 * row, no tuning, no long-row handling.  Scratch of the backward call: sar_gat_storing_workspace_bytes
 * (4 bytes per (edge, head) plus 4 bytes per edge), 16-byte aligned.  Errors as for sar_gat_fwd / sar_gat_bwd.
 * ------------------------------------------------------------------------------------------- */
SAR_API size_t sar_gat_storing_workspace_bytes(const sar_part *g, int32_t H);
SAR_API sar_status sar_gat_fwd_storing(const sar_part *g, const void *feat, const float *el, const float *er,
                                       int32_t H, int32_t F, sar_dtype t, float slope, float *alpha, void *out,
                                       void *stream);
SAR_API sar_status sar_gat_bwd_storing(const sar_part *g, const void *feat, const float *el, const float *er,
                                       const float *alpha, const void *gout, int32_t H, int32_t F, sar_dtype t,
                                       float slope, void *dfeat, float *del, float *der, void *workspace,
                                       size_t workspace_bytes, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Sum aggregation (Eq. 2; Sec. 3.2 "case 1").  out[i,:] (+)= sum over this partition's in-edges of
 * feat_q[j,:]; feat_q [n_src,F], out [n_dst,F], both of type t, float32 accumulation within the
 * call.  SAR_FIRST overwrites out, otherwise the partition's sum is added to it.  Between
 * calls the running sum lives in `out` itself, i.e. in the storage type: with bf16 storage a sum over K partitions is
 * rounded K times (half a bf16 ulp of the running sum each), a sum over one partition once.  SAR_MEAN with
 * SAR_LAST divides the result by deg_total[i] (int64 [n_dst] total in-degree over all partitions;
 * rows with degree 0 stay 0).  The backward pass of the sum is this same call on the transposed
 * partition applied to gout. */
SAR_API sar_status sar_spmm_agg(const sar_part *g, const void *feat_q, int32_t F, sar_dtype t, uint32_t flags,
                        const int64_t *deg_total, void *out, void *workspace, size_t workspace_bytes,
                        void *stream);
SAR_API size_t sar_spmm_workspace_bytes(const sar_part *g, int32_t F, sar_dtype t);

/* Weighted sum aggregation: out[i,:] (+)= dst_scale[i] * sum over this partition's in-edges of
 * src_scale[j] * feat_q[j,:] - the propagation step X <- S X with S = diag(dst_scale) A diag(src_scale),
 * e.g. the symmetrically normalised adjacency (both scales = degree^-1/2) of the label-propagation
 * post-processing the paper combines SAR with (Sec. 4.2).  src_scale [n_src] and dst_scale [n_dst] are
 * float32 DEVICE arrays; either may be NULL (= all ones).  The factors are applied on the fly, nothing of
 * size E is stored.  SAR_FIRST overwrites out, otherwise the partition's weighted sum is added; SAR_MEAN is
 * not accepted (SAR_ERR_INVALID_ARG).  Workspace and other conventions as for sar_spmm_agg.  The backward
 * pass is this call on the transposed partition with the two scale arrays exchanged. */
SAR_API sar_status sar_spmm_agg_scaled(const sar_part *g, const void *feat_q, int32_t F, sar_dtype t, uint32_t flags,
                                       const float *src_scale, const float *dst_scale, void *out, void *workspace,
                                       size_t workspace_bytes, void *stream);

/* ---------------------------------------------------------------------------------------------
 * The rest of a GAT layer around the aggregation (Eq. 3; Eq. 1's f_node reduced to a ReLU).
 *   sar_gat_project      el[i,h] = <z[i,h,:], a_l[h,:]>, er[i,h] = <z[i,h,:], a_r[h,:]>: the two halves of
 *                        a^T (z_i || z_j) in Eq. 3.  z [n,H,F] (type t); a_l, a_r [H,F] float32.
 *   sar_gat_project_bwd  chain rule through the projection: dz[i,h,:] += a_l[h,:]*del[i,h] + a_r[h,:]*der[i,h]
 *                        (dz is the dfeat the aggregation's backward pass wrote, updated in place) and
 *                        da_l[h,:] = sum_i del[i,h]*z[i,h,:], da_r likewise (written; fixed summation order,
 *                        no atomics).  Needs sar_gat_project_workspace_bytes(H, F) bytes of scratch.
 *   sar_relu             x = max(x, 0) in place (NaN -> 0).   sar_relu_bwd: g = 0 where y <= 0, y being the
 *                        layer's output after the ReLU.
 * flags = SAR_GLUE_RELU folds the ReLU that closes the previous layer into these two calls, saving its own
 * pass over the node features: sar_gat_project then first writes z = max(z, 0) in place (the only case in
 * which it writes z) and projects the result; sar_gat_project_bwd, after the update of dz, zeroes dz where
 * z <= 0 (what sar_relu_bwd(z, dz) would do).  Any other flag bit: SAR_ERR_INVALID_ARG.
 * All pointers are DEVICE memory owned by the caller.  n = 0 is allowed (node buffers may then be NULL;
 * da_l, da_r are still written, as zeros).  Rows whose head slice F*sizeof(t) is a multiple of 16 bytes
 * with 16-byte aligned z / dz take the vector kernels, everything else a scalar path.
 * Errors: SAR_ERR_INVALID_ARG (NULL pointer with n > 0, H or F < 1, unknown t), SAR_ERR_ALIGNMENT
 * (float arrays not 4-byte aligned), SAR_ERR_WORKSPACE (scratch missing, misaligned or too small).
 * ------------------------------------------------------------------------------------------- */
SAR_API size_t sar_gat_project_workspace_bytes(int32_t H, int32_t F);
#define SAR_GLUE_RELU 1u
#define SAR_GLUE_DROPOUT 2u /* only for the sar_bn_*_act calls */
SAR_API sar_status sar_gat_project(int64_t n, int32_t H, int32_t F, sar_dtype t, void *z, const float *a_l,
                                   const float *a_r, float *el, float *er, uint32_t flags, void *stream);
SAR_API sar_status sar_gat_project_bwd(int64_t n, int32_t H, int32_t F, sar_dtype t, const void *z, const float *a_l,
                                       const float *a_r, const float *del, const float *der, void *dz, float *da_l,
                                       float *da_r, uint32_t flags, void *workspace, size_t workspace_bytes,
                                       void *stream);
SAR_API sar_status sar_relu(int64_t n_elems, sar_dtype t, void *x, void *stream);
/* Dropout between layers (Sec. 4.2: "batch normalization and dropout between all layers"), counter-based so
 * that nothing is kept for the backward pass: element i is KEPT (and multiplied by 1/(1-p)) when the top
 * 24 bits of the (i+1)-th output of SplitMix64 started at `seed` (z = seed + (i+1)*0x9E3779B97F4A7C15, then
 * the generator's two multiply-xorshift rounds) are >= floor(p * 2^24); otherwise y[i] = 0.  0 <= p < 1.
 * y may be x.  The backward pass is the same call on the upstream gradient with the same seed and p. */
SAR_API sar_status sar_dropout(int64_t n_elems, sar_dtype t, const void *x, float p, uint64_t seed, void *y,
                               void *stream);
SAR_API sar_status sar_relu_bwd(int64_t n_elems, sar_dtype t, const void *y, void *g, void *stream);
/* y = a*x + b*y element-wise (float32 arithmetic; x, y of type t, n_elems each, DEVICE memory, x != y): the mixing
 * step of an iterated propagation X <- (1-alpha) X0 + alpha S X (Sec. 4.2: label-propagation post-processing), whose
 * product S X is sar_spmm_agg_scaled. */
SAR_API sar_status sar_axpby(int64_t n_elems, sar_dtype t, float a, const void *x, float b, void *y, void *stream);
/* The sum of the error contributions a worker receives for its own rows (Algorithm 2: every other worker returns the
 * error of this worker's features with respect to its part of the output).
 *   sar_accumulate  acc[i] += x[i], or acc[i] = x[i] with flags = SAR_FIRST; x of type t, acc float32 (the sum of K
 *                   terms is formed in float32 whatever the storage type), n_elems each, DEVICE memory.
 *   sar_round_to    y[i] = acc[i] rounded to type t. */
SAR_API sar_status sar_accumulate(int64_t n_elems, sar_dtype t, const void *x, float *acc, uint32_t flags, void *stream);
SAR_API sar_status sar_round_to(int64_t n_elems, sar_dtype t, const float *acc, void *y, void *stream);

/* ---------------------------------------------------------------------------------------------
 * The dense projection of a layer, z = h W (Eq. 1 / Eq. 3 apply a weight matrix to every node's features
 * before the aggregation), and its backward pass: the one dense contraction around the aggregation.  It
 * runs on the tensor cores (tcgen05 MMA, accumulators in tensor memory, operands staged by TMA; CUTLASS
 * sm100 collectives instantiated in the library), bf16 operands with float32 accumulation.
 *   sar_linear             z[n, d_out]  = h[n, d_in] W[d_in, d_out]          (bf16 out)
 *   sar_linear_accumulate  z[n, d_out] += h[n, d_in] W[d_in, d_out]          (z read and written, bf16: the sum
 *                          over relations of Appendix A's layer, one call per relation)
 *   sar_linear_project     z = h W as sar_linear with d_out = H F, and in the same kernel the two halves of Eq. 3's
 *                          a^T (z_i || z_j): el[i,h] = <z[i,h,:], a_l[h,:]>, er[i,h] = <z[i,h,:], a_r[h,:]> taken of
 *                          the bf16-rounded z while the accumulator tile leaves tensor memory (what sar_linear
 *                          followed by sar_gat_project computes, without reading z back).  a_l, a_r [H,F] and el, er
 *                          [n,H] float32.  F must be a multiple of 8 that divides 128 (a head may not straddle the
 *                          128-column tiles), else SAR_ERR_UNSUPPORTED.  flag (DEVICE int, may be NULL) is set to 1
 *                          if the epilogue's thread layout does not give every row to one thread (el, er are then
 *                          not written for the rows concerned); the library's tests check that it stays 0.
 *   sar_linear_bwd_input   dh[n, d_in]  = dz[n, d_out] W^T                   (bf16 out)
 *   sar_linear_bwd_input_relu  the same followed by the backward of the ReLU that produced the layer's input h:
 *                          dh[i, c] = 0 where y[i, c] <= 0, y [n, d_in] (bf16) being that ReLU's output (= h); the
 *                          mask is applied in the GEMM's epilogue (what sar_relu_bwd(y, dh) would do in a pass of
 *                          its own)
 *   sar_linear_bwd_weight  dw[d_in, d_out] = h^T dz                          (float32 out; the n-long
 *                          contraction is cut across the SMs and the partial tiles are reduced in the scratch)
 * All arrays row-major DEVICE memory, 16-byte aligned; t must be SAR_BF16 and d_in, d_out multiples of 8
 * (SAR_ERR_UNSUPPORTED otherwise); n <= 2^31-1.  Scratch: sar_linear_workspace_bytes(n, d_in, d_out) covers
 * all of these calls.  n = 0 is allowed (dw is then written as zeros).
 * ------------------------------------------------------------------------------------------- */
SAR_API size_t sar_linear_workspace_bytes(int64_t n, int32_t d_in, int32_t d_out);
SAR_API sar_status sar_linear_bwd_input_relu(int64_t n, int32_t d_in, int32_t d_out, sar_dtype t, const void *dz,
                                             const void *w, const void *y, void *dh, void *workspace,
                                             size_t workspace_bytes, void *stream);
SAR_API sar_status sar_linear_project(int64_t n, int32_t d_in, int32_t H, int32_t F, sar_dtype t, const void *h,
                                      const void *w, const float *a_l, const float *a_r, void *z, float *el, float *er,
                                      int32_t *flag, void *workspace, size_t workspace_bytes, void *stream);
SAR_API sar_status sar_linear(int64_t n, int32_t d_in, int32_t d_out, sar_dtype t, const void *h, const void *w,
                              void *z, void *workspace, size_t workspace_bytes, void *stream);
SAR_API sar_status sar_linear_accumulate(int64_t n, int32_t d_in, int32_t d_out, sar_dtype t, const void *h,
                                         const void *w, void *z, void *workspace, size_t workspace_bytes,
                                         void *stream);
SAR_API sar_status sar_linear_bwd_input(int64_t n, int32_t d_in, int32_t d_out, sar_dtype t, const void *dz,
                                        const void *w, void *dh, void *workspace, size_t workspace_bytes,
                                        void *stream);
SAR_API sar_status sar_linear_bwd_weight(int64_t n, int32_t d_in, int32_t d_out, sar_dtype t, const void *h,
                                         const void *dz, float *dw, void *workspace, size_t workspace_bytes,
                                         void *stream);

/* ---------------------------------------------------------------------------------------------
 * Relational layer (Appendix A): h'_i = sigma( sum_r sum_{j in N^r_i} W_r h_j / |N^r_i| ), one graph per
 * relation r.  The layer is a sequence of calls of this library, per relation: the mean aggregation of h over
 * the relation's graph (sar_spmm_agg with SAR_MEAN, partition by partition), then z += agg_r W_r
 * (sar_linear / sar_linear_accumulate).  Backward, per relation: the aggregate is rebuilt from h (the
 * input features are needed again, as the appendix notes - nothing of size R x n is kept), dW_r = agg_r^T dz
 * (sar_linear_bwd_weight), dagg_r = dz W_r^T (sar_linear_bwd_input), and dh (+)= the sum over the relation's
 * out-edges of dagg_r[i] / |N^r_i| (sar_spmm_agg_scaled on the transposed partition with src_scale from
 * sar_degree_scale).  The two helpers below are what is not covered by those calls.
 *   sar_degree_scale    scale[i] = deg(i)^power with deg(i) = indptr[i+1] - indptr[i], 0 where deg(i) = 0;
 *                       power <= 0 (-1: the mean's factor, -0.5: the symmetric normalisation of Sec. 4.2's
 *                       propagation).  indptr [n+1] int64, scale [n] float32.
 *   sar_rgcn_basis      W[r,:] = sum_b a[r,b] V[b,:] (the appendix's second equation): a [R,B], V [B,size]
 *                       float32, W [R,size] of type t (bf16 for the contraction), size = d_in*d_out.
 *   sar_rgcn_basis_bwd  da[r,b] = <dW[r,:], V[b,:]>, dV[b,:] = sum_r a[r,b] dW[r,:]; all float32, written.
 * All pointers DEVICE memory owned by the caller; n = 0 / size = 0 allowed.
 * ------------------------------------------------------------------------------------------- */
SAR_API sar_status sar_degree_scale(int64_t n, const int64_t *indptr, float power, float *scale, void *stream);
SAR_API sar_status sar_rgcn_basis(int32_t R, int32_t B, int64_t size, sar_dtype t, const float *a, const float *V,
                                  void *W, void *stream);
SAR_API sar_status sar_rgcn_basis_bwd(int32_t R, int32_t B, int64_t size, const float *a, const float *V,
                                      const float *dW, float *da, float *dV, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Batch normalisation over the node dimension (Sec. 3.4, "Batch normalization"): y[i,c] =
 * (x[i,c] - mean[c]) * rstd[c] * gamma[c] + beta[c] with mean and variance taken over ALL rows of
 * x [n, C] (type t).  A worker that holds only some of the rows computes LOCAL statistics, combines them
 * with the other workers' (a few floats per column: that is all that is communicated), and applies the
 * global ones; the entry points are split accordingly.  All arrays are DEVICE memory; [C] arrays are
 * float32; gamma / beta may be NULL (1 / 0); y may be x, gx may be gy.  Scratch for the two *_stats
 * calls: sar_bn_workspace_bytes(C).  Sums are formed in a fixed order (no atomics), block partials are
 * added in float64.
 *   sar_bn_stats      mean[c] = (1/n) sum_i x[i,c] and m2[c] = sum_i (x[i,c] - mean[c])^2 of the n local rows
 *                     (two passes, no cancellation).  Workers combine (n, mean, m2) triples by the pairwise
 *                     rule mean = sum n_r mean_r / N, m2 = sum [m2_r + n_r (mean_r - mean)^2]; the variance
 *                     is m2 / N and rstd = 1 / sqrt(variance + eps).
 *   sar_bn_rstd       rstd[c] = 1 / sqrt(m2[c] / count + eps) from the (global) m2 and row count.
 *   sar_bn_apply      the normalisation with given (global) mean and rstd.
 *   sar_bn_bwd_stats  sum_gy[c] = sum_i gy[i,c] (= d beta) and sum_gy_xhat[c] = sum_i gy[i,c] * xhat[i,c]
 *                     (= d gamma) over the local rows, xhat = (x - mean) * rstd; workers add these up.
 *   sar_bn_bwd_apply  gx = gamma * rstd * (gy - sum_gy * inv_count - xhat * sum_gy_xhat * inv_count) with
 *                     the GLOBAL sums and inv_count = 1 / N, N the global row count: the gradients through
 *                     the mean and the variance, scaled by the number of rows everywhere, as the paper
 *                     requires of the distributed backward pass.
 * n = 0 is allowed (statistics and sums are written as zeros).  Errors as for the other streaming calls.
 * ------------------------------------------------------------------------------------------- */
SAR_API size_t sar_bn_workspace_bytes(int32_t C);
/* The combination rule across R workers (Sec. 3.4, "Batch normalization"), on HOST arrays: what is communicated
 * is a few floats per column, so the workers gather each other's triples with whatever transport they use and
 * every worker evaluates the same rule in the same (rank) order, in float64.
 *   sar_bn_combine_moments  n_r [R], mean_r [R,C], m2_r [R,C] (row r = worker r's local statistics from
 *                           sar_bn_stats) -> *n_all = sum n_r, mean[c] = sum_r n_r mean_r / n_all,
 *                           m2[c] = sum_r [ m2_r + n_r (mean_r - mean)^2 ]  (all rows of all workers).
 *   sar_bn_combine_sums     sums_r [R,count] -> sums[i] = sum_r sums_r[r,i] (the backward statistics).
 * No device work, no stream.  Errors: SAR_ERR_INVALID_ARG (R < 1, negative counts, NULL arrays). */
SAR_API sar_status sar_bn_combine_moments(int32_t R, int32_t C, const int64_t *n_r, const float *mean_r,
                                          const float *m2_r, int64_t *n_all, float *mean, float *m2);
SAR_API sar_status sar_bn_combine_sums(int32_t R, int64_t count, const float *sums_r, float *sums);
SAR_API sar_status sar_bn_stats(int64_t n, int32_t C, sar_dtype t, const void *x, float *mean, float *m2,
                                void *workspace, size_t workspace_bytes, void *stream);
SAR_API sar_status sar_bn_rstd(int32_t C, const float *m2, int64_t count, float eps, float *rstd, void *stream);
SAR_API sar_status sar_bn_apply(int64_t n, int32_t C, sar_dtype t, const void *x, const float *mean,
                                const float *rstd, const float *gamma, const float *beta, void *y, void *stream);
SAR_API sar_status sar_bn_bwd_stats(int64_t n, int32_t C, sar_dtype t, const void *x, const float *mean,
                                    const float *rstd, const void *gy, float *sum_gy, float *sum_gy_xhat,
                                    void *workspace, size_t workspace_bytes, void *stream);
SAR_API sar_status sar_bn_bwd_apply(int64_t n, int32_t C, sar_dtype t, const void *x, const float *mean,
                                    const float *rstd, const float *gamma, const void *gy, const float *sum_gy,
                                    const float *sum_gy_xhat, float inv_count, void *gx, void *stream);

/* The same three calls with the chain that follows the normalisation in the paper's networks (Sec. 4.2: batch
 * normalisation and dropout between all layers) folded in, so that the node array is read and written once instead
 * of three times: y = dropout(relu(bn(x))), with flags = SAR_GLUE_RELU and / or SAR_GLUE_DROPOUT choosing the links
 * (0: plain sar_bn_apply).  The dropout is sar_dropout's: element i (flat index into [n, C]) is kept and scaled by
 * 1/(1-p) when the top 24 bits of SplitMix64's (i+1)-th output for `seed` reach p * 2^24.
 * Backward: gy is the gradient with respect to y; both calls first take it back through the dropout (same seed)
 * and the ReLU and then proceed as sar_bn_bwd_stats / sar_bn_bwd_apply.  `post` is y as the forward call left it
 * (needed when SAR_GLUE_RELU is set: the ReLU passed where y > 0; with both flags y > 0 also tells which elements
 * the mask kept, so no random number is drawn).  gx may be gy.  Other flag bits: SAR_ERR_INVALID_ARG. */
SAR_API sar_status sar_bn_apply_act(int64_t n, int32_t C, sar_dtype t, const void *x, const float *mean,
                                    const float *rstd, const float *gamma, const float *beta, uint32_t flags, float p,
                                    uint64_t seed, void *y, void *stream);
SAR_API sar_status sar_bn_bwd_stats_act(int64_t n, int32_t C, sar_dtype t, const void *x, const float *mean,
                                        const float *rstd, const void *gy, const void *post, uint32_t flags, float p,
                                        uint64_t seed, float *sum_gy, float *sum_gy_xhat, void *workspace,
                                        size_t workspace_bytes, void *stream);
SAR_API sar_status sar_bn_bwd_apply_act(int64_t n, int32_t C, sar_dtype t, const void *x, const float *mean,
                                        const float *rstd, const float *gamma, const void *gy, const void *post,
                                        uint32_t flags, float p, uint64_t seed, const float *sum_gy,
                                        const float *sum_gy_xhat, float inv_count, void *gx, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Backward pass without any caller-provided scratch.  (The paper has no counterpart: this is a
 * convenience of this library.)
 *
 * Some callers have no way to give the library working memory: code that runs where cudaMalloc is off
 * limits (inside a latency-critical loop, because cudaMalloc synchronises the whole device; in a plug-in
 * whose host owns the allocator and hands out only the input and output buffers; in a process that has
 * pinned its memory budget at start-up).  For them this entry point runs the whole-graph backward pass of
 * sar_gat_bwd (one partition holding all sources, D rebuilt from the edges) with its scratch taken from a
 * fixed array of SAR_NOALLOC_SCRATCH_BYTES that is part of the library's device image.  It calls no
 * cudaMalloc / cudaFree and no allocating library routine; inputs and outputs are the caller's, exactly
 * as for sar_gat_bwd.
 *
 *   - Limit: sar_gat_workspace_bytes(g, H, F, t) must not exceed SAR_NOALLOC_SCRATCH_BYTES (16 bytes per
 *     (destination, head) plus the long-row partials); larger problems return SAR_ERR_WORKSPACE and launch
 *     nothing.  Every GPU that loads the library carries the array until the process exits.
 *   - The first call on each device looks up the array's device address (with that device current) and
 *     remembers it for the life of the process; make that first call before any stream capture begins.
 *     The remembered address belongs to the device's context at that time: after a cudaDeviceReset of
 *     that device it is stale, and this entry point must not be called on that device again.
 *   - All calls on a device share the one array, which keeps whatever the previous call left in it.  The
 *     pass writes every byte of it that it later reads, so nothing needs clearing between calls; but two
 *     calls whose kernels overlap on the GPU (different streams, no dependency) race on it: keep calls to
 *     this entry point ordered.
 * ------------------------------------------------------------------------------------------- */
#define SAR_NOALLOC_SCRATCH_BYTES (16u << 20)
SAR_API size_t sar_gat_bwd_noalloc_limit(void); /* = SAR_NOALLOC_SCRATCH_BYTES */
SAR_API sar_status sar_gat_bwd_noalloc(const sar_part *g, const void *feat, const float *el, const float *er,
                                       const float *m, const float *d, const void *gout, int32_t H, int32_t F,
                                       sar_dtype t, float slope, void *dfeat, float *del, float *der, void *stream);

/* ---------------------------------------------------------------------------------------------
 * A stack of L aggregation layers with HOST buffers (the 3-layer GAT of the paper's Sec. 4.2 reduced
 * to its aggregation steps): layer l computes out^l from feat^l = out^(l-1) (feat^0 given) with its
 * own el^l, er^l; the backward pass feeds dfeat^(l+1) as gout of layer l.  The kernels are enqueued on
 * `stream`; the host->device copies of the inputs and the device->host copies of the results run on two
 * side streams of the library (created on first use, one pair per device) so that they overlap with the
 * kernels, ordered after the work already queued on `stream`, and `stream` waits for the last copy:
 * once `stream` has completed, every output is in host memory.  Returns without synchronising; use
 * pinned host memory for the copies to be asynchronous.  The host inputs must stay unchanged, and
 * `arena` untouched, until then.
 *
 * Pipelined mode (io->flags = SAR_STACK_PIPELINED) for a sequence of calls, e.g. one per training step:
 * `arena` holds TWO working sets (2 x sar_gat_stack_arena_bytes) used alternately, so that the input
 * copies of call t+1 run while the kernels of call t are still busy and its results are still on their
 * way back.  In this mode
 *   - the input copies are NOT ordered after earlier work on `stream` (only the kernels are): the host
 *     inputs must already hold their values when the call is made;
 *   - `stream` does not wait for the result copies of the call: sar_gat_stack_host_wait(stream) makes it
 *     wait for everything the pipelined calls on this device have in flight (call it before reading
 *     results on the host, reusing the host inputs, freeing the arena, or switching mode);
 *   - results of successive calls arrive in call order (one copy stream), so calls may share their host
 *     output buffers if only the last result matters.
 * ------------------------------------------------------------------------------------------- */
#define SAR_STACK_PIPELINED 1u
typedef struct {
    int32_t L, H, F;
    sar_dtype t;
    float slope;
    /* HOST inputs */
    const void *feat0;        /* [n,H,F] type t                                          */
    const float *const *el;   /* HOST array of L HOST pointers, each [n,H]               */
    const float *const *er;   /* idem                                                    */
    const void *gout;         /* [n,H,F] type t: gradient w.r.t. the last layer's output */
    /* HOST outputs (any may be NULL to skip its copy) */
    void *out_last;           /* [n,H,F] type t                                          */
    void *dfeat0;             /* [n,H,F] type t                                          */
    float *const *del;        /* HOST array of L HOST pointers, each [n,H], or NULL      */
    float *const *der;        /* idem                                                    */
    uint32_t flags;           /* 0 or SAR_STACK_PIPELINED                                */
} sar_stack_host_io;

/* DEVICE bytes sar_gat_stack_host needs in `arena` for this graph and shape. */
SAR_API size_t sar_gat_stack_arena_bytes(const sar_part *g, int32_t L, int32_t H, int32_t F, sar_dtype t);

/* `g` is the un-split graph (DEVICE arrays), partitions as in sar_gat_fwd_fused; `arena` is DEVICE
 * scratch of at least sar_gat_stack_arena_bytes, 256-byte aligned. */
SAR_API sar_status sar_gat_stack_host(const sar_part *g, int32_t k, const int64_t *bounds,
                                      const sar_stack_host_io *io, void *arena, size_t arena_bytes,
                                      void *stream);

/* Makes `stream` wait for every copy that pipelined calls of sar_gat_stack_host on the current device
 * still have in flight.  Does not block the host. */
SAR_API sar_status sar_gat_stack_host_wait(void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SAR_H_ */

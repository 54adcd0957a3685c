/*
 * CPU oracle for the graph-attention aggregation of SAR (arXiv 2111.06483).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, float64 restatement of
 * what the CUDA library must compute.  It shares no code with the CUDA path and is
 * never called by it; only the tests, the smoke check and the benchmark's
 * "cpu_baseline"/reference arm may execute it.
 *
 * Conventions (the same ones the library's header states):
 *   - a graph is a CSR by DESTINATION: row i lists the sources j of the edges j -> i;
 *     indptr is int64[n_dst+1], indices is int32[nnz];
 *   - feat is [n_src, H, F] row-major, el is [n_dst, H] (destination term of the score),
 *     er is [n_src, H] (source term of the score);
 *   - inputs are float32 storage (bf16 test inputs are bf16-rounded values held in
 *     float32); every intermediate and every output is float64.
 *
 * Where each function comes from:
 *   oracle_gat_fwd      Eq. 3 (GAT layer), written as the definition: per-edge score,
 *                       row-wise softmax over the in-neighbourhood, weighted sum.  The
 *                       per-edge arrays e[E,H] and alpha[E,H] ARE materialised.
 *   oracle_gat_bwd      chain rule applied to Eq. 3 (the error Algorithm 2 pushes through
 *                       the aggregation gap), again with per-edge arrays.
 *   oracle_gat_fwd_seq  Algorithm 1 with the running-max correction of Sec. 3.4 ("Stable
 *                       softmax"): partitions are visited one after the other; numerator
 *                       and normaliser are accumulated separately and divided at the end
 *                       (Sec. 3.2).
 *   oracle_spmm         the neighbour sum of Eq. 2 (GraphSage aggregation, without the
 *                       1/|N(i)| factor unless asked for).
 *   oracle_csr_*        construction of the per-partition subgraphs G_{p,q} of Sec. 3.2
 *                       for one worker owning every destination and K contiguous source
 *                       ranges.
 *
 * Readings taken where the paper is silent (same on both sides):
 *   - the LeakyReLU slope is a parameter; its derivative at 0 is the slope;
 *   - a destination without in-edges gets out = 0, d = 0, m = -inf and contributes no
 *     gradient;
 *   - duplicate edges are kept and count separately;
 *   - the running max is treated as a constant in the backward pass.
 *
 * Pins (tests/test_oracle_*.py): dense masked-softmax brute force, scipy.sparse products,
 * central finite differences, torch CPU autograd over a dense formulation, closed-form
 * fixtures in tests/golden/, and algebraic invariants.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_BAD_ARG 1
#define ORACLE_NO_MEM 2

static double leaky_relu(double s, double slope) { return s > 0.0 ? s : slope * s; }
static double leaky_relu_grad(double s, double slope) { return s > 0.0 ? 1.0 : slope; }

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* ------------------------------------------------------------------------------------
 * Integer side (Sec. 3.2: the subgraphs G_{p,q}).
 * ---------------------------------------------------------------------------------- */

static int cmp_i32(const void *a, const void *b) {
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

/* COO edge list (src[t] -> dst[t]) to CSR by destination.  Within a row the sources
 * ascend; duplicates stay, next to one another. */
int oracle_csr_from_coo(int64_t n_dst, int64_t n_src, int64_t nnz, const int32_t *src, const int32_t *dst,
                        int64_t *indptr, int32_t *indices) {
    if (n_dst < 0 || n_src < 0 || nnz < 0) return ORACLE_BAD_ARG;
    for (int64_t i = 0; i <= n_dst; ++i) indptr[i] = 0;
    for (int64_t t = 0; t < nnz; ++t) {
        if (dst[t] < 0 || dst[t] >= n_dst || src[t] < 0 || src[t] >= n_src) return ORACLE_BAD_ARG;
        indptr[dst[t] + 1] += 1;
    }
    for (int64_t i = 0; i < n_dst; ++i) indptr[i + 1] += indptr[i];
    int64_t *cursor = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n_dst > 0 ? n_dst : 1));
    if (!cursor) return ORACLE_NO_MEM;
    for (int64_t i = 0; i < n_dst; ++i) cursor[i] = indptr[i];
    for (int64_t t = 0; t < nnz; ++t) indices[cursor[dst[t]]++] = src[t];
    free(cursor);
    for (int64_t i = 0; i < n_dst; ++i)
        qsort(indices + indptr[i], (size_t)(indptr[i + 1] - indptr[i]), sizeof(int32_t), cmp_i32);
    return ORACLE_OK;
}

/* Transpose of a CSR with n_rows rows and n_cols columns: row c of the result lists, in
 * ascending order, the rows r of the input that contain column c (once per occurrence). */
int oracle_csr_transpose(int64_t n_rows, int64_t n_cols, const int64_t *indptr, const int32_t *indices,
                         int64_t *t_indptr, int32_t *t_indices) {
    if (n_rows < 0 || n_cols < 0) return ORACLE_BAD_ARG;
    for (int64_t c = 0; c <= n_cols; ++c) t_indptr[c] = 0;
    for (int64_t r = 0; r < n_rows; ++r)
        for (int64_t t = indptr[r]; t < indptr[r + 1]; ++t) {
            if (indices[t] < 0 || indices[t] >= n_cols) return ORACLE_BAD_ARG;
            t_indptr[indices[t] + 1] += 1;
        }
    for (int64_t c = 0; c < n_cols; ++c) t_indptr[c + 1] += t_indptr[c];
    int64_t *cursor = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n_cols > 0 ? n_cols : 1));
    if (!cursor) return ORACLE_NO_MEM;
    for (int64_t c = 0; c < n_cols; ++c) cursor[c] = t_indptr[c];
    for (int64_t r = 0; r < n_rows; ++r)
        for (int64_t t = indptr[r]; t < indptr[r + 1]; ++t) t_indices[cursor[indices[t]]++] = (int32_t)r;
    free(cursor);
    return ORACLE_OK;
}

/* Contiguous source ranges: s_q = floor(q * n / k), q = 0..k. */
int oracle_partition_bounds(int64_t n, int32_t k, int64_t *bounds) {
    if (n < 0 || k < 1) return ORACLE_BAD_ARG;
    for (int32_t q = 0; q <= k; ++q) bounds[q] = (int64_t)(((__int128)q * (__int128)n) / (__int128)k);
    return ORACLE_OK;
}

/* Split a CSR by source range.  Partition q keeps, for every row, the edges whose source j
 * satisfies bounds[q] <= j < bounds[q+1], in row order, renumbered to j - bounds[q].
 * Output: indptr_all is k consecutive arrays of n_dst+1 entries (each starting at 0);
 * indices_all is the k index arrays back to back; nnz_off[q] is where partition q's
 * indices begin in indices_all (nnz_off[k] = nnz). */
int oracle_csr_split(int64_t n_dst, const int64_t *indptr, const int32_t *indices, int32_t k,
                     const int64_t *bounds, int64_t *indptr_all, int32_t *indices_all, int64_t *nnz_off) {
    if (n_dst < 0 || k < 1) return ORACLE_BAD_ARG;
    int64_t written = 0;
    for (int32_t q = 0; q < k; ++q) {
        int64_t *ip = indptr_all + (int64_t)q * (n_dst + 1);
        nnz_off[q] = written;
        ip[0] = 0;
        for (int64_t i = 0; i < n_dst; ++i) {
            int64_t cnt = 0;
            for (int64_t t = indptr[i]; t < indptr[i + 1]; ++t) {
                int64_t j = indices[t];
                if (j >= bounds[q] && j < bounds[q + 1]) {
                    indices_all[written++] = (int32_t)(j - bounds[q]);
                    ++cnt;
                }
            }
            ip[i + 1] = ip[i] + cnt;
        }
    }
    nnz_off[k] = written;
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------
 * Forward, the definition (Eq. 3).
 *   s[t,h]     = el[i,h] + er[j,h]               i = destination of edge t, j = its source
 *   e[t,h]     = LeakyReLU(s[t,h])
 *   mx[i,h]    = max over the edges t of row i of e[t,h]
 *   w[t,h]     = exp(e[t,h] - mx[i,h])
 *   den[i,h]   = sum over the row of w[t,h]
 *   alpha[t,h] = w[t,h] / den[i,h]
 *   out[i,h,:] = sum over the row of alpha[t,h] * feat[j,h,:]
 * e_out and alpha_out are [nnz,H]; out is [n_dst,H,F]; m_out, d_out are [n_dst,H].
 * ---------------------------------------------------------------------------------- */
int oracle_gat_fwd(int64_t n_dst, const int64_t *indptr, const int32_t *indices, const float *feat,
                   const float *el, const float *er, int32_t H, int32_t F, double slope, double *e_out,
                   double *alpha_out, double *out, double *m_out, double *d_out) {
    if (n_dst < 0 || H < 1 || F < 1) return ORACLE_BAD_ARG;
    const int64_t HF = (int64_t)H * F;
#pragma omp parallel for schedule(dynamic, 256)
    for (int64_t i = 0; i < n_dst; ++i) {
        const int64_t beg = indptr[i], end = indptr[i + 1];
        for (int32_t h = 0; h < H; ++h) {
            double mx = -INFINITY;
            for (int64_t t = beg; t < end; ++t) {
                const int64_t j = indices[t];
                const double s = (double)el[i * H + h] + (double)er[j * H + h];
                const double e = leaky_relu(s, slope);
                e_out[t * H + h] = e;
                if (e > mx) mx = e;
            }
            double den = 0.0;
            for (int64_t t = beg; t < end; ++t) {
                const double w = exp(e_out[t * H + h] - mx);
                alpha_out[t * H + h] = w; /* normalised just below */
                den += w;
            }
            for (int64_t t = beg; t < end; ++t) alpha_out[t * H + h] /= den;
            m_out[i * H + h] = mx;
            d_out[i * H + h] = den;
            for (int32_t f = 0; f < F; ++f) {
                double acc = 0.0;
                for (int64_t t = beg; t < end; ++t) {
                    const int64_t j = indices[t];
                    acc += alpha_out[t * H + h] * (double)feat[j * HF + (int64_t)h * F + f];
                }
                out[i * HF + (int64_t)h * F + f] = acc;
            }
        }
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------
 * Backward, the definition (chain rule on Eq. 3; what Algorithm 2 back-propagates).
 * Given gout = dLoss/dout and the per-edge alpha of the forward pass:
 *   dalpha[t,h] = <gout[i,h,:], feat[j,h,:]>
 *   D[i,h]      = sum over row i of alpha[t,h] * dalpha[t,h]
 *   de[t,h]     = alpha[t,h] * (dalpha[t,h] - D[i,h])                (softmax Jacobian)
 *   ds[t,h]     = de[t,h] * (s[t,h] > 0 ? 1 : slope)                 (LeakyReLU)
 *   del[i,h]    = sum over the in-edges of i of ds[t,h]
 *   der[j,h]    = sum over the out-edges of j of ds[t,h]
 *   dfeat[j,h,:]= sum over the out-edges of j of alpha[t,h] * gout[i,h,:]
 * D is [n_dst,H]; dfeat is [n_src,H,F]; del is [n_dst,H]; der is [n_src,H].
 * The scatter over sources runs serially so that the sums have one fixed order.
 * ---------------------------------------------------------------------------------- */
int oracle_gat_bwd(int64_t n_dst, int64_t n_src, const int64_t *indptr, const int32_t *indices,
                   const float *feat, const float *el, const float *er, const double *alpha,
                   const float *gout, int32_t H, int32_t F, double slope, double *D_out, double *dfeat,
                   double *del, double *der) {
    if (n_dst < 0 || n_src < 0 || H < 1 || F < 1) return ORACLE_BAD_ARG;
    const int64_t HF = (int64_t)H * F;
    const int64_t nnz = indptr[n_dst];
    double *ds = (double *)malloc(sizeof(double) * (size_t)(nnz * H > 0 ? nnz * H : 1));
    if (!ds) return ORACLE_NO_MEM;
    memset(dfeat, 0, sizeof(double) * (size_t)(n_src * HF));
    memset(der, 0, sizeof(double) * (size_t)(n_src * H));
#pragma omp parallel for schedule(dynamic, 256)
    for (int64_t i = 0; i < n_dst; ++i) {
        const int64_t beg = indptr[i], end = indptr[i + 1];
        for (int32_t h = 0; h < H; ++h) {
            double Dih = 0.0;
            for (int64_t t = beg; t < end; ++t) {
                const int64_t j = indices[t];
                double dalpha = 0.0;
                for (int32_t f = 0; f < F; ++f)
                    dalpha += (double)gout[i * HF + (int64_t)h * F + f] * (double)feat[j * HF + (int64_t)h * F + f];
                ds[t * H + h] = dalpha; /* holds dalpha for now */
                Dih += alpha[t * H + h] * dalpha;
            }
            D_out[i * H + h] = Dih;
            double acc = 0.0;
            for (int64_t t = beg; t < end; ++t) {
                const int64_t j = indices[t];
                const double s = (double)el[i * H + h] + (double)er[j * H + h];
                const double de = alpha[t * H + h] * (ds[t * H + h] - Dih);
                ds[t * H + h] = de * leaky_relu_grad(s, slope);
                acc += ds[t * H + h];
            }
            del[i * H + h] = acc;
        }
    }
    for (int64_t i = 0; i < n_dst; ++i)
        for (int64_t t = indptr[i]; t < indptr[i + 1]; ++t) {
            const int64_t j = indices[t];
            for (int32_t h = 0; h < H; ++h) {
                der[j * H + h] += ds[t * H + h];
                const double a = alpha[t * H + h];
                for (int32_t f = 0; f < F; ++f)
                    dfeat[j * HF + (int64_t)h * F + f] += a * (double)gout[i * HF + (int64_t)h * F + f];
            }
        }
    free(ds);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------
 * Forward, the sequential form (Algorithm 1 with the running max of Sec. 3.4).
 * K partitions in the layout oracle_csr_split writes.  feat and er are the full arrays;
 * partition q's local source id l means global source bounds[q] + l.  The partitions are
 * visited in the order given by order[0..K-1].  Per (i,h):
 *     M = -inf, d = 0, acc = 0
 *     for each visited partition with at least one edge in row i:
 *         mq = max of e over the row's edges in this partition
 *         Mn = max(M, mq);  c = (M == -inf) ? 0 : exp(M - Mn)
 *         acc = acc*c + sum exp(e - Mn) * feat[j];   d = d*c + sum exp(e - Mn);   M = Mn
 *     out = acc / d   (0 when d == 0)
 * ---------------------------------------------------------------------------------- */
int oracle_gat_fwd_seq(int64_t n_dst, int32_t K, const int64_t *bounds, const int32_t *order,
                       const int64_t *indptr_all, const int32_t *indices_all, const int64_t *nnz_off,
                       const float *feat, const float *el, const float *er, int32_t H, int32_t F,
                       double slope, double *out, double *m_out, double *d_out) {
    if (n_dst < 0 || K < 1 || H < 1 || F < 1) return ORACLE_BAD_ARG;
    const int64_t HF = (int64_t)H * F;
#pragma omp parallel for schedule(dynamic, 256)
    for (int64_t i = 0; i < n_dst; ++i) {
        for (int32_t h = 0; h < H; ++h) {
            double M = -INFINITY, d = 0.0;
            double *acc = out + i * HF + (int64_t)h * F; /* numerator lives in out until the end */
            for (int32_t f = 0; f < F; ++f) acc[f] = 0.0;
            for (int32_t v = 0; v < K; ++v) {
                const int32_t q = order[v];
                const int64_t *ip = indptr_all + (int64_t)q * (n_dst + 1);
                const int32_t *idx = indices_all + nnz_off[q];
                const int64_t beg = ip[i], end = ip[i + 1];
                if (beg == end) continue;
                double mq = -INFINITY;
                for (int64_t t = beg; t < end; ++t) {
                    const int64_t j = bounds[q] + idx[t];
                    const double e = leaky_relu((double)el[i * H + h] + (double)er[j * H + h], slope);
                    if (e > mq) mq = e;
                }
                const double Mn = M > mq ? M : mq;
                const double c = (M == -INFINITY) ? 0.0 : exp(M - Mn);
                d *= c;
                for (int32_t f = 0; f < F; ++f) acc[f] *= c;
                for (int64_t t = beg; t < end; ++t) {
                    const int64_t j = bounds[q] + idx[t];
                    const double e = leaky_relu((double)el[i * H + h] + (double)er[j * H + h], slope);
                    const double w = exp(e - Mn);
                    d += w;
                    for (int32_t f = 0; f < F; ++f) acc[f] += w * (double)feat[j * HF + (int64_t)h * F + f];
                }
                M = Mn;
            }
            for (int32_t f = 0; f < F; ++f) acc[f] = d > 0.0 ? acc[f] / d : 0.0;
            m_out[i * H + h] = M;
            d_out[i * H + h] = d;
        }
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------
 * Neighbour sum (Eq. 2 without the non-linearity and residual): out[i,:] = sum of feat[j,:]
 * over the in-edges of i; with mean != 0 the sum is divided by the in-degree (rows without
 * in-edges stay 0).  The backward pass of the sum is the same routine on the transposed
 * graph applied to gout ("case 1" of Sec. 3.2: no input features needed).
 * ---------------------------------------------------------------------------------- */
int oracle_spmm(int64_t n_dst, const int64_t *indptr, const int32_t *indices, const float *feat, int32_t F,
                int32_t mean, double *out) {
    if (n_dst < 0 || F < 1) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(dynamic, 256)
    for (int64_t i = 0; i < n_dst; ++i) {
        const int64_t beg = indptr[i], end = indptr[i + 1];
        for (int32_t f = 0; f < F; ++f) {
            double acc = 0.0;
            for (int64_t t = beg; t < end; ++t) acc += (double)feat[(int64_t)indices[t] * F + f];
            if (mean && end > beg) acc /= (double)(end - beg);
            out[i * (int64_t)F + f] = acc;
        }
    }
    return ORACLE_OK;
}

// Graph preparation on the device: edge list -> CSR / CSC, split by source range, long-row plan,
// validation.  Integer work whose results are unique.  Sorting and prefix sums are CUB device
// primitives; everything else is small kernels in this file.  Contracts are in include/sar.h.
#include <cub/device/device_radix_sort.cuh>
#include <cub/device/device_scan.cuh>
#include <cub/device/device_select.cuh>
#include <thrust/iterator/counting_iterator.h>

#include "sar_common.cuh"

namespace sar {

struct Bounds {
    int k;
    long long s[SAR_MAX_PARTS + 1];
};

__global__ void make_keys_kernel(long long nnz, const int32_t *__restrict__ row, const int32_t *__restrict__ col,
                                 unsigned long long *__restrict__ keys) {
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t < nnz) keys[t] = ((unsigned long long)(unsigned)row[t] << 32) | (unsigned)col[t];
}

// keys of the transpose: (column << 32) | row, the row of edge t found by bisection of indptr
__global__ void make_transposed_keys_kernel(long long nnz, long long n_rows, const int64_t *__restrict__ indptr,
                                            const int32_t *__restrict__ indices,
                                            unsigned long long *__restrict__ keys) {
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= nnz) return;
    long long lo = 0, hi = n_rows;  // last r with indptr[r] <= t
    while (hi - lo > 1) {
        const long long mid = (lo + hi) >> 1;
        if (indptr[mid] <= t) lo = mid; else hi = mid;
    }
    keys[t] = ((unsigned long long)(unsigned)indices[t] << 32) | (unsigned)lo;
}

// sorted keys -> indices (low word) and indptr (first position of each high word)
__global__ void keys_to_csr_kernel(long long nnz, long long n_rows, const unsigned long long *__restrict__ keys,
                                   int64_t *__restrict__ indptr, int32_t *__restrict__ indices) {
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t > nnz) return;
    const long long r_cur = t < nnz ? (long long)(keys[t] >> 32) : n_rows;
    const long long r_prev = t > 0 ? (long long)(keys[t - 1] >> 32) : -1;
    for (long long r = r_prev + 1; r <= r_cur; ++r) indptr[r] = t;
    if (t < nnz) indices[t] = (int32_t)(unsigned)(keys[t] & 0xffffffffull);
}

__device__ __forceinline__ long long lower_bound_row(const int32_t *__restrict__ idx, long long lo, long long hi,
                                                     long long key) {
    while (lo < hi) {
        const long long mid = (lo + hi) >> 1;
        if (idx[mid] < key) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// counts of row i's edges per source range, written one slot to the right (ready for an inclusive scan)
__global__ void split_count_kernel(long long n_dst, const int64_t *__restrict__ indptr,
                                   const int32_t *__restrict__ indices, Bounds b, int64_t *__restrict__ indptr_all) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_dst) return;
    const long long beg = indptr[i], end = indptr[i + 1];
    long long prev = beg;
    for (int q = 0; q < b.k; ++q) {
        const long long pos = q + 1 == b.k ? end : lower_bound_row(indices, prev, end, b.s[q + 1]);
        indptr_all[(long long)q * (n_dst + 1) + i + 1] = pos - prev;
        if (i == 0) indptr_all[(long long)q * (n_dst + 1)] = 0;
        prev = pos;
    }
}

__global__ void split_fill_kernel(long long n_dst, const int64_t *__restrict__ indptr,
                                  const int32_t *__restrict__ indices, Bounds b, Bounds off,
                                  const int64_t *__restrict__ indptr_all, int32_t *__restrict__ indices_all) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_dst) return;
    const long long end = indptr[i + 1];
    long long t = indptr[i];
    for (int q = 0; q < b.k && t < end; ++q) {
        long long w = off.s[q] + indptr_all[(long long)q * (n_dst + 1) + i];
        while (t < end && indices[t] < b.s[q + 1]) indices_all[w++] = (int32_t)(indices[t++] - b.s[q]);
    }
}

// out[i] = in[i] - in[0]: the offsets of a run of consecutive rows, counted from the run's first edge
__global__ void rebase_kernel(long long count, const int64_t *__restrict__ in, int64_t *__restrict__ out) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) out[i] = in[i] - in[0];
}

struct IsLongRow {
    const int64_t *indptr;
    int threshold;
    __device__ bool operator()(int r) const { return indptr[r + 1] - indptr[r] > threshold; }
};

__global__ void plan_count_kernel(long long n_rows, const int64_t *__restrict__ indptr, int threshold,
                                  unsigned long long *__restrict__ counts) {
    const long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    long long deg = 0;
    if (r < n_rows) deg = indptr[r + 1] - indptr[r];
    const bool is_long = deg > threshold;
    const unsigned ballot = __ballot_sync(0xffffffffu, is_long);
    long long segs = is_long ? (deg + threshold - 1) / threshold : 0;
    for (int o = 16; o > 0; o >>= 1) segs += __shfl_down_sync(0xffffffffu, segs, o);
    if ((threadIdx.x & 31) == 0 && ballot) {  // integer sums: order does not matter
        atomicAdd(counts, (unsigned long long)__popc(ballot));
        atomicAdd(counts + 1, (unsigned long long)segs);
    }
}

__global__ void plan_segcount_kernel(int n_long, const int32_t *__restrict__ long_row,
                                     const int64_t *__restrict__ indptr, int threshold, int64_t *__restrict__ segs) {
    const int lr = blockIdx.x * blockDim.x + threadIdx.x;
    if (lr > n_long) return;
    if (lr == n_long) {
        segs[lr] = 0;
        return;
    }
    const long long deg = indptr[long_row[lr] + 1] - indptr[long_row[lr]];
    segs[lr] = (deg + threshold - 1) / threshold;
}

__global__ void validate_kernel(long long n_rows, long long n_cols, long long nnz, const int64_t *__restrict__ indptr,
                                const int32_t *__restrict__ indices, int32_t *flag) {
    const long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= n_rows) return;
    const long long beg = indptr[r], end = indptr[r + 1];
    bool bad = beg > end || beg < 0 || end > nnz;
    if (r == 0 && beg != 0) bad = true;
    if (r == n_rows - 1 && end != nnz) bad = true;
    if (!bad)
        for (long long t = beg; t < end; ++t) {
            const long long j = indices[t];
            if (j < 0 || j >= n_cols || (t > beg && indices[t - 1] > j)) {
                bad = true;
                break;
            }
        }
    if (bad) *flag = 1;  // every writer stores the same value
}


// ---- message-flow pruning (Appendix B) ------------------------------------------------------------
// One warp per destination row: an active row marks itself and every source it reads.  All writers
// store the same value 1, so the races are benign and the result does not depend on the schedule.
__global__ void mfg_frontier_kernel(long long n, const int64_t *__restrict__ indptr, const int32_t *__restrict__ indices,
                                    const uint8_t *__restrict__ need_out, uint8_t *__restrict__ need_in) {
    const long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= n || !need_out[row]) return;
    if (lane == 0) need_in[row] = 1;
    const long long beg = indptr[row], end = indptr[row + 1];
    for (long long t = beg + lane; t < end; t += 32) need_in[indices[t]] = 1;
}

// degrees of the kept rows, one slot to the right (ready for an inclusive scan)
__global__ void filter_count_kernel(long long n, const int64_t *__restrict__ indptr, const uint8_t *__restrict__ keep,
                                    int64_t *__restrict__ indptr_out) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    indptr_out[i + 1] = keep[i] ? indptr[i + 1] - indptr[i] : 0;
    if (i == 0) indptr_out[0] = 0;
}

__global__ void filter_fill_kernel(long long n, const int64_t *__restrict__ indptr, const int32_t *__restrict__ indices,
                                   const int64_t *__restrict__ indptr_out, int32_t *__restrict__ indices_out) {
    const long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= n) return;
    const long long w = indptr_out[row], cnt = indptr_out[row + 1] - w, beg = indptr[row];
    for (long long t = lane; t < cnt; t += 32) indices_out[w + t] = indices[beg + t];
}

// ---- node order by degree ---------------------------------------------------------------------------------------
// degree of a node = edges it is the source of + edges it is the destination of (integer atomics: order-independent)
__global__ void degree_count_kernel(long long e, const int32_t *__restrict__ src, const int32_t *__restrict__ dst,
                                    unsigned *__restrict__ deg) {
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= e) return;
    atomicAdd(deg + src[t], 1u);
    atomicAdd(deg + dst[t], 1u);
}

// key of node i: (2^32 - 1 - degree) in the high word, i in the low word: ascending keys = descending degree, ties by id
__global__ void order_keys_kernel(long long n, const unsigned *__restrict__ deg, unsigned long long *__restrict__ keys) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) keys[i] = ((unsigned long long)(0xffffffffu - deg[i]) << 32) | (unsigned)i;
}

__global__ void order_from_keys_kernel(long long n, const unsigned long long *__restrict__ keys,
                                       int32_t *__restrict__ order, int32_t *__restrict__ rank) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int32_t old = (int32_t)(unsigned)(keys[i] & 0xffffffffull);
    order[i] = old;
    rank[old] = (int32_t)i;
}

__global__ void relabel_kernel(long long e, const int32_t *__restrict__ ids, const int32_t *__restrict__ rank,
                               int32_t *__restrict__ out) {
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t < e) out[t] = rank[ids[t]];
}

// out row i = in row index[i]; W = the widest word that divides the row
template <typename W>
__global__ void permute_rows_kernel(long long n, long long words, const int32_t *__restrict__ index,
                                    const W *__restrict__ in, W *__restrict__ out) {
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n * words) return;
    const long long i = t / words, w = t - i * words;
    out[t] = in[(long long)index[i] * words + w];
}

static inline unsigned nblk(long long n) { return (unsigned)((n + 255) / 256); }

static size_t sort_temp_bytes(long long nnz) {
    size_t bytes = 0;
    unsigned long long *nullk = nullptr;
    if (cub::DeviceRadixSort::SortKeys(nullptr, bytes, nullk, nullk, nnz > 0 ? nnz : 1, 0, 64) != cudaSuccess) {
        (void)cudaGetLastError();
        bytes = (size_t)(nnz / 512 + 4096) * 4096;  // no device to ask: generous guess
    }
    return bytes;
}

static size_t scan_temp_bytes(long long n) {
    size_t bytes = 0;
    int64_t *nullp = nullptr;
    if (cub::DeviceScan::InclusiveSum(nullptr, bytes, nullp, nullp, n > 0 ? n : 1) != cudaSuccess) {
        (void)cudaGetLastError();
        bytes = (size_t)(n / 256 + 4096) * 64;
    }
    return bytes;
}

static size_t select_temp_bytes(long long n) {
    size_t bytes = 0;
    int32_t *nullo = nullptr;
    int *nulln = nullptr;
    IsLongRow pred{nullptr, 1};
    if (cub::DeviceSelect::If(nullptr, bytes, thrust::counting_iterator<int>(0), nullo, nulln, (int)(n > 0 ? n : 1),
                              pred) != cudaSuccess) {
        (void)cudaGetLastError();
        bytes = (size_t)(n / 256 + 4096) * 64;
    }
    return bytes;
}

// sort the keys held in ws[0 .. 8*nnz) into ws[8*nnz .. 16*nnz), CUB scratch behind them
static sar_status sort_keys(long long nnz, int key_bits, void *ws, size_t ws_bytes, cudaStream_t st,
                            unsigned long long **sorted) {
    const size_t kb = sar_round_up((size_t)nnz * 8, 256);
    unsigned long long *in = static_cast<unsigned long long *>(ws);
    unsigned long long *out = reinterpret_cast<unsigned long long *>(static_cast<char *>(ws) + kb);
    void *temp = static_cast<char *>(ws) + 2 * kb;
    size_t temp_bytes = ws_bytes - 2 * kb;
    size_t need = 0;
    SAR_CUDA_TRY(cub::DeviceRadixSort::SortKeys(nullptr, need, in, out, nnz, 0, key_bits, st));
    if (need > temp_bytes) return SAR_ERR_WORKSPACE;
    SAR_CUDA_TRY(cub::DeviceRadixSort::SortKeys(temp, need, in, out, nnz, 0, key_bits, st));
    *sorted = out;
    return SAR_OK;
}

static int bits_for(long long n) {
    int b = 1;
    while (b < 32 && (1LL << b) < n) ++b;
    return b;
}

}  // namespace sar

using namespace sar;

extern "C" {

size_t sar_graph_workspace_bytes(int64_t nnz, int64_t n_rows) {
    if (nnz < 0 || n_rows < 0) return 0;
    size_t temp = sort_temp_bytes(nnz);
    const size_t a = scan_temp_bytes(n_rows + 1), b = select_temp_bytes(n_rows);
    if (a > temp) temp = a;
    if (b > temp) temp = b;
    return 2 * sar_round_up((size_t)nnz * 8, 256) + sar_round_up(temp, 256) + sar_round_up((size_t)(n_rows + 1) * 8, 256) + 512;
}

sar_status sar_csr_from_coo(int64_t n_rows, int64_t n_cols, int64_t nnz, const int32_t *row, const int32_t *col,
                            int64_t *indptr, int32_t *indices, void *workspace, size_t workspace_bytes,
                            void *stream) {
    if (n_rows < 0 || n_cols < 0 || nnz < 0 || !indptr) return SAR_ERR_INVALID_ARG;
    if (n_rows > INT32_MAX || n_cols > INT32_MAX) return SAR_ERR_UNSUPPORTED;
    if (nnz > 0 && (!row || !col || !indices)) return SAR_ERR_INVALID_ARG;
    if (!sar_aligned(indptr, 8) || !sar_aligned(indices, 4) || !sar_aligned(row, 4) || !sar_aligned(col, 4))
        return SAR_ERR_ALIGNMENT;
    const size_t kb = sar_round_up((size_t)nnz * 8, 256);
    if (!workspace || !sar_aligned(workspace, 256) || workspace_bytes < 2 * kb) return SAR_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned long long *keys = static_cast<unsigned long long *>(workspace);
    unsigned long long *sorted = keys;
    if (nnz > 0) {
        make_keys_kernel<<<nblk(nnz), 256, 0, st>>>(nnz, row, col, keys);
        SAR_TRY(sar_after_launch());
        SAR_TRY(sort_keys(nnz, 32 + bits_for(n_rows), workspace, workspace_bytes, st, &sorted));
    }
    keys_to_csr_kernel<<<nblk(nnz + 1), 256, 0, st>>>(nnz, n_rows, sorted, indptr, indices);
    return sar_after_launch();
}

sar_status sar_csr_transpose(int64_t n_rows, int64_t n_cols, const int64_t *indptr, const int32_t *indices,
                             int64_t *t_indptr, int32_t *t_indices, void *workspace, size_t workspace_bytes,
                             void *stream) {
    if (n_rows < 0 || n_cols < 0 || !indptr || !t_indptr) return SAR_ERR_INVALID_ARG;
    if (n_rows > INT32_MAX || n_cols > INT32_MAX) return SAR_ERR_UNSUPPORTED;
    if (!sar_aligned(indptr, 8) || !sar_aligned(indices, 4) || !sar_aligned(t_indptr, 8) || !sar_aligned(t_indices, 4))
        return SAR_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the edge count lives on the device; fetch it (this call is preparation, not the hot path)
    int64_t nnz = 0;
    SAR_CUDA_TRY(cudaMemcpyAsync(&nnz, indptr + n_rows, 8, cudaMemcpyDeviceToHost, st));
    SAR_CUDA_TRY(cudaStreamSynchronize(st));
    if (nnz < 0) return SAR_ERR_BAD_GRAPH;
    if (nnz > 0 && (!indices || !t_indices)) return SAR_ERR_INVALID_ARG;
    const size_t kb = sar_round_up((size_t)nnz * 8, 256);
    if (!workspace || !sar_aligned(workspace, 256) || workspace_bytes < 2 * kb) return SAR_ERR_WORKSPACE;
    unsigned long long *keys = static_cast<unsigned long long *>(workspace);
    unsigned long long *sorted = keys;
    if (nnz > 0) {
        make_transposed_keys_kernel<<<nblk(nnz), 256, 0, st>>>(nnz, n_rows, indptr, indices, keys);
        SAR_TRY(sar_after_launch());
        SAR_TRY(sort_keys(nnz, 32 + bits_for(n_cols), workspace, workspace_bytes, st, &sorted));
    }
    keys_to_csr_kernel<<<nblk(nnz + 1), 256, 0, st>>>(nnz, n_cols, sorted, t_indptr, t_indices);
    return sar_after_launch();
}

sar_status sar_partition_bounds(int64_t n, int32_t k, int64_t *bounds) {
    if (n < 0 || k < 1 || !bounds) return SAR_ERR_INVALID_ARG;
    for (int32_t q = 0; q <= k; ++q) bounds[q] = (int64_t)(((__int128)q * (__int128)n) / (__int128)k);
    return SAR_OK;
}

static sar_status load_bounds(int32_t k, const int64_t *bounds, Bounds *b) {
    if (k < 1 || !bounds) return SAR_ERR_INVALID_ARG;
    if (k > SAR_MAX_PARTS) return SAR_ERR_UNSUPPORTED;
    b->k = k;
    for (int q = 0; q <= k; ++q) {
        if (q > 0 && bounds[q] < bounds[q - 1]) return SAR_ERR_INVALID_ARG;
        b->s[q] = bounds[q];
    }
    return SAR_OK;
}

sar_status sar_csr_split_indptr(int64_t n_dst, const int64_t *indptr, const int32_t *indices, int32_t k,
                                const int64_t *bounds, int64_t *indptr_all, void *workspace, size_t workspace_bytes,
                                void *stream) {
    if (n_dst < 0 || !indptr || !indptr_all) return SAR_ERR_INVALID_ARG;
    Bounds b;
    SAR_TRY(load_bounds(k, bounds, &b));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n_dst == 0) {
        SAR_CUDA_TRY(cudaMemsetAsync(indptr_all, 0, (size_t)k * 8, st));
        return SAR_OK;
    }
    split_count_kernel<<<nblk(n_dst), 256, 0, st>>>(n_dst, indptr, indices, b, indptr_all);
    SAR_TRY(sar_after_launch());
    size_t need = 0;
    SAR_CUDA_TRY(cub::DeviceScan::InclusiveSum(nullptr, need, indptr_all, indptr_all, n_dst + 1, st));
    if (!workspace || workspace_bytes < need) return SAR_ERR_WORKSPACE;
    for (int q = 0; q < k; ++q) {
        int64_t *p = indptr_all + (long long)q * (n_dst + 1);
        SAR_CUDA_TRY(cub::DeviceScan::InclusiveSum(workspace, need, p, p, n_dst + 1, st));
    }
    return SAR_OK;
}

sar_status sar_csr_split_indices(int64_t n_dst, const int64_t *indptr, const int32_t *indices, int32_t k,
                                 const int64_t *bounds, const int64_t *indptr_all, const int64_t *nnz_off,
                                 int32_t *indices_all, void *stream) {
    if (n_dst < 0 || !indptr || !indptr_all || !nnz_off) return SAR_ERR_INVALID_ARG;
    Bounds b, off;
    SAR_TRY(load_bounds(k, bounds, &b));
    SAR_TRY(load_bounds(k, nnz_off, &off));
    if (n_dst == 0 || nnz_off[k] == 0) return SAR_OK;
    if (!indices || !indices_all) return SAR_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    split_fill_kernel<<<nblk(n_dst), 256, 0, st>>>(n_dst, indptr, indices, b, off, indptr_all, indices_all);
    return sar_after_launch();
}

sar_status sar_csc_slice_indptr(int64_t s0, int64_t s1, const int64_t *t_indptr, int64_t *t_indptr_q, void *stream) {
    if (s0 < 0 || s1 < s0 || !t_indptr || !t_indptr_q) return SAR_ERR_INVALID_ARG;
    if (!sar_aligned(t_indptr, 8) || !sar_aligned(t_indptr_q, 8)) return SAR_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rebase_kernel<<<nblk(s1 - s0 + 1), 256, 0, st>>>(s1 - s0 + 1, t_indptr + s0, t_indptr_q);
    return sar_after_launch();
}

sar_status sar_mfg_frontier(int64_t n, const int64_t *indptr, const int32_t *indices, const uint8_t *need_out,
                            uint8_t *need_in, void *stream) {
    if (n < 0 || (n > 0 && (!indptr || !need_out || !need_in))) return SAR_ERR_INVALID_ARG;
    if (n > INT32_MAX) return SAR_ERR_UNSUPPORTED;
    if (!sar_aligned(indptr, 8) || !sar_aligned(indices, 4)) return SAR_ERR_ALIGNMENT;
    if (n == 0) return SAR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SAR_CUDA_TRY(cudaMemsetAsync(need_in, 0, (size_t)n, st));
    mfg_frontier_kernel<<<nblk(n * 32), 256, 0, st>>>(n, indptr, indices, need_out, need_in);
    return sar_after_launch();
}

sar_status sar_csr_filter_rows_indptr(int64_t n, const int64_t *indptr, const uint8_t *keep, int64_t *indptr_out,
                                      void *workspace, size_t workspace_bytes, void *stream) {
    if (n < 0 || !indptr_out || (n > 0 && (!indptr || !keep))) return SAR_ERR_INVALID_ARG;
    if (!sar_aligned(indptr, 8) || !sar_aligned(indptr_out, 8)) return SAR_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n == 0) {
        SAR_CUDA_TRY(cudaMemsetAsync(indptr_out, 0, 8, st));
        return SAR_OK;
    }
    filter_count_kernel<<<nblk(n), 256, 0, st>>>(n, indptr, keep, indptr_out);
    SAR_TRY(sar_after_launch());
    size_t need = 0;
    SAR_CUDA_TRY(cub::DeviceScan::InclusiveSum(nullptr, need, indptr_out, indptr_out, n + 1, st));
    if (!workspace || workspace_bytes < need) return SAR_ERR_WORKSPACE;
    SAR_CUDA_TRY(cub::DeviceScan::InclusiveSum(workspace, need, indptr_out, indptr_out, n + 1, st));
    return SAR_OK;
}

sar_status sar_csr_filter_rows_indices(int64_t n, const int64_t *indptr, const int32_t *indices,
                                       const int64_t *indptr_out, int32_t *indices_out, void *stream) {
    if (n < 0 || (n > 0 && (!indptr || !indptr_out))) return SAR_ERR_INVALID_ARG;
    if (n == 0) return SAR_OK;
    if (!indices || !indices_out) return SAR_ERR_INVALID_ARG;
    if (!sar_aligned(indices, 4) || !sar_aligned(indices_out, 4)) return SAR_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    filter_fill_kernel<<<nblk(n * 32), 256, 0, st>>>(n, indptr, indices, indptr_out, indices_out);
    return sar_after_launch();
}

sar_status sar_validate_part(const sar_part *g, int32_t *flag, void *stream) {
    if (!g || !flag || !g->indptr) return SAR_ERR_INVALID_ARG;
    if (g->n_dst < 0 || g->n_src < 0 || g->nnz < 0) return SAR_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SAR_CUDA_TRY(cudaMemsetAsync(flag, 0, 4, st));
    if (g->n_dst > 0) {
        validate_kernel<<<nblk(g->n_dst), 256, 0, st>>>(g->n_dst, g->n_src, g->nnz, g->indptr, g->indices, flag);
        SAR_TRY(sar_after_launch());
    }
    if (g->t_indptr && g->n_src > 0) {
        validate_kernel<<<nblk(g->n_src), 256, 0, st>>>(g->n_src, g->n_dst, g->nnz, g->t_indptr, g->t_indices, flag);
        SAR_TRY(sar_after_launch());
    }
    int32_t h = 0;
    SAR_CUDA_TRY(cudaMemcpyAsync(&h, flag, 4, cudaMemcpyDeviceToHost, st));
    SAR_CUDA_TRY(cudaStreamSynchronize(st));
    if (g->n_dst == 0 && g->nnz != 0) h = 1;
    return h ? SAR_ERR_BAD_GRAPH : SAR_OK;
}

sar_status sar_plan_count(int64_t n_rows, const int64_t *indptr, int32_t threshold, int64_t *counts, int32_t *n_long,
                          int64_t *n_seg, void *stream) {
    if (n_rows < 0 || !indptr || threshold < 1 || !counts || !n_long || !n_seg) return SAR_ERR_INVALID_ARG;
    if (n_rows > INT32_MAX) return SAR_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SAR_CUDA_TRY(cudaMemsetAsync(counts, 0, 16, st));
    if (n_rows > 0) {
        plan_count_kernel<<<nblk(n_rows), 256, 0, st>>>(n_rows, indptr, threshold,
                                                        reinterpret_cast<unsigned long long *>(counts));
        SAR_TRY(sar_after_launch());
    }
    int64_t h[2] = {0, 0};
    SAR_CUDA_TRY(cudaMemcpyAsync(h, counts, 16, cudaMemcpyDeviceToHost, st));
    SAR_CUDA_TRY(cudaStreamSynchronize(st));
    *n_long = (int32_t)h[0];
    *n_seg = h[1];
    return SAR_OK;
}

sar_status sar_plan_fill(int64_t n_rows, const int64_t *indptr, int32_t threshold, int32_t n_long, int32_t *long_row,
                         int64_t *long_seg, void *workspace, size_t workspace_bytes, void *stream) {
    if (n_rows < 0 || !indptr || threshold < 1 || n_long < 0 || !long_seg) return SAR_ERR_INVALID_ARG;
    if (n_rows > INT32_MAX) return SAR_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n_long == 0) {
        SAR_CUDA_TRY(cudaMemsetAsync(long_seg, 0, 8, st));
        return SAR_OK;
    }
    if (!long_row) return SAR_ERR_INVALID_ARG;
    if (!workspace || !sar_aligned(workspace, 256) || workspace_bytes < 256) return SAR_ERR_WORKSPACE;
    int *n_selected = static_cast<int *>(workspace);
    void *temp = static_cast<char *>(workspace) + 256;
    size_t temp_bytes = workspace_bytes - 256, need = 0;
    IsLongRow pred{indptr, threshold};
    thrust::counting_iterator<int> rows(0);
    SAR_CUDA_TRY(cub::DeviceSelect::If(nullptr, need, rows, long_row, n_selected, (int)n_rows, pred, st));
    if (need > temp_bytes) return SAR_ERR_WORKSPACE;
    SAR_CUDA_TRY(cub::DeviceSelect::If(temp, need, rows, long_row, n_selected, (int)n_rows, pred, st));
    plan_segcount_kernel<<<nblk(n_long + 1), 256, 0, st>>>(n_long, long_row, indptr, threshold, long_seg);
    SAR_TRY(sar_after_launch());
    SAR_CUDA_TRY(cub::DeviceScan::ExclusiveSum(nullptr, need, long_seg, long_seg, n_long + 1, st));
    if (need > temp_bytes) return SAR_ERR_WORKSPACE;
    SAR_CUDA_TRY(cub::DeviceScan::ExclusiveSum(temp, need, long_seg, long_seg, n_long + 1, st));
    return SAR_OK;
}

size_t sar_degree_order_workspace_bytes(int64_t n) {
    if (n < 0) return 0;
    return 2 * sar_round_up((size_t)n * 8, 256) + sar_round_up(sort_temp_bytes(n), 256) + sar_round_up((size_t)n * 4, 256) + 512;
}

sar_status sar_degree_order(int64_t n, int64_t e, const int32_t *src, const int32_t *dst, int32_t *order, int32_t *rank,
                            void *workspace, size_t workspace_bytes, void *stream) {
    if (n < 0 || e < 0 || (n > 0 && (!order || !rank)) || (e > 0 && (!src || !dst))) return SAR_ERR_INVALID_ARG;
    if (n > INT32_MAX) return SAR_ERR_UNSUPPORTED;
    if (!sar_aligned(src, 4) || !sar_aligned(dst, 4) || !sar_aligned(order, 4) || !sar_aligned(rank, 4)) return SAR_ERR_ALIGNMENT;
    if (n == 0) return SAR_OK;
    const size_t kb = sar_round_up((size_t)n * 8, 256), db = sar_round_up((size_t)n * 4, 256);
    if (!workspace || !sar_aligned(workspace, 256) || workspace_bytes < 2 * kb + db) return SAR_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // layout: keys | sorted keys | CUB scratch ... | degrees (last)
    unsigned *deg = reinterpret_cast<unsigned *>(static_cast<char *>(workspace) + workspace_bytes - db - (workspace_bytes - db) % 256);
    if (reinterpret_cast<char *>(deg) < static_cast<char *>(workspace) + 2 * kb) return SAR_ERR_WORKSPACE;
    const size_t sort_bytes = (size_t)(reinterpret_cast<char *>(deg) - static_cast<char *>(workspace));
    SAR_CUDA_TRY(cudaMemsetAsync(deg, 0, (size_t)n * 4, st));
    if (e > 0) {
        degree_count_kernel<<<nblk(e), 256, 0, st>>>(e, src, dst, deg);
        SAR_TRY(sar_after_launch());
    }
    unsigned long long *keys = static_cast<unsigned long long *>(workspace);
    order_keys_kernel<<<nblk(n), 256, 0, st>>>(n, deg, keys);
    SAR_TRY(sar_after_launch());
    unsigned long long *sorted = keys;
    SAR_TRY(sort_keys(n, 64, workspace, sort_bytes, st, &sorted));
    order_from_keys_kernel<<<nblk(n), 256, 0, st>>>(n, sorted, order, rank);
    return sar_after_launch();
}

sar_status sar_relabel(int64_t e, const int32_t *ids, const int32_t *rank, int32_t *out, void *stream) {
    if (e < 0 || (e > 0 && (!ids || !rank || !out))) return SAR_ERR_INVALID_ARG;
    if (!sar_aligned(ids, 4) || !sar_aligned(rank, 4) || !sar_aligned(out, 4)) return SAR_ERR_ALIGNMENT;
    if (e == 0) return SAR_OK;
    relabel_kernel<<<nblk(e), 256, 0, static_cast<cudaStream_t>(stream)>>>(e, ids, rank, out);
    return sar_after_launch();
}

sar_status sar_permute_rows(int64_t n, int64_t row_bytes, const int32_t *index, const void *in, void *out, void *stream) {
    if (n < 0 || row_bytes < 1 || (n > 0 && (!index || !in || !out))) return SAR_ERR_INVALID_ARG;
    if (in == out) return SAR_ERR_INVALID_ARG;
    if (n == 0) return SAR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (row_bytes % 16 == 0 && sar_aligned(in, 16) && sar_aligned(out, 16)) {
        const long long w = row_bytes / 16;
        permute_rows_kernel<uint4><<<nblk(n * w), 256, 0, st>>>(n, w, index, static_cast<const uint4 *>(in), static_cast<uint4 *>(out));
    } else if (row_bytes % 4 == 0 && sar_aligned(in, 4) && sar_aligned(out, 4)) {
        const long long w = row_bytes / 4;
        permute_rows_kernel<uint32_t><<<nblk(n * w), 256, 0, st>>>(n, w, index, static_cast<const uint32_t *>(in), static_cast<uint32_t *>(out));
    } else {
        permute_rows_kernel<uint8_t><<<nblk(n * row_bytes), 256, 0, st>>>(n, row_bytes, index, static_cast<const uint8_t *>(in), static_cast<uint8_t *>(out));
    }
    return sar_after_launch();
}

}  // extern "C"

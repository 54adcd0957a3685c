// Host-buffer entry point: a stack of aggregation layers with the copies inside the call.
// Contracts are in include/sar.h.
#include <mutex>
#include <vector>

#include "sar_common.cuh"

namespace {

struct Arena {
    char *base;
    size_t used, cap;
    void *take(size_t bytes) {
        const size_t b = sar_round_up(bytes, 256);
        if (used + b > cap) return nullptr;
        void *p = base + used;
        used += b;
        return p;
    }
};

// Two non-blocking side streams per device for the copies, created on first use and kept.
struct Copies {
    cudaStream_t up = nullptr, down = nullptr;
    // pipelined mode: the two halves of the arena alternate; half_done[i] follows the last result copy of the
    // latest call that used half i
    cudaEvent_t half_done[2] = {nullptr, nullptr};
    bool half_used[2] = {false, false};
    unsigned long long calls = 0;
    // held for the whole of a call: the pipelined state above is read at its start and advanced at its end, so two
    // host threads that call on the same device take turns
    std::mutex call_mutex;
};
constexpr int kMaxDevices = 64;
Copies g_copies[kMaxDevices];
std::mutex g_copies_mutex;

sar_status copies_for_current_device(Copies **out) {
    int dev = -1;
    SAR_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SAR_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_copies_mutex);
    Copies &c = g_copies[dev];
    if (!c.up) SAR_CUDA_TRY(cudaStreamCreateWithFlags(&c.up, cudaStreamNonBlocking));
    if (!c.down) SAR_CUDA_TRY(cudaStreamCreateWithFlags(&c.down, cudaStreamNonBlocking));
    for (int i = 0; i < 2; ++i)
        if (!c.half_done[i]) SAR_CUDA_TRY(cudaEventCreateWithFlags(&c.half_done[i], cudaEventDisableTiming));
    *out = &c;
    return SAR_OK;
}

size_t stack_bytes(const sar_part *g, int32_t L, int32_t H, int32_t F, sar_dtype t) {
    const size_t n = (size_t)g->n_dst;
    const size_t row = sar_round_up(n * H * F * sar_elem_size(t), 256);
    const size_t nh = sar_round_up(n * H * 4, 256);
    return (size_t)(L + 1) * row + 2 * row + (size_t)L * 6 * nh + sar_round_up(sar_gat_workspace_bytes(g, H, F, t), 256) + 256;
}

}  // namespace

extern "C" {

size_t sar_gat_stack_arena_bytes(const sar_part *g, int32_t L, int32_t H, int32_t F, sar_dtype t) {
    if (!g || L < 1 || H < 1 || F < 1) return 0;
    return stack_bytes(g, L, H, F, t);
}

sar_status sar_gat_stack_host(const sar_part *g, int32_t k, const int64_t *bounds, const sar_stack_host_io *io,
                              void *arena, size_t arena_bytes, void *stream) {
    if (!g || !io || !bounds || k < 1) return SAR_ERR_INVALID_ARG;
    const int32_t L = io->L, H = io->H, F = io->F;
    if (L < 1 || L > 64 || H < 1 || F < 1) return SAR_ERR_INVALID_ARG;
    if (g->n_dst != g->n_src) return SAR_ERR_INVALID_ARG;  // layers chain: outputs become inputs
    if (!io->feat0 || !io->el || !io->er || !io->gout) return SAR_ERR_INVALID_ARG;
    for (int l = 0; l < L; ++l)
        if (!io->el[l] || !io->er[l] || (io->del && !io->del[l]) || (io->der && !io->der[l])) return SAR_ERR_INVALID_ARG;
    if (io->flags & ~(uint32_t)SAR_STACK_PIPELINED) return SAR_ERR_INVALID_ARG;
    const bool pipelined = (io->flags & SAR_STACK_PIPELINED) != 0;
    const size_t one = sar_round_up(stack_bytes(g, L, H, F, io->t), 256);
    if (!arena || !sar_aligned(arena, 256) || arena_bytes < (pipelined ? 2 * one : one)) return SAR_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t n = (size_t)g->n_dst;
    const size_t row_b = n * H * F * sar_elem_size(io->t), nh_b = n * H * 4;

    Copies *cp = nullptr;
    SAR_TRY(copies_for_current_device(&cp));
    std::lock_guard<std::mutex> call_lock(cp->call_mutex);
    const int half = pipelined ? (int)(cp->calls & 1ull) : 0;
    Arena a{static_cast<char *>(arena) + (size_t)half * one, 0, one};
    std::vector<void *> feat(L + 1);
    std::vector<float *> el(L), er(L), m(L), d(L), del(L), der(L);
    for (int l = 0; l <= L; ++l) feat[l] = a.take(row_b);
    void *ga = a.take(row_b), *gb = a.take(row_b);
    for (int l = 0; l < L; ++l) {
        el[l] = static_cast<float *>(a.take(nh_b));
        er[l] = static_cast<float *>(a.take(nh_b));
        m[l] = static_cast<float *>(a.take(nh_b));
        d[l] = static_cast<float *>(a.take(nh_b));
        del[l] = static_cast<float *>(a.take(nh_b));
        der[l] = static_cast<float *>(a.take(nh_b));
    }
    const size_t ws_bytes = sar_gat_workspace_bytes(g, H, F, io->t);
    void *ws = a.take(ws_bytes);
    if (!ws || !gb) return SAR_ERR_WORKSPACE;

    // Copies run on two side streams of the library so that they overlap with the kernels (PCIe is full
    // duplex): `up` brings the inputs in layer order, `down` returns each result as soon as it exists.
    // Everything is ordered after the work already queued on `st`, and `st` finally waits for the last
    // copy, so that completion of `st` still means "all done".
    cudaStream_t up = cp->up, down = cp->down;
    std::vector<cudaEvent_t> ev;
    auto new_event = [&](cudaEvent_t *e) -> sar_status {
        SAR_CUDA_TRY(cudaEventCreateWithFlags(e, cudaEventDisableTiming));
        ev.push_back(*e);
        return SAR_OK;
    };
    auto cleanup = [&]() {
        for (cudaEvent_t e : ev) cudaEventDestroy(e);  // released by the runtime once the work that uses them is done
    };
#define SAR_STEP(expr)                    \
    do {                                  \
        sar_status st__ = (expr);         \
        if (st__ != SAR_OK) {             \
            cleanup();                    \
            return st__;                  \
        }                                 \
    } while (0)
#define SAR_CUDA_STEP(expr) SAR_STEP((expr) == cudaSuccess ? SAR_OK : SAR_ERR_CUDA)

    cudaEvent_t e_start, e_gout, e_done;
    std::vector<cudaEvent_t> e_in(L), e_bwd(L);
    SAR_STEP(new_event(&e_start));
    SAR_STEP(new_event(&e_gout));
    SAR_STEP(new_event(&e_done));
    for (int l = 0; l < L; ++l) {
        SAR_STEP(new_event(&e_in[l]));
        SAR_STEP(new_event(&e_bwd[l]));
    }
    if (pipelined) {
        // this half's previous user must be completely done (kernels and result copies) before anything is
        // written into it; nothing else of the earlier calls is waited for
        if (cp->half_used[half]) {
            SAR_CUDA_STEP(cudaStreamWaitEvent(up, cp->half_done[half], 0));
            SAR_CUDA_STEP(cudaStreamWaitEvent(st, cp->half_done[half], 0));
        }
    } else {
        // a plain call after pipelined ones: let those finish first (they may be using this part of the arena)
        for (int i = 0; i < 2; ++i)
            if (cp->half_used[i]) {
                SAR_CUDA_STEP(cudaStreamWaitEvent(st, cp->half_done[i], 0));
                cp->half_used[i] = false;
            }
        cp->calls = 0;
        SAR_CUDA_STEP(cudaEventRecord(e_start, st));
        SAR_CUDA_STEP(cudaStreamWaitEvent(up, e_start, 0));
        SAR_CUDA_STEP(cudaStreamWaitEvent(down, e_start, 0));
    }

    // host -> device, in the order the layers need them
    SAR_CUDA_STEP(cudaMemcpyAsync(feat[0], io->feat0, row_b, cudaMemcpyHostToDevice, up));
    for (int l = 0; l < L; ++l) {
        SAR_CUDA_STEP(cudaMemcpyAsync(el[l], io->el[l], nh_b, cudaMemcpyHostToDevice, up));
        SAR_CUDA_STEP(cudaMemcpyAsync(er[l], io->er[l], nh_b, cudaMemcpyHostToDevice, up));
        SAR_CUDA_STEP(cudaEventRecord(e_in[l], up));
    }
    SAR_CUDA_STEP(cudaMemcpyAsync(ga, io->gout, row_b, cudaMemcpyHostToDevice, up));
    SAR_CUDA_STEP(cudaEventRecord(e_gout, up));

    for (int l = 0; l < L; ++l) {
        SAR_CUDA_STEP(cudaStreamWaitEvent(st, e_in[l], 0));
        SAR_STEP(sar_gat_fwd_fused(g, k, bounds, feat[l], el[l], er[l], H, F, io->t, io->slope, m[l], d[l],
                                   feat[l + 1], ws, ws_bytes, st));
    }
    if (io->out_last) {
        cudaEvent_t e_out;
        SAR_STEP(new_event(&e_out));
        SAR_CUDA_STEP(cudaEventRecord(e_out, st));
        SAR_CUDA_STEP(cudaStreamWaitEvent(down, e_out, 0));
        SAR_CUDA_STEP(cudaMemcpyAsync(io->out_last, feat[L], row_b, cudaMemcpyDeviceToHost, down));
    }
    SAR_CUDA_STEP(cudaStreamWaitEvent(st, e_gout, 0));
    void *gin = ga, *gout = gb;
    for (int l = L - 1; l >= 0; --l) {
        SAR_STEP(sar_gat_bwd_fused(g, k, bounds, feat[l], el[l], er[l], m[l], d[l], gin, H, F, io->t, io->slope, gout,
                                   del[l], der[l], ws, ws_bytes, st));
        SAR_CUDA_STEP(cudaEventRecord(e_bwd[l], st));
        SAR_CUDA_STEP(cudaStreamWaitEvent(down, e_bwd[l], 0));
        if (io->del) SAR_CUDA_STEP(cudaMemcpyAsync(io->del[l], del[l], nh_b, cudaMemcpyDeviceToHost, down));
        if (io->der) SAR_CUDA_STEP(cudaMemcpyAsync(io->der[l], der[l], nh_b, cudaMemcpyDeviceToHost, down));
        void *tmp = gin;
        gin = gout;
        gout = tmp;
    }
    // gin now holds dfeat of layer 0 (the last backward call has been waited for by `down` above)
    if (io->dfeat0) SAR_CUDA_STEP(cudaMemcpyAsync(io->dfeat0, gin, row_b, cudaMemcpyDeviceToHost, down));
    if (pipelined) {
        // the half changes hands only once its completion event is in place: a call that failed earlier leaves the
        // parity where it was, and the next call takes the same half again
        SAR_CUDA_STEP(cudaEventRecord(cp->half_done[half], down));
        cp->half_used[half] = true;
        ++cp->calls;
    } else {
        SAR_CUDA_STEP(cudaEventRecord(e_done, down));
        SAR_CUDA_STEP(cudaStreamWaitEvent(st, e_done, 0));
    }
    cleanup();
#undef SAR_STEP
#undef SAR_CUDA_STEP
    return SAR_OK;
}

sar_status sar_gat_stack_host_wait(void *stream) {
    Copies *cp = nullptr;
    SAR_TRY(copies_for_current_device(&cp));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaEvent_t e = nullptr;
    SAR_CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    // the copy streams run their work in order, so their current ends cover every call made so far
    cudaError_t err = cudaEventRecord(e, cp->up);
    if (err == cudaSuccess) err = cudaStreamWaitEvent(st, e, 0);
    if (err == cudaSuccess) err = cudaEventRecord(e, cp->down);
    if (err == cudaSuccess) err = cudaStreamWaitEvent(st, e, 0);
    cudaEventDestroy(e);
    return err == cudaSuccess ? SAR_OK : SAR_ERR_CUDA;
}

}  // extern "C"

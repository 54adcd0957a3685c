// sar_gat_bwd_noalloc: the whole-graph backward pass for callers that cannot hand the library any
// scratch memory.  The scratch lives in a fixed array in this library's device image instead.
// Contract and rationale are in include/sar.h.
#include <mutex>

#include "sar_common.cuh"

// The scratch itself.  One copy exists on every GPU that loads the library and stays until the
// process exits.  In HOST code the name below is only a handle for the runtime (a stand-in, not a
// device address): kernels must be given the address cudaGetSymbolAddress returns for it.
static __device__ __align__(256) unsigned char g_noalloc_scratch[SAR_NOALLOC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
void *g_scratch_ptr[kMaxDevices];  // device address of the array, per device ordinal (null: not looked up yet)
std::mutex g_scratch_mutex;

// Device address of the scratch array on the CURRENT device; looked up once per device.
sar_status scratch_for_current_device(void **out) {
    int dev = -1;
    SAR_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SAR_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return SAR_ERR_CUDA;
        }
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return SAR_OK;
}

}  // namespace

extern "C" {

size_t sar_gat_bwd_noalloc_limit(void) { return SAR_NOALLOC_SCRATCH_BYTES; }

sar_status sar_gat_bwd_noalloc(const sar_part *g, const void *feat, const float *el, const float *er, const float *m,
                               const float *d, const void *gout, int32_t H, int32_t F, sar_dtype t, float slope,
                               void *dfeat, float *del, float *der, void *stream) {
    if (!g || H < 1 || F < 1) return SAR_ERR_INVALID_ARG;
    // what the ordinary entry point would ask its caller for; it must fit the fixed array
    const size_t need = sar_gat_workspace_bytes(g, H, F, t);
    if (need == 0) return SAR_ERR_INVALID_ARG;
    if (need > SAR_NOALLOC_SCRATCH_BYTES) return SAR_ERR_WORKSPACE;
    void *scratch = nullptr;
    SAR_TRY(scratch_for_current_device(&scratch));
    // Whole graph in one call: the destination-major pass writes every record and every long-row
    // partial before anything reads them, so whatever an earlier call left in the array is never read
    // and nothing has to be cleared.
    return sar_gat_bwd(g, feat, el, er, m, d, gout, H, F, t, slope, SAR_FIRST | SAR_LAST, dfeat, del, der, scratch,
                       SAR_NOALLOC_SCRATCH_BYTES, stream);
}

}  // extern "C"

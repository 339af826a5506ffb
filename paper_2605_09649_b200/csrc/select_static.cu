// trimkv_select_topk_static: the standalone global selection for callers that may not allocate.
//
// Its scratch memory is a file-scope device array that lives in the library image, so the call needs
// no workspace from the caller and performs no device or host allocation.  Host code cannot hand the
// array's name to a kernel (on the host the name is only a stand-in for the symbol); the device address
// is looked up once per device with cudaGetSymbolAddress and cached.
#include <mutex>

#include "trimkv_internal.cuh"

namespace {

// Scratch needed by the selection for n <= TRIMKV_SELECT_STATIC_MAX_N scores: the same layout and size formula as the
// workspace of trimkv_select_topk (state, histograms, the candidate list of n / 16 + 16384 keys): about 2.4 MB.
constexpr size_t STATIC_SCRATCH_BYTES = tkv::flat_select_workspace_bytes(TRIMKV_SELECT_STATIC_MAX_N);
static_assert(STATIC_SCRATCH_BYTES < (3u << 20), "the built-in scratch array is meant to stay small");

static __device__ __align__(256) unsigned char g_select_scratch[STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
std::mutex g_setup_lock;
void* g_scratch_addr[MAX_DEVICES] = {};   // device address of g_select_scratch, per device ordinal

// Device address of the scratch array on the current device; looked up on the first call per device.
cudaError_t scratch_address(void** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> guard(g_setup_lock);
    if (g_scratch_addr[dev]) {
        // a cudaDeviceReset since the look-up would have destroyed the context the address belongs to: check it still
        // names device memory (a query, no allocation) and look it up again if not
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, g_scratch_addr[dev]) != cudaSuccess || attr.type != cudaMemoryTypeDevice) {
            cudaGetLastError();
            g_scratch_addr[dev] = nullptr;
        }
    }
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_select_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" TRIMKV_API trimkv_status trimkv_select_topk_static(const float* scores, int64_t n, int64_t k_keep,
                                                              uint64_t* keep_bits, int32_t* status_out, void* stream) {
    if (n < 0) {
        tkv::set_last_error("n must not be negative");
        return TRIMKV_E_ARG;
    }
    if (n > (int64_t)TRIMKV_SELECT_STATIC_MAX_N || trimkv_select_workspace_bytes(n) > STATIC_SCRATCH_BYTES) {
        tkv::set_last_error("n = %lld exceeds the built-in scratch array's limit of %lld scores; use trimkv_select_topk "
                            "with a caller-provided workspace", (long long)n, (long long)TRIMKV_SELECT_STATIC_MAX_N);
        return TRIMKV_E_UNSUPPORTED;
    }
    void* scratch = nullptr;
    const cudaError_t e = scratch_address(&scratch);
    if (e != cudaSuccess) {
        cudaGetLastError();
        tkv::set_last_error("cudaGetSymbolAddress of the built-in scratch array failed: %s", cudaGetErrorString(e));
        return TRIMKV_E_CUDA;
    }
    // The selection's first kernel clears, on `stream`, every counter and histogram that must start at zero; the
    // candidate lists are written before they are read.
    return trimkv_select_topk(scores, n, k_keep, keep_bits, scratch, STATIC_SCRATCH_BYTES, status_out, stream);
}

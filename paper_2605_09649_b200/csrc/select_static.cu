// trimkv_select_topk_static: the standalone global selection for callers that may not allocate.
//
// Its scratch memory is a file-scope device array that lives in the library image, so the call needs
// no workspace from the caller and performs no device or host allocation.  Host code cannot hand the
// array's name to a kernel (on the host the name is only a stand-in for the symbol); the device address
// is looked up once per device with cudaGetSymbolAddress and cached.
#include <mutex>

#include "trimkv_internal.cuh"

namespace {

// Scratch needed by the selection for n <= TRIMKV_SELECT_STATIC_MAX_N scores: 1 KB of state, the
// 4096-bin histogram and 16384 candidate records of 16 bytes, plus alignment slack.
constexpr size_t STATIC_SCRATCH_BYTES = 1024 + (size_t)tkv::NB * sizeof(uint32_t) + 16384 * sizeof(tkv::Cand) + 256;

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
    // The selection clears the state words and the histogram it needs at zero on `stream` before its
    // kernels run; the candidate records are written before they are read.
    return trimkv_select_topk(scores, n, k_keep, keep_bits, scratch, STATIC_SCRATCH_BYTES, status_out, stream);
}

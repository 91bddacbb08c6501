// eta_decode_static: eta_decode for callers that cannot supply scratch memory.
//
// Some hosts of this library have no way to hand it a device buffer: a serving
// process that gave every byte of HBM to its KV-cache pool at start-up, a
// plug-in that is passed tensors but no allocator, a decode loop that must not
// enter the CUDA allocator because cudaMalloc synchronises the device and can
// fail once memory is fragmented.  For them the scratch eta_decode needs lives
// here, in a file-scope __device__ array that the CUDA module carries: it is
// reserved on every GPU on which the module gets loaded (with CUDA's default
// lazy loading: at the library's first kernel launch or symbol look-up on that
// device, so a caller makes one warm-up call before it gives the rest of the
// memory away), until the process exits, and no call allocates or frees
// anything.
#include <mutex>

#include "eta_common.cuh"

namespace eta {

constexpr size_t STATIC_SCRATCH_BYTES = ETA_STATIC_SCRATCH_BYTES;
constexpr int MAX_DEVICES = 64;

// In host code this name is only a handle for cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

static std::mutex g_static_mutex;
static void* g_static_ptr[MAX_DEVICES] = {};

// Device address of the scratch array on the current device, looked up once per device.
static int static_scratch_ptr(void** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { set_cuda_error(e, "eta_decode_static: cudaGetDevice"); return ETA_ERR_CUDA; }
    if (dev < 0 || dev >= MAX_DEVICES) return ETA_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) {
            set_cuda_error(e != cudaSuccess ? e : cudaErrorUnknown, "eta_decode_static: cudaGetSymbolAddress");
            return ETA_ERR_CUDA;
        }
        g_static_ptr[dev] = p;
    }
    *out = g_static_ptr[dev];
    return ETA_OK;
}

}  // namespace eta

extern "C" {

size_t eta_static_scratch_bytes(void) { return eta::STATIC_SCRATCH_BYTES; }

int eta_decode_static(const eta_cache_desc* desc, const eta_params* params, const void* q, const void* K,
                      const void* V, const int32_t* seq_lens, const void* musig, const float* mnorm,
                      const float* tau, const float* head_const, float* out, uint8_t* sel_mask, int32_t* stats,
                      uint32_t* status_dev, void* stream) {
    size_t need = 0;
    int rc = eta_workspace_bytes(desc, &need);
    if (rc != ETA_OK) return rc;
    if (need > eta::STATIC_SCRATCH_BYTES) return ETA_ERR_WORKSPACE;   // shape needs more scratch than is built in
    void* scratch = nullptr;
    rc = eta::static_scratch_ptr(&scratch);
    if (rc != ETA_OK) return rc;
    // every word of the scratch that a kernel reads is written earlier in the same call (counts, lists and window
    // statistics by the screening kernel, partial slots by the streaming kernel), so nothing carried over from
    // the previous call is ever consumed
    return eta_decode(desc, params, q, K, V, seq_lens, musig, mnorm, tau, head_const, out, sel_mask, stats,
                      status_dev, scratch, eta::STATIC_SCRATCH_BYTES, stream);
}

}  // extern "C"

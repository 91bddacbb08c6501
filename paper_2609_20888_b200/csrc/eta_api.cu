// Host-side plumbing of the C ABI: status text, argument validation and the
// scratch layout shared by the kernels of eta_decode.
#include <stdio.h>
#include <string.h>

#include "eta_common.cuh"

namespace eta {

static thread_local char g_cuda_error[256] = "";

void set_pdl(bool on);

void set_cuda_error(cudaError_t e, const char* where) {
    snprintf(g_cuda_error, sizeof g_cuda_error, "%s: %s", where, cudaGetErrorString(e));
}

int validate_desc(const eta_cache_desc* d) {
    if (!d) return ETA_ERR_INVALID_ARG;
    if (d->batch <= 0 || d->n_q_heads <= 0 || d->n_kv_heads <= 0 || d->t_cap <= 0 || d->nb_cap <= 0)
        return ETA_ERR_INVALID_ARG;
    if (d->n_q_heads % d->n_kv_heads != 0) return ETA_ERR_INVALID_ARG;
    int G = d->n_q_heads / d->n_kv_heads;
    if (G != 1 && G != 2 && G != 4 && G != 8) return ETA_ERR_UNSUPPORTED;
    if (d->head_dim != 64 && d->head_dim != 128) return ETA_ERR_UNSUPPORTED;
    if (d->block_size != 32 && d->block_size != 64 && d->block_size != 128) return ETA_ERR_UNSUPPORTED;
    if ((int64_t)d->nb_cap * d->block_size < d->t_cap - d->block_size + 1) return ETA_ERR_INVALID_ARG;
    if (d->nb_cap >= (1 << 24)) return ETA_ERR_UNSUPPORTED;   // block index shares a word with the head bits
    if ((int64_t)d->batch * d->n_kv_heads > MAX_ROWS) return ETA_ERR_UNSUPPORTED;
    if (d->k_stride_t % 8 || d->k_stride_h % 8 || d->k_stride_b % 8) return ETA_ERR_UNSUPPORTED;
    if (d->v_stride_t % 8 || d->v_stride_h % 8 || d->v_stride_b % 8) return ETA_ERR_UNSUPPORTED;
    if (d->k_stride_t < d->head_dim || d->v_stride_t < d->head_dim) return ETA_ERR_INVALID_ARG;
    return ETA_OK;
}

// Optional per-kernel timing: host-side CUDA events recorded between the launches of one decode step
// (append, predict, then the three kernels of eta_decode).  Event k is recorded just before launch k; event 5
// after the last launch.
constexpr int N_MARKS = 6;
static bool g_profile = false;
static cudaEvent_t g_ev[N_MARKS];
static bool g_ev_made = false;
static unsigned g_ev_seen = 0;

void profile_mark(int k, cudaStream_t s) {
    if (!g_profile) return;
    if (!g_ev_made) {
        for (int i = 0; i < N_MARKS; ++i) cudaEventCreate(&g_ev[i]);
        g_ev_made = true;
    }
    // inside a stream capture the record must be an "external" node to stay a real, timeable event at replay
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    cudaStreamIsCapturing(s, &cap);
    if (cap == cudaStreamCaptureStatusActive) cudaEventRecordWithFlags(g_ev[k], s, cudaEventRecordExternal);
    else cudaEventRecord(g_ev[k], s);
    g_ev_seen |= 1u << k;
}

static unsigned long long* g_timeline = nullptr;
unsigned long long* debug_timeline() { return g_timeline; }
static bool g_pdl = true;
bool pdl_enabled() { return g_pdl; }
void set_pdl(bool on) { g_pdl = on; }

void prefer_max_shared(const void* kernel) {
    static const void* seen[64];
    static int n_seen = 0;
    for (int k = 0; k < n_seen; ++k)
        if (seen[k] == kernel) return;
    cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (n_seen < 64) seen[n_seen++] = kernel;
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

WsLayout ws_layout(const eta_cache_desc* d) {
    WsLayout L;
    int G = d->n_q_heads / d->n_kv_heads;
    L.rows = d->batch * d->n_kv_heads;
    L.nseg = (d->nb_cap + SEG - 1) / SEG;
    L.entries = L.rows * (L.nseg + 2);
    size_t off = 0;
    L.seg_count = off;  off = align_up(off + sizeof(int32_t) * (size_t)L.rows * L.nseg, 256);
    L.seg_list = off;   off = align_up(off + sizeof(int32_t) * (size_t)L.rows * L.nseg * LSTRIDE, 256);
    L.seg_resc = off;   off = align_up(off + sizeof(RescueRec) * (size_t)L.rows * L.nseg * G, 256);
    L.row_span = off;   off = align_up(off + sizeof(int2) * (size_t)L.rows, 256);
    L.tau_eff = off;    off = align_up(off + sizeof(float) * (size_t)d->batch * d->n_q_heads, 256);
    size_t slots = ((size_t)MAX_CTAS + L.rows) * DECODE_GROUPS;
    L.part_ml = off;    off = align_up(off + sizeof(float2) * slots * G, 256);
    L.part_o = off;     off = align_up(off + sizeof(float) * slots * G * d->head_dim, 256);
    L.total = off;
    return L;
}

}  // namespace eta

extern "C" {

int eta_workspace_bytes(const eta_cache_desc* desc, size_t* out_bytes) {
    if (!out_bytes) return ETA_ERR_INVALID_ARG;
    int rc = eta::validate_desc(desc);
    if (rc != ETA_OK) return rc;
    *out_bytes = eta::ws_layout(desc).total;
    return ETA_OK;
}

const char* eta_strerror(int code) {
    switch (code) {
        case ETA_OK: return "ok";
        case ETA_ERR_INVALID_ARG: return "invalid argument";
        case ETA_ERR_UNSUPPORTED: return "unsupported shape or alignment";
        case ETA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case ETA_ERR_CUDA: return "CUDA error (see eta_last_cuda_error)";
        default: return "unknown status";
    }
}

const char* eta_last_cuda_error(void) { return eta::g_cuda_error; }

int eta_debug_timeline(void* dev_buffer) {
    eta::g_timeline = static_cast<unsigned long long*>(dev_buffer);
    return ETA_OK;
}

int eta_set_pdl(int on) {
    eta::set_pdl(on != 0);
    return ETA_OK;
}

int eta_profile_enable(int on) {
    if (on && !eta::g_profile) eta::g_ev_seen = 0;     // a new profiled run starts; a finished one stays readable
    eta::g_profile = on != 0;
    return ETA_OK;
}

int eta_profile_read(float* ms, int n) {
    using namespace eta;
    if (!ms || n < N_MARKS - 1) return ETA_ERR_INVALID_ARG;
    if ((g_ev_seen & 0x3c) != 0x3c) return ETA_ERR_INVALID_ARG;      // no profiled eta_decode yet
    cudaError_t e = cudaEventSynchronize(g_ev[5]);
    for (int k = 0; k < N_MARKS - 1 && e == cudaSuccess; ++k) {
        ms[k] = 0.f;
        // append / predict are separate calls: timed only when they were made in the same profiled step; an
        // interval runs to the next mark that was recorded
        if (!((g_ev_seen >> k) & 1)) continue;
        int j = k + 1;
        while (j < N_MARKS - 1 && !((g_ev_seen >> j) & 1)) ++j;
        e = cudaEventElapsedTime(&ms[k], g_ev[k], g_ev[j]);
    }
    if (e != cudaSuccess) { set_cuda_error(e, "eta_profile_read"); return ETA_ERR_CUDA; }
    return N_MARKS - 1;
}

const char* eta_profile_kernel_name(int k) {
    static const char* names[5] = {"append_summary_kernel", "predict_threshold_kernel", "screen_kernel",
                                   "decode_kernel", "merge_kernel"};
    return (k >= 0 && k < 5) ? names[k] : "";
}

}  // extern "C"

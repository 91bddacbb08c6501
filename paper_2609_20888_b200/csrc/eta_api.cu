// Host-side plumbing of the C ABI: status text, argument validation and the
// scratch layout shared by the kernels of eta_decode.
#include <stdio.h>
#include <string.h>

#include <mutex>

#include "eta_common.cuh"
#include "eta_timeline.h"

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
static std::mutex g_profile_mutex;       // the marks are process-wide state: serialised, meant for one measuring thread
static bool g_profile = false;
static cudaEvent_t g_ev[N_MARKS];
static bool g_ev_made = false;
static unsigned g_ev_seen = 0;

void profile_mark(int k, cudaStream_t s) {
    if (!g_profile) return;
    std::lock_guard<std::mutex> lock(g_profile_mutex);
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

#ifdef ETA_TIMELINE
static unsigned long long* g_timeline = nullptr;
unsigned long long* debug_timeline() { return g_timeline; }
#endif
static bool g_pdl = true;
bool pdl_enabled() { return g_pdl; }
void set_pdl(bool on) { g_pdl = on; }

// ---- per-device kernel attributes
// cudaFuncAttributeMaxDynamicSharedMemorySize and the shared-memory carve-out belong to a (device, kernel) pair: a
// process that uses a second GPU has to set them there again.  The table below remembers, per device ordinal and
// kernel, the dynamic shared memory already granted and whether the carve-out was asked for; look-ups and updates
// are serialised by a mutex (two host threads may launch at once).  The setter is a parameter so that the
// bookkeeping can be exercised without a device.
int KernelAttrTable::configure(int dev, const void* kernel, size_t dyn_smem, Setter set, void* ctx) {
    std::lock_guard<std::mutex> lock(mu_);
    Entry* e = nullptr;
    if (dev >= 0 && dev < MAX_DEVICES) {
        for (int k = 0; k < n_[dev]; ++k)
            if (tab_[dev][k].kernel == kernel) e = &tab_[dev][k];
        if (!e && n_[dev] < MAX_KERNELS) {
            e = &tab_[dev][n_[dev]++];
            e->kernel = kernel; e->smem = 0; e->carveout = false;
        }
    }
    // a device or kernel beyond the table's capacity is configured on every call: slower, never wrong
    if (!e || !e->carveout) {
        const int rc = set(ctx, kernel, ATTR_CARVEOUT, 0);
        if (rc != 0) return rc;
        if (e) e->carveout = true;
    }
    if (dyn_smem > DEFAULT_DYN_SMEM && (!e || dyn_smem > e->smem)) {
        const int rc = set(ctx, kernel, ATTR_MAX_DYN_SMEM, dyn_smem);
        if (rc != 0) return rc;
        if (e) e->smem = dyn_smem;
    }
    return 0;
}

static KernelAttrTable g_attr_table;

static int cuda_setter(void*, const void* kernel, int attr, size_t value) {
    const cudaError_t e = (attr == KernelAttrTable::ATTR_CARVEOUT)
        ? cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared)
        : cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)value);
    if (e != cudaSuccess) { set_cuda_error(e, "kernel attribute"); return ETA_ERR_CUDA; }
    return 0;
}

int configure_kernel(const void* kernel, size_t dyn_smem) {
    int dev = 0;
    const cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { set_cuda_error(e, "cudaGetDevice"); return ETA_ERR_CUDA; }
    return g_attr_table.configure(dev, kernel, dyn_smem, cuda_setter, nullptr);
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

// Host-only check of the per-device attribute bookkeeping with a recording setter and made-up device ordinals
// (no device is touched).  Not part of the public interface; called by the CPU test-suite.  -> 0, or the number of
// the first expectation that failed.
int eta_selftest_kernel_attr_table(void) {
    using T = eta::KernelAttrTable;
    struct Log { int carve = 0, smem = 0; size_t last = 0; } log;
    auto rec = [](void* ctx, const void*, int attr, size_t v) {
        Log* l = static_cast<Log*>(ctx);
        if (attr == T::ATTR_CARVEOUT) ++l->carve; else { ++l->smem; l->last = v; }
        return 0;
    };
    static T t;                        // own instance: the library's table is left alone
    int ka = 0, kb = 0;
    const void *A = &ka, *B = &kb;
    if (t.configure(0, A, 200 * 1024, rec, &log) != 0 || log.carve != 1 || log.smem != 1) return 1;
    if (t.configure(0, A, 200 * 1024, rec, &log) != 0 || log.carve != 1 || log.smem != 1) return 2;   // remembered
    if (t.configure(1, A, 200 * 1024, rec, &log) != 0 || log.carve != 2 || log.smem != 2) return 3;   // second device: again
    if (t.configure(1, A, 100 * 1024, rec, &log) != 0 || log.smem != 2) return 4;                      // smaller: nothing
    if (t.configure(1, A, 220 * 1024, rec, &log) != 0 || log.smem != 3 || log.last != 220 * 1024) return 5;
    if (t.configure(0, B, 16 * 1024, rec, &log) != 0 || log.carve != 3 || log.smem != 3) return 6;     // under 48 KB: carve-out only
    if (t.configure(T::MAX_DEVICES + 3, A, 200 * 1024, rec, &log) != 0 || log.carve != 4 || log.smem != 4) return 7;
    if (t.configure(T::MAX_DEVICES + 3, A, 200 * 1024, rec, &log) != 0 || log.carve != 5 || log.smem != 5) return 8;  // untracked: every call
    auto fail = [](void*, const void*, int, size_t) { return -4; };
    int kc = 0;
    if (t.configure(2, &kc, 200 * 1024, fail, nullptr) != -4) return 9;
    if (t.configure(2, &kc, 200 * 1024, rec, &log) != 0 || log.carve != 6 || log.smem != 6) return 10;  // a failure is not remembered
    return 0;
}

#ifdef ETA_TIMELINE
int eta_debug_timeline(void* dev_buffer) {
    eta::g_timeline = static_cast<unsigned long long*>(dev_buffer);
    return ETA_OK;
}
#endif

int eta_set_pdl(int on) {
    eta::set_pdl(on != 0);
    return ETA_OK;
}

int eta_profile_enable(int on) {
    std::lock_guard<std::mutex> lock(eta::g_profile_mutex);
    if (on && !eta::g_profile) eta::g_ev_seen = 0;     // a new profiled run starts; a finished one stays readable
    eta::g_profile = on != 0;
    return ETA_OK;
}

int eta_profile_read(float* ms, int n) {
    using namespace eta;
    if (!ms || n < N_MARKS - 1) return ETA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_profile_mutex);
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

// Shared declarations of the ETA decode library: status plumbing, the scratch
// layout every kernel of eta_decode agrees on, and thin wrappers over the PTX
// the kernels use (mbarrier, bulk / tensor TMA copies, warp MMA).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>
#include <utility>

#include "../../include/eta.h"

namespace eta {

// ---------------------------------------------------------------- host side
void set_cuda_error(cudaError_t e, const char* where);
inline int check_launch(const char* where) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_cuda_error(e, where); return ETA_ERR_CUDA; }
    return ETA_OK;
}
int validate_desc(const eta_cache_desc* d);
int validate_pages(const eta_cache_desc* desc, const eta_page_table* pages);
// Measurement aid: when profiling is enabled, records timing event k on the stream (see eta_profile_enable).
void profile_mark(int k, cudaStream_t s);

// Screening works on segments of SEG consecutive block records of one
// (sequence, KV head) row; a segment's survivors are compacted into a list of
// LSTRIDE slots (SEG plus room for one rescued block per query head).
constexpr int SEG = 64;
constexpr int LSTRIDE = SEG + 8;
constexpr int MAX_CTAS = 256;        // upper bound on streaming CTAs (sizes the scratch; a B200 has 148 SMs)
constexpr int MAX_ROWS = 1024;        // rows (batch * n_kv_heads) whose unit prefix a streaming CTA keeps in shared memory
constexpr int DECODE_GROUPS = 3;     // consumer groups per streaming CTA, each with its own partial per piece

// Scratch layout (byte offsets from a 256-byte aligned base).
struct WsLayout {
    int rows;        // batch * n_kv_heads
    int nseg;        // segments per row
    int entries;     // rows * (nseg + 2): per row its segments, a rescue pseudo-entry and a tail pseudo-entry
    size_t seg_count;   // int32 [rows * nseg]
    size_t seg_list;    // int32 [rows * nseg * LSTRIDE]: block index | head bits << 24
    size_t seg_resc;    // {int cnt; float maxb; int arg; int pad} [rows * nseg * G]
    size_t row_span;    // int2 [rows]: first streaming CTA that holds units of the row, number of such CTAs (written by the streaming kernel)
    size_t tau_eff;     // float [batch * n_q_heads]
    size_t part_ml;     // float2 [(MAX_CTAS + rows) * DECODE_GROUPS * G]
    size_t part_o;      // float [(MAX_CTAS + rows) * DECODE_GROUPS * G * d]
    size_t total;
};
WsLayout ws_layout(const eta_cache_desc* d);

struct RescueRec { int cnt; float maxb; int arg; int pad; };

// Division by a run-time constant as multiply-high + shift (exact for 0 <= n < 2^31): integer division costs
// dozens of instructions, and the single-warp set-up code of the kernels divides by the same few numbers.
struct FastDiv {
    uint32_t d, mul, shr;
    FastDiv() : d(1), mul(0), shr(0) {}
    explicit FastDiv(int divisor) : d((uint32_t)divisor), mul(0), shr(0) {
        if (d > 1) {
            uint32_t lg = 0;
            while ((1ull << lg) < d) ++lg;
            const uint32_t p = 31 + lg;
            mul = (uint32_t)(((1ull << p) + d - 1) / d);
            shr = p - 32;
        }
    }
#ifdef __CUDACC__
    __device__ __forceinline__ int div(int n) const { return d == 1 ? n : (int)(__umulhi((uint32_t)n, mul) >> shr); }
    __device__ __forceinline__ void divmod(int n, int& q, int& r) const { q = div(n); r = n - q * (int)d; }
#endif
};



// Arguments of the screening kernel (defined in eta_screen.cu, launched from eta_decode).
struct ScreenArgs {
    const __nv_bfloat16* q;
    const __half* musig;
    const float* mnorm;
    const int32_t* seq_lens;
    const float* tau;
    const float* head_const;
    float z, a, scale;
    int lwb, rescue_window;
    uint32_t flags;
    int Hq, Hkv, b, b_shift, t_cap, nb_cap, nseg, rows;
    int n_early, per_early, per_late;     // item split over the CTAs: the first n_early share per_early items evenly, the rest take per_late each
    FastDiv div_nseg, div_hkv;
    int32_t* seg_count;
    int32_t* seg_list;
    RescueRec* seg_resc;
    float* tau_eff;
    uint8_t* sel_mask;
    uint32_t* status;
    unsigned long long* timeline;
};
int launch_screen(const ScreenArgs& a, int rows, int D, int G, int n_ctas, cudaStream_t s);

// Launch with programmatic dependent launch allowed: the grid may start while its predecessor in the stream is
// still draining, and must call pdl_wait() before touching anything the predecessor wrote.
// Per-CTA %globaltimer stamps exist in development builds only (-DETA_TIMELINE, see eta_timeline.h): in the shipped
// build ETA_TL() is a constant null pointer, so every `if (tl && ...)` below it is compiled out.
#ifdef ETA_TIMELINE
#define ETA_TL(expr) (expr)
unsigned long long* debug_timeline();   // device buffer for the stamps, or nullptr
#else
#define ETA_TL(expr) (static_cast<unsigned long long*>(nullptr))
inline unsigned long long* debug_timeline() { return nullptr; }
#endif
bool pdl_enabled();          // false after eta_set_pdl(0): every launch is then fully serialised
// Per-(device, kernel) attribute set-up, remembered per device ordinal under a mutex (see eta_api.cu).
// Every kernel of a step asks for the largest shared-memory carve-out: the streaming kernel needs it, and when its
// neighbours in the stream run with another split of the SM's L1/shared memory, an SM has to drain and reconfigure
// before the first CTA of the next kernel can start on it, which showed as ~2 us between the last CTA of one kernel
// and the first of the next.  None of the kernels of a step depends on L1 capacity.  dyn_smem above 48 KB is granted
// with cudaFuncAttributeMaxDynamicSharedMemorySize.  -> ETA_OK or ETA_ERR_CUDA.
int configure_kernel(const void* kernel, size_t dyn_smem);

class KernelAttrTable {
public:
    static constexpr int MAX_DEVICES = 64, MAX_KERNELS = 64;
    static constexpr size_t DEFAULT_DYN_SMEM = 48 * 1024;
    enum { ATTR_CARVEOUT = 0, ATTR_MAX_DYN_SMEM = 1 };
    typedef int (*Setter)(void* ctx, const void* kernel, int attr, size_t value);
    int configure(int dev, const void* kernel, size_t dyn_smem, Setter set, void* ctx);
private:
    struct Entry { const void* kernel; size_t smem; bool carveout; };
    std::mutex mu_;
    Entry tab_[MAX_DEVICES][MAX_KERNELS] = {};
    int n_[MAX_DEVICES] = {};
};

template <typename... KArgs, typename... Args>
inline int launch_pdl(const char* what, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                      Args&&... args) {
    const int rc = configure_kernel(reinterpret_cast<const void*>(kernel), smem);
    if (rc != ETA_OK) return rc;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl_enabled() ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
    if (e != cudaSuccess) { set_cuda_error(e, what); return ETA_ERR_CUDA; }
    return check_launch(what);
}

// -------------------------------------------------------------- device side
#ifdef __CUDACC__

// Programmatic dependent launch: let the next kernel of the stream start its prologue now / wait until the
// previous kernel of the stream has completed and its writes are visible.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

#ifndef ETA_WAIT_LIMIT
#define ETA_WAIT_LIMIT (1u << 24)
#endif
constexpr uint32_t WAIT_LIMIT = ETA_WAIT_LIMIT;   // polls before a bounded wait gives up

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false when the limit ran out (the caller then abandons the work
// and reports ETA_DEV_TIMEOUT instead of spinning forever).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it >= 2) __nanosleep(40);      // leave the issue slots to the warps that have work
    }
    return false;
}

// 1-D bulk copy global -> shared, completion counted on an mbarrier.
// Both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void tma_load_1d(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// 4-D tiled copy global -> shared through a tensor map, into this CTA's shared memory only.
__device__ __forceinline__ void tma_load_4d(void* dst, const void* tmap, int x, int y, int z, int w, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(tmap), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
// 5-D tiled copy (this CTA's shared memory only): used with the head_dim split into 64-column halves as an extra dimension, so one
// instruction brings both swizzled half tiles of a K or V tile.
__device__ __forceinline__ void tma_load_5d(void* dst, const void* tmap, int c0, int c1, int c2, int c3, int c4,
                                            uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.5d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(tmap), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const void* tmap) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(tmap) : "memory");
}

// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
// (d0, d1) += (a0, a1) * (b0, b1): the packed fp32 fma of sm_100, two independent round-to-nearest fmas per issue
__device__ __forceinline__ void fma2(float& d0, float& d1, float a0, float a1, float b0, float b1) {
    asm("{\n\t.reg .b64 ra, rb, rc;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%0, %1};\n\t"
        "fma.rn.f32x2 rc, ra, rb, rc;\n\t"
        "mov.b64 {%0, %1}, rc;\n\t}"
        : "+f"(d0), "+f"(d1) : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}

// (d0, d1) += (a0, a1): the packed fp32 add of sm_100
__device__ __forceinline__ void add2(float& d0, float& d1, float a0, float a1) {
    asm("{\n\t.reg .b64 ra, rc;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rc, {%0, %1};\n\t"
        "add.rn.f32x2 rc, rc, ra;\n\t"
        "mov.b64 {%0, %1}, rc;\n\t}"
        : "+f"(d0), "+f"(d1) : "f"(a0), "f"(a1));
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void mma_f16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ int ld_volatile(const int* p) { return *reinterpret_cast<const volatile int*>(p); }
__device__ __forceinline__ void st_volatile(int* p, int v) { *reinterpret_cast<volatile int*>(p) = v; }

// e4m3 (8-bit float: 4 exponent bits, 3 fraction bits, largest finite value 448, 0x7f = NaN), the storage type of sigma in
// packed summaries.  Two values at a time -> fp16 (exact: every e4m3 value is an fp16 value).
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t two_bytes) {
    uint32_t r;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"((unsigned short)two_bytes));
    return r;
}
// eight e4m3 values (bytes 0 .. 7 of v) -> fp32, in order
__device__ __forceinline__ void e4m3x8_to_f32(uint2 v, float (&out)[8]) {
    const uint32_t h[4] = {e4m3x2_to_f16x2(v.x & 0xffffu), e4m3x2_to_f16x2(v.x >> 16), e4m3x2_to_f16x2(v.y & 0xffffu),
                           e4m3x2_to_f16x2(v.y >> 16)};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&h[k]));
        out[2 * k] = f.x; out[2 * k + 1] = f.y;
    }
}
// The smallest e4m3 value that is >= x, for x >= 0 (rounding toward +infinity: a packed sigma must not fall below
// the sigma it stands for); x above 448 or NaN gives the NaN code, which the screening rule reads as "admit".
__device__ __forceinline__ uint32_t f32_to_e4m3_up(float x) {
    if (!(x <= 448.f)) return 0x7fu;
    unsigned short pair;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(pair) : "f"(0.f), "f"(x));        // low byte: nearest to x
    uint32_t code = pair & 0xffu;
    const uint32_t back = e4m3x2_to_f16x2(code);
    const float nearest = __half2float(*reinterpret_cast<const __half*>(&back));
    return nearest < x ? code + 1u : code;      // positive codes ascend with their values
}

__device__ __forceinline__ float bf16_lo(uint32_t p) { return __uint_as_float(p << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t p) { return __uint_as_float(p & 0xffff0000u); }

#endif  // __CUDACC__
}  // namespace eta

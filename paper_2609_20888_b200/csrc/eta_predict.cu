// Threshold predictor, Eq. tau_pred: tau = qbar W + bias with qbar the
// head-major concatenation of the post-RoPE query heads of one sequence.
//
// W is small (n_q_heads^2 * head_dim floats) but a decode step waits for tau, so
// the kernel is built for latency, not bandwidth: the rows of W are split over
// the CTAs of a thread-block cluster (one cluster per sequence) so that no SM
// reads more than 1/8 of W and every thread has all of its loads in flight at
// once; the per-CTA partial sums meet in the shared memory of the cluster's
// first CTA and are added there in a fixed order, so the result does not depend
// on scheduling.
#include <cooperative_groups.h>

#include <stdint.h>

#include "eta_common.cuh"
#include "eta_timeline.h"

namespace cg = cooperative_groups;

namespace eta {

constexpr int PRED_THREADS = 512;
constexpr int PRED_CLUSTER = 8;

__global__ void __launch_bounds__(PRED_THREADS) predict_threshold_kernel(
    const __nv_bfloat16* __restrict__ q, const float* __restrict__ W, const float* __restrict__ bias,
    float* __restrict__ tau, int Hq, int rows, int vec4, unsigned long long* timeline) {
    extern __shared__ float sm[];
    unsigned long long* const tl = ETA_TL((timeline && blockIdx.y * PRED_CLUSTER + blockIdx.x < TL_PREDICT_N)
                                              ? timeline + (size_t)(TL_PREDICT + blockIdx.y * PRED_CLUSTER + blockIdx.x) * 8 : nullptr);
    if (tl && threadIdx.x == 0) tl[0] = globaltimer_ns();
    const int NRG = PRED_THREADS / Hq;           // row groups inside a CTA
    float* part = sm;                            // [max(NRG, warps)][Hq] partial sums of this CTA
    float* cpart = sm + max(NRG, PRED_THREADS / 32) * Hq;      // [PRED_CLUSTER][Hq], used in the cluster's first CTA
    pdl_trigger();
    cg::cluster_group cluster = cg::this_cluster();
    const int crank = (int)cluster.block_rank();
    const int i = blockIdx.y;
    const int per_cta = (rows + PRED_CLUSTER - 1) / PRED_CLUSTER;
    const int r_begin = crank * per_cta, r_end = min(rows, r_begin + per_cta);
    const __nv_bfloat16* qi = q + (int64_t)i * rows;
    const int h = threadIdx.x % Hq, rg = threadIdx.x / Hq;

    if (vec4) {
        // Four heads per thread: a row of W is read as 16-byte pieces, so a warp instruction covers 512 bytes and the
        // CTA needs a quarter of the load instructions of the scalar form (the kernel's time is the number of requests
        // its SM's load unit has to take, not bytes).  Thread (rl, cg): heads 4 cg .. 4 cg + 3 of rows rl, rl + RL, ...
        const int CG = Hq >> 2, RL = PRED_THREADS / CG;
        const int cg4 = threadIdx.x % CG, rl = threadIdx.x / CG;
        float a4[4] = {0.f, 0.f, 0.f, 0.f};
        if (rl < RL) {
            for (int r0 = r_begin + rl; r0 < r_end; r0 += 8 * RL) {
                float4 w[8];
                float x[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int r = min(r0 + k * RL, r_end - 1);
                    w[k] = __ldg(reinterpret_cast<const float4*>(W + (int64_t)r * Hq) + cg4);
                    x[k] = (r0 + k * RL < r_end) ? __bfloat162float(qi[r]) : 0.f;
                }
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    a4[0] = fmaf(x[k], w[k].x, a4[0]);
                    a4[1] = fmaf(x[k], w[k].y, a4[1]);
                    a4[2] = fmaf(x[k], w[k].z, a4[2]);
                    a4[3] = fmaf(x[k], w[k].w, a4[3]);
                }
            }
        }
        // rows of one warp first (lanes that share cg: exchanges at distance CG, 2 CG, ...), then the warps in order
        for (int s = CG; s < 32; s <<= 1) {
#pragma unroll
            for (int j = 0; j < 4; ++j) a4[j] += __shfl_xor_sync(0xffffffffu, a4[j], s);
        }
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        if (lane < CG) {
#pragma unroll
            for (int j = 0; j < 4; ++j) part[warp * Hq + 4 * lane + j] = a4[j];
        }
        if (tl && threadIdx.x == 0) tl[1] = globaltimer_ns();
        __syncthreads();
        if (tl && threadIdx.x == 0) tl[2] = globaltimer_ns();
        if (threadIdx.x < Hq) {
            float s = 0.f;
            for (int k = 0; k < PRED_THREADS / 32; ++k) s += part[k * Hq + threadIdx.x];
            float* dst = cluster.map_shared_rank(cpart, 0);
            dst[crank * Hq + threadIdx.x] = s;
        }
    } else {
        // any other number of heads: a head per thread, sixteen loads in flight per pass
        float acc = 0.f;
        if (rg < NRG) {
            for (int r0 = r_begin + rg; r0 < r_end; r0 += 16 * NRG) {
                float w[16], x[16];
#pragma unroll
                for (int k = 0; k < 16; ++k) {
                    const int r = r0 + k * NRG;
                    const bool in = r < r_end;
                    w[k] = in ? __ldg(W + (int64_t)r * Hq + h) : 0.f;
                    x[k] = in ? __bfloat162float(qi[r]) : 0.f;
                }
#pragma unroll
                for (int k = 0; k < 16; ++k) acc = fmaf(x[k], w[k], acc);
            }
            part[rg * Hq + h] = acc;
        }
        if (tl && threadIdx.x == 0) tl[1] = globaltimer_ns();
        __syncthreads();
        if (tl && threadIdx.x == 0) tl[2] = globaltimer_ns();
        if (threadIdx.x < Hq) {
            float s = 0.f;
            for (int k = 0; k < NRG; ++k) s += part[k * Hq + threadIdx.x];
            float* dst = cluster.map_shared_rank(cpart, 0);
            dst[crank * Hq + threadIdx.x] = s;
        }
    }
    cluster.sync();
    if (tl && threadIdx.x == 0) tl[3] = globaltimer_ns();
    if (crank == 0 && threadIdx.x < Hq) {
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < PRED_CLUSTER; ++c) s += cpart[c * Hq + threadIdx.x];
        tau[(int64_t)i * Hq + threadIdx.x] = s + bias[threadIdx.x];
    }
    if (tl && threadIdx.x == 0) tl[4] = globaltimer_ns();
    if (threadIdx.x == 0) pdl_wait();
    if (tl && threadIdx.x == 0) tl[5] = globaltimer_ns();
}

// Copy of a step's queries from page-locked host memory to device memory by a kernel: for a few tens of
// kilobytes a kernel's loads over the interconnect cost less than setting up a copy engine.  The kernel never
// signals its dependents early, so whatever follows it in the stream starts after the copy is complete.
__global__ void __launch_bounds__(256) stage_query_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, int n16) {
    for (int k = blockIdx.x * blockDim.x + threadIdx.x; k < n16; k += gridDim.x * blockDim.x) {
        uint4 v;
        asm volatile("ld.global.cv.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(src + k));
        dst[k] = v;
    }
}

}  // namespace eta

extern "C" int eta_stage_query(int32_t batch, int32_t n_q_heads, int32_t head_dim, const void* q_host, void* q_dev,
                               void* stream) {
    if (!q_host || !q_dev || batch <= 0 || n_q_heads <= 0 || head_dim <= 0) return ETA_ERR_INVALID_ARG;
    const size_t bytes = (size_t)batch * n_q_heads * head_dim * 2;
    if (bytes % 16 || ((uintptr_t)q_host & 15) || ((uintptr_t)q_dev & 15)) return ETA_ERR_UNSUPPORTED;
    if (bytes / 16 > 0x7fffffffu) return ETA_ERR_UNSUPPORTED;
    const int n16 = (int)(bytes / 16);
    int grid = (n16 + 255) / 256;
    if (grid > 296) grid = 296;
    const int rc = eta::configure_kernel(reinterpret_cast<const void*>(eta::stage_query_kernel), 0);
    if (rc != ETA_OK) return rc;
    eta::stage_query_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const uint4*>(q_host),
                                                                                 static_cast<uint4*>(q_dev), n16);
    return eta::check_launch("eta_stage_query");
}

extern "C" int eta_predict_threshold(int32_t batch, int32_t n_q_heads, int32_t head_dim, const void* q,
                                     const float* W, const float* bias, float* tau, void* stream) {
    if (!q || !W || !bias || !tau) return ETA_ERR_INVALID_ARG;
    if (batch <= 0 || n_q_heads <= 0 || head_dim <= 0) return ETA_ERR_INVALID_ARG;
    if (n_q_heads > eta::PRED_THREADS || batch > 65535) return ETA_ERR_UNSUPPORTED;
    const int rows = n_q_heads * head_dim;
    const int NRG = eta::PRED_THREADS / n_q_heads;
    const int part_rows = NRG > eta::PRED_THREADS / 32 ? NRG : eta::PRED_THREADS / 32;
    const size_t smem = sizeof(float) * ((size_t)part_rows * n_q_heads + (size_t)eta::PRED_CLUSTER * n_q_heads);
    // four heads per thread need a power-of-two head count (4 .. 128) and 16-byte aligned rows of W
    const int vec4 = (n_q_heads >= 4 && n_q_heads <= 128 && (n_q_heads & (n_q_heads - 1)) == 0 &&
                      (reinterpret_cast<uintptr_t>(W) & 15) == 0) ? 1 : 0;
    if (smem > 48 * 1024) return ETA_ERR_UNSUPPORTED;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(eta::PRED_CLUSTER, batch, 1);
    cfg.blockDim = dim3(eta::PRED_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = eta::PRED_CLUSTER;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // the predictor reads nothing an earlier kernel of the stream writes, so it may run beside its predecessor
    // (typically the summary append); it only waits for it before it exits, which keeps "this kernel is complete"
    // meaning "everything before it is complete" for whoever comes next
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = eta::pdl_enabled() ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    const int rc = eta::configure_kernel(reinterpret_cast<const void*>(eta::predict_threshold_kernel), smem);
    if (rc != ETA_OK) return rc;
    eta::profile_mark(1, cfg.stream);
    cudaError_t e = cudaLaunchKernelEx(&cfg, eta::predict_threshold_kernel, static_cast<const __nv_bfloat16*>(q), W,
                                       bias, tau, (int)n_q_heads, rows, vec4, eta::debug_timeline());
    if (e != cudaSuccess) { eta::set_cuda_error(e, "eta_predict_threshold"); return ETA_ERR_CUDA; }
    return eta::check_launch("eta_predict_threshold");
}

// Threshold predictor, Eq. tau_pred: tau = qbar W + bias with qbar the
// head-major concatenation of the post-RoPE query heads of one sequence.
//
// One CTA per sequence.  Thread (rg, h) accumulates column h of W over the rows
// r = rg, rg + NRG, ... so that a warp reads whole rows of W (coalesced), then
// the NRG partial sums of a column are added in a fixed order: the result does
// not depend on scheduling.
#include "eta_common.cuh"

namespace eta {

constexpr int PRED_THREADS = 1024;

__global__ void __launch_bounds__(PRED_THREADS) predict_threshold_kernel(
    const __nv_bfloat16* __restrict__ q, const float* __restrict__ W, const float* __restrict__ bias,
    float* __restrict__ tau, int Hq, int rows) {
    extern __shared__ float sm[];
    float* qs = sm;                 // [rows] the concatenated query in fp32
    float* part = sm + rows;        // [NRG][Hq]
    const int i = blockIdx.x;
    const __nv_bfloat16* qi = q + (int64_t)i * rows;
    for (int r = threadIdx.x; r < rows; r += PRED_THREADS) qs[r] = __bfloat162float(qi[r]);
    __syncthreads();
    const int NRG = PRED_THREADS / Hq;
    const int h = threadIdx.x % Hq, rg = threadIdx.x / Hq;
    float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
    if (rg < NRG) {
        int r = rg;
        for (; r + 3 * NRG < rows; r += 4 * NRG) {
            float w0 = __ldg(W + (int64_t)r * Hq + h);
            float w1 = __ldg(W + (int64_t)(r + NRG) * Hq + h);
            float w2 = __ldg(W + (int64_t)(r + 2 * NRG) * Hq + h);
            float w3 = __ldg(W + (int64_t)(r + 3 * NRG) * Hq + h);
            acc0 = fmaf(qs[r], w0, acc0);
            acc1 = fmaf(qs[r + NRG], w1, acc1);
            acc2 = fmaf(qs[r + 2 * NRG], w2, acc2);
            acc3 = fmaf(qs[r + 3 * NRG], w3, acc3);
        }
        for (; r < rows; r += NRG) acc0 = fmaf(qs[r], __ldg(W + (int64_t)r * Hq + h), acc0);
        part[rg * Hq + h] = (acc0 + acc1) + (acc2 + acc3);
    }
    __syncthreads();
    if (threadIdx.x < Hq) {
        float s = 0.f;
        for (int g = 0; g < NRG; ++g) s += part[g * Hq + threadIdx.x];
        tau[(int64_t)i * Hq + threadIdx.x] = s + bias[threadIdx.x];
    }
}

}  // namespace eta

extern "C" int eta_predict_threshold(int32_t batch, int32_t n_q_heads, int32_t head_dim, const void* q,
                                     const float* W, const float* bias, float* tau, void* stream) {
    if (!q || !W || !bias || !tau) return ETA_ERR_INVALID_ARG;
    if (batch <= 0 || n_q_heads <= 0 || head_dim <= 0) return ETA_ERR_INVALID_ARG;
    if (n_q_heads > eta::PRED_THREADS) return ETA_ERR_UNSUPPORTED;
    const int rows = n_q_heads * head_dim;
    const int NRG = eta::PRED_THREADS / n_q_heads;
    const size_t smem = sizeof(float) * ((size_t)rows + (size_t)NRG * n_q_heads);
    if (smem > 48 * 1024) return ETA_ERR_UNSUPPORTED;
    eta::predict_threshold_kernel<<<batch, eta::PRED_THREADS, smem, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const __nv_bfloat16*>(q), W, bias, tau, n_q_heads, rows);
    return eta::check_launch("eta_predict_threshold");
}

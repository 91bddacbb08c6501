// Offline threshold calibration (appendix "Offline Threshold Calibration via
// 1/t-Weighted Histograms", Algorithm "Density-Matched Offline Threshold
// Calibration"): one pass over a calibration split builds, per query head, the
// 1/t-weighted histogram of the raw causal scores S_ts = s <q_t, k_s> and the
// density the dynamic thresholds realise; a bisection on the histogram then
// finds the static constant with the same density.
//
// calib_hist_kernel: a CTA per (64-query tile, head, sequence).  The scores of a
// 64 x 64 tile are a small dense contraction and go through the tensor cores
// (mma.m16n8k16, bf16 in, fp32 out; the whole pass is a few GFLOP, so nothing
// heavier is warranted); each score is binned into a histogram in shared memory.
// The causal row weight 1/t is added as the integer round(2^40 / t), so the
// histogram does not depend on the order in which the atomics land; the gates
// sigmoid(beta (S - tau_t)) are summed per row and reduced in a fixed order.
// calib_bisect_kernel: a CTA per head normalises the histogram and bisects
// g(c) = sum_b H[b] sigmoid(beta (s_b - c)) = dbar in double precision.
#include "eta_common.cuh"

namespace eta {

constexpr int CAL_TILE = 64;          // queries and keys per tile
constexpr int CAL_THREADS = 128;      // four warps: 16 query rows each
constexpr int CAL_WSHIFT = 40;        // row weights are integers: round(2^40 / t)
constexpr int CAL_BISECT_THREADS = 256;

template <int D>
__global__ void __launch_bounds__(CAL_THREADS) calib_hist_kernel(
    const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K, const float* __restrict__ tau,
    int Hq, int Hkv, int T, float beta, float scale, int n_bins, float s_min, float inv_w,
    unsigned long long* __restrict__ hist, double* __restrict__ dpart) {
    constexpr int KS = D + 8;            // padded row of the key tile: conflict-free fragment reads
    extern __shared__ unsigned char cal_raw[];
    __nv_bfloat16* sK = reinterpret_cast<__nv_bfloat16*>(cal_raw);
    unsigned long long* sh = reinterpret_cast<unsigned long long*>(cal_raw + CAL_TILE * KS * 2);
    __shared__ double s_red[CAL_THREADS / 32];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, tq = lane & 3;
    const int ttile = blockIdx.x, h = blockIdx.y, x = blockIdx.z;
    const int hk = h / (Hq / Hkv);
    const int t0 = ttile * CAL_TILE;
    const __nv_bfloat16* Qh = Q + (((int64_t)x * Hq + h) * T) * D;
    const __nv_bfloat16* Kh = K + (((int64_t)x * Hkv + hk) * T) * D;
    const float* tauh = tau + ((int64_t)x * Hq + h) * T;

    for (int b = tid; b < n_bins; b += CAL_THREADS) sh[b] = 0ull;

    // this thread's two query rows and their A fragments (row-major 16 x 16 per k-step)
    const int r0 = t0 + warp * 16 + g, r1 = r0 + 8;
    uint32_t qa[D / 16][4];
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
        const int c = 16 * kk + 2 * tq;
        qa[kk][0] = (r0 < T) ? *reinterpret_cast<const uint32_t*>(Qh + (int64_t)r0 * D + c) : 0u;
        qa[kk][1] = (r1 < T) ? *reinterpret_cast<const uint32_t*>(Qh + (int64_t)r1 * D + c) : 0u;
        qa[kk][2] = (r0 < T) ? *reinterpret_cast<const uint32_t*>(Qh + (int64_t)r0 * D + c + 8) : 0u;
        qa[kk][3] = (r1 < T) ? *reinterpret_cast<const uint32_t*>(Qh + (int64_t)r1 * D + c + 8) : 0u;
    }
    const float tau0 = (r0 < T) ? tauh[r0] : 0.f, tau1 = (r1 < T) ? tauh[r1] : 0.f;
    // t counts from 1: row index r is decoding step t = r + 1
    const unsigned long long w0 = (r0 < T) ? (((1ull << CAL_WSHIFT) + (unsigned)(r0 + 1) / 2) / (unsigned)(r0 + 1)) : 0ull;
    const unsigned long long w1 = (r1 < T) ? (((1ull << CAL_WSHIFT) + (unsigned)(r1 + 1) / 2) / (unsigned)(r1 + 1)) : 0ull;
    double gate0 = 0.0, gate1 = 0.0;       // sum of the gates of the two rows

    for (int s0 = 0; s0 <= t0 && s0 < T; s0 += CAL_TILE) {
        __syncthreads();                   // the previous tile has been read (and the histogram is zeroed)
        // key tile -> shared memory, 16 bytes at a time; rows past the end read as zero
        for (int p = tid; p < CAL_TILE * (D / 8); p += CAL_THREADS) {
            const int row = p / (D / 8), piece = p % (D / 8);
            uint4 v = make_uint4(0, 0, 0, 0);
            if (s0 + row < T) v = *reinterpret_cast<const uint4*>(Kh + (int64_t)(s0 + row) * D + piece * 8);
            *reinterpret_cast<uint4*>(sK + row * KS + piece * 8) = v;
        }
        __syncthreads();
#pragma unroll 2
        for (int nn = 0; nn < CAL_TILE / 8; ++nn) {
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            const __nv_bfloat16* krow = sK + (nn * 8 + g) * KS + 2 * tq;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t b0 = *reinterpret_cast<const uint32_t*>(krow + 16 * kk);
                const uint32_t b1 = *reinterpret_cast<const uint32_t*>(krow + 16 * kk + 8);
                mma_bf16_16816(acc, qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], b0, b1);
            }
            // acc[0], acc[1]: row r0, keys col, col + 1; acc[2], acc[3]: row r1
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int r = (e < 2) ? r0 : r1;
                const int sidx = s0 + nn * 8 + 2 * tq + (e & 1);
                if (r < T && sidx <= r) {
                    const float S = acc[e] * scale;
                    int b = (int)floorf((S - s_min) * inv_w);
                    b = b < 0 ? 0 : (b >= n_bins ? n_bins - 1 : b);
                    atomicAdd(&sh[b], (e < 2) ? w0 : w1);
                    const float m = 1.f / (1.f + __expf(-beta * (S - ((e < 2) ? tau0 : tau1))));
                    if (e < 2) gate0 += (double)m; else gate1 += (double)m;
                }
            }
        }
    }
    __syncthreads();
    // density contribution of this tile: sum over its rows of (1/t) * (sum of the row's gates), fixed order
    double dsum = 0.0;
    if (r0 < T) dsum += gate0 / (double)(r0 + 1);
    if (r1 < T) dsum += gate1 / (double)(r1 + 1);
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, s);
    if (lane == 0) s_red[warp] = dsum;
    for (int b = tid; b < n_bins; b += CAL_THREADS) {
        const unsigned long long v = sh[b];
        if (v) atomicAdd(&hist[(int64_t)h * n_bins + b], v);
    }
    __syncthreads();
    if (tid == 0) {
        double tot = 0.0;
        for (int w = 0; w < CAL_THREADS / 32; ++w) tot += s_red[w];
        dpart[((int64_t)x * Hq + h) * gridDim.x + ttile] = tot;
    }
}

__device__ __forceinline__ double sigmoid_d(double v) {
    if (v >= 0) return 1.0 / (1.0 + exp(-v));
    const double e = exp(v);
    return e / (1.0 + e);
}

// Fixed-order sum of one value per thread over the block; every thread gets the result.
__device__ double block_sum_fixed(double v, double* scratch) {
    const int tid = threadIdx.x;
    scratch[tid] = v;
    __syncthreads();
    for (int s = CAL_BISECT_THREADS / 2; s >= 1; s >>= 1) {
        if (tid < s) scratch[tid] += scratch[tid + s];
        __syncthreads();
    }
    const double r = scratch[0];
    __syncthreads();
    return r;
}

__global__ void __launch_bounds__(CAL_BISECT_THREADS) calib_bisect_kernel(
    const unsigned long long* __restrict__ hist, const double* __restrict__ dpart, int Hq, int n_seq, int n_ttiles,
    int T, int n_bins, double s_min, double s_max, double beta, int iters, float* __restrict__ head_const,
    float* __restrict__ dbar_out, double* __restrict__ head_const_d) {
    extern __shared__ unsigned char bis_raw[];
    double* Hn = reinterpret_cast<double*>(bis_raw);
    __shared__ double scratch[CAL_BISECT_THREADS];
    __shared__ double s_lo, s_hi;
    const int tid = threadIdx.x, h = blockIdx.x;
    const unsigned long long* Hh = hist + (int64_t)h * n_bins;

    // total weight (an integer: exact whatever the order), then the normalised histogram
    unsigned long long part = 0;
    for (int b = tid; b < n_bins; b += CAL_BISECT_THREADS) part += Hh[b];
    __shared__ unsigned long long s_tot[CAL_BISECT_THREADS];
    s_tot[tid] = part;
    __syncthreads();
    for (int s = CAL_BISECT_THREADS / 2; s >= 1; s >>= 1) {
        if (tid < s) s_tot[tid] += s_tot[tid + s];
        __syncthreads();
    }
    const double tot = (double)s_tot[0];
    for (int b = tid; b < n_bins; b += CAL_BISECT_THREADS) Hn[b] = tot > 0.0 ? (double)Hh[b] / tot : 0.0;
    // target density: partial sums of every (sequence, tile) of this head, in a fixed order
    double d = 0.0;
    for (int k = tid; k < n_seq * n_ttiles; k += CAL_BISECT_THREADS) {
        const int x = k / n_ttiles, tt = k % n_ttiles;
        d += dpart[((int64_t)x * Hq + h) * n_ttiles + tt];
    }
    const double target = block_sum_fixed(d, scratch) / ((double)n_seq * (double)T);

    const double w = (s_max - s_min) / n_bins;
    if (tid == 0) { s_lo = s_min - 40.0 / beta; s_hi = s_max + 40.0 / beta; }
    __syncthreads();
    for (int it = 0; it < iters; ++it) {
        const double mid = 0.5 * (s_lo + s_hi);
        double gsum = 0.0;
        for (int b = tid; b < n_bins; b += CAL_BISECT_THREADS)
            gsum += Hn[b] * sigmoid_d(beta * (s_min + (b + 0.5) * w - mid));
        const double gmid = block_sum_fixed(gsum, scratch);
        if (tid == 0) { if (gmid > target) s_lo = mid; else s_hi = mid; }
        __syncthreads();
    }
    if (tid == 0) {
        const double c = 0.5 * (s_lo + s_hi);
        head_const[h] = (float)c;
        if (dbar_out) dbar_out[h] = (float)target;
        if (head_const_d) head_const_d[h] = c;
    }
}

static size_t cal_align(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace eta

extern "C" {

int eta_calibration_workspace_bytes(int32_t n_seq, int32_t seq_len, int32_t n_q_heads, int32_t n_bins,
                                    size_t* out_bytes) {
    if (!out_bytes || n_seq <= 0 || seq_len <= 0 || n_q_heads <= 0 || n_bins < 2) return ETA_ERR_INVALID_ARG;
    const size_t n_ttiles = (size_t)(seq_len + eta::CAL_TILE - 1) / eta::CAL_TILE;
    *out_bytes = eta::cal_align(sizeof(unsigned long long) * (size_t)n_q_heads * n_bins) +
                 eta::cal_align(sizeof(double) * (size_t)n_seq * n_q_heads * n_ttiles) +
                 eta::cal_align(sizeof(double) * (size_t)n_q_heads);
    return ETA_OK;
}

int eta_calibrate_head_const(int32_t n_seq, int32_t seq_len, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                             const void* Q, const void* K, const float* tau, float beta, float scale, int32_t n_bins,
                             float s_min, float s_max, float* head_const, float* dbar, void* workspace,
                             size_t workspace_bytes, void* stream) {
    using namespace eta;
    if (!Q || !K || !tau || !head_const) return ETA_ERR_INVALID_ARG;
    if (n_seq <= 0 || seq_len <= 0 || n_q_heads <= 0 || n_kv_heads <= 0 || n_q_heads % n_kv_heads != 0)
        return ETA_ERR_INVALID_ARG;
    if (!(beta > 0.f) || !(s_max > s_min) || n_bins < 2) return ETA_ERR_INVALID_ARG;
    if ((head_dim != 64 && head_dim != 128) || n_bins > 4096 || n_seq > 65535 || n_q_heads > 65535)
        return ETA_ERR_UNSUPPORTED;
    if ((int64_t)n_seq * seq_len > (1ll << 22)) return ETA_ERR_UNSUPPORTED;        // keeps the integer weights in 64 bits
    if ((reinterpret_cast<uintptr_t>(Q) | reinterpret_cast<uintptr_t>(K)) & 15) return ETA_ERR_UNSUPPORTED;
    size_t need = 0;
    int rc = eta_calibration_workspace_bytes(n_seq, seq_len, n_q_heads, n_bins, &need);
    if (rc != ETA_OK) return rc;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < need) return ETA_ERR_WORKSPACE;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int n_ttiles = (seq_len + CAL_TILE - 1) / CAL_TILE;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    unsigned long long* hist = reinterpret_cast<unsigned long long*>(ws);
    const size_t hist_bytes = cal_align(sizeof(unsigned long long) * (size_t)n_q_heads * n_bins);
    double* dpart = reinterpret_cast<double*>(ws + hist_bytes);
    double* hc_d = reinterpret_cast<double*>(ws + hist_bytes + cal_align(sizeof(double) * (size_t)n_seq * n_q_heads * n_ttiles));
    cudaError_t e = cudaMemsetAsync(hist, 0, hist_bytes, s);
    if (e != cudaSuccess) { set_cuda_error(e, "calibration memset"); return ETA_ERR_CUDA; }

    const float sc = scale > 0.f ? scale : 1.0f / sqrtf((float)head_dim);
    const float inv_w = (float)n_bins / (s_max - s_min);
    const dim3 grid((unsigned)n_ttiles, (unsigned)n_q_heads, (unsigned)n_seq);
    const size_t smem = (size_t)CAL_TILE * (head_dim + 8) * 2 + sizeof(unsigned long long) * (size_t)n_bins;
    auto Qp = static_cast<const __nv_bfloat16*>(Q);
    auto Kp = static_cast<const __nv_bfloat16*>(K);
    if (head_dim == 128) {
        rc = configure_kernel(reinterpret_cast<const void*>(calib_hist_kernel<128>), 64 * 1024);
        if (rc != ETA_OK) return rc;
        calib_hist_kernel<128><<<grid, CAL_THREADS, smem, s>>>(Qp, Kp, tau, n_q_heads, n_kv_heads, seq_len, beta, sc,
                                                               n_bins, s_min, inv_w, hist, dpart);
    } else {
        rc = configure_kernel(reinterpret_cast<const void*>(calib_hist_kernel<64>), 64 * 1024);
        if (rc != ETA_OK) return rc;
        calib_hist_kernel<64><<<grid, CAL_THREADS, smem, s>>>(Qp, Kp, tau, n_q_heads, n_kv_heads, seq_len, beta, sc,
                                                              n_bins, s_min, inv_w, hist, dpart);
    }
    rc = check_launch("calibration histogram");
    if (rc != ETA_OK) return rc;
    calib_bisect_kernel<<<n_q_heads, CAL_BISECT_THREADS, sizeof(double) * (size_t)n_bins, s>>>(
        hist, dpart, n_q_heads, n_seq, n_ttiles, seq_len, n_bins, (double)s_min, (double)s_max, (double)beta, 80,
        head_const, dbar, hc_d);
    return check_launch("calibration bisection");
}

}  // extern "C"

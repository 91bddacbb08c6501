// Block-summary kernels: the dual probabilistic-geometric index of Section 3
// (centroid, coordinate-wise population standard deviation, largest key norm),
// built in one pass over K at prefill and extended by one block whenever a
// decode step completes a block.
//
// One CTA of eight warps owns one block of b keys; warp w takes the b/8
// consecutive rows [w*b/8, (w+1)*b/8).  A row of d bf16 values is read by d/8
// lanes as 16-byte vectors, every load of the block is issued before the first
// one is used (one HBM round trip per block, which is what the per-step append
// waits for), and the block stays in registers for the second pass (deviations
// about the mean), so K is read from HBM exactly once.  Warp partials meet in
// shared memory and are added in a fixed order.  Arithmetic is fp32.
#include "eta_common.cuh"

namespace eta {

constexpr int SUM_WARPS = 8;
constexpr int SUM_THREADS = 32 * SUM_WARPS;

// NLW: 16-byte pieces per lane = (b / SUM_WARPS) / (rows per warp instruction)
template <int D, int NLW>
__device__ __forceinline__ void summarize_block_cta(const __nv_bfloat16* __restrict__ blk, int64_t stride_t,
                                                    bool envelope, __half* __restrict__ rec, float* __restrict__ mn) {
    constexpr int LPR = D / 8;            // lanes per row
    constexpr int RPP = 32 / LPR;         // rows per warp instruction
    constexpr int RPW = NLW * RPP;        // rows per warp
    constexpr int b = RPW * SUM_WARPS;
    static_assert(RPW % 4 == 0, "a warp must own whole 4-token sub-blocks");
    __shared__ float psum[SUM_WARPS][D];
    __shared__ float pdev[SUM_WARPS][D];
    __shared__ float pmax[SUM_WARPS];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int cc = lane % LPR, ro = lane / LPR;
    const __nv_bfloat16* base = blk + (int64_t)(warp * RPW + ro) * stride_t + cc * 8;
    uint4 v[NLW];
#pragma unroll
    for (int k = 0; k < NLW; ++k) v[k] = __ldg(reinterpret_cast<const uint4*>(base + (int64_t)(k * RPP) * stride_t));

    // pass 1: coordinate sums and the largest row norm of this warp's rows
    float sum[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) sum[k] = 0.f;
    float maxn2 = 0.f;
#pragma unroll
    for (int u = 0; u < NLW; ++u) {
        const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
        float n2 = 0.f;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float lo = bf16_lo(w[k]), hi = bf16_hi(w[k]);
            sum[2 * k] += lo;
            sum[2 * k + 1] += hi;
            n2 = fmaf(lo, lo, n2);
            n2 = fmaf(hi, hi, n2);
        }
#pragma unroll
        for (int s = 1; s < LPR; s <<= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, s);
        maxn2 = fmaxf(maxn2, n2);
    }
#pragma unroll
    for (int s = LPR; s < 32; s <<= 1) {
#pragma unroll
        for (int k = 0; k < 8; ++k) sum[k] += __shfl_xor_sync(0xffffffffu, sum[k], s);
        maxn2 = fmaxf(maxn2, __shfl_xor_sync(0xffffffffu, maxn2, s));
    }
    if (ro == 0) {
#pragma unroll
        for (int k = 0; k < 8; ++k) psum[warp][cc * 8 + k] = sum[k];
    }
    if (lane == 0) pmax[warp] = maxn2;
    __syncthreads();
    float mean[8];
    const float inv_b = 1.0f / (float)b;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < SUM_WARPS; ++w) s += psum[w][cc * 8 + k];
        mean[k] = s * inv_b;
    }

    // pass 2, from registers: squared deviations about the block mean; per 4-token sub-block for the envelope
    float dev[8], sub[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) { dev[k] = 0.f; sub[k] = 0.f; }
#pragma unroll
    for (int u = 0; u < NLW; ++u) {
        const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float dl = bf16_lo(w[k]) - mean[2 * k], dh = bf16_hi(w[k]) - mean[2 * k + 1];
            sub[2 * k] = fmaf(dl, dl, sub[2 * k]);
            sub[2 * k + 1] = fmaf(dh, dh, sub[2 * k + 1]);
        }
        if ((u + 1) % (4 / RPP) == 0) {
            // the row groups of the warp together hold one whole 4-token sub-block here
            if (envelope) {
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    float s4 = sub[k];
#pragma unroll
                    for (int s = LPR; s < 32; s <<= 1) s4 += __shfl_xor_sync(0xffffffffu, s4, s);
                    dev[k] = fmaxf(dev[k], s4);       // envelope: largest sub-block sum
                    sub[k] = 0.f;
                }
            } else {
#pragma unroll
                for (int k = 0; k < 8; ++k) { dev[k] += sub[k]; sub[k] = 0.f; }
            }
        }
    }
    if (!envelope) {
#pragma unroll
        for (int s = LPR; s < 32; s <<= 1) {
#pragma unroll
            for (int k = 0; k < 8; ++k) dev[k] += __shfl_xor_sync(0xffffffffu, dev[k], s);
        }
    }
    if (ro == 0) {
#pragma unroll
        for (int k = 0; k < 8; ++k) pdev[warp][cc * 8 + k] = dev[k];
    }
    __syncthreads();

    // one thread per coordinate writes mu and sigma (two coalesced runs of the record); thread 0 writes M
    const int c = threadIdx.x;
    if (c < D) {
        float s = 0.f, d2 = 0.f;
#pragma unroll
        for (int w = 0; w < SUM_WARPS; ++w) {
            s += psum[w][c];
            d2 = envelope ? fmaxf(d2, pdev[w][c]) : d2 + pdev[w][c];
        }
        rec[c] = __float2half_rn(s * inv_b);
        rec[D + c] = __float2half_rn(envelope ? sqrtf(d2 * 0.25f) : sqrtf(d2 * inv_b));
    }
    if (threadIdx.x == 0) {
        float m2 = 0.f;
#pragma unroll
        for (int w = 0; w < SUM_WARPS; ++w) m2 = fmaxf(m2, pmax[w]);
        *mn = sqrtf(m2);
    }
}

template <int D>
__device__ __forceinline__ void summarize_dispatch(const __nv_bfloat16* blk, int64_t st, int b, bool envelope,
                                                   __half* rec, float* mn) {
    constexpr int RPP = 32 / (D / 8);
    const int nlw = b / SUM_WARPS / RPP;       // b in {32, 64, 128}: 1, 2, 4 (d=64) or 2, 4, 8 (d=128)
    if (nlw == 1) {
        if constexpr (RPP == 4) summarize_block_cta<D, 1>(blk, st, envelope, rec, mn);
    } else if (nlw == 2) {
        summarize_block_cta<D, 2>(blk, st, envelope, rec, mn);
    } else if (nlw == 4) {
        summarize_block_cta<D, 4>(blk, st, envelope, rec, mn);
    } else if (nlw == 8) {
        if constexpr (RPP == 2) summarize_block_cta<D, 8>(blk, st, envelope, rec, mn);
    }
}

template <int D>
__global__ void __launch_bounds__(SUM_THREADS) build_summaries_kernel(
    const __nv_bfloat16* __restrict__ K, int64_t sb, int64_t sh, int64_t st, int Hkv, int b, int t_cap, int nb_cap,
    int nb_max, const int32_t* __restrict__ seq_lens, int envelope, __half* __restrict__ musig,
    float* __restrict__ mnorm) {
    const int j = blockIdx.x, r = blockIdx.y;
    const int i = r / Hkv, hk = r % Hkv;
    int T = seq_lens[i];
    T = T < 0 ? 0 : (T > t_cap ? t_cap : T);
    if (j >= T / b || j >= nb_cap) return;
    const __nv_bfloat16* blk = K + i * sb + hk * sh + (int64_t)j * b * st;
    const int64_t rec = (int64_t)r * nb_cap + j;
    summarize_dispatch<D>(blk, st, b, envelope != 0, musig + rec * 2 * D, mnorm + rec);
}

template <int D>
__global__ void __launch_bounds__(SUM_THREADS) append_summary_kernel(
    const __nv_bfloat16* __restrict__ K, int64_t sb, int64_t sh, int64_t st, int Hkv, int b, int t_cap, int nb_cap,
    const int32_t* __restrict__ seq_lens, int envelope, __half* __restrict__ musig, float* __restrict__ mnorm) {
    const int r = blockIdx.x;
    const int i = r / Hkv, hk = r % Hkv;
    pdl_trigger();       // nothing later in a decode step needs this kernel's output before it has waited for it
    const int T = seq_lens[i];
    if (T <= 0 || T > t_cap || T % b != 0) return;
    const int j = T / b - 1;
    if (j >= nb_cap) return;
    const __nv_bfloat16* blk = K + i * sb + hk * sh + (int64_t)j * b * st;
    const int64_t rec = (int64_t)r * nb_cap + j;
    summarize_dispatch<D>(blk, st, b, envelope != 0, musig + rec * 2 * D, mnorm + rec);
}

}  // namespace eta

extern "C" {

int eta_build_block_summaries(const eta_cache_desc* desc, const void* K, const int32_t* seq_lens, void* musig,
                              float* mnorm, uint32_t flags, void* stream) {
    int rc = eta::validate_desc(desc);
    if (rc != ETA_OK) return rc;
    if (!K || !seq_lens || !musig || !mnorm) return ETA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(musig)) & 15) return ETA_ERR_UNSUPPORTED;
    const int rows = desc->batch * desc->n_kv_heads;
    const int nb_max = desc->t_cap / desc->block_size;
    if (nb_max == 0) return ETA_OK;
    if (rows > 65535) return ETA_ERR_UNSUPPORTED;
    dim3 grid(nb_max, rows);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int env = (flags & ETA_BUILD_SIGMA_ENVELOPE) ? 1 : 0;
    auto Kp = static_cast<const __nv_bfloat16*>(K);
    auto mp = static_cast<__half*>(musig);
    if (desc->head_dim == 128)
        eta::build_summaries_kernel<128><<<grid, eta::SUM_THREADS, 0, s>>>(Kp, desc->k_stride_b, desc->k_stride_h,
            desc->k_stride_t, desc->n_kv_heads, desc->block_size, desc->t_cap, desc->nb_cap, nb_max, seq_lens, env, mp,
            mnorm);
    else
        eta::build_summaries_kernel<64><<<grid, eta::SUM_THREADS, 0, s>>>(Kp, desc->k_stride_b, desc->k_stride_h,
            desc->k_stride_t, desc->n_kv_heads, desc->block_size, desc->t_cap, desc->nb_cap, nb_max, seq_lens, env, mp,
            mnorm);
    return eta::check_launch("eta_build_block_summaries");
}

int eta_append_summary(const eta_cache_desc* desc, const void* K, const int32_t* seq_lens_after, void* musig,
                       float* mnorm, uint32_t flags, void* stream) {
    int rc = eta::validate_desc(desc);
    if (rc != ETA_OK) return rc;
    if (!K || !seq_lens_after || !musig || !mnorm) return ETA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(musig)) & 15) return ETA_ERR_UNSUPPORTED;
    const int rows = desc->batch * desc->n_kv_heads;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int env = (flags & ETA_BUILD_SIGMA_ENVELOPE) ? 1 : 0;
    auto Kp = static_cast<const __nv_bfloat16*>(K);
    auto mp = static_cast<__half*>(musig);
    eta::profile_mark(0, s);
    if (desc->head_dim == 128)
        eta::append_summary_kernel<128><<<rows, eta::SUM_THREADS, 0, s>>>(Kp, desc->k_stride_b, desc->k_stride_h,
            desc->k_stride_t, desc->n_kv_heads, desc->block_size, desc->t_cap, desc->nb_cap, seq_lens_after, env, mp,
            mnorm);
    else
        eta::append_summary_kernel<64><<<rows, eta::SUM_THREADS, 0, s>>>(Kp, desc->k_stride_b, desc->k_stride_h,
            desc->k_stride_t, desc->n_kv_heads, desc->block_size, desc->t_cap, desc->nb_cap, seq_lens_after, env, mp,
            mnorm);
    return eta::check_launch("eta_append_summary");
}

}  // extern "C"

// Block-summary kernels: the dual probabilistic-geometric index of Section 3
// (centroid, coordinate-wise population standard deviation, largest key norm),
// built in one pass over K at prefill and extended by one block whenever a
// decode step completes a block.
//
// One warp owns one block of b keys.  A row of d bf16 values is read by d/8
// lanes as 16-byte vectors, so a warp covers 32/(d/8) rows per load
// instruction and every 32-byte sector of the block is requested exactly once
// from HBM; eight such loads are in flight per lane.  The plain sigma needs
// one pass (deviations about the block's first key); the sub-block envelope
// takes a second pass (deviations about the mean) that re-reads the block
// from L1/L2.  Arithmetic is fp32.  Build and append share these routines, so
// appending a block gives the same bytes as rebuilding the index.
#include "eta_common.cuh"
#include "eta_timeline.h"

namespace eta {

// One pass over the block for centroid, sigma and the largest norm: squared deviations are taken about the block's
// first key k0 instead of the (not yet known) mean,
//   mu = S / b,   sigma^2 = S2 / b - (mu - k0)^2,   S = sum k,  S2 = sum (k - k0)^2,
// which is exact for identical keys and loses only a factor 1 + (mu - k0)^2 / sigma^2 (a few units for a key drawn
// from the block) of fp32's 24 bits against the fp16 the result is stored in.  The centroid comes from the plain
// sum: bf16 keys have 8 significant bits, so fp32 partial sums of a block's keys are exact or nearly so, which the
// shifted sum (whose partial sums grow like t (mu - k0)) would not be for a centroid close to zero.  Packed fp32
// arithmetic: two coordinates per issue.
//
// Lane (cc, ro) of a warp holds the 16-byte piece cc of the rows ro, ro + RPP, ... (RPP = 32 / (d / 8) rows per
// warp instruction) and adds them up in ascending order; the two or four row groups meet in a shuffle tree at the
// end.  The prefill build (a warp per block) and the append (four warps per block) go through the same three
// routines below in the same order, so appending a block gives the bytes rebuilding it would.

// minus the coordinates of the block's first key, for this lane's piece
__device__ __forceinline__ void first_key_negated(const uint4& v0, float (&nk0)[8]) {
    const uint32_t w[4] = {v0.x, v0.y, v0.z, v0.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) { nk0[2 * k] = -bf16_lo(w[k]); nk0[2 * k + 1] = -bf16_hi(w[k]); }
}

// squared norm of a row: this lane's piece first, then the LPR lanes of the row
template <int LPR>
__device__ __forceinline__ float row_norm2(const uint4& v) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    float na = 0.f, nb = 0.f;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float lo = bf16_lo(w[k]), hi = bf16_hi(w[k]);
        fma2(na, nb, lo, hi, lo, hi);
    }
    float n2 = na + nb;
#pragma unroll
    for (int s = 1; s < LPR; s <<= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, s);
    return n2;
}

// adds one row's piece to the running coordinate sums s1 and shifted squared sums s2
__device__ __forceinline__ void accumulate_row(const uint4& v, const float (&nk0)[8], float (&s1)[8], float (&s2)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float lo = bf16_lo(w[k]), hi = bf16_hi(w[k]);
        add2(s1[2 * k], s1[2 * k + 1], lo, hi);
        float dl = lo, dh = hi;
        add2(dl, dh, nk0[2 * k], nk0[2 * k + 1]);
        fma2(s2[2 * k], s2[2 * k + 1], dl, dh, dl, dh);
    }
}

// Lane (cc, ro < 2) stores its piece of a record: row group 0 the centroid's piece cc (fp16), row group 1 sigma's.
// Compact layout: mu fp16[d] | sigma fp16[d]; packed layout: mu fp16[d] | sigma e4m3[d], sigma rounded up.
template <int D>
__device__ __forceinline__ void store_record_piece(unsigned char* __restrict__ rec, bool packed, int ro, int cc,
                                                   const float (&src)[8]) {
    if (ro == 1 && packed) {
        uint32_t c[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) c[k] = f32_to_e4m3_up(src[k]);
        uint2 o;
        o.x = c[0] | (c[1] << 8) | (c[2] << 16) | (c[3] << 24);
        o.y = c[4] | (c[5] << 8) | (c[6] << 16) | (c[7] << 24);
        *reinterpret_cast<uint2*>(rec + 2 * D + cc * 8) = o;
        return;
    }
    __half2 h[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) h[k] = __floats2half2_rn(src[2 * k], src[2 * k + 1]);
    uint4 o;
    o.x = *reinterpret_cast<uint32_t*>(&h[0]);
    o.y = *reinterpret_cast<uint32_t*>(&h[1]);
    o.z = *reinterpret_cast<uint32_t*>(&h[2]);
    o.w = *reinterpret_cast<uint32_t*>(&h[3]);
    *reinterpret_cast<uint4*>(rec + ro * 2 * D + cc * 16) = o;
}

// row groups meet, then mean / sigma / largest norm are stored: one contiguous record
template <int D>
__device__ __forceinline__ void finish_block(float (&s1)[8], float (&s2)[8], float maxn2, const float (&nk0)[8], int b,
                                             unsigned char* __restrict__ rec, bool packed, float* __restrict__ mn) {
    constexpr int LPR = D / 8;
    const int lane = threadIdx.x & 31;
    const int cc = lane % LPR, ro = lane / LPR;
#pragma unroll
    for (int s = LPR; s < 32; s <<= 1) {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            s1[k] += __shfl_xor_sync(0xffffffffu, s1[k], s);
            s2[k] += __shfl_xor_sync(0xffffffffu, s2[k], s);
        }
        maxn2 = fmaxf(maxn2, __shfl_xor_sync(0xffffffffu, maxn2, s));
    }
    const float inv_b = 1.0f / (float)b;
    if (ro < 2) {
        float src[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const float mean = s1[k] * inv_b;
            const float m1 = mean + nk0[k];
            src[k] = (ro == 0) ? mean : sqrtf(fmaxf(fmaf(-m1, m1, s2[k] * inv_b), 0.f));
        }
        store_record_piece<D>(rec, packed, ro, cc, src);
    }
    if (lane == 0) *mn = sqrtf(maxn2);
}

// A warp summarises a block straight from global memory, eight rows per lane in flight (the throughput-bound
// prefill build: many warps per SM hide the latency).
template <int D>
__device__ __forceinline__ void summarize_block_onepass(const __nv_bfloat16* __restrict__ blk, int64_t stride_t, int b,
                                                        unsigned char* __restrict__ rec, bool packed, float* __restrict__ mn) {
    constexpr int LPR = D / 8;        // lanes per row
    constexpr int RPP = 32 / LPR;     // rows per pass
    const int lane = threadIdx.x & 31;
    const int cc = lane % LPR, ro = lane / LPR;
    const __nv_bfloat16* base = blk + cc * 8;

    float nk0[8];
    first_key_negated(__ldg(reinterpret_cast<const uint4*>(base)), nk0);
    float s1[8], s2[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) { s1[k] = 0.f; s2[k] = 0.f; }
    float maxn2 = 0.f;
    for (int t0 = ro; t0 < b; t0 += 8 * RPP) {      // b is a multiple of 8 * RPP for every supported block size
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = __ldg(reinterpret_cast<const uint4*>(base + (int64_t)(t0 + u * RPP) * stride_t));
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            // row_norm2 and accumulate_row in one sweep over the row's words (the same operations on the same
            // operands; written out so that a word is unpacked once)
            const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
            float na = 0.f, nb = 0.f;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float lo = bf16_lo(w[k]), hi = bf16_hi(w[k]);
                fma2(na, nb, lo, hi, lo, hi);
                add2(s1[2 * k], s1[2 * k + 1], lo, hi);
                float dl = lo, dh = hi;
                add2(dl, dh, nk0[2 * k], nk0[2 * k + 1]);
                fma2(s2[2 * k], s2[2 * k + 1], dl, dh, dl, dh);
            }
            float n2 = na + nb;
#pragma unroll
            for (int s = 1; s < LPR; s <<= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, s);
            maxn2 = fmaxf(maxn2, n2);
        }
    }
    finish_block<D>(s1, s2, maxn2, nk0, b, rec, packed, mn);
}

// b is a multiple of 8 * (rows per warp instruction) for every supported block size, so the loops need no guards.
template <int D, bool envelope>
__device__ __forceinline__ void summarize_block_t(const __nv_bfloat16* __restrict__ blk, int64_t stride_t, int b,
                                                  unsigned char* __restrict__ rec, bool packed, float* __restrict__ mn) {
    constexpr int LPR = D / 8;        // lanes per row
    constexpr int RPP = 32 / LPR;     // rows per pass
    const int lane = threadIdx.x & 31;
    const int cc = lane % LPR, ro = lane / LPR;
    const __nv_bfloat16* base = blk + cc * 8;

    float sum[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) sum[k] = 0.f;
    float maxn2 = 0.f;
    // pass 1: coordinate sums and row norms, eight rows per lane in flight
    for (int t0 = ro; t0 < b; t0 += 8 * RPP) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            int t = t0 + u * RPP;
            v[u] = __ldg(reinterpret_cast<const uint4*>(base + (int64_t)t * stride_t));
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
            float n2 = 0.f;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                float lo = bf16_lo(w[k]), hi = bf16_hi(w[k]);
                sum[2 * k] += lo;
                sum[2 * k + 1] += hi;
                n2 = fmaf(lo, lo, n2);
                n2 = fmaf(hi, hi, n2);
            }
#pragma unroll
            for (int s = 1; s < LPR; s <<= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, s);
            maxn2 = fmaxf(maxn2, n2);
        }
    }
#pragma unroll
    for (int s = LPR; s < 32; s <<= 1) {
#pragma unroll
        for (int k = 0; k < 8; ++k) sum[k] += __shfl_xor_sync(0xffffffffu, sum[k], s);
        maxn2 = fmaxf(maxn2, __shfl_xor_sync(0xffffffffu, maxn2, s));
    }
    float mean[8];
    const float inv_b = 1.0f / (float)b;
#pragma unroll
    for (int k = 0; k < 8; ++k) mean[k] = sum[k] * inv_b;

    // pass 2: squared deviations about the mean
    float dev[8], env[8], sub[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) { dev[k] = 0.f; env[k] = 0.f; sub[k] = 0.f; }
    for (int t0 = ro; t0 < b; t0 += 8 * RPP) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            int t = t0 + u * RPP;
            v[u] = __ldg(reinterpret_cast<const uint4*>(base + (int64_t)t * stride_t));
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            {
                const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    float dl = bf16_lo(w[k]) - mean[2 * k], dh = bf16_hi(w[k]) - mean[2 * k + 1];
                    if (envelope) {
                        sub[2 * k] = fmaf(dl, dl, sub[2 * k]);
                        sub[2 * k + 1] = fmaf(dh, dh, sub[2 * k + 1]);
                    } else {
                        dev[2 * k] = fmaf(dl, dl, dev[2 * k]);
                        dev[2 * k + 1] = fmaf(dh, dh, dev[2 * k + 1]);
                    }
                }
            }
            // a 4-token sub-block ends after 4/RPP of this lane's rows (u counts them: t = ro + (8*it+u)*RPP)
            if (envelope && ((u + 1) % (4 / RPP) == 0)) {
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    float s4 = sub[k];
#pragma unroll
                    for (int s = LPR; s < 32; s <<= 1) s4 += __shfl_xor_sync(0xffffffffu, s4, s);
                    env[k] = fmaxf(env[k], s4);
                    sub[k] = 0.f;
                }
            }
        }
    }
#pragma unroll
    for (int s = LPR; s < 32; s <<= 1) {
#pragma unroll
        for (int k = 0; k < 8; ++k) dev[k] += __shfl_xor_sync(0xffffffffu, dev[k], s);
    }
    float sg[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) sg[k] = envelope ? sqrtf(env[k] * 0.25f) : sqrtf(dev[k] * inv_b);

    // row group 0 stores the centroid chunk, row group 1 the sigma chunk: one contiguous record
    if (ro < 2) {
        float src[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) src[k] = (ro == 0) ? mean[k] : sg[k];
        store_record_piece<D>(rec, packed, ro, cc, src);
    }
    if (lane == 0) *mn = sqrtf(maxn2);
}

template <int D>
__device__ __forceinline__ void summarize_block(const __nv_bfloat16* __restrict__ blk, int64_t stride_t, int b,
                                                bool envelope, unsigned char* __restrict__ rec, bool packed,
                                                float* __restrict__ mn) {
    if (envelope) summarize_block_t<D, true>(blk, stride_t, b, rec, packed, mn);
    else summarize_block_onepass<D>(blk, stride_t, b, rec, packed, mn);
}

// Eight CTAs (32 warps) per SM: the kernel is bound by memory latency at the bytes it keeps in flight, and 64
// registers per thread (a few spilled words) buy one more CTA than the 72 the routine would take.
template <int D>
__global__ void __launch_bounds__(128, 8) build_summaries_kernel(
    const __nv_bfloat16* __restrict__ K, int64_t sb, int64_t sh, int64_t st, int Hkv, int b, int t_cap, int nb_cap,
    int nb_max, int rows, const int32_t* __restrict__ seq_lens, int mode, unsigned char* __restrict__ musig,
    float* __restrict__ mnorm, const int32_t* __restrict__ table, int table_stride) {
    const int64_t wid = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (wid >= (int64_t)rows * nb_max) return;
    const int r = (int)(wid / nb_max), j = (int)(wid % nb_max);
    const int i = r / Hkv, hk = r % Hkv;
    int T = seq_lens[i];
    T = T < 0 ? 0 : (T > t_cap ? t_cap : T);
    if (j >= T / b || j >= nb_cap) return;
    // contiguous cache: block j of sequence i; paged cache: the page the table names for it
    const __nv_bfloat16* blk = table ? K + (int64_t)table[(int64_t)i * table_stride + j] * sb + hk * sh
                                     : K + i * sb + hk * sh + (int64_t)j * b * st;
    const int64_t rec = (int64_t)r * nb_cap + j;
    const bool packed = (mode & 2) != 0;      // mode: bit 0 sub-block envelope, bit 1 packed records
    summarize_block<D>(blk, st, b, (mode & 1) != 0, musig + rec * (packed ? 3 * D : 4 * D), packed, mnorm + rec);
}

// The append: one CTA of four warps per (sequence, KV head) row whose newest token completed a block.  A decode step
// waits for this kernel (the thresholds' consumer needs the new record), so it is built for latency: the block is
// requested at once by all four warps (one round trip to HBM), every warp takes the norms of the rows it loaded
// while it parks them in shared memory, and the first warp then runs the coordinate sums over the parked rows in
// the order of the prefill build, in a short loop (a fully unrolled body costs more in instruction fetches than in
// arithmetic when it runs once).  Same routines, same order of sums: the same bytes as a rebuild.
template <int D>
__global__ void __launch_bounds__(128) append_summary_kernel(
    const __nv_bfloat16* __restrict__ K, int64_t sb, int64_t sh, int64_t st, int Hkv, int b, int t_cap, int nb_cap,
    int rows, const int32_t* __restrict__ seq_lens, int mode, unsigned char* __restrict__ musig,
    float* __restrict__ mnorm, const int32_t* __restrict__ table, int table_stride, unsigned long long* timeline) {
    constexpr int LPR = D / 8;            // lanes per row
    constexpr int RPP = 32 / LPR;         // rows per warp instruction
    constexpr int RPC = 128 / LPR;        // rows per CTA instruction
    __shared__ uint4 s_rows[128 * LPR];   // the block's rows, piece by piece (up to 128 rows)
    __shared__ float s_max[4];
    const int r = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned long long* const tl = ETA_TL((timeline && r < TL_APPEND_N) ? timeline + (size_t)(TL_APPEND + r) * 8 : nullptr);
    if (tl && tid == 0) tl[0] = globaltimer_ns();
    pdl_trigger();       // nothing later in a decode step needs this kernel's output before it has waited for it
    const int i = r / Hkv, hk = r % Hkv;
    const int T = seq_lens[i];
    if (T <= 0 || T > t_cap || T % b != 0) return;
    const int j = T / b - 1;
    if (j >= nb_cap) return;
    const __nv_bfloat16* blk = table ? K + (int64_t)table[(int64_t)i * table_stride + j] * sb + hk * sh
                                     : K + i * sb + hk * sh + (int64_t)j * b * st;
    const int64_t rec = (int64_t)r * nb_cap + j;
    const bool packed = (mode & 2) != 0;      // mode: bit 0 sub-block envelope, bit 1 packed records
    unsigned char* const recp = musig + rec * (packed ? 3 * D : 4 * D);
    if (tl && tid == 0) tl[1] = globaltimer_ns();
    if (mode & 1) {
        // the sub-block envelope keeps its own (two-pass, single-warp) routine
        if (warp == 0) summarize_block_t<D, true>(blk, st, b, recp, packed, mnorm + rec);
        return;
    }
    // ---- all four warps: the whole block in flight at once, parked in shared memory; then the norms of the rows a
    // thread parked (whole warps are in or out of range together: b is a multiple of the rows per CTA instruction)
    {
        const int cc = tid % LPR, t_first = tid / LPR;
        const __nv_bfloat16* base = blk + cc * 8;
        constexpr int MAXL = 128 / RPC;       // loads per thread for the largest block
        uint4 v[MAXL];
#pragma unroll
        for (int u = 0; u < MAXL; ++u)
            if (t_first + u * RPC < b) v[u] = __ldg(reinterpret_cast<const uint4*>(base + (int64_t)(t_first + u * RPC) * st));
#pragma unroll
        for (int u = 0; u < MAXL; ++u)
            if (t_first + u * RPC < b) s_rows[(t_first + u * RPC) * LPR + cc] = v[u];
        float maxn2 = 0.f;
#pragma unroll 2
        for (int t = t_first; t < b; t += RPC) maxn2 = fmaxf(maxn2, row_norm2<LPR>(s_rows[t * LPR + cc]));
#pragma unroll
        for (int s = 16; s >= 1; s >>= 1) maxn2 = fmaxf(maxn2, __shfl_xor_sync(0xffffffffu, maxn2, s));
        if (lane == 0) s_max[warp] = maxn2;
    }
    __syncthreads();
    if (tl && tid == 0) tl[3] = globaltimer_ns();
    if (warp != 0) return;
    // ---- first warp: the sums, in the build's order (lane (cc, ro): rows ro, ro + RPP, ... ascending)
    {
        const int cc = lane % LPR, ro = lane / LPR;
        float nk0[8];
        first_key_negated(s_rows[cc], nk0);
        float s1[8], s2[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) { s1[k] = 0.f; s2[k] = 0.f; }
#pragma unroll 2
        for (int t = ro; t < b; t += RPP) accumulate_row(s_rows[t * LPR + cc], nk0, s1, s2);
        const float maxn2 = fmaxf(fmaxf(s_max[0], s_max[1]), fmaxf(s_max[2], s_max[3]));
        finish_block<D>(s1, s2, maxn2, nk0, b, recp, packed, mnorm + rec);
    }
    if (tl && tid == 0) tl[2] = globaltimer_ns();
}

int validate_pages(const eta_cache_desc* desc, const eta_page_table* pages) {
    if (!pages || !pages->block_table || pages->n_pages <= 0) return ETA_ERR_INVALID_ARG;
    if ((int64_t)pages->table_stride * desc->block_size < desc->t_cap) return ETA_ERR_INVALID_ARG;
    return ETA_OK;
}

static int build_impl(const eta_cache_desc* desc, const eta_page_table* pages, const void* K, const int32_t* seq_lens,
                      void* musig, float* mnorm, uint32_t flags, void* stream) {
    int rc = eta::validate_desc(desc);
    if (rc != ETA_OK) return rc;
    if (pages && (rc = validate_pages(desc, pages)) != ETA_OK) return rc;
    const int32_t* table = pages ? pages->block_table : nullptr;
    const int tstride = pages ? pages->table_stride : 0;
    if (!K || !seq_lens || !musig || !mnorm) return ETA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(musig)) & 15) return ETA_ERR_UNSUPPORTED;
    const int rows = desc->batch * desc->n_kv_heads;
    const int nb_max = desc->t_cap / desc->block_size;
    if (nb_max == 0) return ETA_OK;
    const int64_t warps = (int64_t)rows * nb_max;
    const unsigned grid = (unsigned)((warps + 3) / 4);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int env = ((flags & ETA_BUILD_SIGMA_ENVELOPE) ? 1 : 0) | ((flags & ETA_BUILD_PACKED_SIGMA) ? 2 : 0);
    auto Kp = static_cast<const __nv_bfloat16*>(K);
    auto mp = static_cast<unsigned char*>(musig);
    if (desc->head_dim == 128)
        eta::build_summaries_kernel<128><<<grid, 128, 0, s>>>(Kp, desc->k_stride_b, desc->k_stride_h, desc->k_stride_t,
            desc->n_kv_heads, desc->block_size, desc->t_cap, desc->nb_cap, nb_max, rows, seq_lens, env, mp, mnorm,
            table, tstride);
    else
        eta::build_summaries_kernel<64><<<grid, 128, 0, s>>>(Kp, desc->k_stride_b, desc->k_stride_h, desc->k_stride_t,
            desc->n_kv_heads, desc->block_size, desc->t_cap, desc->nb_cap, nb_max, rows, seq_lens, env, mp, mnorm,
            table, tstride);
    return eta::check_launch("eta_build_block_summaries");
}

static int append_impl(const eta_cache_desc* desc, const eta_page_table* pages, const void* K,
                       const int32_t* seq_lens_after, void* musig, float* mnorm, uint32_t flags, void* stream) {
    int rc = eta::validate_desc(desc);
    if (rc != ETA_OK) return rc;
    if (pages && (rc = validate_pages(desc, pages)) != ETA_OK) return rc;
    const int32_t* table = pages ? pages->block_table : nullptr;
    const int tstride = pages ? pages->table_stride : 0;
    if (!K || !seq_lens_after || !musig || !mnorm) return ETA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(musig)) & 15) return ETA_ERR_UNSUPPORTED;
    const int rows = desc->batch * desc->n_kv_heads;
    const unsigned grid = (unsigned)rows;      // a CTA of four warps per (sequence, KV head) row
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int env = ((flags & ETA_BUILD_SIGMA_ENVELOPE) ? 1 : 0) | ((flags & ETA_BUILD_PACKED_SIGMA) ? 2 : 0);
    auto Kp = static_cast<const __nv_bfloat16*>(K);
    auto mp = static_cast<unsigned char*>(musig);
    rc = eta::configure_kernel(desc->head_dim == 128 ? reinterpret_cast<const void*>(eta::append_summary_kernel<128>)
                                                     : reinterpret_cast<const void*>(eta::append_summary_kernel<64>), 0);
    if (rc != ETA_OK) return rc;
    eta::profile_mark(0, s);
    if (desc->head_dim == 128)
        eta::append_summary_kernel<128><<<grid, 128, 0, s>>>(Kp, desc->k_stride_b, desc->k_stride_h, desc->k_stride_t,
            desc->n_kv_heads, desc->block_size, desc->t_cap, desc->nb_cap, rows, seq_lens_after, env, mp, mnorm,
            table, tstride, eta::debug_timeline());
    else
        eta::append_summary_kernel<64><<<grid, 128, 0, s>>>(Kp, desc->k_stride_b, desc->k_stride_h, desc->k_stride_t,
            desc->n_kv_heads, desc->block_size, desc->t_cap, desc->nb_cap, rows, seq_lens_after, env, mp, mnorm,
            table, tstride, eta::debug_timeline());
    return eta::check_launch("eta_append_summary");
}

}  // namespace eta

extern "C" {

int eta_build_block_summaries(const eta_cache_desc* desc, const void* K, const int32_t* seq_lens, void* musig,
                              float* mnorm, uint32_t flags, void* stream) {
    return eta::build_impl(desc, nullptr, K, seq_lens, musig, mnorm, flags, stream);
}

int eta_build_block_summaries_paged(const eta_cache_desc* desc, const eta_page_table* pages, const void* K_pool,
                                    const int32_t* seq_lens, void* musig, float* mnorm, uint32_t flags, void* stream) {
    if (!pages) return ETA_ERR_INVALID_ARG;
    return eta::build_impl(desc, pages, K_pool, seq_lens, musig, mnorm, flags, stream);
}

int eta_append_summary(const eta_cache_desc* desc, const void* K, const int32_t* seq_lens_after, void* musig,
                       float* mnorm, uint32_t flags, void* stream) {
    return eta::append_impl(desc, nullptr, K, seq_lens_after, musig, mnorm, flags, stream);
}

int eta_append_summary_paged(const eta_cache_desc* desc, const eta_page_table* pages, const void* K_pool,
                             const int32_t* seq_lens_after, void* musig, float* mnorm, uint32_t flags, void* stream) {
    if (!pages) return ETA_ERR_INVALID_ARG;
    return eta::append_impl(desc, pages, K_pool, seq_lens_after, musig, mnorm, flags, stream);
}

}  // extern "C"

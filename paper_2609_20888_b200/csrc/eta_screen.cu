// Screening stage of eta_decode (Eq. dual_bound_eq; Algorithm 3, screening and
// rescue lines) and the planning step that turns its output into balanced work
// for the streaming kernel.
//
// screen_kernel: one CTA per (row = sequence x KV head, segment of SEG block
// records).  The segment's records (centroid and sigma, fp16) are one
// contiguous run of HBM, staged into shared memory with four 1-D bulk copies so
// that arithmetic on the first quarter overlaps the arrival of the rest.  Each
// record is evaluated once for all G query heads of the group: d/8 lanes share
// a record (16-byte shared-memory loads), each lane forms partial sums of
// <q,mu> and sum q^2 sigma^2 for the G heads in fp32, and a transposed
// butterfly leaves every lane with the two complete sums of one
// (record, head) pair.  Admission bits are gathered with a ballot; survivors
// are compacted per segment with ballot + popc prefix sums.  Nothing returns
// to the host.
//
// plan_kernel: a single CTA.  Resolves top-1 rescue per query head, scans the
// per-segment survivor counts into a global unit prefix and gives each
// streaming CTA an equal, contiguous share of the units.
#include "eta_common.cuh"

namespace eta {

// min that keeps a NaN (so that "not below the threshold" admits the block)
__device__ __forceinline__ float min_keep_nan(float g, float s) {
    return (g < s) ? g : ((s < g) ? s : ((g != g) ? g : s));
}

template <int D, int G>
__global__ void __launch_bounds__(256) screen_kernel(const ScreenArgs a) {
    constexpr int LPR = D / 8;            // lanes sharing one record
    constexpr int RPW = 32 / LPR;         // records per warp instruction
    constexpr int NI = LPR / G;           // iterations whose partial sums are reduced together
    constexpr int NV = 2 * LPR;           // partial sums per lane before the butterfly
    constexpr int RB = RPW * NI;          // records per warp per batch
    constexpr int REC_BYTES = 4 * D;      // fp16 mu[d] + fp16 sigma[d]
    constexpr bool USE_Q2 = (G <= 4);
    static_assert(NI >= 1, "group size too large for this head_dim");

    __shared__ __align__(128) unsigned char srec[SEG * REC_BYTES];
    __shared__ __align__(8) uint64_t bars[4];
    __shared__ float sbound[SEG][G];
    __shared__ float smn[SEG];
    __shared__ uint8_t smask[SEG];

    const int seg = blockIdx.x, r = blockIdx.y;
    const int i = r / a.Hkv, hk = r % a.Hkv;
    int T = a.seq_lens[i];
    T = T < 0 ? 0 : (T > a.t_cap ? a.t_cap : T);
    const int NB = min(T / a.b, a.nb_cap);
    const int j0 = seg * SEG;
    const int n_rec = max(0, min(SEG, NB - j0));
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool dense = (a.flags & ETA_FLAG_DENSE) != 0;

    // thresholds of the G heads of this group (tau_eff = tau - a)
    const int cc = lane % LPR, rg = lane / LPR;
    const int my_g = cc % G;
    const int my_h = hk * G + my_g;
    float my_te = (a.tau ? a.tau[(int64_t)i * a.Hq + my_h] : a.head_const[my_h]) - a.a;
    if (dense) my_te = -INFINITY;
    if (seg == 0 && tid < G) {
        int h = hk * G + tid;
        float te = (a.tau ? a.tau[(int64_t)i * a.Hq + h] : a.head_const[h]) - a.a;
        a.tau_eff[(int64_t)i * a.Hq + h] = dense ? -INFINITY : te;
    }
    // mask entries of this segment that are not full blocks read as "not attended"
    if (tid < SEG && tid >= n_rec && j0 + tid < a.nb_cap) a.sel_mask[(int64_t)r * a.nb_cap + j0 + tid] = 0;
    if (n_rec == 0) {
        if (tid == 0) a.seg_count[r * a.nseg + seg] = 0;
        return;
    }

    if (!dense) {
        if (tid == 0) {
#pragma unroll
            for (int c = 0; c < 4; ++c) mbar_init(&bars[c], 1);
            fence_barrier_init();
        }
        __syncthreads();
        if (tid == 0) {
            const unsigned char* src = reinterpret_cast<const unsigned char*>(a.musig) +
                                       ((int64_t)r * a.nb_cap + j0) * REC_BYTES;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                int n = min(16, n_rec - 16 * c);
                if (n > 0) {
                    mbar_arrive_expect_tx(&bars[c], n * REC_BYTES);
                    tma_load_1d(srec + c * 16 * REC_BYTES, src + (size_t)c * 16 * REC_BYTES, n * REC_BYTES, &bars[c]);
                }
            }
        }
        if (tid < n_rec) smn[tid] = a.mnorm[(int64_t)r * a.nb_cap + j0 + tid];

        // this lane's slice of the G query vectors, in fp32
        float qf[G][8], q2[USE_Q2 ? G : 1][8], qn[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(a.q + ((int64_t)i * a.Hq + hk * G + g) * D + cc * 8));
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
            float n2 = 0.f;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                qf[g][2 * k] = bf16_lo(w[k]);
                qf[g][2 * k + 1] = bf16_hi(w[k]);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                n2 = fmaf(qf[g][k], qf[g][k], n2);
                if (USE_Q2) q2[g][k] = qf[g][k] * qf[g][k];
            }
#pragma unroll
            for (int s = 1; s < LPR; s <<= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, s);
            qn[g] = sqrtf(n2);
        }
        float my_qn = qn[0];
#pragma unroll
        for (int g = 1; g < G; ++g) my_qn = (my_g == g) ? qn[g] : my_qn;
        __syncthreads();   // smn visible

        for (int base = warp * RB; base < n_rec; base += 8 * RB) {
            // wait (bounded) for the chunks this batch reads
            const int c_lo = base / 16, c_hi = min(3, (min(base + RB, n_rec) - 1) / 16);
            bool ok = true;
            for (int c = c_lo; c <= c_hi; ++c) ok = mbar_wait(&bars[c], 0) && ok;
            ok = __all_sync(0xffffffffu, ok);
            // a wait that ran out: admit everything in this batch (errs toward loading) - never seen in practice
            float v[NV];
#pragma unroll
            for (int it = 0; it < NI; ++it) {
                const int rec = base + it * RPW + rg;
                float mu[8], s2[8];
                if (rec < n_rec && ok) {
                    const uint32_t addr = smem_u32(srec) + rec * REC_BYTES + cc * 16;
                    const uint4 m4 = lds128(addr), s4 = lds128(addr + 2 * D);
                    const uint32_t mw[4] = {m4.x, m4.y, m4.z, m4.w}, sw[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        float2 mf = __half22float2(*reinterpret_cast<const __half2*>(&mw[k]));
                        float2 sf = __half22float2(*reinterpret_cast<const __half2*>(&sw[k]));
                        mu[2 * k] = mf.x; mu[2 * k + 1] = mf.y;
                        s2[2 * k] = USE_Q2 ? sf.x * sf.x : sf.x;
                        s2[2 * k + 1] = USE_Q2 ? sf.y * sf.y : sf.y;
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < 8; ++k) { mu[k] = 0.f; s2[k] = 0.f; }
                }
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    float dot = 0.f, var = 0.f;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        dot = fmaf(qf[g][k], mu[k], dot);
                        if (USE_Q2) {
                            var = fmaf(q2[g][k], s2[k], var);
                        } else {
                            const float t = qf[g][k] * s2[k];
                            var = fmaf(t, t, var);
                        }
                    }
                    v[(it * G + g) * 2] = dot;
                    v[(it * G + g) * 2 + 1] = var;
                }
            }
            // transposed butterfly over the LPR lanes of a record: halves the values held at every step
#pragma unroll
            for (int s = LPR / 2, n = NV / 2; s >= 1; s >>= 1, n >>= 1) {
                const bool upper = (lane & s) != 0;
#pragma unroll
                for (int k = 0; k < n; ++k) {
                    const float send = upper ? v[k] : v[k + n];
                    const float keep = upper ? v[k + n] : v[k];
                    v[k] = keep + __shfl_xor_sync(0xffffffffu, send, s);
                }
            }
            // lane cc now holds (dot, var) of pair cc = it * G + g
            const int it = cc / G;
            const int rec = base + it * RPW + rg;
            const bool valid = rec < n_rec;
            const float mnv = valid ? smn[rec] : 0.f;
            const float bound = a.scale * min_keep_nan(v[0] + a.z * sqrtf(v[1]), my_qn * mnv);
            const bool pinned = (j0 + rec) >= NB - a.lwb;
            const bool admit = valid && (!(bound < my_te) || pinned || !ok);
            if (valid) sbound[rec][my_g] = bound;
            const unsigned bal = __ballot_sync(0xffffffffu, admit);
            if (valid && my_g == 0) smask[rec] = (uint8_t)((bal >> lane) & ((1u << G) - 1u));
        }
    } else {
        if (tid < n_rec) smask[tid] = (uint8_t)((1u << G) - 1u);
    }
    __syncthreads();

    // user-visible admission bits
    if (tid < n_rec) a.sel_mask[(int64_t)r * a.nb_cap + j0 + tid] = smask[tid];

    // segment-local compaction of the union (ballot + popc prefix), ascending block order
    if (warp == 7) {
        int carry = 0;
        int32_t* list = a.seg_list + ((int64_t)r * a.nseg + seg) * LSTRIDE;
#pragma unroll
        for (int half = 0; half < SEG / 32; ++half) {
            const int rec = half * 32 + lane;
            const unsigned m = (rec < n_rec) ? smask[rec] : 0u;
            const unsigned nz = __ballot_sync(0xffffffffu, m != 0);
            if (m) list[carry + __popc(nz & ((1u << lane) - 1u))] = (j0 + rec) | (int)(m << 24);
            carry += __popc(nz);
        }
        if (lane == 0) a.seg_count[r * a.nseg + seg] = carry;
    }

    // rescue statistics of the part of the rescue window inside this segment, per query head
    const int Wr = min(a.rescue_window, NB);
    if (j0 < Wr && warp < G) {
        const int g = warp;
        const int nwin = min(n_rec, Wr - j0);
        int cnt = 0, arg = 0x7fffffff;
        float best = -INFINITY;
#pragma unroll
        for (int half = 0; half < SEG / 32; ++half) {
            const int rec = half * 32 + lane;
            if (rec < nwin) {
                cnt += (smask[rec] >> g) & 1;
                const float bd = dense ? 0.f : sbound[rec][g];
                if (bd > best) { best = bd; arg = rec; }
            }
        }
#pragma unroll
        for (int s = 16; s >= 1; s >>= 1) {
            cnt += __shfl_xor_sync(0xffffffffu, cnt, s);
            const float ob = __shfl_xor_sync(0xffffffffu, best, s);
            const int oa = __shfl_xor_sync(0xffffffffu, arg, s);
            if (ob > best || (ob == best && oa < arg)) { best = ob; arg = oa; }
        }
        if (lane == 0) {
            RescueRec rr;
            rr.cnt = cnt; rr.maxb = best; rr.arg = (arg == 0x7fffffff) ? -1 : (j0 + arg); rr.pad = 0;
            a.seg_resc[((int64_t)r * a.nseg + seg) * G + g] = rr;
        }
    }
}

__global__ void __launch_bounds__(1024) plan_kernel(const PlanArgs a) {
    extern __shared__ int32_t pref_s[];          // [entries + 1]
    __shared__ int32_t warp_sum[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // partial slots a streaming group never writes must read as "absent" in the merge
    for (int k = tid; k < a.n_part; k += 1024) a.part_ml[k] = make_float2(-INFINITY, 0.f);

    // ---- top-1 rescue, one warp per row (Algorithm 3: rescue phase of the first chunk).  Lane (g, s) reads the
    // window statistics of head g in window segment s, all at once; four segments (256 blocks) per pass.
    for (int r = warp; r < a.rows; r += 32) {
        const int i = r / a.Hkv;
        int T = a.seq_lens[i];
        if (lane == 0 && a.status) {
            if (T > a.t_cap) atomicOr(a.status, ETA_DEV_LEN_CLAMPED);
            if (T <= 0) atomicOr(a.status, ETA_DEV_EMPTY_ROW);
        }
        T = T < 0 ? 0 : (T > a.t_cap ? a.t_cap : T);
        const int NB = min(T / a.b, a.nb_cap);
        const int Wr = min(a.rescue_window, NB);
        const int nsw = (Wr + SEG - 1) / SEG;
        if (Wr <= 0) continue;
        const int g = lane >> 2, s4 = lane & 3;
        int cnt = 0, arg = 0x7fffffff;
        float best = -INFINITY;
        if (g < a.G) {
            for (int s = s4; s < nsw; s += 4) {
                const RescueRec rr = a.seg_resc[((int64_t)r * a.nseg + s) * a.G + g];
                cnt += rr.cnt;
                if (rr.arg >= 0 && rr.maxb > best) { best = rr.maxb; arg = rr.arg; }
            }
        }
#pragma unroll
        for (int s = 1; s <= 2; s <<= 1) {
            cnt += __shfl_xor_sync(0xffffffffu, cnt, s);
            const float ob = __shfl_xor_sync(0xffffffffu, best, s);
            const int oa = __shfl_xor_sync(0xffffffffu, arg, s);
            if (ob > best || (ob == best && oa < arg)) { best = ob; arg = oa; }
        }
        unsigned need = __ballot_sync(0xffffffffu, g < a.G && s4 == 0 && cnt == 0);
        while (need) {
            const int src = __ffs(need) - 1;
            need &= need - 1;
            const int gg = src >> 2;
            const int ja = __shfl_sync(0xffffffffu, arg, src);
            const int j = (ja == 0x7fffffff) ? 0 : ja;
            const int s = j / SEG;
            int32_t* list = a.seg_list + ((int64_t)r * a.nseg + s) * LSTRIDE;
            const int n = a.seg_count[r * a.nseg + s];
            int found = -1;
            for (int k = lane; k < n; k += 32)
                if ((list[k] & 0xffffff) == j) found = k;
            const unsigned fb = __ballot_sync(0xffffffffu, found >= 0);
            if (fb) {
                if (found >= 0) list[found] |= 1 << (24 + gg);
            } else if (lane == 0) {
                list[n] = j | (1 << (24 + gg));
                a.seg_count[r * a.nseg + s] = n + 1;
            }
            if (lane == 0) a.sel_mask[(int64_t)r * a.nb_cap + j] |= (uint8_t)(1u << gg);
            __threadfence_block();
            __syncwarp();
        }
    }
    __syncthreads();

    // ---- exclusive prefix of units over (row, segment) entries; the last entry of a row is its tail unit
    const int E = a.entries;
    const int per = (E + 1023) / 1024;
    const int e0 = min(E, tid * per), e1 = min(E, e0 + per);
    int local = 0;
    for (int e = e0; e < e1; ++e) {
        const int r = e / (a.nseg + 1), s = e % (a.nseg + 1);
        int c;
        if (s < a.nseg) {
            c = a.seg_count[r * a.nseg + s];
        } else {
            int T = a.seq_lens[r / a.Hkv];
            T = T < 0 ? 0 : (T > a.t_cap ? a.t_cap : T);
            c = (T % a.b) ? 1 : 0;
        }
        pref_s[e] = c;      // own slots only; turned into the prefix below
        local += c;
    }
    int incl = local;
    for (int s = 1; s < 32; s <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, incl, s);
        if (lane >= s) incl += o;
    }
    if (lane == 31) warp_sum[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = warp_sum[lane];
        int wi = w;
        for (int s = 1; s < 32; s <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, wi, s);
            if (lane >= s) wi += o;
        }
        warp_sum[lane] = wi - w;   // exclusive
    }
    __syncthreads();
    int run = warp_sum[warp] + incl - local;
    for (int e = e0; e < e1; ++e) {
        const int c = pref_s[e];
        pref_s[e] = run;
        a.pref[e] = run;
        run += c;
    }
    if (tid == 1023) { pref_s[E] = run; a.pref[E] = run; }
    __syncthreads();

    const int U = pref_s[E];
    if (tid == 0) { a.hdr[0] = U; a.hdr[1] = a.n_ctas; }
    if (a.stats) {
        for (int r = tid; r < a.rows; r += 1024) {
            int T = a.seq_lens[r / a.Hkv];
            T = T < 0 ? 0 : (T > a.t_cap ? a.t_cap : T);
            a.stats[r] = pref_s[(r + 1) * (a.nseg + 1)] - pref_s[r * (a.nseg + 1)] - ((T % a.b) ? 1 : 0);
        }
    }
    // ---- equal contiguous shares of the unit sequence for the streaming CTAs
    for (int c = tid; c < a.n_ctas; c += 1024) {
        const int u0 = (int)(((int64_t)c * U) / a.n_ctas), u1 = (int)(((int64_t)(c + 1) * U) / a.n_ctas);
        int lo = 0, hi = E;              // last e with pref[e] <= u0
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (pref_s[mid] <= u0) lo = mid; else hi = mid - 1;
        }
        a.cta_start[c] = make_int4(u0, u1, min(lo, E - 1), 0);
    }
}

// Diagnostic evaluation of Eq. dual_bound_eq: one warp per (sequence, query head, block).
__global__ void __launch_bounds__(128) score_dual_kernel(
    const __nv_bfloat16* __restrict__ q, const __half* __restrict__ musig, const float* __restrict__ mnorm,
    const int32_t* __restrict__ seq_lens, int B, int Hq, int Hkv, int d, int b, int t_cap, int nb_cap, float z,
    float scale, float* __restrict__ bound) {
    const int64_t wid = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (wid >= (int64_t)B * Hq * nb_cap) return;
    const int j = (int)(wid % nb_cap);
    const int h = (int)((wid / nb_cap) % Hq);
    const int i = (int)(wid / ((int64_t)nb_cap * Hq));
    int T = seq_lens[i];
    T = T < 0 ? 0 : (T > t_cap ? t_cap : T);
    if (j >= T / b) return;
    const int G = Hq / Hkv;
    const int64_t rec = ((int64_t)i * Hkv + h / G) * nb_cap + j;
    const __nv_bfloat16* qv = q + ((int64_t)i * Hq + h) * d;
    float dot = 0.f, var = 0.f, n2 = 0.f;
    for (int c = lane; c < d; c += 32) {
        const float x = __bfloat162float(qv[c]);
        const float m = __half2float(musig[rec * 2 * d + c]);
        const float s = __half2float(musig[rec * 2 * d + d + c]);
        dot = fmaf(x, m, dot);
        var = fmaf(x * x, s * s, var);
        n2 = fmaf(x, x, n2);
    }
    for (int s = 16; s >= 1; s >>= 1) {
        dot += __shfl_xor_sync(0xffffffffu, dot, s);
        var += __shfl_xor_sync(0xffffffffu, var, s);
        n2 += __shfl_xor_sync(0xffffffffu, n2, s);
    }
    if (lane == 0) bound[wid] = scale * min_keep_nan(dot + z * sqrtf(var), sqrtf(n2) * mnorm[rec]);
}

// ------------------------------------------------------------------ launchers (host)

template <int D, int G>
static void launch_screen_t(const ScreenArgs& a, int rows, cudaStream_t s) {
    dim3 grid(a.nseg, rows);
    screen_kernel<D, G><<<grid, 256, 0, s>>>(a);
}

int launch_screen(const ScreenArgs& a, int rows, int D, int G, cudaStream_t s) {
#define ETA_CASE(DD, GG) if (D == DD && G == GG) { launch_screen_t<DD, GG>(a, rows, s); return check_launch("screen"); }
    ETA_CASE(128, 1) ETA_CASE(128, 2) ETA_CASE(128, 4) ETA_CASE(128, 8)
    ETA_CASE(64, 1) ETA_CASE(64, 2) ETA_CASE(64, 4) ETA_CASE(64, 8)
#undef ETA_CASE
    return ETA_ERR_UNSUPPORTED;
}

int launch_plan(const PlanArgs& a, cudaStream_t s) {
    const size_t smem = sizeof(int32_t) * ((size_t)a.entries + 1);
    if (a.entries > MAX_ENTRIES) return ETA_ERR_UNSUPPORTED;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) { set_cuda_error(e, "plan smem attribute"); return ETA_ERR_CUDA; }
    }
    plan_kernel<<<1, 1024, smem, s>>>(a);
    return check_launch("plan");
}

}  // namespace eta

extern "C" int eta_score_dual(const eta_cache_desc* desc, const eta_params* params, const void* q,
                              const int32_t* seq_lens, const void* musig, const float* mnorm, float* bound,
                              void* stream) {
    int rc = eta::validate_desc(desc);
    if (rc != ETA_OK) return rc;
    if (!params || !q || !seq_lens || !musig || !mnorm || !bound) return ETA_ERR_INVALID_ARG;
    const float scale = params->scale > 0.f ? params->scale : 1.0f / sqrtf((float)desc->head_dim);
    const int64_t warps = (int64_t)desc->batch * desc->n_q_heads * desc->nb_cap;
    eta::score_dual_kernel<<<(unsigned)((warps + 3) / 4), 128, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const __nv_bfloat16*>(q), static_cast<const __half*>(musig), mnorm, seq_lens, desc->batch,
        desc->n_q_heads, desc->n_kv_heads, desc->head_dim, desc->block_size, desc->t_cap, desc->nb_cap, params->z,
        scale, bound);
    return eta::check_launch("eta_score_dual");
}

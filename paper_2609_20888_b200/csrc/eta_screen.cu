// Screening stage of eta_decode (Eq. dual_bound_eq; Algorithm 3, screening and
// rescue lines).
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
// The CTA that finishes a row last (a ticket per row) closes the row: it
// resolves top-1 rescue per query head from the per-segment window statistics
// and scans the row's survivor counts into a per-row unit prefix, which is all
// the streaming kernel needs to split the work evenly.
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
    const int cta_lin = blockIdx.y * gridDim.x + blockIdx.x;
    unsigned long long* tl = (a.timeline && cta_lin < 512) ? a.timeline + (size_t)(512 + cta_lin) * 8 : nullptr;
    if (tl && tid == 0) tl[0] = globaltimer_ns();

    const int cc = lane % LPR, rg = lane / LPR;
    const int my_g = cc % G;
    const int my_h = hk * G + my_g;
    // everything above reads only the caller's inputs; the summaries and thresholds may still be in the making
    pdl_wait();
    if (tl && tid == 0) tl[1] = globaltimer_ns();
    // thresholds of the G heads of this group (tau_eff = tau - a)
    float my_te = (a.tau ? a.tau[(int64_t)i * a.Hq + my_h] : a.head_const[my_h]) - a.a;
    if (dense) my_te = -INFINITY;
    if (seg == 0 && tid < G) {
        int h = hk * G + tid;
        float te = (a.tau ? a.tau[(int64_t)i * a.Hq + h] : a.head_const[h]) - a.a;
        a.tau_eff[(int64_t)i * a.Hq + h] = dense ? -INFINITY : te;
    }
    // mask entries of this segment that are not full blocks read as "not attended"
    if (tid < SEG && tid >= n_rec && j0 + tid < a.nb_cap) a.sel_mask[(int64_t)r * a.nb_cap + j0 + tid] = 0;
    if (n_rec == 0 && tid == 0) a.seg_count[r * a.nseg + seg] = 0;
    if (seg == 0 && tid == 0 && a.status) {
        const int Traw = a.seq_lens[i];
        if (Traw > a.t_cap) atomicOr(a.status, ETA_DEV_LEN_CLAMPED);
        if (Traw <= 0) atomicOr(a.status, ETA_DEV_EMPTY_ROW);
    }

    if (n_rec > 0) {
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
        if (tl && tid == 0) tl[2] = globaltimer_ns();

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
    if (tl && tid == 0) tl[3] = globaltimer_ns();
    pdl_trigger();       // the bulk of this CTA's work is done: the plan kernel may start to set up

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
        if (tl && lane == 0) tl[4] = globaltimer_ns();
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
    }   // n_rec > 0

    // ---- row ticket: the CTA that finishes this row last closes it
    __shared__ int s_last;
    __shared__ int s_warp_sum[8];
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(a.row_ticket + r, 1) == a.nseg - 1) ? 1 : 0;
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    // top-1 rescue (Algorithm 3, rescue phase of the first chunk): warp 0, lane (g, s) reads the window statistics
    // of head g in window segment s; four segments (256 blocks) per pass
    const int Wr_row = min(a.rescue_window, NB);
    if (warp == 0 && Wr_row > 0) {
        const int nsw = (Wr_row + SEG - 1) / SEG;
        const int g = lane >> 2, s4 = lane & 3;
        int cnt = 0, arg = 0x7fffffff;
        float best = -INFINITY;
        if (g < G) {
            for (int s = s4; s < nsw; s += 4) {
                const RescueRec* rp = a.seg_resc + ((int64_t)r * a.nseg + s) * G + g;
                const int4 raw = __ldcg(reinterpret_cast<const int4*>(rp));
                cnt += raw.x;
                const float mb = __int_as_float(raw.y);
                if (raw.z >= 0 && mb > best) { best = mb; arg = raw.z; }
            }
        }
#pragma unroll
        for (int s = 1; s <= 2; s <<= 1) {
            cnt += __shfl_xor_sync(0xffffffffu, cnt, s);
            const float ob = __shfl_xor_sync(0xffffffffu, best, s);
            const int oa = __shfl_xor_sync(0xffffffffu, arg, s);
            if (ob > best || (ob == best && oa < arg)) { best = ob; arg = oa; }
        }
        unsigned need = __ballot_sync(0xffffffffu, g < G && s4 == 0 && cnt == 0);
        while (need) {
            const int src = __ffs(need) - 1;
            need &= need - 1;
            const int gg = src >> 2;
            const int ja = __shfl_sync(0xffffffffu, arg, src);
            const int j = (ja == 0x7fffffff) ? 0 : ja;
            const int s = j / SEG;
            int32_t* list = a.seg_list + ((int64_t)r * a.nseg + s) * LSTRIDE;
            const int n = __ldcg(a.seg_count + r * a.nseg + s);
            int found = -1;
            for (int k = lane; k < n; k += 32)
                if ((__ldcg(list + k) & 0xffffff) == j) found = k;
            const unsigned fb = __ballot_sync(0xffffffffu, found >= 0);
            if (fb) {
                if (found >= 0) list[found] = __ldcg(list + found) | (1 << (24 + gg));
            } else if (lane == 0) {
                list[n] = j | (1 << (24 + gg));
                a.seg_count[r * a.nseg + s] = n + 1;
            }
            if (lane == 0) {
                uint8_t* mp = a.sel_mask + (int64_t)r * a.nb_cap + j;
                const unsigned w = *reinterpret_cast<volatile uint8_t*>(mp);
                *mp = (uint8_t)(w | (1u << gg));
            }
            __threadfence();
            __syncwarp();
        }
    }
    __syncthreads();

    // exclusive prefix of the row's survivor counts; the entry after the last segment holds the block total
    int32_t* rp = a.row_pref + (int64_t)r * (a.nseg + 1);
    int carry = 0;
    for (int s0 = 0; s0 < a.nseg; s0 += 256) {
        const int sgi = s0 + tid;
        const int c = (sgi < a.nseg) ? __ldcg(a.seg_count + r * a.nseg + sgi) : 0;
        int incl = c;
#pragma unroll
        for (int s = 1; s < 32; s <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, incl, s);
            if (lane >= s) incl += o;
        }
        if (lane == 31) s_warp_sum[warp] = incl;
        __syncthreads();
        int wbase = 0, tot = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            const int v = s_warp_sum[w];
            if (w < warp) wbase += v;
            tot += v;
        }
        if (sgi < a.nseg) rp[sgi] = carry + wbase + incl - c;
        carry += tot;
        __syncthreads();
    }
    if (tid == 0) {
        rp[a.nseg] = carry;
        a.row_total[r] = carry + ((T % a.b) ? 1 : 0);      // the tail, when there is one, is one more unit
        if (a.stats) a.stats[r] = carry;
        a.row_ticket[r] = 0;                                // ready for the next call
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
    cudaError_t e = launch_pdl(screen_kernel<D, G>, grid, dim3(256), 0, s, a);
    if (e != cudaSuccess) set_cuda_error(e, "screen launch");
}

int launch_screen(const ScreenArgs& a, int rows, int D, int G, cudaStream_t s) {
#define ETA_CASE(DD, GG) if (D == DD && G == GG) { launch_screen_t<DD, GG>(a, rows, s); return check_launch("screen"); }
    ETA_CASE(128, 1) ETA_CASE(128, 2) ETA_CASE(128, 4) ETA_CASE(128, 8)
    ETA_CASE(64, 1) ETA_CASE(64, 2) ETA_CASE(64, 4) ETA_CASE(64, 8)
#undef ETA_CASE
    return ETA_ERR_UNSUPPORTED;
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

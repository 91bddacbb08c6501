// Screening stage of eta_decode (Eq. dual_bound_eq; Algorithm 3, screening and
// rescue lines).
//
// screen_kernel is persistent: two CTAs per SM, each owning a contiguous range
// of items, an item being one segment of SEG consecutive block records of one
// (sequence, KV head) row.  A segment's records (centroid and sigma, fp16) are
// one contiguous run of HBM; they travel into a ring of NBUF shared-memory
// buffers by 1-D bulk copies (with the group's queries behind them), ahead of
// the item being worked on.  Each record is evaluated once for all G
// query heads of the group.  Phase 1 (bounds; needs neither thresholds nor the
// newest summary) runs item by item with one CTA barrier per item; phase 2
// (admission, pinning, mask, ballot + popc compaction, rescue-window
// statistics) takes a warp per item after the dependency wait.  Nothing
// returns to the host.
//
// Top-1 rescue needs the whole rescue window of a head, which may span several
// segments: this kernel only leaves per-segment window statistics (admitted
// count, largest bound and its index per head); the streaming kernel combines
// them when it lays out its work.
#include "eta_common.cuh"
#include "eta_timeline.h"

namespace eta {

// min that keeps a NaN (so that "not below the threshold" admits the block)
__device__ __forceinline__ float min_keep_nan(float g, float s) {
    return (g < s) ? g : ((s < g) ? s : ((g != g) ? g : s));
}

// sigma's piece cc (eight coordinates) of a record, as fp32: from the compact record (fp16) or the packed one (e4m3)
template <int D, bool PACKED>
__device__ __forceinline__ void sigma_piece_shared(uint32_t rec_addr, int cc, float (&sg)[8]) {
    if constexpr (PACKED) {
        uint2 v;
        asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(rec_addr + 2 * D + cc * 8));
        e4m3x8_to_f32(v, sg);
    } else {
        const uint4 s4 = lds128(rec_addr + 2 * D + cc * 16);
        const uint32_t sw[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            const float2 sf = __half22float2(*reinterpret_cast<const __half2*>(&sw[kk]));
            sg[2 * kk] = sf.x; sg[2 * kk + 1] = sf.y;
        }
    }
}
template <int D, bool PACKED>
__device__ __forceinline__ void sigma_piece_global(const unsigned char* rec, int cc, float (&sg)[8]) {
    if constexpr (PACKED) {
        e4m3x8_to_f32(__ldcg(reinterpret_cast<const uint2*>(rec + 2 * D + cc * 8)), sg);
    } else {
        const uint4 s4 = __ldcg(reinterpret_cast<const uint4*>(rec + 2 * D + cc * 16));
        const uint32_t sw[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            const float2 sf = __half22float2(*reinterpret_cast<const __half2*>(&sw[kk]));
            sg[2 * kk] = sf.x; sg[2 * kk + 1] = sf.y;
        }
    }
}

constexpr int SCR_GROUP = 8;       // items whose bounds are kept before their admission is decided: one per warp

template <int D, int G, bool PACKED>
struct ScreenSmem {
    static constexpr int REC_BYTES = PACKED ? 3 * D : 4 * D;   // fp16 mu[d] + fp16 (packed: e4m3) sigma[d]
    static constexpr int BUF_BYTES = SEG * REC_BYTES + G * D * 2;   // a segment's records, then the group's queries
    // ring of record buffers: the copies of NBUF - 1 items are in flight while one item is worked on (a third buffer
    // was measured and gained nothing: the kernel is bound by the latency of its arithmetic, not by bytes in flight)
    static constexpr int FIXED_BYTES = 32 + SCR_GROUP * 4 * SEG * G + 2 * 4 * SEG + 4 * SCR_GROUP + 4 * MAX_ROWS + 8 * G * D * 2 + 128;
    static constexpr int NBUF = 2;
    static constexpr int BAR_OFF = NBUF * BUF_BYTES;
    static constexpr int BOUND_OFF = BAR_OFF + 32;             // float [SCR_GROUP][SEG][G]: bounds of a group's items
    static constexpr int MN_OFF = BOUND_OFF + SCR_GROUP * 4 * SEG * G;   // float [2][SEG]: largest key norms
    static constexpr int OK_OFF = MN_OFF + 2 * 4 * SEG;        // int [SCR_GROUP]: 0 where the wait for an item's records ran out
    static constexpr int LEN_OFF = OK_OFF + 4 * SCR_GROUP;     // int32 clamped sequence lengths [MAX_ROWS]
    static constexpr int QW_OFF = LEN_OFF + 4 * MAX_ROWS;      // bf16 [8 warps][G][D]: a warp's queries for phase 2's recomputation
    static constexpr int BYTES = QW_OFF + 8 * G * D * 2 + 128; // + slack for the 128-byte alignment of the base
    static_assert(BYTES == BAR_OFF + FIXED_BYTES, "shared-memory layout and its size formula disagree");
};

// Persistent screening kernel.  Every CTA owns a contiguous range of (row, segment) items and works through it in
// groups of up to SCR_GROUP items, in two phases.
//   Phase 1, item by item: the records (and the group's queries) arrive by double-buffered 1-D bulk copies and
//   the bound of every (record, head) pair is computed and kept in shared memory.  Nothing here needs the
//   thresholds, so under programmatic dependent launch this phase runs while the predictor is still at work.
//   Phase 2, a warp per item: admission against the thresholds, pinning, the user-visible mask, compaction of the
//   union in ascending block order, and the rescue-window statistics.
template <int D, int G, bool PACKED>
__global__ void __launch_bounds__(256, 2) screen_kernel(const ScreenArgs a) {
    using L = ScreenSmem<D, G, PACKED>;
    constexpr int NBUF = L::NBUF;
    constexpr int LPR = D / 8;            // lanes sharing one record
    constexpr int RPW = 32 / LPR;         // records per warp instruction
    constexpr int NI = LPR / G;           // iterations whose partial sums are reduced together
    constexpr int NV = 2 * LPR;           // partial sums per lane before the butterfly
    constexpr int RB = RPW * NI;          // records per warp per batch
    constexpr int REC_BYTES = L::REC_BYTES;
    constexpr bool USE_Q2 = (G <= 4);
    // head_dim 128 with 4 heads per group (every benchmark configuration): the centroid term <q, mu> of a warp's
    // eight records is one 16 x 8 x 128 tensor-core product (fp16 operands, fp32 accumulation; bf16 -> fp16 is
    // exact from 2^-17 up), which leaves the fp32 pipe the variance term only
    constexpr bool USE_MMA = (D == 128 && G == 4);
    static_assert(NI >= 1, "group size too large for this head_dim");

    extern __shared__ unsigned char scr_raw[];
    unsigned char* sm = scr_raw + ((128u - (smem_u32(scr_raw) & 127u)) & 127u);
    uint64_t* bars = reinterpret_cast<uint64_t*>(sm + L::BAR_OFF);
    float (*sbound_all)[G] = reinterpret_cast<float (*)[G]>(sm + L::BOUND_OFF);
    float* smn_all = reinterpret_cast<float*>(sm + L::MN_OFF);
    int* s_ok = reinterpret_cast<int*>(sm + L::OK_OFF);
    int* s_len = reinterpret_cast<int*>(sm + L::LEN_OFF);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool dense = (a.flags & ETA_FLAG_DENSE) != 0;
    unsigned long long* const tl = ETA_TL((a.timeline && blockIdx.x < TL_SCREEN_N) ? a.timeline + (size_t)(TL_SCREEN + blockIdx.x) * 8 : nullptr);
    if (tl && tid == 0) tl[0] = globaltimer_ns();

    const int n_items = a.rows * a.nseg;
    const int c = blockIdx.x;
    // a.per_early holds the number of items the first n_early CTAs share evenly; the others take per_late each
    int it0, it1;
    if (c < a.n_early) {
        it0 = (int)(((int64_t)c * a.per_early) / a.n_early);
        it1 = (int)(((int64_t)(c + 1) * a.per_early) / a.n_early);
    } else {
        it0 = min(n_items, a.per_early + (c - a.n_early) * a.per_late);
        it1 = min(n_items, it0 + a.per_late);
    }
    const int cc = lane % LPR, rg = lane / LPR;
    const int my_g = cc % G;

    __shared__ int s_abort;               // set when a bounded wait ran out: no further copies are issued
    if (tid == 0) {
        s_abort = 0;
#pragma unroll
        for (int k = 0; k < NBUF; ++k) mbar_init(&bars[k], 1);
        fence_barrier_init();
        // The copy of the CTA's first item starts before the sequence lengths are known: it takes every record of
        // the segment that the summary array holds (how many of them are blocks of the sequence only matters
        // when the bounds are computed), which saves the round trip for the lengths ahead of the first copy.
        if (it0 < it1 && !dense) {
            int r0, seg0, i0, hk0;
            a.div_nseg.divmod(it0, r0, seg0);
            a.div_hkv.divmod(r0, i0, hk0);
            const int n_spec = min(SEG, a.nb_cap - seg0 * SEG);
            const unsigned char* src = reinterpret_cast<const unsigned char*>(a.musig) +
                                       ((int64_t)r0 * a.nb_cap + seg0 * SEG) * REC_BYTES;
            mbar_arrive_expect_tx(&bars[0], n_spec * REC_BYTES + G * D * 2);
            tma_load_1d(sm, src, n_spec * REC_BYTES, &bars[0]);
            tma_load_1d(sm + SEG * REC_BYTES, a.q + ((int64_t)i0 * a.Hq + hk0 * G) * D, G * D * 2, &bars[0]);
        }
    }
    if (tid < SCR_GROUP) s_ok[tid] = 1;
    // sequence lengths (a caller input) of every row, clamped, once: the per-item geometry then needs no global load
    for (int rr = tid; rr < a.rows; rr += 256) {
        const int T = a.seq_lens[rr / a.Hkv];
        s_len[rr] = T < 0 ? 0 : (T > a.t_cap ? a.t_cap : T);
    }
    __syncthreads();
    if (it0 >= it1) return;

    // geometry of an item, computed once per item (multiply-high divisions; b is a power of two)
    struct Geom { int r, seg, i, hk, T, NB, j0, n_rec; };
    auto item_geom = [&](int item) {
        Geom g;
        a.div_nseg.divmod(item, g.r, g.seg);
        a.div_hkv.divmod(g.r, g.i, g.hk);
        g.T = s_len[g.r];
        g.NB = min(g.T >> a.b_shift, a.nb_cap);
        g.j0 = g.seg * SEG;
        g.n_rec = max(0, min(SEG, g.NB - g.j0));
        return g;
    };
    // one thread starts the copies of an item into buffer `buf`
    int last_issued = 0;                  // (thread 0) newest item, counted from it0, whose copies were started
    auto issue = [&](const Geom& g, int k) {
        if (s_abort) return;              // a wait ran out earlier: nothing is issued (or waited for) any more
        const int buf = k % NBUF;
        last_issued = k;
        if (g.n_rec > 0 && !dense) {
            unsigned char* dst = sm + buf * L::BUF_BYTES;
            const unsigned char* src = reinterpret_cast<const unsigned char*>(a.musig) +
                                       ((int64_t)g.r * a.nb_cap + g.j0) * REC_BYTES;
            mbar_arrive_expect_tx(&bars[buf], g.n_rec * REC_BYTES + G * D * 2);
            tma_load_1d(dst, src, g.n_rec * REC_BYTES, &bars[buf]);
            tma_load_1d(dst + SEG * REC_BYTES, a.q + ((int64_t)g.i * a.Hq + g.hk * G) * D, G * D * 2, &bars[buf]);
        } else {
            mbar_arrive(&bars[buf]);      // nothing to copy: the phase completes at once
        }
    };
    // The summaries and thresholds may still be in the making when this kernel starts (programmatic dependent
    // launch): the append kernel writes the record and the norm of a block that has just filled up, the predictor
    // writes tau.  Everything else this kernel reads is final.  Phase 1 therefore never waits: the one record per
    // row that may be stale (the newest block of a just-completed length) gets a bound there like any other, and
    // the warp that handles its item in phase 2, after the wait, recomputes that bound from global memory.
    auto load_mn = [&](const Geom& g) {        // largest-norm entry of record `tid` of the item
        return (tid < g.n_rec && !dense) ? __ldg(a.mnorm + (int64_t)g.r * a.nb_cap + g.j0 + tid) : 0.f;
    };

    float qf[G][8], q2[USE_Q2 ? G : 1][8], qn[G], my_qn = 0.f;
    uint32_t qa[USE_MMA ? 8 : 1][2];       // A fragments of the centroid product: head lane / 4, one pair of registers per k-step
    float qa_inv = 1.f;                    // undoes the power-of-two scaling of the A fragments (head lane / 4)
    int q_row = -1;
    bool waited = false;
    Geom gc = item_geom(it0);
    if (tid == 0) {
        if (dense) mbar_arrive(&bars[0]);              // (otherwise the first item's copy is already on its way)
        for (int k = 1; k < NBUF - 1 && it0 + k < it1; ++k) issue(item_geom(it0 + k), k);
    }
    {
        const float mn0 = load_mn(gc);
        if (tid < SEG) smn_all[tid] = mn0;
    }
    int first_failed = -1;                // (thread 0) item, counted from it0, whose wait ran out
    __syncthreads();

    for (int gs = it0; gs < it1; gs += SCR_GROUP) {
        const int ge = min(it1, gs + SCR_GROUP);
        // ------------------------------------------------------------ phase 1: bounds of the group's items
        for (int item = gs; item < ge; ++item) {
            const int k = item - it0, buf = k % NBUF, npar = k & 1, slot = item - gs;
            float (*sbound)[G] = sbound_all + slot * SEG;
            const float* smn = smn_all + npar * SEG;
            const int r = gc.r, n_rec = gc.n_rec;
            Geom gn = gc;
            float mn_next = 0.f;
            // the copies of item k + NBUF - 1 go into the buffer item k - 1 was read from (its reads ended at the
            // barrier that closed item k - 1)
            if (tid == 0 && item + NBUF - 1 < it1) issue(item_geom(item + NBUF - 1), k + NBUF - 1);
            if (item + 1 < it1) {
                gn = item_geom(item + 1);
                mn_next = load_mn(gn);
            }
            if (tl && tid == 0 && item == it0 + 1) tl[6] = globaltimer_ns();
            // A wait that runs out: the item's blocks are all admitted (the safe direction), the call reports
            // ETA_DEV_TIMEOUT, and the CTA stops issuing copies and waiting for them; copies already on their way
            // are given time to land before the CTA leaves (end of the kernel).
            bool ok = !ld_volatile(&s_abort) && mbar_wait(&bars[buf], (k / NBUF) & 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) {
                if (lane == 0) s_ok[slot] = 0;
                if (tid == 0 && first_failed < 0) {
                    first_failed = k;
                    s_abort = 1;
                    if (a.status) atomicOr(a.status, ETA_DEV_TIMEOUT);
                }
            }
            if (tl && tid == 0 && item == it0 + 1) tl[7] = globaltimer_ns();

            if (n_rec > 0 && !dense && ok) {
                const uint32_t rec_base = smem_u32(sm + buf * L::BUF_BYTES);
                // this lane's slice of the G query vectors, in fp32: kept across the items of one row
                if (r != q_row) {
                    q_row = r;
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const uint4 v = lds128(rec_base + SEG * REC_BYTES + (g * D + cc * 8) * 2);
                        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
                        float n2 = 0.f;
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) {
                            qf[g][2 * kk] = bf16_lo(w[kk]);
                            qf[g][2 * kk + 1] = bf16_hi(w[kk]);
                        }
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {
                            n2 = fmaf(qf[g][kk], qf[g][kk], n2);
                            if (USE_Q2) q2[g][kk] = qf[g][kk] * qf[g][kk];
                        }
#pragma unroll
                        for (int s = 1; s < LPR; s <<= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, s);
                        qn[g] = sqrtf(n2);
                    }
                    my_qn = qn[0];
#pragma unroll
                    for (int g = 1; g < G; ++g) my_qn = (my_g == g) ? qn[g] : my_qn;
                    if constexpr (USE_MMA) {
                        // A[head][k]: lane (t = lane % 4, head = lane / 4 < G) holds, for k-steps 2j and 2j + 1, the
                        // eight dimensions 8 (4 j + t) .. + 7 of its head: the same dimensions the B fragments below
                        // take from one 16-byte load of a record (a dot product does not care about the order of k)
                        //
                        // fp16 holds neither the large nor the tiny end of bf16's range, so the head's query is first
                        // scaled by a power of two that puts its norm in [2^13, 2^14) (every component then fits,
                        // and one that falls below fp16's normal range is below 2^-27 of the norm), and the product
                        // is scaled back: both scalings are exact.  A norm that overflowed fp32 gives a NaN bound
                        // (the block is admitted); one that underflowed to zero gives a zero centroid term.
                        const int t4 = lane & 3, hd = lane >> 2;
                        float qn_h = qn[0];
#pragma unroll
                        for (int g = 1; g < G; ++g) qn_h = (hd == g) ? qn[g] : qn_h;
                        const int ef = (__float_as_int(qn_h) >> 23) & 0xff;
                        const int sh = min(max(140 - ef, -120), 120);
                        float q_sc = __int_as_float((127 + sh) << 23);           // 2^sh
                        qa_inv = __int_as_float((127 - sh) << 23);               // 2^-sh
                        if (ef == 255) q_sc = __int_as_float(0x7fc00000);
                        if (ef == 0) { q_sc = 0.f; qa_inv = 0.f; }
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            uint4 v = make_uint4(0, 0, 0, 0);
                            if (hd < G) v = lds128(rec_base + SEG * REC_BYTES + (hd * D + 8 * (4 * j + t4)) * 2);
                            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
                            uint32_t h[4];
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk) {
                                const __half2 hh = __floats2half2_rn(bf16_lo(w[kk]) * q_sc, bf16_hi(w[kk]) * q_sc);
                                h[kk] = *reinterpret_cast<const uint32_t*>(&hh);
                            }
                            qa[2 * j][0] = h[0]; qa[2 * j][1] = h[1];
                            qa[2 * j + 1][0] = h[2]; qa[2 * j + 1][1] = h[3];
                        }
                    }
                }

                if constexpr (USE_MMA) {
                    const int base = warp * RB;            // RB = 8 records per warp: one n-tile of the product
                    if (base < n_rec) {
                        // centroid term: D[head][record] += q[head][k] * mu[record][k] over 8 k-steps
                        float c[4] = {0.f, 0.f, 0.f, 0.f};
                        {
                            const int t4 = lane & 3, n8 = lane >> 2;
                            const uint32_t mu_addr = rec_base + (base + n8) * REC_BYTES + t4 * 16;
                            uint4 bq[4];
#pragma unroll
                            for (int j = 0; j < 4; ++j) bq[j] = lds128(mu_addr + j * 64);
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                mma_f16_16816(c, qa[2 * j][0], 0u, qa[2 * j][1], 0u, bq[j].x, bq[j].y);
                                mma_f16_16816(c, qa[2 * j + 1][0], 0u, qa[2 * j + 1][1], 0u, bq[j].z, bq[j].w);
                            }
                        }
                        // variance term on the fp32 pipe, two heads per packed fma: lane (cc, rg) takes dimensions
                        // 8 cc .. + 7 of record base + it * RPW + rg
                        float v[NI * G];
#pragma unroll
                        for (int it = 0; it < NI; ++it) {
                            const int rec = base + it * RPW + rg;
                            float s2[8];
                            if (rec < n_rec) {
                                float sg[8];
                                sigma_piece_shared<D, PACKED>(rec_base + rec * REC_BYTES, cc, sg);
#pragma unroll
                                for (int kk = 0; kk < 8; ++kk) s2[kk] = sg[kk] * sg[kk];
                            } else {
#pragma unroll
                                for (int kk = 0; kk < 8; ++kk) s2[kk] = 0.f;
                            }
                            float var[G];
#pragma unroll
                            for (int g = 0; g < G; ++g) var[g] = 0.f;
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk)
#pragma unroll
                                for (int g = 0; g < G; g += 2)
                                    fma2(var[g], var[g + 1], q2[g][kk], q2[g + 1][kk], s2[kk], s2[kk]);
#pragma unroll
                            for (int g = 0; g < G; ++g) v[it * G + g] = var[g];
                        }
                        // transposed butterfly over the LPR lanes of a record: lane cc ends with the variance term
                        // of pair cc = it * G + g
#pragma unroll
                        for (int s = LPR / 2, n = NI * G / 2; s >= 1; s >>= 1, n >>= 1) {
                            const bool upper = (lane & s) != 0;
#pragma unroll
                            for (int kk = 0; kk < n; ++kk) {
                                const float send = upper ? v[kk] : v[kk + n];
                                const float keep = upper ? v[kk + n] : v[kk];
                                v[kk] = keep + __shfl_xor_sync(0xffffffffu, send, s);
                            }
                        }
                        // the centroid term of (record base + 2 it + rg, head g) sits in lane 4 g + it, element rg
                        const int it = cc / G;
                        const float d0 = __shfl_sync(0xffffffffu, c[0] * qa_inv, 4 * my_g + it);
                        const float d1 = __shfl_sync(0xffffffffu, c[1] * qa_inv, 4 * my_g + it);
                        const float dot = rg ? d1 : d0;
                        const int rec = base + it * RPW + rg;
                        if (rec < n_rec)
                            sbound[rec][my_g] = a.scale * min_keep_nan(dot + a.z * sqrtf(v[0]), my_qn * smn[rec]);
                    }
                } else
                for (int base = warp * RB; base < n_rec; base += 8 * RB) {
                    float v[NV];
#pragma unroll
                    for (int it = 0; it < NI; ++it) {
                        const int rec = base + it * RPW + rg;
                        float mu[8], s2[8];
                        if (rec < n_rec) {
                            const uint32_t addr = rec_base + rec * REC_BYTES + cc * 16;
                            const uint4 m4 = lds128(addr);
                            const uint32_t mw[4] = {m4.x, m4.y, m4.z, m4.w};
                            float sg[8];
                            sigma_piece_shared<D, PACKED>(rec_base + rec * REC_BYTES, cc, sg);
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk) {
                                float2 mf = __half22float2(*reinterpret_cast<const __half2*>(&mw[kk]));
                                mu[2 * kk] = mf.x; mu[2 * kk + 1] = mf.y;
                            }
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk) s2[kk] = USE_Q2 ? sg[kk] * sg[kk] : sg[kk];
                        } else {
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk) { mu[kk] = 0.f; s2[kk] = 0.f; }
                        }
#pragma unroll
                        for (int g = 0; g < G; ++g) {
                            float dot = 0.f, var = 0.f;
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk) {
                                if (USE_Q2) {
                                    // (dot, var) += (q, q^2) * (mu, sigma^2): one packed instruction, each half
                                    // rounded like a scalar fma
                                    fma2(dot, var, qf[g][kk], q2[g][kk], mu[kk], s2[kk]);
                                } else {
                                    dot = fmaf(qf[g][kk], mu[kk], dot);
                                    const float t = qf[g][kk] * s2[kk];
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
                        for (int kk = 0; kk < n; ++kk) {
                            const float send = upper ? v[kk] : v[kk + n];
                            const float keep = upper ? v[kk + n] : v[kk];
                            v[kk] = keep + __shfl_xor_sync(0xffffffffu, send, s);
                        }
                    }
                    // lane cc now holds (dot, var) of pair cc = it * G + g
                    const int it = cc / G;
                    const int rec = base + it * RPW + rg;
                    if (rec < n_rec)
                        sbound[rec][my_g] = a.scale * min_keep_nan(v[0] + a.z * sqrtf(v[1]), my_qn * smn[rec]);
                }
            }
            // the next item's key norms (fetched at the top of this iteration) go to its parity before the barrier
            if (item + 1 < it1 && tid < SEG) smn_all[(npar ^ 1) * SEG + tid] = mn_next;
            // the one CTA-wide barrier of an item: its bounds are complete, and every read of the record buffer the
            // next copy goes into (and of the norms two items back) is over
            __syncthreads();
            if (tl && tid == 0 && item == it0 + 1) tl[1] = globaltimer_ns();
            gc = gn;
        }

        // ------------------------------------------------------------ phase 2: a warp per item of the group
        // What does not depend on the predecessor kernels is done ahead of the wait: the item's geometry and, for the
        // one record per row that may have been copied stale, the group's queries (a caller input) into shared memory.
        const bool p2 = gs + warp < ge;
        const int slot = warp;
        const Geom g = item_geom(min(gs + slot, n_items - 1));
        const int r = g.r, seg = g.seg, NB = g.NB, j0 = g.j0, n_rec = g.n_rec;
        const bool recompute = p2 && !dense && n_rec > 0 && (g.T & (a.b - 1)) == 0 && j0 + n_rec == NB;
        uint4* qw = reinterpret_cast<uint4*>(sm + L::QW_OFF) + warp * (G * D / 8);
        if (recompute) {
            const uint4* qsrc = reinterpret_cast<const uint4*>(a.q + ((int64_t)g.i * a.Hq + g.hk * G) * D);
            for (int k = lane; k < G * D / 8; k += 32) qw[k] = __ldg(qsrc + k);
            __syncwarp();
        }
        if (tl && tid == 0 && !waited) tl[2] = globaltimer_ns();
        if (!waited) { pdl_wait(); waited = true; }       // the thresholds (and the newest summaries) are final now
        if (tl && tid == 0 && gs == it0) tl[3] = globaltimer_ns();
        if (p2) {
            const float (*sbound)[G] = sbound_all + slot * SEG;
            const bool ok = s_ok[slot] != 0;
            // an ungated newest token must be attended: when it closes a full block, that block counts as pinned
            const int lwb_item = ((a.flags & ETA_FLAG_UNGATE_LAST) && g.T > 0 && (g.T & (a.b - 1)) == 0 && a.lwb < 1) ? 1 : a.lwb;
            // All loads that had to wait are issued together: lane gq < G fetches the effective threshold of head gq of
            // the item's group, and, where the newest record has to be bounded again, every lane its pieces of it.
            // (That record was possibly copied before the append kernel wrote it: its bound is computed again here,
            // from global memory past the L1, in fp32 throughout; a difference of a rounding from the tensor-core value
            // is far inside the near-tie band.)
            float te_l = -INFINITY;
            if (!dense && lane < G) {
                const int h = g.hk * G + lane;
                te_l = (a.tau ? __ldcg(a.tau + (int64_t)g.i * a.Hq + h) : __ldg(a.head_const + h)) - a.a;
            }
            const int cl = lane % LPR;
            if (recompute && ok) {
                const int rec = n_rec - 1;
                const unsigned char* src = reinterpret_cast<const unsigned char*>(a.musig) +
                                           ((int64_t)r * a.nb_cap + j0 + rec) * REC_BYTES;
                const uint4 m4 = __ldcg(reinterpret_cast<const uint4*>(src + cl * 16));
                const float mn = __ldcg(a.mnorm + (int64_t)r * a.nb_cap + j0 + rec);
                const uint32_t mw[4] = {m4.x, m4.y, m4.z, m4.w};
                float mu[8], s2[8], sg[8];
                sigma_piece_global<D, PACKED>(src, cl, sg);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    float2 mf = __half22float2(*reinterpret_cast<const __half2*>(&mw[kk]));
                    mu[2 * kk] = mf.x; mu[2 * kk + 1] = mf.y;
                }
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) s2[kk] = sg[kk] * sg[kk];
#pragma unroll 1
                for (int gq = 0; gq < G; ++gq) {
                    const uint4 qv = qw[gq * LPR + cl];
                    const uint32_t qq[4] = {qv.x, qv.y, qv.z, qv.w};
                    float dot = 0.f, var = 0.f, n2 = 0.f;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const float x = (kk & 1) ? bf16_hi(qq[kk >> 1]) : bf16_lo(qq[kk >> 1]);
                        n2 = fmaf(x, x, n2);
                        dot = fmaf(x, mu[kk], dot);
                        var = fmaf(x * x, s2[kk], var);
                    }
#pragma unroll
                    for (int sh = 1; sh < LPR; sh <<= 1) {
                        n2 += __shfl_xor_sync(0xffffffffu, n2, sh);
                        dot += __shfl_xor_sync(0xffffffffu, dot, sh);
                        var += __shfl_xor_sync(0xffffffffu, var, sh);
                    }
                    if (lane == 0)
                        sbound_all[slot * SEG + rec][gq] = a.scale * min_keep_nan(dot + a.z * sqrtf(var), sqrtf(n2) * mn);
                }
                __syncwarp();
            }
            float te_g[G];
#pragma unroll
            for (int gq = 0; gq < G; ++gq) te_g[gq] = __shfl_sync(0xffffffffu, te_l, gq);
            if (seg == 0) {
                if (lane < G) a.tau_eff[(int64_t)g.i * a.Hq + g.hk * G + lane] = te_l;
                if (lane == 0 && a.status) {
                    const int Traw = __ldg(a.seq_lens + g.i);
                    if (Traw > a.t_cap) atomicOr(a.status, ETA_DEV_LEN_CLAMPED);
                    if (Traw <= 0) atomicOr(a.status, ETA_DEV_EMPTY_ROW);
                }
            }
            // admission bits of records lane and lane + 32
            unsigned m[SEG / 32];
#pragma unroll
            for (int half = 0; half < SEG / 32; ++half) {
                const int rec = half * 32 + lane;
                m[half] = 0;
                if (rec < n_rec) {
                    const bool pinned = (j0 + rec) >= NB - lwb_item;
#pragma unroll
                    for (int gq = 0; gq < G; ++gq)
                        if (dense || !ok || pinned || !(sbound[rec][gq] < te_g[gq])) m[half] |= 1u << gq;
                }
                // user-visible bits; entries of this segment that are not full blocks read as "not attended"
                if (j0 + rec < a.nb_cap) a.sel_mask[(int64_t)r * a.nb_cap + j0 + rec] = (uint8_t)m[half];
            }
            // segment-local compaction of the union (ballot + popc prefix), ascending block order
            {
                int carry = 0;
                int32_t* list = a.seg_list + ((int64_t)r * a.nseg + seg) * LSTRIDE;
#pragma unroll
                for (int half = 0; half < SEG / 32; ++half) {
                    const unsigned nz = __ballot_sync(0xffffffffu, m[half] != 0);
                    if (m[half]) list[carry + __popc(nz & ((1u << lane) - 1u))] = (j0 + half * 32 + lane) | (int)(m[half] << 24);
                    carry += __popc(nz);
                }
                if (lane == 0) a.seg_count[r * a.nseg + seg] = carry;
            }
            // rescue statistics of the part of the rescue window inside this segment, per query head: how many of its
            // blocks the head admits, the largest bound and the first block that attains it.  Bounds are compared as
            // order-preserving integers (one hardware max-reduction and one ballot per head instead of a shuffle tree).
            const int Wr = min(a.rescue_window, NB);
            if (j0 < Wr && n_rec > 0) {
                const int nwin = min(n_rec, Wr - j0);
#pragma unroll 1
                for (int gq = 0; gq < G; ++gq) {
                    uint32_t key = 0;                 // 0: no record of the window in this lane
                    int arg = 0x7fffffff;
#pragma unroll
                    for (int half = 0; half < SEG / 32; ++half) {
                        const int rec = half * 32 + lane;
                        if (rec < nwin) {
                            const float bd = ((dense || !ok) ? 0.f : sbound[rec][gq]) + 0.f;        // (-0 counts as +0)
                            const uint32_t u = __float_as_uint(bd);
                            uint32_t k2 = (u & 0x80000000u) ? ~u : (u | 0x80000000u);           // ascending with the value
                            if (bd != bd) k2 = 1;                                               // a NaN bound never wins
                            if (k2 > key) { key = k2; arg = rec; }                              // ties keep the lower index
                        }
                    }
                    const int cnt = __popc(__ballot_sync(0xffffffffu, (m[0] >> gq) & 1 && lane < nwin)) +
                                    __popc(__ballot_sync(0xffffffffu, (m[1] >> gq) & 1 && lane + 32 < nwin));
                    const uint32_t kmax = __reduce_max_sync(0xffffffffu, key);
                    // among the lanes that hold the maximum the lowest record index wins: a lane's own candidate is its
                    // lower record unless the higher one is strictly larger, so compare the candidates' indices
                    const int amin = __reduce_min_sync(0xffffffffu, key == kmax ? arg : 0x7fffffff);
                    if (lane == 0) {
                        RescueRec rr;
                        float best = -INFINITY;
                        if (kmax > 1) {
                            const uint32_t u = (kmax & 0x80000000u) ? (kmax & 0x7fffffffu) : ~kmax;
                            best = __uint_as_float(u);
                        }
                        rr.cnt = cnt; rr.maxb = best;
                        rr.arg = (kmax <= 1 || amin == 0x7fffffff) ? -1 : (j0 + amin);
                        rr.pad = 0;
                        a.seg_resc[((int64_t)r * a.nseg + seg) * G + gq] = rr;
                    }
                }
            }
        }
        if (ge < it1) {
            __syncthreads();          // the bounds of this group have been read: the next group may overwrite them
            if (tid < SCR_GROUP) s_ok[tid] = 1;
        }
    }
    if (tid == 0 && first_failed >= 0) {
        // bounded wait for the copies that were in flight when a wait gave up, so that none lands in shared memory
        // the next CTA on this SM already owns
        for (int k = first_failed; k <= last_issued; ++k) mbar_wait(&bars[k % NBUF], (k / NBUF) & 1);
    }
    if (tl && tid == 0) tl[5] = globaltimer_ns();
    pdl_trigger();
}

// Diagnostic evaluation of Eq. dual_bound_eq: one warp per (sequence, query head, block).
__global__ void __launch_bounds__(128) score_dual_kernel(
    const __nv_bfloat16* __restrict__ q, const unsigned char* __restrict__ musig, const float* __restrict__ mnorm,
    const int32_t* __restrict__ seq_lens, int B, int Hq, int Hkv, int d, int b, int t_cap, int nb_cap, float z,
    float scale, int packed, float* __restrict__ bound) {
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
        const unsigned char* rp = musig + rec * (packed ? 3 * d : 4 * d);
        const float m = __half2float(reinterpret_cast<const __half*>(rp)[c]);
        float s;
        if (packed) {
            const uint32_t h2 = e4m3x2_to_f16x2(rp[2 * d + c]);
            s = __half2float(*reinterpret_cast<const __half*>(&h2));
        } else {
            s = __half2float(reinterpret_cast<const __half*>(rp)[d + c]);
        }
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

template <int D, int G, bool PACKED>
static int launch_screen_t(const ScreenArgs& a, int rows, int n_ctas, cudaStream_t s) {
    const size_t smem = ScreenSmem<D, G, PACKED>::BYTES;
    // The slowest CTA sets the kernel's end.  All CTAs are resident at once (n_ctas = two per SM), but under
    // programmatic dependent launch the kernel starts while its predecessors (summary append, threshold predictor)
    // still hold some SMs, where no CTA of this kernel fits until they exit: the CTAs dispatched last (the
    // highest indices) start late, by the time `lag` items take (measured at d = 128: 7.6 us against 1.4 us per
    // item with the tensor-core centroid term at G = 4, 1.9 us without), and get that many items fewer, down to
    // none.  With x items for an early CTA all end together when  n_early x + n_late max(x - lag, 0) = n_items.
    const int n_items = rows * a.nseg;
    ScreenArgs b2 = a;
    int grid = 0, n_late = 0;
    if (pdl_enabled()) {
        const int batch = rows / a.Hkv;
        n_late = 2 * ((rows + 3) / 4 + (a.tau ? 8 * batch : 0));      // two slots per CTA of the append / predictor kernel
        if (n_late > n_ctas / 3) n_late = n_ctas / 3;
    }
    const int lag = (D == 128 && G == 4) ? 5 : 2;
    int x = (n_items + lag * n_late + n_ctas - 1) / n_ctas;
    if (x <= lag) x = (n_items + (n_ctas - n_late) - 1) / (n_ctas - n_late);      // the late CTAs take nothing
    if (n_late > 0 && x >= 3) {
        grid = n_ctas;
        b2.per_late = x > lag ? x - lag : 0;
        b2.n_early = grid - n_late;
        b2.per_early = n_items - n_late * b2.per_late;       // shared evenly by the early CTAs
        if (b2.per_early < b2.n_early) n_late = 0;
        else if (b2.per_late == 0) grid = b2.n_early;        // nothing to launch the late CTAs for
    } else {
        n_late = 0;
    }
    if (n_late == 0) {
        // every CTA gets the same number of items (the last ones one fewer)
        const int per_cta = (n_items + n_ctas - 1) / n_ctas;
        grid = (n_items + per_cta - 1) / per_cta;
        b2.per_late = per_cta;
        b2.n_early = grid;
        b2.per_early = n_items;
    }
    return launch_pdl("screen launch", screen_kernel<D, G, PACKED>, dim3(grid), dim3(256), smem, s, b2);
}

int launch_screen(const ScreenArgs& a, int rows, int D, int G, int n_ctas, cudaStream_t s) {
    const bool packed = (a.flags & ETA_FLAG_PACKED_SIGMA) != 0;
#define ETA_CASE(DD, GG) if (D == DD && G == GG) return packed ? launch_screen_t<DD, GG, true>(a, rows, n_ctas, s) \
                                                                : launch_screen_t<DD, GG, false>(a, rows, n_ctas, s);
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
        static_cast<const __nv_bfloat16*>(q), static_cast<const unsigned char*>(musig), mnorm, seq_lens, desc->batch,
        desc->n_q_heads, desc->n_kv_heads, desc->head_dim, desc->block_size, desc->t_cap, desc->nb_cap, params->z,
        scale, (params->flags & ETA_FLAG_PACKED_SIGMA) ? 1 : 0, bound);
    return eta::check_launch("eta_score_dual");
}

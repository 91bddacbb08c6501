// Single-kernel path of eta_decode: screening (Eq. dual_bound_eq; Algorithm 3,
// screening and rescue lines) and streaming (Algorithm 3, attention lines and tail
// phase) run side by side in one persistent kernel, so the first K/V tiles are on
// their way while most of the block summaries are still being screened.
//
// Work is claimed, not laid out in advance.  A claim is a run of items (FSEG
// consecutive block records of one (sequence, KV head) row): the items of a row's
// rescue window form one claim, every other item is a claim of its own.  Each CTA
// starts with three claims fixed by its index and then takes further claims from
// a counter in global memory, so a CTA whose items hold many survivors simply
// claims fewer items.  Inside a CTA
//   - three screening warps evaluate the bound of every record of an item for the
//     G query heads of the group, compact the survivors, resolve the top-1 rescue
//     of a window claim, append the row's tail, and push the item's list to a
//     ring in shared memory in chunks of at most FCH entries;
//   - one producer warp pops chunks, hands each to one of the three consumer
//     groups and issues the tiled TMA copies of its K/V tiles (and one bulk copy
//     of the group's queries per chunk) into the ring of stages;
//   - the consumer groups run the packed-GQA attention of the streaming kernel
//     and store one partial (m, l, O) per (chunk, query head).
// A chunk's partial depends only on the chunk's list, never on which CTA or group
// processed it, and the merge kernel adds the partials of a row in list order, so
// the result does not depend on how the claims fell.
//
// The claim counter is the only state that outlives a call: the merge kernel
// zeroes it and writes a magic number beside it; a kernel that does not find the
// magic number (first use of a workspace) falls back to a fixed assignment of
// claims for that call.
#include <cuda.h>

#include "eta_common.cuh"

namespace eta {

int make_tmap(CUtensorMap* tm, const void* base, const eta_cache_desc* d, int64_t sb, int64_t sh, int64_t st, int TS);

struct FusedArgs {
    const __nv_bfloat16* q;
    const __half* musig;
    const float* mnorm;
    const int32_t* seq_lens;
    const float* tau;
    const float* head_const;
    uint8_t* sel_mask;
    int32_t* f_hdr;
    int32_t* f_count;
    float2* part_ml;
    float* part_o;
    uint32_t* status;
    unsigned long long* timeline;
    float z, a, scale, beta;
    int lwb, rescue_window;
    int Hq, Hkv, b, b_shift, t_cap, nb_cap, nfs, rows, nwi, spr, n_claims;
    FastDiv div_hkv, div_spr;
};

constexpr int F_GROUPS = 3;                      // consumer groups (= chunks in progress) per CTA
constexpr int F_WPG = 4;                         // warps per consumer group
constexpr int F_PRODUCER_WARP = F_GROUPS * F_WPG;
constexpr int F_SCR_WARP0 = F_PRODUCER_WARP + 1;
constexpr int F_SCR_WARPS = 3;
constexpr int F_SCR_THREADS = 32 * F_SCR_WARPS;
constexpr int F_THREADS = 32 * (F_SCR_WARP0 + F_SCR_WARPS);
constexpr int F_NSB = F_SCR_WARPS;               // record buffers: one per screening warp
constexpr int F_RING = 8;                        // chunk records between the screening warps and the producer
constexpr int F_BACKLOG = 8;                     // list entries pushed but not yet issued above which screening pauses
constexpr int F_LIST = FSEG + 12;
constexpr uint32_t FD_END = 1u, FD_SKIP = 2u, FD_NEW = 4u, FD_LAST = 8u;

struct ChunkRec { int row, slot, n, pad; int ent[FCH]; float te[8]; };
struct LaneState { int n, k, sub, row, slot, nchunks, pad0, pad1; };

// control words in shared memory
enum { C_HEAD = 0, C_RESERVE, C_DONE, C_PUSHED, C_ISSUED, C_FAIL, C_FILL, C_WORDS = 8 };

template <int D, int TS, int NSTAGE, int G>
struct FusedSmem {
    static constexpr int HALVES = D / 64;
    static constexpr int TILE_BYTES = TS * 128;
    static constexpr int STAGE_BYTES = 2 * HALVES * TILE_BYTES;
    static constexpr int REC_BYTES = 4 * D;
    static constexpr int QB_BYTES = G * D * 2;
    static constexpr int SBUF_BYTES = FSEG * REC_BYTES + QB_BYTES;
    static constexpr int NQB = NSTAGE / 3 + 1;
    static constexpr int SBUF_OFF = NSTAGE * STAGE_BYTES;
    static constexpr int QBUF_OFF = SBUF_OFF + F_NSB * SBUF_BYTES;
    static constexpr int BAR_OFF = QBUF_OFF + F_GROUPS * NQB * QB_BYTES;       // full, empty, sbar
    static constexpr int DESC_OFF = BAR_OFF + 8 * ((2 * NSTAGE + F_NSB + F_GROUPS + 1) & ~1);
    static constexpr int HTE_OFF = DESC_OFF + 16 * NSTAGE;                     // float [groups][NQB][8]
    static constexpr int RING_OFF = HTE_OFF + 4 * F_GROUPS * NQB * 8;
    static constexpr int LST_OFF = RING_OFF + (int)sizeof(ChunkRec) * F_RING;
    static constexpr int LENT_OFF = LST_OFF + (int)sizeof(LaneState) * F_GROUPS;
    static constexpr int CTRL_OFF = LENT_OFF + 4 * F_GROUPS * FCH;
    static constexpr int READY_OFF = CTRL_OFF + 4 * C_WORDS;                   // int [F_RING]: slot + 1 once its record is written
    static constexpr int LIST_OFF = READY_OFF + 4 * F_RING;                    // int [F_SCR_WARPS][F_LIST]
    static constexpr int ML_OFF = LIST_OFF + 4 * F_LIST * F_SCR_WARPS;         // float [groups][2][F_WPG][8]
    static constexpr int LEN_OFF = ML_OFF + 4 * F_GROUPS * 2 * F_WPG * 8;      // int len[rows], float te[rows * G]
    static size_t bytes(int rows) { return 1024 + LEN_OFF + (size_t)4 * rows * (1 + G); }
};

template <int D, int TS, int NSTAGE, int G>
__global__ void __launch_bounds__(F_THREADS, 1)
fused_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const FusedArgs a) {
    using L = FusedSmem<D, TS, NSTAGE, G>;
    constexpr int HALVES = L::HALVES;
    constexpr int NQB = L::NQB;
    constexpr int WT = TS / F_WPG;              // tokens per consumer warp per tile
    constexpr int NT = WT / 8;
    static_assert(NT == 1 || NT == 2, "tile must give each warp 8 or 16 tokens");
    static_assert(4 * G * D <= D * TS, "a warp's partial must fit the part of a stage it owns");

    extern __shared__ unsigned char fsm_raw[];
    unsigned char* smem = fsm_raw + ((1024u - (smem_u32(fsm_raw) & 1023u)) & 1023u);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::BAR_OFF);
    uint64_t* empty = full + NSTAGE;
    uint64_t* sbar = empty + NSTAGE;
    uint64_t* flushbar = sbar + F_NSB;         // one per consumer group: its four warps meet here at the end of a chunk
    int4* desc = reinterpret_cast<int4*>(smem + L::DESC_OFF);
    float* hte = reinterpret_cast<float*>(smem + L::HTE_OFF);
    ChunkRec* ring = reinterpret_cast<ChunkRec*>(smem + L::RING_OFF);
    LaneState* lst = reinterpret_cast<LaneState*>(smem + L::LST_OFF);
    int* lent = reinterpret_cast<int*>(smem + L::LENT_OFF);
    int* ctrl = reinterpret_cast<int*>(smem + L::CTRL_OFF);
    int* s_len = reinterpret_cast<int*>(smem + L::LEN_OFF);
    float* s_te = reinterpret_cast<float*>(s_len + a.rows);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // development aid: with bit 0 of the time-stamp pointer set, the slots hold progress markers instead (volatile
    // stores, so that a host that maps the buffer can look at them while the kernel runs)
    const bool progress = (reinterpret_cast<uintptr_t>(a.timeline) & 1) != 0;
    volatile unsigned long long* pg = progress ? reinterpret_cast<unsigned long long*>(reinterpret_cast<uintptr_t>(a.timeline) & ~(uintptr_t)7) + (size_t)blockIdx.x * 8 : nullptr;
    unsigned long long* tl = (a.timeline && !progress) ? a.timeline + (size_t)blockIdx.x * 8 : nullptr;
    unsigned long long* xt = tl ? a.timeline + 2048 + (size_t)blockIdx.x * 16 : nullptr;   // phase stamps of one item
    if (tl && tid == 0) tl[0] = globaltimer_ns();
    if (pg && tid == 0) pg[0] = 1;
    if (tid == 0) {
        for (int s = 0; s < NSTAGE; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], F_WPG); }
        for (int k = 0; k < F_NSB; ++k) mbar_init(&sbar[k], 1);
        for (int k = 0; k < F_GROUPS; ++k) mbar_init(&flushbar[k], 32 * F_WPG);
        fence_barrier_init();
        prefetch_tmap(&tmK);
        prefetch_tmap(&tmV);
        for (int k = 0; k < C_WORDS; ++k) ctrl[k] = 0;
        for (int k = 0; k < F_RING; ++k) reinterpret_cast<int*>(smem + L::READY_OFF)[k] = 0;
        for (int k = 0; k < (int)(sizeof(LaneState) / 4) * F_GROUPS; ++k) reinterpret_cast<int*>(lst)[k] = 0;
    }
    // sequence lengths are a caller input: they can be read while the previous kernel is still running
    for (int rr = tid; rr < a.rows; rr += F_THREADS) {
        const int T = __ldg(a.seq_lens + a.div_hkv.div(rr));
        s_len[rr] = T < 0 ? 0 : (T > a.t_cap ? a.t_cap : T);
    }
    __syncthreads();

    if (warp >= F_SCR_WARP0) {
        // ======================================================================= screening warps
        // Each warp works on items of its own: a lane per record.  A lane walks the head_dim of its record in
        // 16-byte pieces, starting at a piece that depends on the lane so that the lanes of a quarter-warp always
        // hit different banks, and keeps the two sums of Eq. dual_bound_eq for the G heads in registers.
        constexpr int REC_BYTES = L::REC_BYTES;
        constexpr int NCH = D / 8;                      // 16-byte pieces per vector
        int* s_list = reinterpret_cast<int*>(smem + L::LIST_OFF) + (warp - F_SCR_WARP0) * F_LIST;
        int* ready = reinterpret_cast<int*>(smem + L::READY_OFF);
        const int sw = warp - F_SCR_WARP0;
        const int P = gridDim.x, NC = a.n_claims;
        const int NSWG = P * F_SCR_WARPS;               // screening warps of the whole grid
        const int wg = blockIdx.x * F_SCR_WARPS + sw;
        unsigned char* buf = smem + L::SBUF_OFF + sw * L::SBUF_BYTES;
        const uint32_t rec_base = smem_u32(buf) + lane * REC_BYTES;
        const uint32_t q_base = smem_u32(buf) + FSEG * REC_BYTES;

        // the first claim is fixed by the warp's index; later ones come from the counter (or, on a workspace that
        // does not carry the magic number yet, from the same fixed pattern)
        bool dynamic = false;
        if (lane == 0) {
            const int m0 = ld_volatile(a.f_hdr), m1 = ld_volatile(a.f_hdr + 1);
            dynamic = ((uint32_t)m0 == F_MAGIC0 && (uint32_t)m1 == F_MAGIC1);
        }
        dynamic = __shfl_sync(0xffffffffu, dynamic ? 1 : 0, 0) != 0;

        struct Geom { int r, fit, i, hk, T, NB, j0, n_rec; };
        auto geom_of = [&](int row, int fit) {
            Geom g;
            g.r = row; g.fit = fit;
            a.div_hkv.divmod(row, g.i, g.hk);
            g.T = s_len[row];
            g.NB = min(g.T >> a.b_shift, a.nb_cap);
            g.j0 = fit * FSEG;
            g.n_rec = max(0, min(FSEG, g.NB - g.j0));
            return g;
        };
        // an item that holds a row's newest block of a just-completed length must not be copied before the
        // summary update of this step is known to be complete
        auto safe_item = [&](const Geom& g) {
            return !(g.n_rec > 0 && (g.T & (a.b - 1)) == 0 && g.j0 + g.n_rec == g.NB);
        };
        bool waited = false;
        auto wait_pred = [&]() {
            if (waited) return;
            pdl_wait();
            waited = true;
        };
        auto issue = [&](const Geom& g) {          // lane 0: copies of an item into this warp's buffer
            if (g.n_rec > 0) {
                const unsigned char* src = reinterpret_cast<const unsigned char*>(a.musig) +
                                           ((int64_t)g.r * a.nb_cap + g.j0) * REC_BYTES;
                mbar_arrive_expect_tx(&sbar[sw], g.n_rec * REC_BYTES + L::QB_BYTES);
                tma_load_1d(buf, src, g.n_rec * REC_BYTES, &sbar[sw]);
                tma_load_1d(buf + FSEG * REC_BYTES, a.q + ((int64_t)g.i * a.Hq + g.hk * G) * D, L::QB_BYTES, &sbar[sw]);
            } else {
                mbar_arrive(&sbar[sw]);
            }
        };
        auto load_mn = [&](const Geom& g) {        // this lane's record's largest key norm
            return (lane < g.n_rec) ? __ldg(a.mnorm + (int64_t)g.r * a.nb_cap + g.j0 + lane) : 0.f;
        };
        auto load_te = [&](const Geom& g) {        // lane g < G: effective threshold of head g of the item's group
            if (lane >= G) return 0.f;
            const int h = g.hk * G + lane;
            return (a.tau ? __ldg(a.tau + (int64_t)g.i * a.Hq + h) : __ldg(a.head_const + h)) - a.a;
        };
        auto claim_items = [&](int cid, int& row, int& it0, int& nit) {
            if (cid < a.rows) { row = cid; it0 = 0; nit = a.nwi; }
            else { a.div_spr.divmod(cid - a.rows, row, it0); it0 += a.nwi; nit = 1; }
        };
        // id of the claim after the current one: asked for (lane 0) as an item starts, used when it ends
        int n_claimed = 1;
        auto ask_claim = [&]() {
            int v = NC;
            if (lane == 0) {
                // pause while the producer has enough to issue: claims taken early are claims taken from others
                for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
                    if (ld_volatile(ctrl + C_PUSHED) - ld_volatile(ctrl + C_ISSUED) < F_BACKLOG) break;
                    __nanosleep(100);
                }
                v = dynamic ? NSWG + atomicAdd(a.f_hdr + 2, 1) : wg + n_claimed * NSWG;
            }
            ++n_claimed;
            return v;
        };

        int cid = wg;
        int row = 0, it0 = 0, nit = 1, pos = 0;
        bool have = cid < NC;
        Geom gc = {};
        float mn_cur = 0.f, te_cur = 0.f;
        bool te_have = false;
        uint32_t n_items = 0;
        if (have) {
            claim_items(cid, row, it0, nit);
            gc = geom_of(row, it0);
            if (!safe_item(gc)) wait_pred();
            if (lane == 0) issue(gc);
            mn_cur = load_mn(gc);
        }
        // window statistics of a rescue-window claim (uniform across the warp)
        int w_cnt[G], w_arg[G];
        float w_best[G];

        while (have) {
            const bool first_of_claim = pos == 0, last_of_claim = pos + 1 == nit;
            const bool win_claim = it0 == 0;
            const int r = gc.r, NB = gc.NB, j0 = gc.j0, n_rec = gc.n_rec;
            if (xt && sw == 0 && lane == 0 && n_items == 3) xt[1] = globaltimer_ns();
            int pend = NC;
            if (last_of_claim) pend = ask_claim();
            if (first_of_claim && win_claim) {
#pragma unroll
                for (int g = 0; g < G; ++g) { w_cnt[g] = 0; w_arg[g] = -1; w_best[g] = -INFINITY; }
            }
            if (xt && sw == 0 && lane == 0 && n_items == 3) xt[2] = globaltimer_ns();
            bool ok = mbar_wait(&sbar[sw], n_items & 1);
            if (!__all_sync(0xffffffffu, ok)) {
                if (lane == 0) { ctrl[C_FAIL] = 1; if (tl) tl[7] = (1ull << 32) | n_items; }
                break;
            }
            if (xt && sw == 0 && lane == 0 && n_items == 3) xt[3] = globaltimer_ns();

            float bound[G];
            if (n_rec > 0) {
                // ||q_g||: the lanes of a half-warp split the pieces of q_g
                float qn[G];
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const uint4 v = lds128(q_base + g * 2 * D + (lane % NCH) * 16);
                    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
                    float n2 = 0.f;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        const float x0 = bf16_lo(w[kk]), x1 = bf16_hi(w[kk]);
                        n2 = fmaf(x0, x0, n2);
                        n2 = fmaf(x1, x1, n2);
                    }
#pragma unroll
                    for (int s = 1; s < NCH; s <<= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, s);
                    qn[g] = sqrtf(n2);
                }
                float dot[G], var[G];
#pragma unroll
                for (int g = 0; g < G; ++g) { dot[g] = 0.f; var[g] = 0.f; }
#pragma unroll 2
                for (int c = 0; c < NCH; ++c) {
                    const int cc = (c + lane) % NCH;
                    const uint4 m4 = lds128(rec_base + cc * 16), s4 = lds128(rec_base + 2 * D + cc * 16);
                    const uint32_t mw[4] = {m4.x, m4.y, m4.z, m4.w}, sw4[4] = {s4.x, s4.y, s4.z, s4.w};
                    float mu[8], sg[8];
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        const float2 mf = __half22float2(*reinterpret_cast<const __half2*>(&mw[kk]));
                        const float2 sf = __half22float2(*reinterpret_cast<const __half2*>(&sw4[kk]));
                        mu[2 * kk] = mf.x; mu[2 * kk + 1] = mf.y;
                        sg[2 * kk] = sf.x; sg[2 * kk + 1] = sf.y;
                    }
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const uint4 q4 = lds128(q_base + g * 2 * D + cc * 16);
                        const uint32_t qw[4] = {q4.x, q4.y, q4.z, q4.w};
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) {
                            const float x0 = bf16_lo(qw[kk]), x1 = bf16_hi(qw[kk]);
                            dot[g] = fmaf(x0, mu[2 * kk], dot[g]);
                            dot[g] = fmaf(x1, mu[2 * kk + 1], dot[g]);
                            const float t0 = x0 * sg[2 * kk], t1 = x1 * sg[2 * kk + 1];
                            var[g] = fmaf(t0, t0, var[g]);
                            var[g] = fmaf(t1, t1, var[g]);
                        }
                    }
                }
#pragma unroll
                for (int g = 0; g < G; ++g)
                    bound[g] = a.scale * min_keep_nan(dot[g] + a.z * sqrtf(var[g]), qn[g] * mn_cur);
            } else {
#pragma unroll
                for (int g = 0; g < G; ++g) bound[g] = 0.f;
            }
            if (xt && sw == 0 && lane == 0 && n_items == 3) xt[4] = globaltimer_ns();

            // ---- the buffer is free: start the copies of the warp's next item
            int nrow = row, nit0 = it0, nnit = nit, npos = pos + 1;
            bool nhave = true;
            if (last_of_claim) {
                const int ncid = __shfl_sync(0xffffffffu, pend, 0);
                nhave = ncid < NC;
                npos = 0;
                if (nhave) claim_items(ncid, nrow, nit0, nnit);
            }
            Geom gn = gc;
            float mn_next = 0.f, te_next = 0.f;
            bool te_next_have = false;
            __syncwarp();
            fence_proxy_async();          // this warp's reads of the buffer are ordered before the next copy into it
            if (nhave) {
                gn = geom_of(nrow, nit0 + npos);
                if (!safe_item(gn)) wait_pred();
                if (lane == 0) issue(gn);
                mn_next = load_mn(gn);
                if (waited) { te_next = load_te(gn); te_next_have = true; }
            }
            // the thresholds of this item, if they could not be fetched ahead (first item of the warp)
            if (!te_have) { wait_pred(); te_cur = load_te(gc); te_have = true; }
            if (xt && sw == 0 && lane == 0 && n_items == 3) xt[5] = globaltimer_ns();

            // ---- admission bits, survivors in ascending order, window statistics
            float te_g[G];
#pragma unroll
            for (int g = 0; g < G; ++g) te_g[g] = __shfl_sync(0xffffffffu, te_cur, g);     // lane g holds head g's
            unsigned m = 0;
            if (lane < n_rec) {
                const bool pinned = (j0 + lane) >= NB - a.lwb;
#pragma unroll
                for (int g = 0; g < G; ++g)
                    if (!(bound[g] < te_g[g]) || pinned) m |= 1u << g;
            }
            if (j0 + lane < a.nb_cap) a.sel_mask[(int64_t)r * a.nb_cap + j0 + lane] = (uint8_t)m;
            const unsigned nz = __ballot_sync(0xffffffffu, m != 0);
            if (m) s_list[__popc(nz & ((1u << lane) - 1u))] = (j0 + lane) | (int)(m << 24);
            int nl = __popc(nz), nblk = nl;
            if (win_claim) {
                // rescue statistics of the part of the rescue window inside this item, per query head
                const int Wr = min(a.rescue_window, NB);
                const int nwin = min(n_rec, Wr - j0);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    int cnt = (lane < nwin) ? (int)((m >> g) & 1u) : 0;
                    float best = (lane < nwin) ? bound[g] : -INFINITY;
                    int arg = (lane < nwin) ? lane : 0x7fffffff;
#pragma unroll
                    for (int s = 16; s >= 1; s >>= 1) {
                        cnt += __shfl_xor_sync(0xffffffffu, cnt, s);
                        const float ob = __shfl_xor_sync(0xffffffffu, best, s);
                        const int oa = __shfl_xor_sync(0xffffffffu, arg, s);
                        if (ob > best || (ob == best && oa < arg)) { best = ob; arg = oa; }
                    }
                    if (nwin > 0) {
                        w_cnt[g] += cnt;
                        if (best > w_best[g] && arg != 0x7fffffff) { w_best[g] = best; w_arg[g] = j0 + arg; }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) {
                if (win_claim && last_of_claim) {
                    // top-1 rescue: a head with no admitted block in the window gets the window's best block
                    const int Wr = min(a.rescue_window, NB);
                    const int n0 = nl;
                    if (Wr > 0) {
#pragma unroll
                        for (int g = 0; g < G; ++g) {
                            if (w_cnt[g] != 0) continue;
                            const int j = w_arg[g] < 0 ? 0 : w_arg[g];
                            uint8_t* mp = a.sel_mask + (int64_t)r * a.nb_cap + j;
                            const unsigned w = *reinterpret_cast<volatile uint8_t*>(mp);
                            if (w == 0) ++nblk;
                            *reinterpret_cast<volatile uint8_t*>(mp) = (uint8_t)(w | (1u << g));
                            bool merged = false;
                            for (int k = n0; k < nl; ++k)
                                if ((s_list[k] & 0xffffff) == j) { s_list[k] |= 1 << (24 + g); merged = true; }
                            if (!merged) s_list[nl++] = j | (1 << (24 + g));
                        }
                    }
                }
                // the row's tail rides with the item of the row's last full block
                const int tail_fit = NB > 0 ? (NB - 1) / FSEG : 0;
                if (gc.fit == tail_fit && gc.T > NB * a.b) s_list[nl++] = NB | (0xff << 24);
                a.f_count[(int64_t)r * a.nfs + gc.fit] = nl | (nblk << 8);
                if (gc.fit == 0 && a.status) {
                    const int Traw = __ldg(a.seq_lens + gc.i);
                    if (Traw > a.t_cap) atomicOr(a.status, ETA_DEV_LEN_CLAMPED);
                    if (Traw <= 0) atomicOr(a.status, ETA_DEV_EMPTY_ROW);
                }
            }
            nl = __shfl_sync(0xffffffffu, nl, 0);
            if (xt && sw == 0 && lane == 0 && n_items == 3) xt[6] = globaltimer_ns();

            // ---- hand the list to the producer in chunks: slots of the ring are reserved in order and filled
            // independently; the producer takes a slot when its owner has marked it ready
            if (nl > 0) {
                const int nch = (nl + FCH - 1) / FCH;
                int slot0 = 0;
                if (lane == 0) slot0 = atomicAdd(ctrl + C_RESERVE, nch);
                slot0 = __shfl_sync(0xffffffffu, slot0, 0);
                bool pushed_ok = true;
                for (int c = 0; c < nch && pushed_ok; ++c) {
                    const int slot = slot0 + c, c0 = c * FCH;
                    const int cn = min(FCH, nl - c0);
                    if (lane == 0) {
                        bool room = false;
                        for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
                            if (slot - ld_volatile(ctrl + C_HEAD) < F_RING) { room = true; break; }
                            __nanosleep(100);
                        }
                        if (!room) { pushed_ok = false; ctrl[C_FAIL] = 1; if (tl) tl[7] = (2ull << 32) | (unsigned)slot; }
                    }
                    pushed_ok = __shfl_sync(0xffffffffu, pushed_ok ? 1 : 0, 0) != 0;
                    if (!pushed_ok) break;
                    ChunkRec* rec = &ring[slot % F_RING];
                    if (lane < cn) rec->ent[lane] = s_list[c0 + lane];
                    if (lane < 8) rec->te[lane] = (lane < G) ? te_cur : 0.f;
                    if (lane == 0) {
                        rec->row = r;
                        rec->slot = (r * a.nfs + gc.fit) * FCPI + c;
                        rec->n = cn;
                    }
                    __syncwarp();
                    if (lane == 0) {
                        __threadfence_block();
                        st_volatile(ready + slot % F_RING, slot + 1);
                        atomicAdd(ctrl + C_PUSHED, cn);
                    }
                    __syncwarp();
                }
                if (!pushed_ok) break;
            }
            if (xt && sw == 0 && lane == 0 && n_items == 3) xt[7] = globaltimer_ns();

            have = nhave;
            row = nrow; it0 = nit0; nit = nnit; pos = npos;
            gc = gn;
            mn_cur = mn_next;
            te_cur = te_next;
            te_have = te_next_have;
            ++n_items;
            if (n_items > (uint32_t)(a.rows * a.nfs)) { if (lane == 0) ctrl[C_FAIL] = 1; break; }     // cannot happen
        }
        if (lane == 0) {
            if (ld_volatile(ctrl + C_FAIL)) {
                if (a.status) atomicOr(a.status, ETA_DEV_TIMEOUT);
                mbar_wait(&sbar[sw], n_items & 1);      // a copy already started must land before the CTA can go
            }
            __threadfence_block();
            atomicAdd(ctrl + C_DONE, 1);
            if (tl && sw == 0) tl[1] = globaltimer_ns();
            if (pg) pg[1] = 0xffff;
        }
        return;
    }

    if (warp == F_PRODUCER_WARP) {
        // ============================================================================== producer
        uint32_t fill = 0;
        int head = 0, done_mask = 0;
        bool ok = true;
        uint32_t idle = 0;
        bool pred_waited = false;
        while (ok) {
            const int Lg = fill % F_GROUPS;
            LaneState* st = &lst[Lg];
            if (pg && lane == 0) pg[2] = ((unsigned long long)fill << 8) | 1;
            uint32_t flags = 0;
            bool skip = false;
            if (st->k >= st->n) {
                // the lane needs a new chunk
                // read in this order: once every screening warp is done, the number of reserved slots is final
                const bool done = ld_volatile(ctrl + C_DONE) == F_SCR_WARPS;
                const int reserved = ld_volatile(ctrl + C_RESERVE);
                if (ld_volatile(reinterpret_cast<int*>(smem + L::READY_OFF) + head % F_RING) == head + 1) {
                    __threadfence_block();             // the record was written before its slot was marked ready
                    const ChunkRec* rec = &ring[head % F_RING];
                    const int qb = st->nchunks % NQB;
                    if (lane < FCH) lent[Lg * FCH + lane] = rec->ent[lane];
                    if (lane < 8) hte[(Lg * NQB + qb) * 8 + lane] = rec->te[lane];
                    __syncwarp();
                    if (lane == 0) {
                        st->n = rec->n; st->k = 0; st->sub = 0; st->row = rec->row; st->slot = rec->slot;
                        st->nchunks = st->nchunks + 1;
                        __threadfence_block();
                        st_volatile(ctrl + C_HEAD, head + 1);
                    }
                    ++head;
                    __syncwarp();
                    flags = FD_NEW | ((uint32_t)qb << 8);
                    idle = 0;
                } else {
                    if (done && head == reserved) done_mask |= 1 << Lg;
                    if (done_mask == (1 << F_GROUPS) - 1) break;
                    bool others = false;
#pragma unroll
                    for (int k = 0; k < F_GROUPS; ++k) others = others || (k != Lg && lst[k].k < lst[k].n);
                    if (!others && !(done && head == reserved)) {
                        if (++idle > WAIT_LIMIT) { ok = false; if (tl && lane == 0) tl[6] = (3ull << 32) | fill; break; }
                        __nanosleep(100);
                        continue;
                    }
                    skip = true;      // the fill still needs a marker: the groups take fills in a fixed rotation
                }
            }
            const int stage = fill % NSTAGE;
            const uint32_t round = fill / NSTAGE;
            if (pg && lane == 0) pg[2] = ((unsigned long long)fill << 8) | (skip ? 3 : 2);
            if (lane == 0) {
                if (!mbar_wait(&empty[stage], (round & 1) ^ 1)) { ok = false; if (tl) tl[6] = (4ull << 32) | fill; }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            if (lane == 0) st_volatile(ctrl + C_FILL, (int)fill + 1);      // see the consumers' wait
            if (skip) {
                if (lane == 0) {
                    desc[stage] = make_int4((int)FD_SKIP, 0, 0, 0);
                    mbar_arrive(&full[stage]);
                }
                ++fill;
                continue;
            }
            if (!pred_waited) { pdl_wait(); pred_waited = true; }
            if (lane == 0) {
                const int r = st->row;
                int i, hk;
                a.div_hkv.divmod(r, i, hk);
                const int T = s_len[r];
                const int ent = lent[Lg * FCH + st->k];
                const int j = ent & 0xffffff;
                const int hmask = (ent >> 24) & 0xff;
                const int nrows = min(a.b, T - j * a.b);
                const int sub = st->sub;
                const int nvalid = min(TS, nrows - sub * TS);
                const bool last_sub = (sub + 1) * TS >= nrows;
                if (last_sub && st->k + 1 == st->n) flags |= FD_LAST;
                if (tl && fill == 0) tl[2] = globaltimer_ns();
                desc[stage] = make_int4((int)flags, st->slot, hmask, nvalid);
                unsigned char* sp = smem + stage * L::STAGE_BYTES;
                mbar_arrive_expect_tx(&full[stage], L::STAGE_BYTES + ((flags & FD_NEW) ? L::QB_BYTES : 0));
                const int y = j * a.b + sub * TS;
                tma_load_5d(sp, &tmK, 0, y, 0, hk, i, &full[stage]);
                tma_load_5d(sp + HALVES * L::TILE_BYTES, &tmV, 0, y, 0, hk, i, &full[stage]);
                if (flags & FD_NEW) {
                    const int qb = (int)(flags >> 8);
                    tma_load_1d(smem + L::QBUF_OFF + (Lg * NQB + qb) * L::QB_BYTES,
                                a.q + ((int64_t)i * a.Hq + hk * G) * D, L::QB_BYTES, &full[stage]);
                }
                if (last_sub) {
                    st->k = st->k + 1; st->sub = 0;
                    st_volatile(ctrl + C_ISSUED, ctrl[C_ISSUED] + 1);
                } else {
                    st->sub = sub + 1;
                }
            }
            __syncwarp();
            ++fill;
        }
        pdl_trigger();
        if (pg && lane == 0) pg[2] = ((unsigned long long)fill << 8) | (ok ? 9 : 10);
        if (pg && lane == 0) pg[6] = ((unsigned long long)head << 32) | ((unsigned)done_mask << 16) | (unsigned)(idle & 0xffff);
        if (pg && lane == 0) pg[7] = ((unsigned long long)ld_volatile(ctrl + C_RESERVE) << 48) | ((unsigned long long)ld_volatile(ctrl + C_DONE) << 40) | ((unsigned long long)(ld_volatile(ctrl + C_PUSHED) & 0xfffff) << 20) | (unsigned)(ld_volatile(ctrl + C_ISSUED) & 0xfffff);
        // one end marker per group (no data): the next F_GROUPS fills reach every group exactly once
        for (int k = 0; k < F_GROUPS && ok; ++k) {
            const int stage = fill % NSTAGE;
            if (lane == 0) {
                if (!mbar_wait(&empty[stage], ((fill / NSTAGE) & 1) ^ 1)) {
                    ok = false;
                } else {
                    st_volatile(ctrl + C_FILL, (int)fill + 1);
                    desc[stage] = make_int4((int)FD_END, 0, 0, 0);
                    mbar_arrive(&full[stage]);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            ++fill;
        }
        if (!ok && lane == 0) {
            if (a.status) atomicOr(a.status, ETA_DEV_TIMEOUT);
            const uint32_t first_fill = fill > NSTAGE ? fill - NSTAGE : 0;
            for (uint32_t f = first_fill; f < fill; ++f) mbar_wait(&full[f % NSTAGE], (f / NSTAGE) & 1);
        }
        return;
    }

    // ================================================================================== consumers
    const int group = warp / F_WPG, wq = warp % F_WPG;
    float* sm_m = reinterpret_cast<float*>(smem + L::ML_OFF) + group * 2 * F_WPG * 8;
    float* sm_l = sm_m + F_WPG * 8;
    const int gtid = tid - group * 32 * F_WPG;
    const int g = lane >> 2, t = lane & 3;
    const int rb = wq * WT;
    const int r0 = rho(2 * t), r1 = rho(2 * t + 1);
    const int vchunk = ((g & 1) << 2) | (g >> 1);
    const float LOG2E = 1.4426950408889634f;
    const bool head = g < G;

    uint32_t koff[NT][2], voff[NT][2];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int krow = rb + nt * 8 + rho(g);
#pragma unroll
        for (int m = 0; m < 2; ++m) koff[nt][m] = krow * 128 + (((4 * m + t) ^ (krow & 7)) << 4);
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            const int vrow = rb + nt * 8 + (c ? r1 : r0);
            voff[nt][c] = vrow * 128 + ((vchunk ^ (vrow & 7)) << 4);
        }
    }
    // a warp's own part of a stage (the token rows it reads of every half tile) doubles as the scratch in which
    // the four warps of a group meet at the end of a chunk: float x of warp w lives at region_off(w, x)
    constexpr int PIECE_BYTES = WT * 128;
    auto region_off = [&](int w, int x) {
        const int byte = 4 * x;
        return (byte / PIECE_BYTES) * L::TILE_BYTES + w * WT * 128 + (byte % PIECE_BYTES);
    };

    uint32_t qa[HALVES][2][4];
    float o[HALVES][4][4];
    float m_run = -INFINITY, l_run = 0.f, te = 0.f;
    bool ok = true;
    uint32_t flush_phase = 0;

    for (uint32_t fill = group;; fill += F_GROUPS) {
        const int stage = fill % NSTAGE;
        if (pg && lane == 0 && wq == 0) pg[3 + group] = ((unsigned long long)fill << 8) | 1;
        volatile unsigned long long* pw = pg ? pg - (size_t)blockIdx.x * 8 + 2048 + (size_t)blockIdx.x * 16 + warp : nullptr;
        if (pw && lane == 0) *pw = ((unsigned long long)fill << 8) | 1;
        // A stage serves different groups in successive rounds (NSTAGE is not a multiple of the number of groups),
        // and a parity wait only tells the current phase from the one before it: a group that is handed markers
        // instead of tiles could otherwise ask for round k of a stage while round k - 1 has not completed and be
        // told "done".  The producer counts a fill as started once the stage's previous round has been consumed;
        // from then on the parity wait means what it should.
        {
            bool started = false;
            for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
                if ((uint32_t)ld_volatile(ctrl + C_FILL) > fill) { started = true; break; }
                __nanosleep(40);
            }
            if (!started) { ok = false; if (tl && lane == 0 && wq == 0) tl[4] = (8ull << 32) | ((unsigned long long)group << 28) | fill; break; }
        }
        if (!mbar_wait(&full[stage], (fill / NSTAGE) & 1)) {
            if (pw && lane == 0) *pw = ((unsigned long long)fill << 8) | 2;
            ok = false;
            if (tl && lane == 0 && wq == 0) tl[4] = (5ull << 32) | ((unsigned long long)group << 28) | fill;
            break;
        }
        const int4 ds = desc[stage];
        const uint32_t flags = (uint32_t)ds.x;
        if (pw && lane == 0) *pw = ((unsigned long long)fill << 8) | 0x10 | (flags & 0xf);
        if (flags & FD_END) {
            pdl_trigger();
            if (tl && warp == 0 && lane == 0) tl[5] = globaltimer_ns();
            break;
        }
        if (flags & FD_SKIP) {
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[stage]);
            continue;
        }
        if (tl && warp == 0 && lane == 0 && fill == 0) tl[3] = globaltimer_ns();
        const int hmask = ds.z, nvalid = ds.w;
        unsigned char* stage_ptr = smem + stage * L::STAGE_BYTES;
        const uint32_t kbase = smem_u32(stage_ptr);
        const uint32_t vbase = kbase + HALVES * L::TILE_BYTES;

        if (flags & FD_NEW) {
            // a new chunk: the group's queries came with this fill
            const int qb = (int)(flags >> 8);
            const uint32_t qbase = smem_u32(smem + L::QBUF_OFF + (group * NQB + qb) * L::QB_BYTES);
#pragma unroll
            for (int hf = 0; hf < HALVES; ++hf)
#pragma unroll
                for (int m = 0; m < 2; ++m) {
                    uint4 v = make_uint4(0, 0, 0, 0);
                    if (head) v = lds128(qbase + ((g * D) + 64 * hf + 32 * m + 8 * t) * 2);
                    qa[hf][m][0] = v.x; qa[hf][m][1] = v.y; qa[hf][m][2] = v.z; qa[hf][m][3] = v.w;
                }
            te = head ? hte[(group * NQB + qb) * 8 + g] : 0.f;
            m_run = -INFINITY;
            l_run = 0.f;
#pragma unroll
            for (int hf = 0; hf < HALVES; ++hf)
#pragma unroll
                for (int mt = 0; mt < 4; ++mt)
#pragma unroll
                    for (int c = 0; c < 4; ++c) o[hf][mt][c] = 0.f;
        }

        // ---- S = q K^T for this warp's WT tokens: heads on M (rows 8..15 are padding), tokens on N
        float sacc[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int c = 0; c < 4; ++c) sacc[nt][c] = 0.f;
        {
            uint4 kv[HALVES][2][NT];
#pragma unroll
            for (int hf = 0; hf < HALVES; ++hf)
#pragma unroll
                for (int m = 0; m < 2; ++m)
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) kv[hf][m][nt] = lds128(kbase + hf * L::TILE_BYTES + koff[nt][m]);
#pragma unroll
            for (int hf = 0; hf < HALVES; ++hf)
#pragma unroll
                for (int m = 0; m < 2; ++m)
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        mma_bf16_16816(sacc[nt], qa[hf][m][0], 0u, qa[hf][m][1], 0u, kv[hf][m][nt].x, kv[hf][m][nt].y);
                        mma_bf16_16816(sacc[nt], qa[hf][m][2], 0u, qa[hf][m][3], 0u, kv[hf][m][nt].z, kv[hf][m][nt].w);
                    }
        }
        uint4 v[HALVES][2 * NT];
#pragma unroll
        for (int hf = 0; hf < HALVES; ++hf)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int c = 0; c < 2; ++c) v[hf][nt * 2 + c] = lds128(vbase + hf * L::TILE_BYTES + voff[nt][c]);

        // ---- gate, mask, online softmax (lane (g,t) holds head g, tokens r0/r1 of each 8-group)
        const bool head_on = head && ((hmask >> g) & 1);
        float sg[NT][2];
        float bmax = -INFINITY;
        const bool gate_on = (te != -INFINITY);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const int trow = rb + nt * 8 + (c ? r1 : r0);
                const float S = sacc[nt][c] * a.scale;
                float gated = S;
                if (gate_on) {
                    const float x = (a.beta == 0.f) ? 0.f : a.beta * (S - te);
                    gated = S * rcp_approx(1.f + exp2f(-x * LOG2E));
                }
                gated = (head_on && trow < nvalid) ? gated : -INFINITY;
                sg[nt][c] = gated;
                bmax = fmaxf(bmax, gated);
            }
        bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 1));
        bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 2));
        const float m_new = fmaxf(m_run, bmax);
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
        const float alpha = (m_run == m_new) ? 1.f : exp2f((m_run - m_use) * LOG2E);
        float p[NT][2], psum = 0.f;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                p[nt][c] = exp2f((sg[nt][c] - m_use) * LOG2E);
                psum += p[nt][c];
            }
        l_run = l_run * alpha + psum;
        m_run = m_new;

        if (__any_sync(0xffffffffu, alpha != 1.f)) {
            const float al0 = __shfl_sync(0xffffffffu, alpha, 8 * t);
            const float al1 = __shfl_sync(0xffffffffu, alpha, 8 * t + 4);
#pragma unroll
            for (int hf = 0; hf < HALVES; ++hf)
#pragma unroll
                for (int mt = 0; mt < 4; ++mt) {
                    o[hf][mt][0] *= al0; o[hf][mt][1] *= al1; o[hf][mt][2] *= al0; o[hf][mt][3] *= al1;
                }
        }

        uint32_t pb_hi[2] = {0u, 0u}, pb_lo[2] = {0u, 0u};
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const __nv_bfloat162 hi = __floats2bfloat162_rn(p[nt][0], p[nt][1]);
            const float2 hf2 = __bfloat1622float2(hi);
            const __nv_bfloat162 lo = __floats2bfloat162_rn(p[nt][0] - hf2.x, p[nt][1] - hf2.y);
            pb_hi[nt] = *reinterpret_cast<const uint32_t*>(&hi);
            pb_lo[nt] = *reinterpret_cast<const uint32_t*>(&lo);
        }

        if (nvalid < TS) {
#pragma unroll
            for (int hf = 0; hf < HALVES; ++hf)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int c = 0; c < 2; ++c)
                        if (rb + nt * 8 + (c ? r1 : r0) >= nvalid) v[hf][nt * 2 + c] = make_uint4(0, 0, 0, 0);
        }
        const bool last = (flags & FD_LAST) != 0;
        // every shared-memory read of this stage has been issued before this point; unless the chunk ends here
        // (the stage then serves as scratch first) the stage goes back to the producer now
        __syncwarp();
        if (!last && lane == 0) mbar_arrive(&empty[stage]);
#pragma unroll
        for (int hf = 0; hf < HALVES; ++hf) {
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) {
                const uint32_t xa = u4_get(v[hf][0], mt), xb = u4_get(v[hf][1], mt);
                const uint32_t a0 = __byte_perm(xa, xb, 0x5410), a1 = __byte_perm(xa, xb, 0x7632);
                uint32_t a2 = 0u, a3 = 0u;
                if (NT == 2) {
                    const uint32_t xc = u4_get(v[hf][2 * (NT - 1)], mt), xd = u4_get(v[hf][2 * (NT - 1) + 1], mt);
                    a2 = __byte_perm(xc, xd, 0x5410);
                    a3 = __byte_perm(xc, xd, 0x7632);
                }
                mma_bf16_16816(o[hf][mt], a0, a1, a2, a3, pb_hi[0], pb_hi[1]);
                mma_bf16_16816(o[hf][mt], a0, a1, a2, a3, pb_lo[0], pb_lo[1]);
            }
        }

        if (last) {
            if (pg && lane == 0) pg[3 + group] = ((unsigned long long)fill << 8) | (4 + wq);
            // ---- the chunk is complete: combine the group's four warps and store (m, l, O) per head
            float lsum = l_run + __shfl_xor_sync(0xffffffffu, l_run, 1);
            lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
            if (t == 0) { sm_m[wq * 8 + g] = m_run; sm_l[wq * 8 + g] = lsum; }
#pragma unroll
            for (int hf = 0; hf < HALVES; ++hf)
#pragma unroll
                for (int mt = 0; mt < 4; ++mt) {
                    const int dcol = 64 * hf + 8 * vchunk + 2 * mt;
                    if (2 * t < G)
                        *reinterpret_cast<float2*>(stage_ptr + region_off(wq, (2 * t) * D + dcol)) = make_float2(o[hf][mt][0], o[hf][mt][2]);
                    if (2 * t + 1 < G)
                        *reinterpret_cast<float2*>(stage_ptr + region_off(wq, (2 * t + 1) * D + dcol)) = make_float2(o[hf][mt][1], o[hf][mt][3]);
                }
            mbar_arrive(&flushbar[group]);
            if (!mbar_wait(&flushbar[group], flush_phase)) { ok = false; if (tl && lane == 0) tl[4] = (6ull << 32) | fill; break; }
            flush_phase ^= 1;
            if (pg && lane == 0 && wq == 0) pg[3 + group] = ((unsigned long long)fill << 8) | 8;
            const int64_t slot = ds.y;
            for (int idx = gtid; idx < G * D; idx += 32 * F_WPG) {
                const int hh = idx / D, dd = idx % D;
                float M = -INFINITY;
#pragma unroll
                for (int w = 0; w < F_WPG; ++w) M = fmaxf(M, sm_m[w * 8 + hh]);
                float acc = 0.f, lacc = 0.f;
                if (M != -INFINITY) {
#pragma unroll
                    for (int w = 0; w < F_WPG; ++w) {
                        const float sc = exp2f((sm_m[w * 8 + hh] - M) * LOG2E);
                        acc = fmaf(*reinterpret_cast<const float*>(stage_ptr + region_off(w, idx)), sc, acc);
                        lacc = fmaf(sm_l[w * 8 + hh], sc, lacc);
                    }
                }
                a.part_o[(slot * G + hh) * D + dd] = acc;
                if (dd == 0) a.part_ml[slot * G + hh] = make_float2(M, lacc);
            }
            mbar_arrive(&flushbar[group]);
            if (!mbar_wait(&flushbar[group], flush_phase)) { ok = false; if (tl && lane == 0) tl[4] = (7ull << 32) | fill; break; }
            flush_phase ^= 1;
            fence_proxy_async();          // the scratch writes are ordered before the next copy into this stage
            if (lane == 0) mbar_arrive(&empty[stage]);
            if (pg && lane == 0 && wq == 0) pg[3 + group] = ((unsigned long long)fill << 8) | 9;
        }
    }
    if (!ok && lane == 0 && a.status) atomicOr(a.status, ETA_DEV_TIMEOUT);
}

// Merge of the single-kernel path: one CTA per (row, query head) adds the partials of the row's chunks in
// list order (Algorithm 3, global reduction):
//   o = sum_k O_k e^{m_k - m*} / sum_k l_k e^{m_k - m*},  m* = max_k m_k.
// It also writes the per-row fetch counts and re-arms the claim counter for the next call.
struct FusedMergeArgs {
    const int32_t* f_count;
    int32_t* f_hdr;
    const float2* part_ml;
    const float* part_o;
    float* out;
    int32_t* stats;
    int Hq, Hkv, G, nfs, rows;
};

constexpr int FM_WARPS = 8;

template <int D>
__global__ void __launch_bounds__(32 * FM_WARPS) fused_merge_kernel(const FusedMergeArgs a) {
    constexpr int VPL = D / 32;
    __shared__ float s_acc[FM_WARPS][D];
    __shared__ float s_l[FM_WARPS];
    __shared__ float s_m[FM_WARPS];
    __shared__ int s_pref[F_MAX_ITEMS_ROW + 1];
    __shared__ int s_wsum[FM_WARPS], s_wblk[FM_WARPS];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int r = blockIdx.x / a.G, gq = blockIdx.x % a.G;
    const int i = r / a.Hkv, hk = r % a.Hkv;
    pdl_wait();          // every partial of the single kernel is in memory from here on
    if (blockIdx.x == 0 && tid == 0) {
        a.f_hdr[2] = 0;
        a.f_hdr[0] = (int)F_MAGIC0;
        a.f_hdr[1] = (int)F_MAGIC1;
        __threadfence();
    }
    pdl_trigger();
    // chunks before item k of the row
    int carry = 0, blk = 0;
    for (int k0 = 0; k0 < a.nfs; k0 += 32 * FM_WARPS) {
        const int k = k0 + tid;
        const int c = (k < a.nfs) ? a.f_count[(int64_t)r * a.nfs + k] : 0;
        const int nch = ((c & 0xff) + FCH - 1) / FCH;
        blk += c >> 8;
        int incl = nch;
#pragma unroll
        for (int s = 1; s < 32; s <<= 1) {
            const int o2 = __shfl_up_sync(0xffffffffu, incl, s);
            if (lane >= s) incl += o2;
        }
        if (lane == 31) s_wsum[warp] = incl;
        __syncthreads();
        int wbase = 0, tot = 0;
        for (int w = 0; w < FM_WARPS; ++w) {
            const int v = s_wsum[w];
            if (w < warp) wbase += v;
            tot += v;
        }
        if (k < a.nfs) s_pref[k] = carry + wbase + incl - nch;
        carry += tot;
        __syncthreads();
    }
    if (tid == 0) s_pref[a.nfs] = carry;
    if (gq == 0 && a.stats) {
#pragma unroll
        for (int s = 16; s >= 1; s >>= 1) blk += __shfl_xor_sync(0xffffffffu, blk, s);
        if (lane == 0) s_wblk[warp] = blk;
    }
    __syncthreads();
    if (gq == 0 && a.stats && tid == 0) {
        int tot = 0;
        for (int w = 0; w < FM_WARPS; ++w) tot += s_wblk[w];
        a.stats[r] = tot;
    }
    const int n_cand = s_pref[a.nfs];

    float acc[VPL];
#pragma unroll
    for (int k = 0; k < VPL; ++k) acc[k] = 0.f;
    float m_w = -INFINITY, l_w = 0.f;
    const int per = (n_cand + FM_WARPS - 1) / FM_WARPS;
    const int k_begin = warp * per, k_end = min(n_cand, k_begin + per);
    for (int k0 = k_begin; k0 < k_end; k0 += 32) {
        const int k = k0 + lane;
        float m_k = -INFINITY, l_k = 0.f;
        int64_t slot = 0;
        if (k < k_end) {
            int lo = 0, hi = a.nfs - 1;          // last item whose first chunk is <= k
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if (s_pref[mid] <= k) lo = mid; else hi = mid - 1;
            }
            slot = ((int64_t)r * a.nfs + lo) * FCPI + (k - s_pref[lo]);
            const float2 ml = a.part_ml[slot * a.G + gq];
            m_k = ml.x; l_k = ml.y;
        }
        float m_round = m_k;
#pragma unroll
        for (int s = 16; s >= 1; s >>= 1) m_round = fmaxf(m_round, __shfl_xor_sync(0xffffffffu, m_round, s));
        const float m_new = fmaxf(m_w, m_round);
        if (m_new == -INFINITY) continue;
        const float rescale = (m_w == -INFINITY) ? 0.f : __expf(m_w - m_new);
        const float w = (m_k == -INFINITY) ? 0.f : __expf(m_k - m_new);
#pragma unroll
        for (int v = 0; v < VPL; ++v) acc[v] *= rescale;
        float lw = l_k * w;
#pragma unroll
        for (int s = 16; s >= 1; s >>= 1) lw += __shfl_xor_sync(0xffffffffu, lw, s);
        l_w = l_w * rescale + lw;
        m_w = m_new;
        const int nk = min(32, k_end - k0);
        for (int j0 = 0; j0 < nk; j0 += 8) {
            float wv[8];
            float xv[8][VPL];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int src = min(j0 + u, 31);
                const float wk = __shfl_sync(0xffffffffu, w, src);
                const int64_t sk = __shfl_sync(0xffffffffu, slot, src);
                wv[u] = (j0 + u < nk) ? wk : 0.f;
#pragma unroll
                for (int v = 0; v < VPL; ++v) xv[u][v] = 0.f;
                if (wv[u] != 0.f) {
                    const float* po = a.part_o + (sk * a.G + gq) * D + lane * VPL;
                    if (VPL == 4) {
                        const float4 x = *reinterpret_cast<const float4*>(po);
                        xv[u][0] = x.x; xv[u][1] = x.y; xv[u][VPL > 2 ? 2 : 0] = x.z; xv[u][VPL > 3 ? 3 : 0] = x.w;
                    } else {
                        const float2 x = *reinterpret_cast<const float2*>(po);
                        xv[u][0] = x.x; xv[u][1] = x.y;
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u)
#pragma unroll
                for (int v = 0; v < VPL; ++v) acc[v] = fmaf(xv[u][v], wv[u], acc[v]);
        }
    }
#pragma unroll
    for (int v = 0; v < VPL; ++v) s_acc[warp][lane * VPL + v] = acc[v];
    if (lane == 0) { s_l[warp] = l_w; s_m[warp] = m_w; }
    __syncthreads();
    if (tid < D) {
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < FM_WARPS; ++w) M = fmaxf(M, s_m[w]);
        float o = 0.f, l = 0.f;
        if (M != -INFINITY) {
#pragma unroll
            for (int w = 0; w < FM_WARPS; ++w) {
                const float sc = (s_m[w] == -INFINITY) ? 0.f : __expf(s_m[w] - M);
                o = fmaf(s_acc[w][tid], sc, o);
                l = fmaf(s_l[w], sc, l);
            }
        }
        a.out[((int64_t)i * a.Hq + hk * a.G + gq) * D + tid] = l > 0.f ? o / l : 0.f;
    }
}

// ------------------------------------------------------------------ host side

template <int D, int TS, int NSTAGE, int G>
static int launch_fused_t(const CUtensorMap& tmK, const CUtensorMap& tmV, const FusedArgs& a, int n_ctas,
                          cudaStream_t s, bool query_only) {
    const size_t smem = FusedSmem<D, TS, NSTAGE, G>::bytes(a.rows);
    if (smem > 227 * 1024) return ETA_ERR_UNSUPPORTED;
    if (query_only) return ETA_OK;
    static size_t configured = 0;
    if (smem > configured) {
        cudaError_t e = cudaFuncSetAttribute(fused_kernel<D, TS, NSTAGE, G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem);
        if (e != cudaSuccess) { set_cuda_error(e, "fused smem attribute"); return ETA_ERR_CUDA; }
        configured = smem;
    }
    cudaError_t e = launch_pdl(fused_kernel<D, TS, NSTAGE, G>, dim3(n_ctas), dim3(F_THREADS), smem, s, tmK, tmV, a);
    if (e != cudaSuccess) { set_cuda_error(e, "fused launch"); return ETA_ERR_CUDA; }
    return check_launch("fused");
}

template <int D, int TS, int NSTAGE>
static int launch_fused_g(const CUtensorMap& tmK, const CUtensorMap& tmV, const FusedArgs& a, int G, int n_ctas,
                          cudaStream_t s, bool query_only) {
    switch (G) {
        case 1: return launch_fused_t<D, TS, NSTAGE, 1>(tmK, tmV, a, n_ctas, s, query_only);
        case 2: return launch_fused_t<D, TS, NSTAGE, 2>(tmK, tmV, a, n_ctas, s, query_only);
        case 4: return launch_fused_t<D, TS, NSTAGE, 4>(tmK, tmV, a, n_ctas, s, query_only);
        default: return ETA_ERR_UNSUPPORTED;
    }
}

// Whether the single-kernel path can run this call: shape limits of its shared-memory tables, a rescue window of
// at most F_MAXWIN items, and a workspace that holds its per-chunk partials.
bool fused_eligible(const eta_cache_desc* d, const eta_params* p, const WsLayout& L, size_t workspace_bytes) {
    if (L.total_fused == L.total || workspace_bytes < L.total_fused) return false;
    const int G = d->n_q_heads / d->n_kv_heads;
    if (G > 4 && !(G == 8 && d->head_dim == 128)) return false;
    const int w_blocks = p->rescue_window < d->nb_cap ? p->rescue_window : d->nb_cap;
    if ((w_blocks + FSEG - 1) / FSEG > F_MAXWIN) return false;
    FusedArgs a = {};
    a.rows = L.rows;
    CUtensorMap dummy = {};
    const int TS = d->block_size < 64 ? d->block_size : 64;
    int rc;
    if (d->head_dim == 128 && TS == 64)
        rc = (G == 8) ? launch_fused_t<128, 64, 4, 8>(dummy, dummy, a, 0, nullptr, true)
                      : launch_fused_g<128, 64, 5>(dummy, dummy, a, G, 0, nullptr, true);
    else if (d->head_dim == 128) rc = launch_fused_g<128, 32, 8>(dummy, dummy, a, G, 0, nullptr, true);
    else if (TS == 64) rc = launch_fused_g<64, 64, 8>(dummy, dummy, a, G, 0, nullptr, true);
    else rc = launch_fused_g<64, 32, 8>(dummy, dummy, a, G, 0, nullptr, true);
    return rc == ETA_OK;
}

// Claims the single-kernel path splits this call into (for the choice between the two paths).
int fused_claims(const eta_cache_desc* d, const eta_params* p, const WsLayout& L) {
    const int w_blocks = p->rescue_window < d->nb_cap ? p->rescue_window : d->nb_cap;
    int nwi = (w_blocks + FSEG - 1) / FSEG;
    if (nwi > L.nfs) nwi = L.nfs;
    if (nwi < 1) nwi = 1;
    return L.rows * (1 + (L.nfs - nwi));
}

int launch_fused_decode(const eta_cache_desc* desc, const eta_params* params, const WsLayout& L, const void* q,
                        const void* K, const void* V, const int32_t* seq_lens, const void* musig, const float* mnorm,
                        const float* tau, const float* head_const, float* out, uint8_t* sel_mask, int32_t* stats,
                        uint32_t* status_dev, unsigned char* ws, int n_ctas, cudaStream_t s) {
    const int D = desc->head_dim, b = desc->block_size;
    const int G = desc->n_q_heads / desc->n_kv_heads;
    const int TS = b < 64 ? b : 64;
    CUtensorMap tmK, tmV;
    int rc = make_tmap(&tmK, K, desc, desc->k_stride_b, desc->k_stride_h, desc->k_stride_t, TS);
    if (rc != ETA_OK) return rc;
    rc = make_tmap(&tmV, V, desc, desc->v_stride_b, desc->v_stride_h, desc->v_stride_t, TS);
    if (rc != ETA_OK) return rc;

    FusedArgs a;
    a.q = static_cast<const __nv_bfloat16*>(q);
    a.musig = static_cast<const __half*>(musig);
    a.mnorm = mnorm;
    a.seq_lens = seq_lens;
    a.tau = tau;
    a.head_const = head_const;
    a.sel_mask = sel_mask;
    a.f_hdr = reinterpret_cast<int32_t*>(ws + L.f_hdr);
    a.f_count = reinterpret_cast<int32_t*>(ws + L.f_count);
    a.part_ml = reinterpret_cast<float2*>(ws + L.f_part_ml);
    a.part_o = reinterpret_cast<float*>(ws + L.f_part_o);
    a.status = status_dev;
    a.timeline = debug_timeline();
    a.z = params->z; a.a = params->a; a.beta = params->beta;
    a.scale = params->scale > 0.f ? params->scale : 1.0f / sqrtf((float)D);
    a.lwb = params->lwb; a.rescue_window = params->rescue_window;
    a.Hq = desc->n_q_heads; a.Hkv = desc->n_kv_heads; a.b = b; a.b_shift = (b == 32) ? 5 : (b == 64 ? 6 : 7);
    a.t_cap = desc->t_cap; a.nb_cap = desc->nb_cap; a.nfs = L.nfs; a.rows = L.rows;
    const int w_blocks = params->rescue_window < desc->nb_cap ? params->rescue_window : desc->nb_cap;
    a.nwi = (w_blocks + FSEG - 1) / FSEG;
    if (a.nwi > L.nfs) a.nwi = L.nfs;
    if (a.nwi < 1) a.nwi = 1;
    a.spr = L.nfs - a.nwi;
    a.n_claims = L.rows * (1 + a.spr);
    a.div_hkv = FastDiv(desc->n_kv_heads);
    a.div_spr = FastDiv(a.spr > 0 ? a.spr : 1);

    profile_mark(2, s);
    profile_mark(3, s);
    if (D == 128 && TS == 64)
        rc = (G == 8) ? launch_fused_t<128, 64, 4, 8>(tmK, tmV, a, n_ctas, s, false)
                      : launch_fused_g<128, 64, 5>(tmK, tmV, a, G, n_ctas, s, false);
    else if (D == 128) rc = launch_fused_g<128, 32, 8>(tmK, tmV, a, G, n_ctas, s, false);
    else if (TS == 64) rc = launch_fused_g<64, 64, 8>(tmK, tmV, a, G, n_ctas, s, false);
    else rc = launch_fused_g<64, 32, 8>(tmK, tmV, a, G, n_ctas, s, false);
    if (rc != ETA_OK) return rc;
    profile_mark(4, s);

    FusedMergeArgs ma;
    ma.f_count = a.f_count; ma.f_hdr = a.f_hdr; ma.part_ml = a.part_ml; ma.part_o = a.part_o; ma.out = out;
    ma.stats = stats; ma.Hq = desc->n_q_heads; ma.Hkv = desc->n_kv_heads; ma.G = G; ma.nfs = L.nfs; ma.rows = L.rows;
    const unsigned mgrid = (unsigned)(L.rows * G);
    cudaError_t me = (D == 128) ? launch_pdl(fused_merge_kernel<128>, dim3(mgrid), dim3(32 * FM_WARPS), 0, s, ma)
                                : launch_pdl(fused_merge_kernel<64>, dim3(mgrid), dim3(32 * FM_WARPS), 0, s, ma);
    if (me != cudaSuccess) { set_cuda_error(me, "fused merge launch"); return ETA_ERR_CUDA; }
    profile_mark(5, s);
    return check_launch("fused merge");
}

}  // namespace eta

// Streaming stage of eta_decode: SiLU-gated attention over the surviving blocks
// (Algorithm 3, attention lines and tail phase; Eq. mult_attn at inference), the
// GQA-grouped execution of the fused-kernel appendix, and the associative
// (m, l, O) merge of its "two-stage reduction".
//
// decode_kernel is persistent, one CTA per SM.  Work is the flattened sequence
// of "units": for each (sequence, KV head) row its surviving blocks (the
// screening kernel's per-segment lists), then its rescued blocks, then its tail.
// Every CTA lays that sequence out for itself from the per-segment counts and
// takes an equal, contiguous share of its COST (units, plus a fixed charge for
// every row boundary inside the share: stream-K), so the load is balanced
// whatever the per-head survivor counts are; a share may cross rows, and a row
// may be split over CTAs; each (CTA, row) piece produces one partial (m, l, O)
// per query head and consumer group.
//
// Inside a CTA one producer warp walks the survivor lists and issues tiled TMA
// copies (5-D tensor maps, 128-byte swizzle) of K and V tiles into a ring of
// shared-memory stages; three consumer groups of four warps take the fills in
// rotation, each warp a quarter of a tile's tokens.  The G query heads of the
// group are packed on the M side of mma.m16n8k16 (bf16 in, fp32 out), tokens on
// N, so each K/V byte is read once from HBM and once from shared memory for all
// heads.  The head_dim and token orders fed to the MMAs are permuted (a dot
// product does not care) so that every shared-memory read is a conflict-free
// 16-byte load of the swizzled tile.  Softmax statistics and accumulators are
// fp32; P is fed to the second MMA as a bf16 high part plus a bf16 residual, so
// the product keeps fp32-level accuracy.  Every wait is bounded.
//
// merge_kernel folds the partials of a (row, head) in a fixed order: a CTA per
// (row, head, slice of head_dim).
#include <cuda.h>

#include "eta_common.cuh"
#include "eta_timeline.h"

namespace eta {

struct DecodeArgs {
    const __nv_bfloat16* q;
    const int32_t* seq_lens;
    const float* tau_eff;
    const int32_t* seg_list;
    const int32_t* seg_count;
    const RescueRec* seg_resc;
    uint8_t* sel_mask;
    int32_t* stats;
    int2* row_span;      // [rows] first streaming CTA that holds units of the row, number of such CTAs
    float2* part_ml;
    float* part_o;
    uint32_t* status;
    float beta, scale;
    int Hq, Hkv, G, b, t_cap, nb_cap, nseg, entries, rows, rescue_window;
    int ungate_last;     // the newest token of every sequence keeps its raw logit (ETA_FLAG_UNGATE_LAST)
    const int32_t* block_table;   // paged cache: [batch, table_stride] page of every block of tokens; null: contiguous
    int table_stride;
    FastDiv div_nseg, div_epr, div_hkv, div_g;
    unsigned long long* timeline;
};

constexpr uint32_t UF_END = 1u;
constexpr int WARPS_PER_GROUP = 4;     // the four warps of a group each take a quarter of a tile's tokens
// Tiles a row boundary inside a CTA's range is worth (flush of the partials, query reload, a pipeline that runs dry
// while a group flushes).  Measured: 3 left the CTAs with several pieces last by 8 us on the mixed-length
// configuration (128 rows); 6, 8, 10 and 14 are within noise of each other on every configuration.
constexpr int PIECE_COST = 8;
constexpr int RESC_ROWS = 8;           // rows (from the CTA's first) whose rescue decisions stay in shared memory
constexpr int PW = 256;                // entries of the unit prefix the producer keeps in shared memory

__device__ __forceinline__ uint32_t u4_get(const uint4& v, int i) {
    return i == 0 ? v.x : (i == 1 ? v.y : (i == 2 ? v.z : v.w));
}
// token row inside an 8-row group that MMA column n reads: bits 0 and 2 of n swapped, so that the two
// rows a quarter-warp touches in one 16-byte load sit in different halves of the swizzle pattern
__device__ __forceinline__ int rho(int n) { return (n & 2) | ((n & 1) << 2) | ((n >> 2) & 1); }
__device__ __forceinline__ float rcp_approx(float x) {
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}


// Top-1 rescue of query head g of row r (Algorithm 3, rescue phase): if none of the first
// Wr = min(rescue_window, NB) blocks was admitted for the head, the first block with the largest bound among them
// is.  Combines the per-segment statistics the screening kernel left.  -> rescued block index, or -1.
__device__ __forceinline__ int rescue_of(const RescueRec* __restrict__ seg_resc, int r, int g, int G, int nseg,
                                          int Wr) {
    if (Wr <= 0) return -1;
    const int nsw = (Wr + SEG - 1) / SEG;
    int cnt = 0, arg = -1;
    float best = -INFINITY;
    for (int s0 = 0; s0 < nsw; s0 += 4) {
        int4 raw[4];
#pragma unroll
        for (int k = 0; k < 4; ++k)          // four segments' statistics in flight at once
            raw[k] = (s0 + k < nsw) ? __ldg(reinterpret_cast<const int4*>(seg_resc + ((int64_t)r * nseg + s0 + k) * G + g))
                                    : make_int4(0, 0, -1, 0);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            cnt += raw[k].x;
            const float mb = __int_as_float(raw[k].y);
            if (raw[k].z >= 0 && mb > best) { best = mb; arg = raw[k].z; }   // ascending segments: ties keep the lowest index
        }
    }
    if (cnt != 0) return -1;
    return arg < 0 ? 0 : arg;
}

// The rescued blocks of a row as fetch units: heads that rescue the same block share one unit.
// -> number of units; unit k is block uj[k] with head bits um[k].
__device__ __forceinline__ int rescue_units(const RescueRec* __restrict__ seg_resc, int r, int G, int nseg, int Wr,
                                            int (&uj)[8], int (&um)[8]) {
    int n = 0;
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        uj[g] = -1; um[g] = 0;
    }
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        if (g < G) {
            const int j = rescue_of(seg_resc, r, g, G, nseg, Wr);
            if (j >= 0) {
                bool merged = false;
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if (k < n && uj[k] == j) { um[k] |= 1 << g; merged = true; }
                if (!merged) {
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        if (k == n) { uj[k] = j; um[k] = 1 << g; }
                    ++n;
                }
            }
        }
    }
    return n;
}

template <int D, int TS, int NSTAGE, int NGROUPS>
struct DecodeSmem {
    static constexpr int HALVES = D / 64;
    static constexpr int TILE_BYTES = TS * 128;                 // one 64-column half tile
    static constexpr int STAGE_BYTES = 2 * HALVES * TILE_BYTES; // K halves then V halves
    static constexpr int BAR_OFF = NSTAGE * STAGE_BYTES;        // full[NSTAGE], empty[NSTAGE], flush[NGROUPS]
    static constexpr int DESC_OFF = BAR_OFF + 8 * (2 * NSTAGE + NGROUPS + (NGROUPS & 1));
    static constexpr int WIN_OFF = DESC_OFF + 16 * NSTAGE;      // int32 pwin[PW + 1] (+3 pad): window of the unit prefix
    static constexpr int ROW_OFF = WIN_OFF + 4 * (PW + 4);      // int32 rowbase[MAX_ROWS + 1]: unit prefix over rows
    static constexpr int INFO_OFF = ROW_OFF + 4 * (MAX_ROWS + 4);   // uint8 per row: rescue units | tail flag << 7
    static constexpr int NZP_OFF = INFO_OFF + MAX_ROWS;         // uint16 per row: rows with at least one unit before the row
    static constexpr int RESC_OFF = NZP_OFF + 2 * MAX_ROWS;     // int32 [RESC_ROWS][8]: rescued block per head, first rows
    static constexpr int ML_OFF = RESC_OFF + 4 * 8 * RESC_ROWS; // float m[NGROUPS][4][8], l[NGROUPS][4][8]
    static constexpr int MO_OFF = ML_OFF + 4 * 2 * NGROUPS * WARPS_PER_GROUP * 8;
    static size_t bytes(int G) { return 1024 + MO_OFF + sizeof(float) * NGROUPS * WARPS_PER_GROUP * G * D; }
};

// The streaming kernel.  Warp roles: NGROUPS consumer groups of four warps, then one producer warp.  Group k
// consumes the stage fills k, k + NGROUPS, ...; with two or three groups every scheduler holds several warps in
// different phases of a tile, which hides the fixed latencies of the MMA / shuffle / exp chains.  Each group
// keeps its own running (m, l, O) and writes its own partial per (CTA, row) piece.
template <int D, int TS, int NSTAGE, int NGROUPS>
__global__ void __launch_bounds__(32 * (WARPS_PER_GROUP * NGROUPS + 1), 1)
decode_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const DecodeArgs a) {
    using L = DecodeSmem<D, TS, NSTAGE, NGROUPS>;
    constexpr int HALVES = L::HALVES;
    constexpr int WT = TS / WARPS_PER_GROUP;    // tokens per consumer warp per tile (8 or 16)
    constexpr int NT = WT / 8;                  // 8-token MMA column tiles per warp
    constexpr int PRODUCER_WARP = WARPS_PER_GROUP * NGROUPS;
    static_assert(NT == 1 || NT == 2, "tile must give each warp 8 or 16 tokens");

    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::BAR_OFF);
    uint64_t* empty = full + NSTAGE;
    uint64_t* flushbar = empty + NSTAGE;
    int4* desc = reinterpret_cast<int4*>(smem + L::DESC_OFF);
    int32_t* pwin = reinterpret_cast<int32_t*>(smem + L::WIN_OFF);
    int32_t* rowbase = reinterpret_cast<int32_t*>(smem + L::ROW_OFF);
    uint8_t* rowinfo = smem + L::INFO_OFF;
    uint16_t* nzp = reinterpret_cast<uint16_t*>(smem + L::NZP_OFF);
    int32_t* resc_tab = reinterpret_cast<int32_t*>(smem + L::RESC_OFF);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned long long* const tl = ETA_TL(a.timeline ? a.timeline + (size_t)(TL_DECODE + blockIdx.x) * 8 : nullptr);
    unsigned long long* const tl2 = ETA_TL(a.timeline ? a.timeline + (size_t)(TL_DECODE2 + blockIdx.x) * 8 : nullptr);
    if (tl && tid == 0) tl[0] = globaltimer_ns();
    // When NSTAGE is not a multiple of NGROUPS a stage serves different groups in successive rounds, and a parity
    // wait only tells the current phase of a barrier from the one before it: a group that runs ahead could ask for
    // round k of a stage while round k - 1 (another group's) has not completed and be told "done".  In those
    // configurations the producer publishes the number of fills it has started (each only after the stage's
    // previous round was consumed) and a consumer looks at its barrier only once its fill is among them.
    constexpr bool SHARED_STAGES = (NSTAGE % NGROUPS) != 0;
    __shared__ int s_fill_started;
    if (tid == 0) {
        s_fill_started = 0;
        for (int s = 0; s < NSTAGE; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], WARPS_PER_GROUP); }
        for (int k = 0; k < NGROUPS; ++k) mbar_init(&flushbar[k], 32 * WARPS_PER_GROUP);
        fence_barrier_init();
        prefetch_tmap(&tmK);
        prefetch_tmap(&tmV);
    }
    // scratch for the layout, in the (still unused) stage memory
    constexpr int NWARPS = WARPS_PER_GROUP * NGROUPS + 1;
    constexpr int NTHREADS = 32 * NWARPS;
    int* resc_j = reinterpret_cast<int*>(smem);                // [rows][8] rescued block per head, -1: none
    int* s_len = resc_j + 8 * MAX_ROWS;                        // [rows] clamped sequence length
    int* rowcnt = s_len + MAX_ROWS;                            // [rows] surviving blocks of the row
    // [rows][nseg + 2] units per entry of the flattened sequence: a row's segments (surviving blocks), then its rescue
    // units, then its tail (0 or 1): what the producer's first prefix window is summed from, one byte load per entry
    uint8_t* cnt8 = reinterpret_cast<uint8_t*>(rowcnt + MAX_ROWS);
    const bool counts_in_smem = (size_t)a.entries + 10 * 4 * MAX_ROWS <= (size_t)NSTAGE * L::STAGE_BYTES;
    // sequence lengths are a caller input: they can be read while the previous kernel is still running
    for (int rr = tid; rr < a.rows; rr += NTHREADS) {
        const int T = __ldg(a.seq_lens + a.div_hkv.div(rr));
        s_len[rr] = T < 0 ? 0 : (T > a.t_cap ? a.t_cap : T);
        rowcnt[rr] = 0;
    }
    __syncthreads();
    pdl_wait();          // the screening kernel's lists, counts and window statistics are complete from here on
    if (tl && tid == 0) tl[7] = globaltimer_ns();
    const unsigned long long clk0 = ETA_TL(reinterpret_cast<unsigned long long*>(1)) ? (unsigned long long)clock64() : 0ull;

    // ---- every CTA lays out the flattened unit sequence for itself: per row the surviving blocks of its
    // segments, then its rescued blocks, then its tail; a scan over the rows gives each row's first unit.
    // The code below runs once per CTA on a cold instruction cache, where every instruction costs tens of cycles:
    // it is written as small loops rather than unrolled, and with as few dependent round trips to L2 as the data
    // allow (one for the counts and window statistics, later one for the first list words).
    __shared__ int s_lay[5];      // rows with units; the CTA's unit range; CTAs that share the units; row of the first unit
    {
        // All loads of the layout are independent and issued together, before any of them is consumed: per thread
        // eight segment counts and, for the thread's (row, head) pair, the window statistics of up to four segments
        // of the rescue window.
        const int n_cnt = a.rows * a.nseg, n_rh = a.rows * a.G;
        auto resc_load = [&](int p, int s0, int4 (&raw)[4], int& Wr) {
            int rr, g;
            a.div_g.divmod(p, rr, g);
            Wr = (p < n_rh) ? min(a.rescue_window, min(s_len[min(rr, a.rows - 1)] / a.b, a.nb_cap)) : 0;
#pragma unroll
            for (int k = 0; k < 4; ++k)
                raw[k] = ((s0 + k) * SEG < Wr)
                    ? __ldg(reinterpret_cast<const int4*>(a.seg_resc + ((int64_t)rr * a.nseg + s0 + k) * a.G + g))
                    : make_int4(0, 0, -1, 0);
        };
        // combines window statistics in ascending segment order: the admitted counts add up, the largest bound
        // wins, the first block among equal bounds
        auto resc_fold = [&](const int4 (&raw)[4], int& cnt, float& best, int& arg) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                cnt += raw[k].x;
                const float mb = __int_as_float(raw[k].y);
                if (raw[k].z >= 0 && mb > best) { best = mb; arg = raw[k].z; }
            }
        };
        auto count_consume = [&](int e, int c) {
            if (e < n_cnt) {
                const int rr = a.div_nseg.div(e);
                if (counts_in_smem) cnt8[e + 2 * rr] = (uint8_t)c;       // entry rr (nseg + 2) + segment
                if (c) atomicAdd(&rowcnt[rr], c);
            }
        };
        int4 raw[4];
        int Wr;
        resc_load(tid, 0, raw, Wr);
        int cv[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int e = tid + k * NTHREADS;
            cv[k] = (e < n_cnt) ? __ldg(a.seg_count + e) : 0;
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) count_consume(tid + k * NTHREADS, cv[k]);
        for (int e0 = tid + 8 * NTHREADS; e0 < n_cnt; e0 += NTHREADS) count_consume(e0, __ldg(a.seg_count + e0));
        // Top-1 rescue of head g of row rr (Algorithm 3, rescue phase): if none of the first
        // Wr = min(rescue_window, NB) blocks was admitted for the head, the first block with the largest bound among
        // them is.  The G heads of a row sit in consecutive lanes of one warp: a head whose block an earlier head of
        // the row rescued too shares that head's fetch unit.
        for (int p0 = 0; p0 < n_rh; p0 += NTHREADS) {
            const int p = p0 + tid;
            if (p0 > 0) resc_load(p, 0, raw, Wr);
            int cnt = 0, arg = -1;
            float best = -INFINITY;
            resc_fold(raw, cnt, best, arg);
            for (int s0 = 4; s0 * SEG < Wr; s0 += 4) {      // windows of more than four segments
                resc_load(p, s0, raw, Wr);
                resc_fold(raw, cnt, best, arg);
            }
            const int rj = (p < n_rh && Wr > 0 && cnt == 0) ? (arg < 0 ? 0 : arg) : -1;
            int rr, g;
            a.div_g.divmod(p, rr, g);
            bool dup = false;
            for (int o = 1; o < a.G; ++o) {
                const int jo = __shfl_up_sync(0xffffffffu, rj, o);
                dup = dup || (o <= g && jo == rj);
            }
            const unsigned uniq = __ballot_sync(0xffffffffu, rj >= 0 && !dup);
            if (p < n_rh) {
                resc_j[rr * 8 + g] = rj;
                if (g == 0) {
                    const int n_resc = __popc((uniq >> (lane & 31)) & ((1u << a.G) - 1u));
                    const int tailf = (s_len[rr] & (a.b - 1)) ? 1 : 0;
                    rowinfo[rr] = (uint8_t)(n_resc | (tailf << 7));
                    if (counts_in_smem) {
                        cnt8[rr * (a.nseg + 2) + a.nseg] = (uint8_t)n_resc;
                        cnt8[rr * (a.nseg + 2) + a.nseg + 1] = (uint8_t)tailf;
                    }
                }
            }
        }
    }
    if (tl2 && tid == 0) tl2[0] = (unsigned long long)clock64() - clk0;
    __syncthreads();
    // Publishing for the merge kernel and the caller is shared out over the CTAs (all of them hold the same layout):
    // CTA c takes the rows c, c + gridDim.x, ...  Here the rescued heads' admission bits and the number of blocks
    // fetched per row; the rows' spans of CTAs follow once the split is known.
    if (warp >= 1) {
        for (int rr = blockIdx.x + (tid - 32) * gridDim.x; rr < a.rows; rr += (NTHREADS - 32) * gridDim.x) {
            int extra = 0;
            for (int g = 0; g < a.G; ++g) {
                const int j = resc_j[rr * 8 + g];
                if (j < 0) continue;
                uint8_t* mp = a.sel_mask + (int64_t)rr * a.nb_cap + j;
                const unsigned w = *mp;
                bool dup = false;
                for (int g2 = 0; g2 < g; ++g2) dup = dup || (resc_j[rr * 8 + g2] == j);
                if (w == 0 && !dup) ++extra;      // a block no head had admitted: one more block fetched
                *mp = (uint8_t)(w | (1u << g));
            }
            if (a.stats) a.stats[rr] = rowcnt[rr] + extra;
        }
    }
    // Equal shares of COST, not of units: a row that starts inside a CTA's range costs that CTA a flush of its
    // partials and a query reload, worth about PIECE_COST tiles.  Row rr spans the cost interval
    // [rowbase[rr] + PIECE_COST * nzp[rr], +PIECE_COST (if it has units) + its units).  The first warp scans the
    // rows, two of its lanes find the CTA's two range ends; everybody else picks them up after the barrier.
    if (warp == 0) {
        int carry_u = 0, carry_z = 0;
        int my_units = 0, my_base = 0, my_nzp = 0;          // of row `lane` (used when there are at most 32 rows)
        for (int r0 = 0; r0 < a.rows; r0 += 32) {
            const int rr = r0 + lane;
            int units = 0;
            if (rr < a.rows) {
                const int info = rowinfo[rr];
                units = rowcnt[rr] + (info & 0x7f) + (info >> 7);      // surviving blocks, rescued blocks, tail
            }
            const int nzf = units > 0 ? 1 : 0;
            int iu = units, iz = nzf;
#pragma unroll
            for (int sft = 1; sft < 32; sft <<= 1) {
                const int ou = __shfl_up_sync(0xffffffffu, iu, sft);
                const int oz = __shfl_up_sync(0xffffffffu, iz, sft);
                if (lane >= sft) { iu += ou; iz += oz; }
            }
            my_units = units; my_base = carry_u + iu - units; my_nzp = carry_z + iz - nzf;
            if (rr < a.rows) { rowbase[rr] = my_base; nzp[rr] = (uint16_t)my_nzp; }
            carry_u += __shfl_sync(0xffffffffu, iu, 31);
            carry_z += __shfl_sync(0xffffffffu, iz, 31);
        }
        if (lane == 0) { rowbase[a.rows] = carry_u; s_lay[0] = carry_z; }
        __syncwarp();
        const int nz_rows = carry_z, U = carry_u;
        // More cost units per CTA than a row's padding (fewer CTAs take part in a tiny problem): then no CTA's
        // range lies inside a padding; the CTAs that meet a row are exactly those between two ends that follow
        // from the row's cost interval in closed form (the merge kernel finds its candidates that way).
        const uint32_t C = (uint32_t)U + (uint32_t)PIECE_COST * (uint32_t)nz_rows;
        const uint32_t P = min((uint32_t)gridDim.x, max(1u, C / (uint32_t)(PIECE_COST + 1)));
        const uint32_t cq = C / P, cr = C - cq * P;
        // cost position x -> unit: the last row rr in [0, rows] whose cost interval starts at or before x holds it
        // (rows start in ascending order of cost).  Up to 32 rows: every lane compares its own row, a ballot counts;
        // more rows: a binary search over the prefix arrays.
        auto cost_to_unit = [&](uint32_t c) {
            if (c >= P) return U;
            const uint32_t x = c * cq + (c * cr) / P;        // floor(c C / P) without a 64-bit division: c cr < 2^16
            int lo, lo_units, lo_base, lo_nzp;
            if (a.rows <= 32) {
                const bool le = lane < a.rows && (uint32_t)my_base + (uint32_t)PIECE_COST * (uint32_t)my_nzp <= x;
                lo = __popc(__ballot_sync(0xffffffffu, le)) - 1;        // x >= 0 = the first row's start: lo >= 0
                if (C <= x) return U;                                   // (cannot happen for c < P; the sentinel row)
                lo_units = __shfl_sync(0xffffffffu, my_units, lo);
                lo_base = __shfl_sync(0xffffffffu, my_base, lo);
                lo_nzp = __shfl_sync(0xffffffffu, my_nzp, lo);
            } else {
                int l2 = 0, h2 = a.rows;
                while (l2 < h2) {
                    const int mid = (l2 + h2 + 1) >> 1;
                    const uint32_t nzb = (mid < a.rows) ? nzp[mid] : (uint32_t)nz_rows;
                    if ((uint32_t)rowbase[mid] + (uint32_t)PIECE_COST * nzb <= x) l2 = mid; else h2 = mid - 1;
                }
                if (l2 >= a.rows) return U;
                lo = l2; lo_base = rowbase[lo]; lo_units = rowbase[lo + 1] - lo_base; lo_nzp = nzp[lo];
            }
            int off = (int)(x - ((uint32_t)lo_base + (uint32_t)PIECE_COST * (uint32_t)lo_nzp)) - (lo_units > 0 ? PIECE_COST : 0);
            off = off < 0 ? 0 : (off > lo_units ? lo_units : off);
            return lo_base + off;
        };
        const int unit0 = cost_to_unit(blockIdx.x), unit1 = cost_to_unit(blockIdx.x + 1);
        // row holding the CTA's first unit: the last row that starts at or before it
        int r_first;
        if (a.rows <= 32) {
            r_first = max(0, __popc(__ballot_sync(0xffffffffu, lane < a.rows && my_base <= unit0)) - 1);
        } else {
            int l2 = 0, h2 = a.rows - 1;
            while (l2 < h2) {
                const int mid = (l2 + h2 + 1) >> 1;
                if (rowbase[mid] <= unit0) l2 = mid; else h2 = mid - 1;
            }
            r_first = l2;
        }
        if (lane == 0) { s_lay[1] = unit0; s_lay[2] = unit1; s_lay[3] = (int)P; s_lay[4] = r_first; }
        if (tl2 && tid == 0) tl2[3] = (unsigned long long)clock64() - clk0;
    }
    __syncthreads();
    if (tl2 && tid == 0) tl2[4] = (unsigned long long)clock64() - clk0;
    const int U = rowbase[a.rows];
    const int u0 = s_lay[1], u1 = s_lay[2];
    const int row0 = s_lay[4];
    if (warp == 1) {
        // For the merge kernel: the streaming CTAs that hold units of each row.  CTA c has the cost interval
        // [floor(c C / P), floor((c + 1) C / P)), row rr the interval [cs, ce) whose first PIECE_COST units are
        // padding, and c holds units of the row exactly when its interval starts before ce and ends after the
        // padding.
        const int64_t C = (int64_t)U + (int64_t)PIECE_COST * s_lay[0];
        const int64_t P = s_lay[3];
        for (int rr = blockIdx.x + lane * gridDim.x; rr < a.rows; rr += 32 * gridDim.x) {
            const int units = rowbase[rr + 1] - rowbase[rr];
            int c_lo = 0, n_span = 0;
            if (units > 0) {
                const int64_t cs = (int64_t)rowbase[rr] + (int64_t)PIECE_COST * nzp[rr], ce = cs + PIECE_COST + units;
                const int c_hi = (int)((ce * P - 1) / C);
                c_lo = (int)(((cs + PIECE_COST + 1) * P + C - 1) / C) - 1;
                n_span = c_hi - c_lo + 1;
            }
            a.row_span[rr] = make_int2(c_lo, n_span);
        }
    }
    if (tl && tid == 0) tl[1] = globaltimer_ns();
    if (u0 >= u1) return;

    if (warp == PRODUCER_WARP) {
        // ------------------------------------------------------------ producer
        // The CTA's units [u0, u1) are located through a shared-memory window of the unit prefix (PW entries from
        // entry e_base on): each lane finds the entry of one unit by binary search in the window and fetches that
        // unit's list word, so a batch of up to 32 units costs one round trip to L2, and the next batch is fetched
        // while the current one is being issued.
        const int EPR = a.nseg + 2;        // per row: its segments, then the rescue entry, then the tail entry
        const int E = a.entries;
        int e_base = row0 * EPR;
        int base_units = rowbase[row0];    // units before entry e_base
        uint32_t fill = 0;
        int piece = -1, prev_row = -1;
        uint32_t piece_f0 = 0;
        bool ok = true;

        // groups that receive no tile of a piece never write its partial: mark those slots "absent" for the merge
        auto close_piece = [&]() {
            if (prev_row < 0) return;
            const uint32_t n = fill - piece_f0;
            for (uint32_t k = n; k < (uint32_t)NGROUPS; ++k) {
                const int grp = (int)((piece_f0 + k) % NGROUPS);
                const int64_t slot = ((int64_t)blockIdx.x + prev_row) * NGROUPS + grp;
                if (lane < a.G) a.part_ml[slot * a.G + lane] = make_float2(-INFINITY, 0.f);
            }
        };

        // units of entry e: survivors of a segment, rescue units of the row, or the row's tail
        bool first_window = counts_in_smem;     // the counts of the layout phase are still in the stage memory
        auto entry_count = [&](int e) {
            if (first_window) return (e < E) ? (int)cnt8[e] : 0;
            int r, sg;
            a.div_epr.divmod(min(e, E - 1), r, sg);
            const bool is_seg = sg < a.nseg;
            int v = 0;
            if (e < E && is_seg) v = __ldg(a.seg_count + r * a.nseg + sg);
            const int info = rowinfo[r];
            return (e >= E) ? 0 : (is_seg ? v : (sg == a.nseg ? (info & 0x7f) : (info >> 7)));
        };
        // pwin[k] = units before entry e_base + k, k = 0 .. PW: lane l counts the PW / 32 consecutive entries from
        // e_base + l PW / 32 on, one warp scan over the lanes' totals gives each lane its first prefix
        auto load_window = [&]() {
            __syncwarp();
            constexpr int EPL = PW / 32;
            int cw[EPL];
#pragma unroll
            for (int m = 0; m < EPL; ++m) cw[m] = entry_count(e_base + EPL * lane + m);   // all loads in flight
            int tot = 0;
#pragma unroll
            for (int m = 0; m < EPL; ++m) tot += cw[m];
            int incl = tot;
#pragma unroll
            for (int sft = 1; sft < 32; sft <<= 1) {
                const int o = __shfl_up_sync(0xffffffffu, incl, sft);
                if (lane >= sft) incl += o;
            }
            int run = base_units + incl - tot;
#pragma unroll
            for (int m = 0; m < EPL; ++m) { pwin[EPL * lane + m] = run; run += cw[m]; }
            if (lane == 31) pwin[PW] = run;
            __syncwarp();
        };
        auto search = [&](int uu) {          // largest k in [0, PW) with pwin[k] <= uu
            int lo = 0, hi = PW - 1;
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if (pwin[mid] <= uu) lo = mid; else hi = mid - 1;
            }
            return lo;
        };
        // make the window hold the entry of unit ub; -> number of units of the batch starting at ub
        auto batch_size = [&](int ub) {
            while (true) {
                const bool reaches_end = (e_base + PW >= E);
                const int wend = pwin[PW];
                const int want = min(32, u1 - ub);
                if (reaches_end || wend >= ub + want) return want;
                if (wend <= ub) { e_base += PW; base_units = wend; load_window(); continue; }
                const int k0 = search(ub);
                if (k0 == 0) return min(want, wend - ub);
                base_units = pwin[k0];
                e_base += k0;
                load_window();
            }
        };
        // per-lane description of unit ub + lane (row < 0: no such unit in this batch)
        auto fetch = [&](int ub, int nb, int& row, int& ent, int& nrows, int& page) {
            row = -1; ent = 0; nrows = 0; page = 0;
            if (lane < nb) {
                const int uu = ub + lane;
                const int k = search(uu);
                const int e = e_base + k;
                int r, sg;
                a.div_epr.divmod(e, r, sg);
                row = r;
                if (sg >= a.nseg) {
                    int T = __ldg(a.seq_lens + a.div_hkv.div(r));
                    T = T < 0 ? 0 : (T > a.t_cap ? a.t_cap : T);
                    const int NB = min(T / a.b, a.nb_cap);
                    if (sg == a.nseg) {
                        // a rescued block, attended by the rescued head(s) only
                        int uj[8], um[8];
                        if (r - row0 < RESC_ROWS) {
                            // same merge of equal blocks as rescue_units, from the table kept in shared memory
                            int n = 0;
#pragma unroll
                            for (int g8 = 0; g8 < 8; ++g8) { uj[g8] = -1; um[g8] = 0; }
#pragma unroll
                            for (int g8 = 0; g8 < 8; ++g8) {
                                const int j8 = resc_tab[(r - row0) * 8 + g8];
                                if (j8 >= 0) {
                                    bool merged = false;
#pragma unroll
                                    for (int q8 = 0; q8 < 8; ++q8)
                                        if (q8 < n && uj[q8] == j8) { um[q8] |= 1 << g8; merged = true; }
                                    if (!merged) {
#pragma unroll
                                        for (int q8 = 0; q8 < 8; ++q8)
                                            if (q8 == n) { uj[q8] = j8; um[q8] = 1 << g8; }
                                        ++n;
                                    }
                                }
                            }
                        } else {
                            rescue_units(a.seg_resc, r, a.G, a.nseg, min(a.rescue_window, NB), uj, um);
                        }
                        const int idx = uu - pwin[k];
                        int j = 0, m = 0;
#pragma unroll
                        for (int q8 = 0; q8 < 8; ++q8)
                            if (q8 == idx) { j = uj[q8]; m = um[q8]; }
                        ent = j | (m << 24);
                        nrows = a.b;
                    } else {
                        ent = NB | (0xff << 24);           // the tail: every head attends it
                        nrows = T - NB * a.b;
                        if (a.ungate_last) nrows |= 0x10000;      // its last token is the sequence's newest
                    }
                } else {
                    ent = __ldg(a.seg_list + ((int64_t)r * a.nseg + sg) * LSTRIDE + (uu - pwin[k]));
                    nrows = a.b;
                    if (a.ungate_last) {
                        int T = __ldg(a.seq_lens + a.div_hkv.div(r));
                        T = T < 0 ? 0 : (T > a.t_cap ? a.t_cap : T);
                        if (((ent & 0xffffff) + 1) * a.b == T) nrows |= 0x10000;   // the block the newest token closes
                    }
                }
                // paged cache: the page that holds the unit's block of tokens (one more dependent load per batch,
                // hidden like the list fetch behind the tiles already on their way)
                if (a.block_table)
                    page = __ldg(a.block_table + (int64_t)a.div_hkv.div(r) * a.table_stride + (ent & 0xffffff));
            }
        };

        // the rescue decisions of the first rows of this CTA's range outlive the layout scratch
        for (int t = lane; t < 8 * RESC_ROWS; t += 32) {
            const int rr = row0 + t / 8;
            resc_tab[t] = (rr < a.rows && (t & 7) < a.G) ? resc_j[rr * 8 + (t & 7)] : -1;
        }
        if (tl2 && lane == 0) tl2[5] = (unsigned long long)clock64() - clk0;
        load_window();
        first_window = false;       // from the first copy on, the stage memory belongs to the tiles
        int u = u0;
        int nb = batch_size(u);
        if (tl2 && lane == 0) tl2[6] = (unsigned long long)clock64() - clk0;
        int c_row, c_ent, c_nrows, c_page;
        fetch(u, nb, c_row, c_ent, c_nrows, c_page);
        if (tl2 && lane == 0) tl2[7] = (unsigned long long)clock64() - clk0 + (c_ent & 0);
        while (u < u1 && ok) {
            // the next batch is fetched once the first tiles of this batch are on their way, so that its loads
            // are in flight while the rest of this batch is issued
            const int un = u + nb;
            int nbn = 0, n_row = -1, n_ent = 0, n_nrows = 0, n_page = 0;
            const int k_prefetch = min(nb, NSTAGE) - 1;
            for (int k = 0; k < nb && ok; ++k) {
                const int r = __shfl_sync(0xffffffffu, c_row, k);
                const int ent = __shfl_sync(0xffffffffu, c_ent, k);
                const int nrows_raw = __shfl_sync(0xffffffffu, c_nrows, k);
                const int page = __shfl_sync(0xffffffffu, c_page, k);
                const int nrows = nrows_raw & 0xffff;
                const bool holds_newest = (nrows_raw >> 16) != 0;
                const int j = ent & 0xffffff;
                const int hmask = (ent >> 24) & 0xff;
                int i, hk;
                a.div_hkv.divmod(r, i, hk);
                if (r != prev_row) {                               // a new (CTA, row) piece starts here
                    close_piece();
                    ++piece; prev_row = r; piece_f0 = fill;
                }
                for (int sub = 0; sub * TS < nrows && ok; ++sub) {
                    const int nvalid = min(TS, nrows - sub * TS);
                    const int stage = fill % NSTAGE;
                    const uint32_t round = fill / NSTAGE;
                    if (lane == 0) {
                        if (tl2 && fill == 0) tl2[1] = (unsigned long long)clock64() - clk0;
                        if (!mbar_wait(&empty[stage], (round & 1) ^ 1)) {
                            ok = false;
                        } else {
                            if (SHARED_STAGES) st_volatile(&s_fill_started, (int)fill + 1);
                            // bits 8..15: row of the tile whose token stays ungated, 0xff: none
                            const int urow = (holds_newest && (sub + 1) * TS >= nrows) ? nvalid - 1 : 0xff;
                            desc[stage] = make_int4(r, piece << 1, hmask | (urow << 8), nvalid);
                            unsigned char* st = smem + stage * L::STAGE_BYTES;
                            mbar_arrive_expect_tx(&full[stage], L::STAGE_BYTES);
                            // one copy per tile: 64 columns x TS tokens x HALVES half tiles, each half swizzled.  The
                            // outermost coordinate is the sequence (contiguous cache: token offset in the sequence) or
                            // the page (paged cache: token offset in the page)
                            const int y = a.block_table ? sub * TS : j * a.b + sub * TS;
                            const int w4 = a.block_table ? page : i;
                            tma_load_5d(st, &tmK, 0, y, 0, hk, w4, &full[stage]);
                            tma_load_5d(st + HALVES * L::TILE_BYTES, &tmV, 0, y, 0, hk, w4, &full[stage]);
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                    ++fill;
                }
                if (k == k_prefetch && un < u1) {
                    nbn = batch_size(un);
                    fetch(un, nbn, n_row, n_ent, n_nrows, n_page);
                }
            }
            u = un;
            nb = nbn; c_row = n_row; c_ent = n_ent; c_nrows = n_nrows; c_page = n_page;
        }
        close_piece();
        pdl_trigger();       // everything is issued: the merge kernel may start to set up
        // one end marker per group (no data): the next NGROUPS fills reach every group exactly once
        for (int k = 0; k < NGROUPS && ok; ++k) {
            const int stage = fill % NSTAGE;
            if (lane == 0) {
                if (!mbar_wait(&empty[stage], ((fill / NSTAGE) & 1) ^ 1)) {
                    ok = false;
                } else {
                    if (SHARED_STAGES) st_volatile(&s_fill_started, (int)fill + 1);
                    desc[stage] = make_int4(0, (int)UF_END, 0, 0);
                    mbar_arrive(&full[stage]);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            ++fill;
        }
        if (!ok) {
            // give up: report, then let copies already issued land before the CTA's shared memory is released
            if (lane == 0) {
                if (a.status) atomicOr(a.status, ETA_DEV_TIMEOUT);
                const uint32_t first_fill = fill > NSTAGE ? fill - NSTAGE : 0;
                for (uint32_t f = first_fill; f < fill; ++f) mbar_wait(&full[f % NSTAGE], (f / NSTAGE) & 1);
            }
        }
        return;
    }

    // ---------------------------------------------------------------- consumers
    const int group = warp / WARPS_PER_GROUP, wq = warp % WARPS_PER_GROUP;
    float* sm_m = reinterpret_cast<float*>(smem + L::ML_OFF) + group * 2 * WARPS_PER_GROUP * 8;
    float* sm_l = sm_m + WARPS_PER_GROUP * 8;
    float* sm_o = reinterpret_cast<float*>(smem + L::MO_OFF) + group * WARPS_PER_GROUP * a.G * D;
    const int gtid = tid - group * 32 * WARPS_PER_GROUP;    // thread index inside the group
    const int g = lane >> 2, t = lane & 3;
    const int rb = wq * WT;                            // first token row of this warp inside a tile
    const int r0 = rho(2 * t), r1 = rho(2 * t + 1);    // token rows (within an 8-group) of MMA columns 2t, 2t+1
    const int vchunk = ((g & 1) << 2) | (g >> 1);      // 16-byte chunk of a V half-row this lane reads
    const float LOG2E = 1.4426950408889634f;
    const bool head = g < a.G;

    // byte offsets inside a half tile of the 16-byte pieces this lane reads (fixed for the whole kernel)
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

    uint32_t qa[HALVES][2][4];
    float o[HALVES][4][4];
    float m_run = -INFINITY, l_run = 0.f, te = 0.f;
    int row = -1, piece = -1, q_row = -1;
    uint32_t flush_phase = 0;
    bool ok = true;

    // query fragments and threshold of a row: head g's slice in the permuted head_dim order of the MMA
    auto load_q = [&](int r) {
        int i, hk;
        a.div_hkv.divmod(r, i, hk);
        const __nv_bfloat16* qp = a.q + ((int64_t)i * a.Hq + hk * a.G + (head ? g : 0)) * D;
#pragma unroll
        for (int hf = 0; hf < HALVES; ++hf)
#pragma unroll
            for (int m = 0; m < 2; ++m) {
                uint4 v = make_uint4(0, 0, 0, 0);
                if (head) v = __ldg(reinterpret_cast<const uint4*>(qp + 64 * hf + 32 * m + 8 * t));
                qa[hf][m][0] = v.x; qa[hf][m][1] = v.y; qa[hf][m][2] = v.z; qa[hf][m][3] = v.w;
            }
        te = head ? __ldg(a.tau_eff + (int64_t)i * a.Hq + hk * a.G + g) : 0.f;
        q_row = r;
    };
    load_q(row0);       // the row of the CTA's first unit: fetched while the producer sets up

    for (uint32_t fill = group;; fill += NGROUPS) {
        const int stage = fill % NSTAGE;
        if (SHARED_STAGES) {
            bool started = false;
            for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
                if ((uint32_t)ld_volatile(&s_fill_started) > fill) { started = true; break; }
                __nanosleep(40);
            }
            if (!started) { ok = false; break; }
        }
        if (!mbar_wait(&full[stage], (fill / NSTAGE) & 1)) { ok = false; break; }
        const int4 ds = desc[stage];
        const bool end = (ds.y & (int)UF_END) != 0;
        const int new_piece = ds.y >> 1;
        if (end) pdl_trigger();
        if (tl && warp == 0 && lane == 0) {
            if (fill == 0) tl[3] = globaltimer_ns();
            if (end) tl[4] = globaltimer_ns();
        }

        // the next piece's query is requested before the finished piece is flushed: the flush does not read the
        // query registers, and its barriers and stores hide the load's latency
        if (!end && new_piece != piece && ds.x != q_row) load_q(ds.x);
        if ((end || new_piece != piece) && piece >= 0) {
            // ---- this group's part of a piece is complete: combine its four warps and store (m, l, O) per head
            float lsum = l_run + __shfl_xor_sync(0xffffffffu, l_run, 1);
            lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
            if (t == 0) { sm_m[wq * 8 + g] = m_run; sm_l[wq * 8 + g] = lsum; }
#pragma unroll
            for (int hf = 0; hf < HALVES; ++hf)
#pragma unroll
                for (int mt = 0; mt < 4; ++mt) {
                    const int dcol = 64 * hf + 8 * vchunk + 2 * mt;
                    if (2 * t < a.G)
                        *reinterpret_cast<float2*>(sm_o + ((wq * a.G + 2 * t) * D + dcol)) = make_float2(o[hf][mt][0], o[hf][mt][2]);
                    if (2 * t + 1 < a.G)
                        *reinterpret_cast<float2*>(sm_o + ((wq * a.G + 2 * t + 1) * D + dcol)) = make_float2(o[hf][mt][1], o[hf][mt][3]);
                }
#ifdef ETA_TEST_SKIP_FLUSH_ARRIVE
            // test build only: one warp of the first CTA never arrives, so that the group's bounded wait runs out and
            // the give-up path (status flag, orderly exit of the whole CTA) executes
            if (!(blockIdx.x == 0 && group == 0 && wq == 1))
#endif
            mbar_arrive(&flushbar[group]);
            if (!mbar_wait(&flushbar[group], flush_phase)) { ok = false; break; }
            flush_phase ^= 1;
            const int64_t slot = ((int64_t)blockIdx.x + row) * NGROUPS + group;
            for (int idx = gtid; idx < a.G * D; idx += 32 * WARPS_PER_GROUP) {
                const int hh = idx / D, dd = idx % D;
                float M = -INFINITY;
#pragma unroll
                for (int w = 0; w < WARPS_PER_GROUP; ++w) M = fmaxf(M, sm_m[w * 8 + hh]);
                float acc = 0.f, lacc = 0.f;
                if (M != -INFINITY) {
#pragma unroll
                    for (int w = 0; w < WARPS_PER_GROUP; ++w) {
                        const float sc = exp2f((sm_m[w * 8 + hh] - M) * LOG2E);
                        acc = fmaf(sm_o[(w * a.G + hh) * D + dd], sc, acc);
                        lacc = fmaf(sm_l[w * 8 + hh], sc, lacc);
                    }
                }
                a.part_o[(slot * a.G + hh) * D + dd] = acc;
                if (dd == 0) a.part_ml[slot * a.G + hh] = make_float2(M, lacc);
            }
            mbar_arrive(&flushbar[group]);
            if (!mbar_wait(&flushbar[group], flush_phase)) { ok = false; break; }
            flush_phase ^= 1;
        }
        if (end) {
            if (tl && warp == 0 && lane == 0) tl[5] = globaltimer_ns();
            break;
        }

        const int hmask = ds.z & 0xff, urow = (ds.z >> 8) & 0xff, nvalid = ds.w;
        const uint32_t kbase = smem_u32(smem + stage * L::STAGE_BYTES);
        const uint32_t vbase = kbase + HALVES * L::TILE_BYTES;

        if (new_piece != piece) {
            piece = new_piece;
            row = ds.x;
            if (row != q_row) load_q(row);
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
        // V pieces are requested now so that their latency hides behind the softmax arithmetic
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
                    gated = S * rcp_approx(1.f + exp2f(-x * LOG2E));      // S * sigmoid(x); exp2(+inf) -> rcp -> 0
                }
                if (trow == urow) gated = S;          // the query's own token (Eq. mult_attn, s = t)
                gated = (head_on && trow < nvalid) ? gated : -INFINITY;
                sg[nt][c] = gated;
                bmax = fmaxf(bmax, gated);
            }
        bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 1));
        bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 2));
        const float m_new = fmaxf(m_run, bmax);
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
        const float alpha = (m_run == m_new) ? 1.f : exp2f((m_run - m_use) * LOG2E);   // m_run = -inf gives 0
        float p[NT][2], psum = 0.f;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                p[nt][c] = exp2f((sg[nt][c] - m_use) * LOG2E);   // -inf gives 0
                psum += p[nt][c];
            }
        l_run = l_run * alpha + psum;
        m_run = m_new;

        // accumulators hold heads 2t, 2t+1 in their columns: fetch those heads' rescale factors
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

        // ---- P as the B operand: bf16 high part and bf16 residual
        uint32_t pb_hi[2] = {0u, 0u}, pb_lo[2] = {0u, 0u};
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const __nv_bfloat162 hi = __floats2bfloat162_rn(p[nt][0], p[nt][1]);
            const float2 hf2 = __bfloat1622float2(hi);
            const __nv_bfloat162 lo = __floats2bfloat162_rn(p[nt][0] - hf2.x, p[nt][1] - hf2.y);
            pb_hi[nt] = *reinterpret_cast<const uint32_t*>(&hi);
            pb_lo[nt] = *reinterpret_cast<const uint32_t*>(&lo);
        }

        // ---- O^T += V^T P : head_dim on M, tokens on K, heads on N
        if (nvalid < TS) {
            // rows past the end of the sequence hold whatever the cache holds: keep them out of the product
#pragma unroll
            for (int hf = 0; hf < HALVES; ++hf)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int c = 0; c < 2; ++c)
                        if (rb + nt * 8 + (c ? r1 : r0) >= nvalid) v[hf][nt * 2 + c] = make_uint4(0, 0, 0, 0);
        }
        // every shared-memory read of this stage has been issued before this point; the arrive (release) orders
        // them before the producer's next copy into the stage
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[stage]);
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

    }
    if (!ok && lane == 0 && a.status) atomicOr(a.status, ETA_DEV_TIMEOUT);
}

// Associative merge of the pieces of one (sequence, query head): Algorithm 3, global reduction.
struct MergeArgs {
    const int2* row_span;
    const float2* part_ml;
    const float* part_o;
    float* out;
    int Hq, Hkv, G, nseg, rows, ngroups;
    unsigned long long* timeline;
};

constexpr int MERGE_WARPS = 8;

// One CTA per (row, query head, slice of head_dim); DS slices of DW = D / DS coordinates each, chosen by the host so
// that a small batch still fills the GPU (with one sequence and four KV heads there are only 16 (row, head) pairs,
// each with up to 3 x 148 partials to fold).  The candidate parts are the (streaming CTA, consumer group) pairs of
// the streaming CTAs that hold units of the row, which the streaming kernel lists per row; a part marked absent
// weighs nothing.  Warp w takes a contiguous share of the candidates, 32 a round: lane k reads the statistics of
// candidate k while O rows are already on their way (a row slice is DW / 4 lanes wide, so a warp instruction
// fetches 128 / DW candidates' slices, eight instructions in flight), the warp takes the largest m of its share,
// weighs and adds the rows; lanes that hold the same coordinates, then the eight warps, are combined in a fixed
// order:  o = sum_k O_k e^{m_k - m*} / sum_k l_k e^{m_k - m*},  m* = max_k m_k.
template <int D, int DS>
__global__ void __launch_bounds__(32 * MERGE_WARPS) merge_kernel(const MergeArgs a) {
    constexpr int DW = D / DS;             // coordinates of this CTA's slice
    constexpr int LPC = DW / 4;            // lanes per candidate row slice (a float4 each)
    constexpr int CPW = 32 / LPC;          // candidates per warp instruction
    static_assert(DW >= 4 && LPC <= 32 && LPC * CPW == 32, "slice must be 4 .. 128 coordinates");
    __shared__ float s_acc[MERGE_WARPS][DW];
    __shared__ float s_l[MERGE_WARPS];
    __shared__ float s_m[MERGE_WARPS];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int pair = blockIdx.x / DS, dpart = blockIdx.x % DS;
    const int r = pair / a.G, gq = pair % a.G;
    const int i = r / a.Hkv, hk = r % a.Hkv;
    unsigned long long* const tl = ETA_TL((a.timeline && blockIdx.x < TL_MERGE_N) ? a.timeline + (size_t)(TL_MERGE + blockIdx.x) * 8 : nullptr);
    if (tl && tid == 0) tl[0] = globaltimer_ns();
    pdl_trigger();
    pdl_wait();          // every partial of the streaming kernel is in memory from here on
    if (tl && tid == 0) tl[1] = globaltimer_ns();
    const int2 span = a.row_span[r];
    const int c_lo = span.x, n_cand = span.y * a.ngroups;
    if (tl && tid == 0) tl[2] = globaltimer_ns() + (n_cand & 0);
    auto slot_of = [&](int k) { return ((int64_t)(c_lo + k / a.ngroups) + r) * a.ngroups + k % a.ngroups; };
    const int sub = lane / LPC, dl = lane % LPC;        // candidate within a warp instruction, float4 within the slice
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    float m_w = -INFINITY, l_w = 0.f;        // this warp's running maximum and weighted l
    const int per = (n_cand + MERGE_WARPS - 1) / MERGE_WARPS;
    const int k_begin = warp * per, k_end = min(n_cand, k_begin + per);
    for (int k0 = k_begin; k0 < k_end; k0 += 32) {
        const int k = k0 + lane;
        const int nk = min(32, k_end - k0);
        float m_k = -INFINITY, l_k = 0.f;
        if (k < k_end) {
            const float2 ml = a.part_ml[slot_of(k) * a.G + gq];
            m_k = ml.x; l_k = ml.y;
        }
        // the first O rows of the round do not wait for the statistics
        float4 xv[8];
        auto load_rows = [&](int j0) {
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int j = j0 + u * CPW + sub;
                xv[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (j < nk)
                    xv[u] = __ldg(reinterpret_cast<const float4*>(a.part_o + (slot_of(k0 + j) * a.G + gq) * D + dpart * DW) + dl);
            }
        };
        load_rows(0);
        float m_round = m_k;
#pragma unroll
        for (int s = 16; s >= 1; s >>= 1) m_round = fmaxf(m_round, __shfl_xor_sync(0xffffffffu, m_round, s));
        const float m_new = fmaxf(m_w, m_round);
        if (m_new == -INFINITY) continue;        // nothing real in this round (warp-uniform)
        const float rescale = (m_w == -INFINITY) ? 0.f : __expf(m_w - m_new);
        const float w = (m_k == -INFINITY) ? 0.f : __expf(m_k - m_new);
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[v] *= rescale;
        float lw = l_k * w;
#pragma unroll
        for (int s = 16; s >= 1; s >>= 1) lw += __shfl_xor_sync(0xffffffffu, lw, s);
        l_w = l_w * rescale + lw;
        m_w = m_new;
        for (int j0 = 0; j0 < nk; j0 += 8 * CPW) {
            if (j0 > 0) load_rows(j0);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int j = j0 + u * CPW + sub;
                const float wk = __shfl_sync(0xffffffffu, w, min(j, 31));
                if (j < nk && wk != 0.f) {       // an absent part's row is stale memory: never touch it
                    acc[0] = fmaf(xv[u].x, wk, acc[0]); acc[1] = fmaf(xv[u].y, wk, acc[1]);
                    acc[2] = fmaf(xv[u].z, wk, acc[2]); acc[3] = fmaf(xv[u].w, wk, acc[3]);
                }
            }
        }
    }
    // lanes that hold the same coordinates of different candidates
#pragma unroll
    for (int o = LPC; o < 32; o <<= 1) {
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[v] += __shfl_xor_sync(0xffffffffu, acc[v], o);
    }
    if (tl && tid == 0) tl[3] = globaltimer_ns() + (__float_as_int(acc[0]) & 0);
    if (sub == 0) {
#pragma unroll
        for (int v = 0; v < 4; ++v) s_acc[warp][dl * 4 + v] = acc[v];
    }
    if (lane == 0) { s_l[warp] = l_w; s_m[warp] = m_w; }
    __syncthreads();
    if (tid < DW) {
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < MERGE_WARPS; ++w) M = fmaxf(M, s_m[w]);
        float o = 0.f, l = 0.f;
        if (M != -INFINITY) {
#pragma unroll
            for (int w = 0; w < MERGE_WARPS; ++w) {
                const float sc = (s_m[w] == -INFINITY) ? 0.f : __expf(s_m[w] - M);
                o = fmaf(s_acc[w][tid], sc, o);
                l = fmaf(s_l[w], sc, l);
            }
        }
        a.out[((int64_t)i * a.Hq + hk * a.G + gq) * D + dpart * DW + tid] = l > 0.f ? o / l : 0.f;
    }
    if (tl && tid == 0) tl[4] = globaltimer_ns();
}

// ------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr);
        if (e != cudaSuccess || qr != cudaDriverEntryPointSuccess || !p) {
            set_cuda_error(e != cudaSuccess ? e : cudaErrorUnknown, "cuTensorMapEncodeTiled lookup");
            return nullptr;
        }
        fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// K or V as a 5-D tensor (c within a 64-column half, t, half, hk, i) of bf16; a box is 64 columns x TS tokens x
// all halves: in shared memory, one 128-byte-swizzled [TS][64] tile per half, back to back.
// Tensor map of a K or V cache: 64 columns x tokens x column halves x KV heads x sequences, or, for a paged cache
// (n_pages > 0), ... x tokens of a page x ... x pages, with sb the stride between pages.
static int make_tmap(CUtensorMap* tm, const void* base, const eta_cache_desc* d, int64_t sb, int64_t sh, int64_t st,
                     int TS, int n_pages) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return ETA_ERR_CUDA;
    const cuuint32_t halves = (cuuint32_t)(d->head_dim / 64);
    cuuint64_t dims[5] = {64, (cuuint64_t)(n_pages > 0 ? d->block_size : d->t_cap), halves, (cuuint64_t)d->n_kv_heads,
                          (cuuint64_t)(n_pages > 0 ? n_pages : d->batch)};
    cuuint64_t strides[4] = {(cuuint64_t)st * 2, 128, (cuuint64_t)sh * 2, (cuuint64_t)sb * 2};
    cuuint32_t box[5] = {64, (cuuint32_t)TS, halves, 1, 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUresult rc = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (rc != CUDA_SUCCESS) {
        set_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
        return ETA_ERR_CUDA;
    }
    return ETA_OK;
}

template <int D, int TS, int NSTAGE, int NGROUPS>
static int launch_decode_t(const CUtensorMap& tmK, const CUtensorMap& tmV, const DecodeArgs& a, int n_ctas,
                           cudaStream_t s) {
    const size_t smem = DecodeSmem<D, TS, NSTAGE, NGROUPS>::bytes(a.G);
    return launch_pdl("decode launch", decode_kernel<D, TS, NSTAGE, NGROUPS>, dim3(n_ctas),
                      dim3(32 * (WARPS_PER_GROUP * NGROUPS + 1)), smem, s, tmK, tmV, a);
}

// eta_decode and eta_decode_paged: `pages` null selects the contiguous cache
static int decode_impl(const eta_cache_desc* desc, const eta_page_table* pages, const eta_params* params, const void* q,
                       const void* K, const void* V, const int32_t* seq_lens, const void* musig, const float* mnorm,
                       const float* tau, const float* head_const, float* out, uint8_t* sel_mask, int32_t* stats,
                       uint32_t* status_dev, void* workspace, size_t workspace_bytes, void* stream) {
    int rc = validate_desc(desc);
    if (rc != ETA_OK) return rc;
    if (pages && (rc = validate_pages(desc, pages)) != ETA_OK) return rc;
    if (!params || !q || !K || !V || !seq_lens || !out || !sel_mask) return ETA_ERR_INVALID_ARG;
    const bool dense = (params->flags & ETA_FLAG_DENSE) != 0;
    if (!dense && (!musig || !mnorm)) return ETA_ERR_INVALID_ARG;
    if ((tau != nullptr) == (head_const != nullptr)) return ETA_ERR_INVALID_ARG;
    if (params->rescue_window < 1 || params->lwb < 0) return ETA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(V) | reinterpret_cast<uintptr_t>(q) |
         reinterpret_cast<uintptr_t>(musig) | reinterpret_cast<uintptr_t>(out)) & 15)
        return ETA_ERR_UNSUPPORTED;
    const WsLayout L = ws_layout(desc);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < L.total)
        return ETA_ERR_WORKSPACE;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    const int D = desc->head_dim, b = desc->block_size;
    const int G = desc->n_q_heads / desc->n_kv_heads;
    const float scale = params->scale > 0.f ? params->scale : 1.0f / sqrtf((float)D);

    int dev = 0, n_sm = 0;
    cudaError_t ce = cudaGetDevice(&dev);
    if (ce == cudaSuccess) ce = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (ce != cudaSuccess) { set_cuda_error(ce, "device query"); return ETA_ERR_CUDA; }
    const int TS = b < 64 ? b : 64;
    int n_ctas = n_sm;                  // one persistent CTA per SM; the shared-memory ring fills the SM
    if (n_ctas > MAX_CTAS) n_ctas = MAX_CTAS;

    ScreenArgs sa;
    sa.q = static_cast<const __nv_bfloat16*>(q);
    sa.musig = static_cast<const __half*>(musig);
    sa.mnorm = mnorm;
    sa.seq_lens = seq_lens;
    sa.tau = tau;
    sa.head_const = head_const;
    sa.z = params->z; sa.a = params->a; sa.scale = scale;
    sa.lwb = params->lwb; sa.rescue_window = params->rescue_window; sa.flags = params->flags;
    sa.Hq = desc->n_q_heads; sa.Hkv = desc->n_kv_heads; sa.b = b; sa.t_cap = desc->t_cap; sa.nb_cap = desc->nb_cap;
    sa.nseg = L.nseg; sa.rows = L.rows;
    sa.b_shift = (b == 32) ? 5 : (b == 64 ? 6 : 7);
    sa.div_nseg = FastDiv(L.nseg); sa.div_hkv = FastDiv(desc->n_kv_heads);
    sa.seg_count = reinterpret_cast<int32_t*>(ws + L.seg_count);
    sa.seg_list = reinterpret_cast<int32_t*>(ws + L.seg_list);
    sa.seg_resc = reinterpret_cast<RescueRec*>(ws + L.seg_resc);
    sa.tau_eff = reinterpret_cast<float*>(ws + L.tau_eff);
    sa.sel_mask = sel_mask;
    sa.timeline = debug_timeline();
    sa.status = status_dev;
    profile_mark(2, s);
    rc = launch_screen(sa, L.rows, D, G, 2 * n_sm, s);
    profile_mark(3, s);
    if (rc != ETA_OK) return rc;

    CUtensorMap tmK, tmV;
    const int n_pages = pages ? pages->n_pages : 0;
    rc = make_tmap(&tmK, K, desc, desc->k_stride_b, desc->k_stride_h, desc->k_stride_t, TS, n_pages);
    if (rc != ETA_OK) return rc;
    rc = make_tmap(&tmV, V, desc, desc->v_stride_b, desc->v_stride_h, desc->v_stride_t, TS, n_pages);
    if (rc != ETA_OK) return rc;

    DecodeArgs da;
    da.q = sa.q; da.seq_lens = seq_lens; da.tau_eff = sa.tau_eff; da.seg_list = sa.seg_list;
    da.seg_count = sa.seg_count; da.seg_resc = sa.seg_resc; da.sel_mask = sel_mask; da.stats = stats;
    da.row_span = reinterpret_cast<int2*>(ws + L.row_span);
    da.part_ml = reinterpret_cast<float2*>(ws + L.part_ml);
    da.part_o = reinterpret_cast<float*>(ws + L.part_o);
    da.status = status_dev;
    da.beta = params->beta; da.scale = scale;
    da.Hq = desc->n_q_heads; da.Hkv = desc->n_kv_heads; da.G = G; da.b = b; da.t_cap = desc->t_cap;
    da.nseg = L.nseg; da.entries = L.entries; da.rows = L.rows; da.nb_cap = desc->nb_cap;
    da.rescue_window = params->rescue_window;
    da.ungate_last = (!dense && (params->flags & ETA_FLAG_UNGATE_LAST)) ? 1 : 0;
    da.block_table = pages ? pages->block_table : nullptr;
    da.table_stride = pages ? pages->table_stride : 0;
    da.div_nseg = FastDiv(L.nseg); da.div_epr = FastDiv(L.nseg + 2); da.div_hkv = FastDiv(desc->n_kv_heads);
    da.div_g = FastDiv(G);
    da.timeline = debug_timeline();
    if (D == 128 && TS == 64) {
        rc = (G == 8) ? launch_decode_t<128, 64, 5, DECODE_GROUPS>(tmK, tmV, da, n_ctas, s)
                      : launch_decode_t<128, 64, 6, DECODE_GROUPS>(tmK, tmV, da, n_ctas, s);
    } else if (D == 128 && TS == 32) {
        rc = launch_decode_t<128, 32, 8, DECODE_GROUPS>(tmK, tmV, da, n_ctas, s);
    } else if (D == 64 && TS == 64) {
        rc = launch_decode_t<64, 64, 8, DECODE_GROUPS>(tmK, tmV, da, n_ctas, s);
    } else {
        rc = launch_decode_t<64, 32, 8, DECODE_GROUPS>(tmK, tmV, da, n_ctas, s);
    }
    if (rc != ETA_OK) return rc;
    profile_mark(4, s);

    MergeArgs ma;
    ma.row_span = da.row_span; ma.part_ml = da.part_ml; ma.part_o = da.part_o; ma.out = out;
    ma.Hq = desc->n_q_heads; ma.Hkv = desc->n_kv_heads; ma.G = G; ma.nseg = L.nseg; ma.rows = L.rows; ma.ngroups = DECODE_GROUPS; ma.timeline = debug_timeline();
    // slices of head_dim per (row, head): enough CTAs to fill the GPU when the batch is small
    const int pairs = L.rows * G;
    const int DS = (pairs * 4 <= n_sm) ? 8 : (pairs * 2 <= n_sm ? 4 : (pairs <= n_sm / 2 ? 2 : 1));
    const dim3 mgrid((unsigned)(pairs * DS)), mblock(32 * MERGE_WARPS);
#define ETA_MERGE(DD, SS) launch_pdl("merge launch", merge_kernel<DD, SS>, mgrid, mblock, 0, s, ma)
    if (D == 128) rc = DS == 8 ? ETA_MERGE(128, 8) : (DS == 4 ? ETA_MERGE(128, 4) : (DS == 2 ? ETA_MERGE(128, 2) : ETA_MERGE(128, 1)));
    else rc = DS == 8 ? ETA_MERGE(64, 8) : (DS == 4 ? ETA_MERGE(64, 4) : (DS == 2 ? ETA_MERGE(64, 2) : ETA_MERGE(64, 1)));
#undef ETA_MERGE
    profile_mark(5, s);
    return rc;
}

}  // namespace eta

extern "C" {

int eta_decode_kernel_count(void) { return 3; }

int eta_decode(const eta_cache_desc* desc, const eta_params* params, const void* q, const void* K, const void* V,
               const int32_t* seq_lens, const void* musig, const float* mnorm, const float* tau,
               const float* head_const, float* out, uint8_t* sel_mask, int32_t* stats, uint32_t* status_dev,
               void* workspace, size_t workspace_bytes, void* stream) {
    return eta::decode_impl(desc, nullptr, params, q, K, V, seq_lens, musig, mnorm, tau, head_const, out, sel_mask, stats,
                            status_dev, workspace, workspace_bytes, stream);
}

int eta_decode_paged(const eta_cache_desc* desc, const eta_page_table* pages, const eta_params* params, const void* q,
                     const void* K_pool, const void* V_pool, const int32_t* seq_lens, const void* musig,
                     const float* mnorm, const float* tau, const float* head_const, float* out, uint8_t* sel_mask,
                     int32_t* stats, uint32_t* status_dev, void* workspace, size_t workspace_bytes, void* stream) {
    if (!pages) return ETA_ERR_INVALID_ARG;
    return eta::decode_impl(desc, pages, params, q, K_pool, V_pool, seq_lens, musig, mnorm, tau, head_const, out, sel_mask,
                            stats, status_dev, workspace, workspace_bytes, stream);
}

}  // extern "C"

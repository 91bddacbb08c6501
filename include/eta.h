/*
 * eta.h - C ABI of the B200 (sm_100a) block-sparse decode attention of
 * Elastic Threshold Attention (ETA).
 *
 * The library covers the inference path of the paper: the dual
 * probabilistic-geometric block index (Section 3), the linear threshold
 * predictor (Eq. tau_pred), O(1)-per-block screening with Score_dual
 * (Eq. dual_bound_eq), and SiLU-gated attention over the surviving blocks with
 * top-1 rescue and tail handling (Algorithm 3), plus the frozen per-head
 * constant-threshold mode (Section 4.5, "Distilling static thresholds").
 *
 * Conventions that hold for every call unless stated otherwise:
 *   - Descriptors (eta_cache_desc, eta_params) are HOST structs read during the
 *     call.  Every other pointer is a DEVICE pointer owned by the caller.
 *   - The library allocates no device memory, never synchronises and never
 *     copies to the host.  All work is enqueued on `stream` (a cudaStream_t
 *     passed as void*; NULL is the default stream).
 *   - Return value: ETA_OK (0) or a negative eta_status.  No exception crosses
 *     the boundary.  Problems only the device can see (a sequence longer than
 *     the cache, a bounded wait that gave up) are OR-ed into *status_dev.
 *   - Layouts (d = head_dim, b = block_size, G = n_q_heads / n_kv_heads;
 *     query head h belongs to KV head h / G):
 *       K, V     bf16, element (i, hk, t, c) at i*stride_b + hk*stride_h + t*stride_t + c
 *                (strides in elements, stride_t a multiple of 8, base 16-byte aligned)
 *       q        bf16 [batch, n_q_heads, d], contiguous
 *       seq_lens int32 [batch]: tokens valid in the cache of each sequence
 *       musig    fp16 [batch, n_kv_heads, nb_cap, 2, d]: centroid, then coordinate-wise
 *                standard deviation (sigma, not the variance) of every full block
 *       mnorm    fp32 [batch, n_kv_heads, nb_cap]: largest key norm of every full block
 *       tau      fp32 [batch, n_q_heads];  head_const fp32 [n_q_heads]
 *       out      fp32 [batch, n_q_heads, d]
 *       sel_mask uint8 [batch, n_kv_heads, nb_cap]: bit g set iff query head hk*G+g attends
 *                full block j.  Tokens past the last full block are always attended.
 *   - Packed summaries (the paper's outlook names "FP8 metadata"; the format is this library's): with
 *     ETA_BUILD_PACKED_SIGMA / ETA_FLAG_PACKED_SIGMA musig is bytes [batch, n_kv_heads, nb_cap, 3 d]: the centroid
 *     as fp16[d], then sigma as e4m3[d] (8-bit float, 4 exponent and 3 fraction bits) rounded UP to the next e4m3
 *     value; mnorm is unchanged.  Score_dual is non-decreasing in sigma, so the packed bound is never below the
 *     bound of the 4 d-byte record: packing adds no false negative, it admits a few more blocks (the variance
 *     term grows by at most one part in eight) and cuts the screening traffic by a quarter.  sigma below 2^-9 is
 *     stored as 2^-9, sigma above 448 as the NaN code (the block is then always admitted).
 *   - Supported shapes: head_dim in {64, 128}; block_size in {32, 64, 128};
 *     G in {1, 2, 4, 8}.  Anything else returns ETA_ERR_UNSUPPORTED.
 */
#ifndef ETA_H_
#define ETA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum eta_status {
    ETA_OK = 0,
    ETA_ERR_INVALID_ARG = -1,   /* NULL pointer, inconsistent sizes, both or neither of tau / head_const */
    ETA_ERR_UNSUPPORTED = -2,   /* shape or alignment outside the supported set */
    ETA_ERR_WORKSPACE = -3,     /* workspace missing, misaligned (256 B) or too small */
    ETA_ERR_CUDA = -4           /* a CUDA call failed; see eta_last_cuda_error() */
} eta_status;

/* bits written to *status_dev by the kernels */
#define ETA_DEV_TIMEOUT      1u  /* a bounded wait inside a kernel ran out; outputs are not valid */
#define ETA_DEV_LEN_CLAMPED  2u  /* some seq_lens[i] exceeded t_cap and was clamped */
#define ETA_DEV_EMPTY_ROW    4u  /* some seq_lens[i] <= 0: that sequence's output is zero */

/* flags of eta_params.flags */
#define ETA_FLAG_DENSE           1u  /* baseline: admit every block and switch the gate off (softmax attention) */
#define ETA_FLAG_PACKED_SIGMA     4u  /* musig holds packed records (see "Packed summaries" below) */
#define ETA_FLAG_UNGATE_LAST     2u  /* Eq. mult_attn leaves the diagonal s = t ungated; at decode time the query's own
                                        token is the newest one: it keeps its raw logit (S~ = S), and when it closes a
                                        full block that block is admitted for every head.  Off: Algorithm 3 as
                                        printed, every token gated */
/* flags of the summary builders */
#define ETA_BUILD_SIGMA_ENVELOPE 1u  /* store the sub-block envelope (Eq. subblock_envelope_appx) instead of sigma */
#define ETA_BUILD_PACKED_SIGMA   2u  /* write packed records (see "Packed summaries" below) */

typedef struct eta_cache_desc {
    int32_t batch, n_q_heads, n_kv_heads, head_dim, block_size;
    int32_t t_cap;                              /* token capacity of the cache along t */
    int32_t nb_cap;                             /* block capacity of musig / mnorm / sel_mask (>= t_cap / block_size) */
    int64_t k_stride_b, k_stride_h, k_stride_t; /* elements */
    int64_t v_stride_b, v_stride_h, v_stride_t; /* elements */
} eta_cache_desc;

typedef struct eta_params {
    float z;                /* z-score of the moment term of Score_dual */
    float a;                /* operating offset: tau_eff = tau - a (Algorithm 3) */
    float beta;             /* gate temperature of Eq. soft_mask at inference */
    float scale;            /* softmax scale s; <= 0 selects 1/sqrt(head_dim) */
    int32_t lwb;            /* the last `lwb` full blocks are always attended */
    int32_t rescue_window;  /* top-1 rescue looks at the first min(rescue_window, NB) blocks; >= 1 */
    uint32_t flags;         /* ETA_FLAG_* */
} eta_params;

/*
 * Bytes of scratch eta_decode needs for this cache shape (independent of the
 * sequence lengths).  The caller allocates it once, 256-byte aligned, and may
 * reuse it across calls on the same stream; it carries no state between calls
 * (every word is written before it is read) and needs no initialisation.
 * No device is touched by this function.
 */
int eta_workspace_bytes(const eta_cache_desc* desc, size_t* out_bytes);

/*
 * Section 3 (dual block index); appendix "End-to-end systems accounting"
 * (prefill indexing: one pass over K).  For every sequence i, KV head hk and
 * full block j < floor(seq_lens[i] / b) writes
 *   mu = mean of the b keys, sigma_c = sqrt(mean_k (k_c - mu_c)^2) (population),
 *   M = max_k ||k||_2
 * as fp16 / fp16 / fp32.  Records of blocks that are not full are left untouched.
 * Arithmetic is fp32 on the bf16 keys, in one pass over the block: mu from the plain
 * coordinate sums, sigma from squared deviations about the block's first key k0,
 *   sigma_c^2 = (1/b) sum_k (k_c - k0_c)^2 - (mu_c - k0_c)^2   (clamped at 0),
 * which is exact for identical keys and otherwise loses a factor
 * 1 + (mu_c - k0_c)^2 / sigma_c^2 of fp32's precision, far inside the fp16 the
 * result is stored in (results are within 1 fp16 ulp of the two-pass definition
 * evaluated in double).
 * flags: ETA_BUILD_SIGMA_ENVELOPE stores max over 4-token sub-blocks of the
 * sub-block RMS deviation from mu instead of sigma (Eq. subblock_envelope_appx;
 * this variant takes a second pass over the block for the deviations about mu).
 */
int eta_build_block_summaries(const eta_cache_desc* desc, const void* K, const int32_t* seq_lens,
                              void* musig, float* mnorm, uint32_t flags, void* stream);

/*
 * Appendix "End-to-end systems accounting" (tail-block metadata update at every
 * decode step).  Call after a token has been appended and seq_lens[i] bumped:
 * for every sequence whose new length is a positive multiple of b, the block
 * that just became full (index seq_lens[i]/b - 1) is summarised exactly as
 * eta_build_block_summaries would; other sequences are untouched.  Stateless and
 * idempotent.
 */
int eta_append_summary(const eta_cache_desc* desc, const void* K, const int32_t* seq_lens_after,
                       void* musig, float* mnorm, uint32_t flags, void* stream);

/*
 * Brings one step's queries (Algorithm 3, "Require: query q_t") from the host to the device with a kernel
 * instead of a copy engine (deployment plumbing; the paper has no counterpart).  q_host: bf16
 * [batch, n_q_heads, head_dim] in page-locked host memory that the device can address (cudaHostAlloc /
 * cudaHostRegister; with unified addressing the host pointer itself); q_dev: the same shape in device memory.
 * Both 16-byte aligned, the size a multiple of 16 bytes (else ETA_ERR_UNSUPPORTED).  Ordered like any kernel on
 * `stream`; the calls that follow on the stream see the complete copy.  The host buffer must stay unchanged until
 * the kernel has run.  In the same way `out` of eta_decode may be page-locked host memory: the merge kernel's
 * stores then go straight to the host and are visible once the stream has been synchronised.
 */
int eta_stage_query(int32_t batch, int32_t n_q_heads, int32_t head_dim, const void* q_host, void* q_dev,
                    void* stream);

/*
 * Eq. tau_pred: tau[i, h] = sum_r qbar[i, r] * W[r, h] + bias[h], with qbar the
 * head-major concatenation of the n_q_heads post-RoPE query vectors of sequence
 * i (length n_q_heads * head_dim).  q bf16 [batch, n_q_heads, head_dim];
 * W fp32 [n_q_heads * head_dim, n_q_heads] row-major; bias fp32 [n_q_heads];
 * tau fp32 [batch, n_q_heads].  fp32 accumulation in a fixed order.
 * Launch order: the kernel is launched with programmatic dependent launch and reads
 * q, W and bias without waiting for the preceding kernel of the stream (it waits for
 * it only before it exits, so that its completion implies its predecessor's).  The
 * producer of q must therefore be complete when that preceding kernel starts: true
 * for copies, for kernels launched without early dependent release (eta_stage_query
 * and eta_append_summary's inputs among them) and for anything ordered by an event
 * or a synchronisation; a kernel that releases its dependents early and then writes
 * q would hand this call a stale query.
 */
int eta_predict_threshold(int32_t batch, int32_t n_q_heads, int32_t head_dim, const void* q,
                          const float* W, const float* bias, float* tau, void* stream);

/*
 * Eq. dual_bound_eq, evaluated for every (sequence, query head, full block):
 *   bound = s * min( <q, mu> + z * sqrt(sum_c q_c^2 sigma_c^2), ||q|| * M ).
 * bound fp32 [batch, n_q_heads, nb_cap]; entries of blocks that are not full are
 * left untouched.  Same arithmetic as the screening stage of eta_decode (packed
 * records with ETA_FLAG_PACKED_SIGMA in params->flags); meant for diagnostics
 * and for calibrating frozen constants, not for the hot loop.
 */
int eta_score_dual(const eta_cache_desc* desc, const eta_params* params, const void* q,
                   const int32_t* seq_lens, const void* musig, const float* mnorm,
                   float* bound, void* stream);

/*
 * Appendix "Offline Threshold Calibration via 1/t-Weighted Histograms", Algorithm
 * "Density-Matched Offline Threshold Calibration": replaces the dynamic predictor
 * by one constant per query head with the same density on a calibration split.
 * For every head h (KV head h / G), over n_seq sequences of seq_len tokens, with
 * raw causal scores S_ts = s <q_t, k_s>, s <= t (t counted from 1):
 *   dbar_h = 1/(n_seq seq_len) sum_x sum_t (1/t) sum_{s<=t} sigmoid(beta (S_ts - tau[x,h,t]))
 *   H_h[bin(S_ts)] += 1/t, then H_h normalised to sum 1
 *   head_const[h] = root of  sum_b H_h[b] sigmoid(beta (s_b - c)) = dbar_h  (bisection, double precision).
 * Bins: n_bins (<= 4096) equal bins on [s_min, s_max], s_b the bin centre; scores
 * outside the range go to the first / last bin (the paper fixes neither).
 * Q bf16 [n_seq, n_q_heads, seq_len, head_dim], K bf16 [n_seq, n_kv_heads, seq_len,
 * head_dim], tau fp32 [n_seq, n_q_heads, seq_len] (the predictor's thresholds),
 * head_const fp32 [n_q_heads] (out), dbar fp32 [n_q_heads] (out, nullable); all
 * device pointers.  Scores are computed in fp32 from the bf16 operands; the row
 * weights are accumulated as integers, so the result does not depend on the
 * order of the atomic updates.  head_dim 64 or 128; n_seq * seq_len <= 2^22.
 * workspace: eta_calibration_workspace_bytes() bytes, 256-byte aligned, no
 * initialisation needed.  Prefill-side tool: not part of a decode step.
 */
int eta_calibration_workspace_bytes(int32_t n_seq, int32_t seq_len, int32_t n_q_heads, int32_t n_bins,
                                    size_t* out_bytes);
int eta_calibrate_head_const(int32_t n_seq, int32_t seq_len, int32_t n_q_heads, int32_t n_kv_heads,
                             int32_t head_dim, const void* Q, const void* K, const float* tau,
                             float beta, float scale, int32_t n_bins, float s_min, float s_max,
                             float* head_const, float* dbar, void* workspace, size_t workspace_bytes,
                             void* stream);

/*
 * Algorithm 3 (screen, top-1 rescue, tail phase, chunk merge) with the
 * GQA-grouped execution of the fused-kernel appendix, for one decode query per
 * sequence.  Per query head h, with tau_eff = (tau[i,h] or head_const[h]) - a:
 *   1. every full block j is admitted unless Score_dual(q_h, j) < tau_eff; the last
 *      `lwb` full blocks are always admitted; if none of the first
 *      min(rescue_window, NB) blocks is admitted the first one with the largest
 *      bound among them is;
 *   2. a block is read from HBM once per KV head if any head of the group admits it;
 *   3. the head attends the tokens of its own admitted blocks and all tokens past
 *      the last full block, with weights exp(S~), S~ = S * sigmoid(beta * (S - tau_eff)),
 *      S = s <q_h, k>; out = sum w v / sum w.
 * Exactly one of tau / head_const must be non-NULL (frozen mode = head_const).
 * sel_mask (required) receives the per-head admission bits; stats (nullable,
 * int32 [batch, n_kv_heads]) the number of blocks fetched per KV head;
 * status_dev (nullable, uint32, caller-zeroed) device-side problems.
 * bf16 operands, fp32 scores / softmax statistics / accumulators; deterministic
 * for a given device (the split of the work depends on its SM count only).
 * workspace: eta_workspace_bytes() bytes.
 * Launch order: the kernels are launched with programmatic dependent launch and read q, seq_lens and every
 * summary except the newest block's before they wait for the preceding kernel of the stream.  Producers of those
 * inputs must therefore be complete when that preceding kernel starts: true for copies, for kernels launched
 * without early dependent release (eta_stage_query among them) and for anything ordered by an event or a
 * synchronisation; only a kernel that releases its dependents early and then writes q would break it.
 */
int eta_decode(const eta_cache_desc* desc, const eta_params* params, const void* q,
               const void* K, const void* V, const int32_t* seq_lens,
               const void* musig, const float* mnorm,
               const float* tau, const float* head_const,
               float* out, uint8_t* sel_mask, int32_t* stats, uint32_t* status_dev,
               void* workspace, size_t workspace_bytes, void* stream);

/*
 * eta_decode for callers that cannot provide scratch memory (the paper has no counterpart: this is a
 * deployment convenience, not part of the method).  Who needs it: a serving process that handed all of its HBM to
 * a KV-cache pool at start-up and has nothing left to carve a workspace from; a plug-in that receives tensors
 * but no allocator; a decode loop that must stay out of the CUDA allocator because cudaMalloc synchronises the
 * device and may fail once memory is fragmented.
 *
 * Same arguments, results and status codes as eta_decode, minus workspace / workspace_bytes.  The scratch is a
 * fixed array of ETA_STATIC_SCRATCH_BYTES (8 MiB) inside the library's CUDA module: every GPU on which the
 * module gets loaded holds it from then until the process exits.  The call allocates and frees nothing.
 *   - Limit: shapes for which eta_workspace_bytes() exceeds ETA_STATIC_SCRATCH_BYTES are refused with
 *     ETA_ERR_WORKSPACE before anything is launched (the five benchmark configurations need 0.8 - 3 MiB).
 *   - Set-up: the first call on each device looks up the array's device address (with that device current).
 *     Make that first call ahead of any stream capture, and ahead of handing the rest of the device's memory
 *     to anybody else: CUDA loads a module lazily by default, so the array is reserved when the library's first
 *     kernel is launched or its first symbol looked up on that device, not when the library is loaded.  A first
 *     call that finds no memory left returns ETA_ERR_CUDA (eta_last_cuda_error names cudaGetSymbolAddress).
 *     The address is looked up once per device and kept; it does not survive a cudaDeviceReset.
 *   - Sharing: all calls on a device use the same array, and it keeps the previous call's contents.  Nothing in
 *     it has to be cleared by the caller: each call writes every word before reading it.  For the same reason
 *     two calls whose kernels can overlap on the GPU (different streams, no dependency between them) race on
 *     the array and corrupt each other; calls on one stream, or otherwise ordered, are fine.
 */
#define ETA_STATIC_SCRATCH_BYTES (8u << 20)
int eta_decode_static(const eta_cache_desc* desc, const eta_params* params, const void* q,
                      const void* K, const void* V, const int32_t* seq_lens,
                      const void* musig, const float* mnorm,
                      const float* tau, const float* head_const,
                      float* out, uint8_t* sel_mask, int32_t* stats, uint32_t* status_dev, void* stream);

/*
 * Paged KV cache (Section 3: the block summaries live "in a held-out table compatible with paged caching").
 * K and V are pools of pages of block_size tokens; page p of KV head hk, token t of the page, is at
 * K + p * k_stride_b + hk * k_stride_h + t * k_stride_t (the descriptor's sequence stride becomes the page
 * stride; same for V).  block_table (device, int32 [batch, table_stride], table_stride >= ceil(t_cap /
 * block_size)) gives, for sequence i and j >= 0, the page that holds tokens [j * block_size, (j + 1) * block_size)
 * of the sequence; entries for j up to floor((T_i - 1) / block_size) must be valid page numbers in [0, n_pages)
 * (the last of them is the partly filled tail page), the others are never read.  The summaries (musig, mnorm) and
 * sel_mask stay indexed by (sequence, KV head, block) as in the contiguous case: they are the held-out table.
 * The three calls compute exactly what their contiguous counterparts compute on the gathered cache, bit for bit.
 * Ownership, alignment, error behaviour: as for the contiguous calls; a NULL table, table_stride too small or
 * n_pages <= 0 return ETA_ERR_INVALID_ARG.  Page numbers are not range-checked on the device.
 */
typedef struct eta_page_table {
    const int32_t* block_table;
    int32_t table_stride;
    int32_t n_pages;
} eta_page_table;

int eta_build_block_summaries_paged(const eta_cache_desc* desc, const eta_page_table* pages, const void* K_pool,
                                    const int32_t* seq_lens, void* musig, float* mnorm, uint32_t flags, void* stream);
int eta_append_summary_paged(const eta_cache_desc* desc, const eta_page_table* pages, const void* K_pool,
                             const int32_t* seq_lens_after, void* musig, float* mnorm, uint32_t flags, void* stream);
int eta_decode_paged(const eta_cache_desc* desc, const eta_page_table* pages, const eta_params* params, const void* q,
                     const void* K_pool, const void* V_pool, const int32_t* seq_lens,
                     const void* musig, const float* mnorm,
                     const float* tau, const float* head_const,
                     float* out, uint8_t* sel_mask, int32_t* stats, uint32_t* status_dev,
                     void* workspace, size_t workspace_bytes, void* stream);

/* Size of the built-in scratch of eta_decode_static, in bytes. */
size_t eta_static_scratch_bytes(void);

/* Number of kernels one eta_decode call launches (for launch accounting). */
int eta_decode_kernel_count(void);

/*
 * Per-kernel timing of a decode step (measurement aid; the paper has no counterpart).  While enabled,
 * eta_append_summary, eta_predict_threshold and eta_decode record host-side CUDA events before each of their
 * kernel launches on the call's stream (inside a stream capture they become nodes of the graph).
 * eta_profile_read waits for the most recent eta_decode to finish and writes the time from each launch to the
 * next, in milliseconds, to ms[0 .. count-1] (n >= 5), in the order append, predict, screen, decode, merge,
 * returning the count, or a negative status when no profiled eta_decode has run.  The first two are 0
 * unless those calls were made, in that order, right before the eta_decode.  Process-wide state (one set of
 * events, created on the device that is current at the first mark; calls are serialised by a lock): for one
 * measuring thread on one device; leave disabled in production.
 */
int eta_profile_enable(int on);
int eta_profile_read(float* ms, int n);
const char* eta_profile_kernel_name(int k);

/*
 * Launch policy (the paper has no counterpart).  By default the kernels of a decode step are launched with
 * programmatic dependent launch: each may start its set-up while its predecessor in the stream drains, and
 * waits for the predecessor's completion before reading anything it wrote.  eta_set_pdl(0) makes every launch
 * wait for the full completion of the previous one instead (for A/B timing and for debugging).  Process-wide.
 */
int eta_set_pdl(int on);

/* Text for an eta_status. */
const char* eta_strerror(int code);

/* Text of the last CUDA error this library saw on the calling thread ("" if none). */
const char* eta_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* ETA_H_ */

/*
 * CPU oracle for the inference path of Elastic Threshold Attention (ETA).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, obviously-correct
 * restatement of the paper's definitions in fp64.  It shares no code with the
 * CUDA library, is never called by the product path, and exists so that the
 * GPU kernels can be compared element by element with something a reader can
 * check against the paper by eye.  The only roundings are the storage
 * roundings the paper states (block summaries kept as fp16 / fp32).
 *
 * Every loop follows the order and the notation of the passage it cites:
 *   - Section 2 (dense attention, threshold prediction, Eq. tau_pred,
 *     Eq. soft_mask, Eq. mult_attn),
 *   - Section 3 (dual block index, Eq. dual_bound_eq),
 *   - Appendix "Inference-Time Block-Sparse Fused Kernel" (Algorithm 3:
 *     screening, top-1 rescue, tail phase; compact metadata layout),
 *   - Appendix "Screening index quality" (Eq. subblock_envelope_appx, lwb),
 *   - Appendix "Train-to-inference consistency" (definitions of o_block,
 *     o_train and the partition sums Z).
 *
 * Parity status: every function here is pinned by tests that do not call it
 * to produce their expectation (closed forms, library routines, brute force,
 * invariants) EXCEPT the general-input sparse output of
 * eta_oracle_gated_block_attention, for which the paper prints no worked
 * example: "parity unpinned" by printed values; it is pinned only through
 * the special cases tau=-inf (softmax), tau=+inf (mean of V), beta=0
 * (half-scale softmax), the exact decomposition identity and a brute-force
 * per-token restatement on tiny inputs.
 *
 * Tensors are dense, row-major, with explicit element strides for K and V
 * so that a cache with spare capacity can be described:
 *   K, V   : bf16 bit patterns (uint16), element (i,h,t,c) at
 *            i*stride_b + h*stride_h + t*stride_t + c
 *   q      : bf16 bit patterns [B, Hq, d]
 *   musig  : fp16 bit patterns [B, Hkv, NBcap, 2, d]  (mu then sigma)
 *   mnorm  : fp32 [B, Hkv, NBcap]
 *   query head h belongs to KV head h / G, G = Hq / Hkv.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------ */
/* storage formats                                                           */
/* ------------------------------------------------------------------------ */

/* bf16 -> double: a bf16 is the upper half of an IEEE binary32. */
double eta_oracle_bf16_to_double(uint16_t bits) {
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* fp16 -> double, IEEE binary16 (1 sign, 5 exponent, 10 fraction bits). */
double eta_oracle_fp16_to_double(uint16_t bits) {
    int sign = (bits >> 15) & 1;
    int expo = (bits >> 10) & 0x1f;
    int frac = bits & 0x3ff;
    double v;
    if (expo == 0) {
        v = ldexp((double)frac, -24);            /* subnormal or zero */
    } else if (expo == 31) {
        v = frac ? NAN : INFINITY;
    } else {
        v = ldexp(1.0 + (double)frac / 1024.0, expo - 15);
    }
    return sign ? -v : v;
}

/* double -> fp16 with a single round-to-nearest-even (no double rounding
 * through binary32); overflow gives infinity. */
uint16_t eta_oracle_double_to_fp16(double x) {
    uint16_t sign = 0;
    if (isnan(x)) return 0x7e00;
    if (signbit(x)) { sign = 0x8000; x = -x; }
    if (isinf(x)) return sign | 0x7c00;
    if (x == 0.0) return sign;
    int e;
    double m = frexp(x, &e);                    /* x = m * 2^e, m in [0.5,1) */
    int expo = e - 1;                            /* x = (2m) * 2^expo         */
    double scaled;
    int biased;
    if (expo < -14) {                            /* subnormal: units of 2^-24 */
        scaled = ldexp(x, 24);
        biased = 0;
    } else {
        scaled = ldexp(2.0 * m, 10);             /* in [1024, 2048)           */
        biased = expo + 15;
    }
    double fl = floor(scaled);
    double rem = scaled - fl;
    long long q = (long long)fl;
    if (rem > 0.5 || (rem == 0.5 && (q & 1))) q += 1;
    if (biased == 0) {
        /* q in [0,1024]; 1024 is the smallest normal and the bit pattern
         * 0x0400 falls out of the addition below. */
        return sign | (uint16_t)q;
    }
    if (q == 2048) { q = 1024; biased += 1; }
    if (biased >= 31) return sign | 0x7c00;
    return sign | (uint16_t)((biased << 10) | (q - 1024));
}

/* e4m3 (8-bit float: 1 sign, 4 exponent bits with bias 7, 3 fraction bits; no
 * infinities, 0x7f / 0xff are NaN, largest finite value 448) -> double. */
double eta_oracle_e4m3_to_double(uint8_t bits) {
    int sign = (bits >> 7) & 1;
    int expo = (bits >> 3) & 0xf;
    int frac = bits & 0x7;
    double v;
    if (expo == 15 && frac == 7) v = NAN;
    else if (expo == 0) v = ldexp((double)frac, -9);          /* subnormal or zero: units of 2^-9 */
    else v = ldexp(1.0 + (double)frac / 8.0, expo - 7);
    return sign ? -v : v;
}

/* The smallest e4m3 value that is >= x, for x >= 0 (rounding toward +infinity);
 * x above the largest finite value (448) or NaN gives the NaN code 0x7f, which
 * the screening rule reads as "admit".  The positive codes 0x00 .. 0x7e are in
 * ascending order of value, so the answer is found by walking them. */
uint8_t eta_oracle_double_to_e4m3_up(double x) {
    if (!(x <= 448.0)) return 0x7f;
    if (x <= 0.0) return 0;
    for (int code = 0; code <= 0x7e; ++code)
        if (eta_oracle_e4m3_to_double((uint8_t)code) >= x) return (uint8_t)code;
    return 0x7f;
}

/*
 * Packed block summaries (the paper's outlook: "FP8 metadata"; the compact
 * layout of the fused-kernel appendix is what it shrinks).  Format "sigma8",
 * chosen by this library: per block and KV head
 *     mu      fp16 [d]   (as in the compact layout)
 *     sigma^  e4m3 [d]   sigma rounded UP to the next e4m3 value
 * (3 d bytes instead of 4 d), M stays fp32.  Score_dual is non-decreasing in
 * every sigma_c, and every e4m3 value is an fp16 value, so with sigma^ >= sigma
 * the packed bound is never below the bound from the fp16 record: packing adds
 * no false negative, it only admits a few more blocks.  sigma beyond 448 becomes
 * the NaN code (bound NaN, block admitted).
 * sigma_raw: the unrounded doubles [B,Hkv,NBcap,d] of eta_oracle_block_summaries;
 * musig: its fp16 records (mu is copied); musig8: bytes [B,Hkv,NBcap,3 d].
 */
void eta_oracle_pack_sigma8(const uint16_t* musig, const double* sigma_raw, int B, int Hkv, int d, int b, int NBcap,
                            const int32_t* seq_lens, uint8_t* musig8)
{
    for (int i = 0; i < B; ++i) {
        int NB = seq_lens[i] / b;
        if (NB > NBcap) NB = NBcap;
        for (int h = 0; h < Hkv; ++h)
            for (int j = 0; j < NB; ++j) {
                int64_t rec = ((int64_t)(i * Hkv + h) * NBcap + j);
                uint8_t* out = musig8 + rec * 3 * d;
                memcpy(out, musig + rec * 2 * d, 2 * (size_t)d);
                for (int c = 0; c < d; ++c) out[2 * d + c] = eta_oracle_double_to_e4m3_up(sigma_raw[rec * d + c]);
            }
    }
}

/* The fp16 record layout with sigma^ in place of sigma (every e4m3 value is exactly
 * an fp16 value; the NaN code becomes an fp16 NaN): what the screening rule
 * evaluates for a packed index.  All records of the arrays are converted. */
void eta_oracle_unpack_sigma8(const uint8_t* musig8, int64_t n_rec, int d, uint16_t* musig)
{
    for (int64_t rec = 0; rec < n_rec; ++rec) {
        memcpy(musig + rec * 2 * d, musig8 + rec * 3 * d, 2 * (size_t)d);
        for (int c = 0; c < d; ++c)
            musig[rec * 2 * d + d + c] = eta_oracle_double_to_fp16(eta_oracle_e4m3_to_double(musig8[rec * 3 * d + 2 * d + c]));
    }
}

/* ------------------------------------------------------------------------ */
/* Section 3: the dual probabilistic-geometric block index                   */
/* ------------------------------------------------------------------------ */

/*
 * For every full block j < floor(T_i / b) of every (sequence, KV head):
 *   mu      = (1/b) sum_k k                    (centroid)
 *   sigma^2 = (1/b) sum_k (k - mu)^2           (coordinate-wise, population)
 *   M       = max_k ||k||_2
 * If envelope != 0, sigma is replaced by the sub-block envelope
 *   sigma~_c = max_m sqrt( (1/4) sum_{k in B_m} (k_c - mu_c)^2 )
 * over the b/4 contiguous 4-token sub-blocks (Eq. subblock_envelope_appx).
 * The record stores sigma (not the variance) in fp16, mu in fp16, M in fp32
 * (compact metadata layout).  mu_raw / sigma_raw / m_raw, when non-NULL,
 * receive the unrounded doubles with the same indexing.
 */
void eta_oracle_block_summaries(
    const uint16_t* K, int64_t stride_b, int64_t stride_h, int64_t stride_t,
    int B, int Hkv, int d, int b, int NBcap, const int32_t* seq_lens,
    int envelope,
    uint16_t* musig, float* mnorm,
    double* mu_raw, double* sigma_raw, double* m_raw)
{
    #pragma omp parallel for collapse(2) schedule(dynamic)
    for (int i = 0; i < B; ++i) {
        for (int h = 0; h < Hkv; ++h) {
            double* mu = (double*)malloc(sizeof(double) * d);
            double* sg = (double*)malloc(sizeof(double) * d);
            int NB = seq_lens[i] / b;
            if (NB > NBcap) NB = NBcap;
            for (int j = 0; j < NB; ++j) {
                const uint16_t* blk = K + i * stride_b + h * stride_h + (int64_t)j * b * stride_t;
                /* centroid */
                for (int c = 0; c < d; ++c) {
                    double s = 0.0;
                    for (int t = 0; t < b; ++t) s += eta_oracle_bf16_to_double(blk[t * stride_t + c]);
                    mu[c] = s / b;
                }
                /* coordinate-wise spread about the centroid */
                for (int c = 0; c < d; ++c) {
                    if (!envelope) {
                        double s = 0.0;
                        for (int t = 0; t < b; ++t) {
                            double dv = eta_oracle_bf16_to_double(blk[t * stride_t + c]) - mu[c];
                            s += dv * dv;
                        }
                        sg[c] = sqrt(s / b);
                    } else {
                        double best = 0.0;
                        for (int m = 0; m < b / 4; ++m) {
                            double s = 0.0;
                            for (int t = 4 * m; t < 4 * m + 4; ++t) {
                                double dv = eta_oracle_bf16_to_double(blk[t * stride_t + c]) - mu[c];
                                s += dv * dv;
                            }
                            double r = sqrt(s / 4.0);
                            if (r > best) best = r;
                        }
                        sg[c] = best;
                    }
                }
                /* largest Euclidean norm */
                double M = 0.0;
                for (int t = 0; t < b; ++t) {
                    double s = 0.0;
                    for (int c = 0; c < d; ++c) {
                        double v = eta_oracle_bf16_to_double(blk[t * stride_t + c]);
                        s += v * v;
                    }
                    double n = sqrt(s);
                    if (n > M) M = n;
                }
                int64_t rec = ((int64_t)(i * Hkv + h) * NBcap + j);
                for (int c = 0; c < d; ++c) {
                    musig[rec * 2 * d + c] = eta_oracle_double_to_fp16(mu[c]);
                    musig[rec * 2 * d + d + c] = eta_oracle_double_to_fp16(sg[c]);
                    if (mu_raw) mu_raw[rec * d + c] = mu[c];
                    if (sigma_raw) sigma_raw[rec * d + c] = sg[c];
                }
                mnorm[rec] = (float)M;
                if (m_raw) m_raw[rec] = M;
            }
            free(mu);
            free(sg);
        }
    }
}

/* ------------------------------------------------------------------------ */
/* Section 2.1: threshold prediction (Eq. tau_pred)                          */
/* ------------------------------------------------------------------------ */

/*
 * qbar_i = [q_{i,1} || ... || q_{i,Hq}]  (head-major concatenation, length Hq*d)
 * tau_i  = qbar_i W + bias,  W is [Hq*d, Hq] row-major, bias is [Hq].
 */
void eta_oracle_predict_threshold(
    const uint16_t* q, const float* W, const float* bias,
    int B, int Hq, int d, double* tau)
{
    for (int i = 0; i < B; ++i) {
        for (int h = 0; h < Hq; ++h) {
            double s = (double)bias[h];
            for (int r = 0; r < Hq * d; ++r)
                s += eta_oracle_bf16_to_double(q[(int64_t)i * Hq * d + r]) * (double)W[(int64_t)r * Hq + h];
            tau[i * Hq + h] = s;
        }
    }
}

/* ------------------------------------------------------------------------ */
/* Eq. dual_bound_eq / Algorithm 3, screening lines                          */
/* ------------------------------------------------------------------------ */

/*
 * bound[i,h,j] = s * min( <q,mu_j> + z*sqrt(sum_c q_c^2 sigma_{j,c}^2),
 *                         ||q|| * M_j )
 * evaluated from the STORED (rounded) record; sigma is squared here, in
 * double.  gauss / spher, when non-NULL, receive the two terms (each already
 * multiplied by s).  Entries j >= floor(T_i/b) are left untouched.
 */
void eta_oracle_score_dual(
    const uint16_t* q, const uint16_t* musig, const float* mnorm,
    int B, int Hq, int Hkv, int d, int b, int NBcap, const int32_t* seq_lens,
    double z, double s,
    double* bound, double* gauss, double* spher)
{
    int G = Hq / Hkv;
    #pragma omp parallel for collapse(2) schedule(dynamic)
    for (int i = 0; i < B; ++i) {
        for (int h = 0; h < Hq; ++h) {
            int hk = h / G;
            int NB = seq_lens[i] / b;
            if (NB > NBcap) NB = NBcap;
            const uint16_t* qv = q + ((int64_t)i * Hq + h) * d;
            double qn = 0.0;
            for (int c = 0; c < d; ++c) {
                double x = eta_oracle_bf16_to_double(qv[c]);
                qn += x * x;
            }
            qn = sqrt(qn);
            for (int j = 0; j < NB; ++j) {
                int64_t rec = ((int64_t)(i * Hkv + hk) * NBcap + j);
                double dot = 0.0, var = 0.0;
                for (int c = 0; c < d; ++c) {
                    double x = eta_oracle_bf16_to_double(qv[c]);
                    double m = eta_oracle_fp16_to_double(musig[rec * 2 * d + c]);
                    double sg = eta_oracle_fp16_to_double(musig[rec * 2 * d + d + c]);
                    dot += x * m;
                    var += x * x * sg * sg;
                }
                double bg = s * (dot + z * sqrt(var));
                double bs = s * qn * (double)mnorm[rec];
                int64_t o = ((int64_t)i * Hq + h) * NBcap + j;
                /* fmin would drop a NaN; keep it so that "not below tau" admits */
                bound[o] = (bg < bs) ? bg : ((bs < bg) ? bs : ((bg != bg) ? bg : bs));
                if (gauss) gauss[o] = bg;
                if (spher) spher[o] = bs;
            }
        }
    }
}

/*
 * Per-query-head selection (Algorithm 3, screening + rescue; lwb pinning from
 * the screening-index appendix):
 *   tau_eff = tau - a
 *   block j admitted  iff  not (bound_j < tau_eff)
 *   the last `lwb` full blocks are always admitted
 *   if none of the first Wr = min(rescue_window, NB) blocks is admitted, the
 *   first index attaining the largest bound among them is admitted
 *   (strict ">" update while scanning upwards).
 * ungate_last (the diagonal case of Eq. mult_attn, M_ts = 1 for s = t, carried
 * over to decoding, where the query's own token is the newest one): when the
 * newest token closes a full block (T mod b == 0) that block is admitted for
 * every head, since an ungated token must be attended.
 * sel[i,hk,j] gets bit g = h - hk*G set for every admitting head.
 * rescued[i,h] (nullable) is set to the rescued index or -1.
 */
void eta_oracle_select(
    const double* bound, const float* tau, const float* head_const,
    int B, int Hq, int Hkv, int b, int NBcap, const int32_t* seq_lens,
    double a, int lwb, int rescue_window, int ungate_last,
    uint8_t* sel, int32_t* rescued)
{
    int G = Hq / Hkv;
    memset(sel, 0, (size_t)B * Hkv * NBcap);
    for (int i = 0; i < B; ++i) {
        for (int h = 0; h < Hq; ++h) {
            int hk = h / G, g = h % G;
            int NB = seq_lens[i] / b;
            if (NB > NBcap) NB = NBcap;
            double t = head_const ? (double)head_const[h] : (double)tau[i * Hq + h];
            double tau_eff = t - a;
            uint8_t* row = sel + (int64_t)(i * Hkv + hk) * NBcap;
            const double* bd = bound + ((int64_t)i * Hq + h) * NBcap;
            int Wr = rescue_window < NB ? rescue_window : NB;
            int attended_in_window = 0;
            double max_bound = -INFINITY;
            int max_idx = -1;
            for (int j = 0; j < NB; ++j) {
                int admit = !(bd[j] < tau_eff);
                if (j >= NB - lwb) admit = 1;
                if (ungate_last && seq_lens[i] > 0 && seq_lens[i] % b == 0 && j == seq_lens[i] / b - 1) admit = 1;
                if (admit) {
                    row[j] |= (uint8_t)(1u << g);
                    if (j < Wr) attended_in_window += 1;
                }
                if (j < Wr && bd[j] > max_bound) { max_bound = bd[j]; max_idx = j; }
            }
            int r = -1;
            if (Wr > 0 && attended_in_window == 0) {
                if (max_idx < 0) max_idx = 0;    /* every bound NaN or -inf */
                row[max_idx] |= (uint8_t)(1u << g);
                r = max_idx;
            }
            if (rescued) rescued[i * Hq + h] = r;
        }
    }
}

/* ------------------------------------------------------------------------ */
/* Eq. mult_attn at inference: S~ = S * sigmoid(beta (S - tau_eff))          */
/* ------------------------------------------------------------------------ */

double eta_oracle_gate(double S, double tau_eff, double beta) {
    double x = beta * (S - tau_eff);
    double sig;
    if (x != x) {
        /* beta = 0 against an infinite threshold: sigmoid(0 * inf) is read
         * as the limit beta -> 0, i.e. one half. */
        sig = 0.5;
    } else if (x >= 0) {
        sig = 1.0 / (1.0 + exp(-x));
    } else {
        double e = exp(x);
        sig = e / (1.0 + e);
    }
    if (sig == 0.0) return 0.0;                  /* avoids (-inf)*0 */
    return S * sig;
}

/*
 * o_block for every query head (Algorithm 3, attention lines; definition of
 * o_block in the consistency appendix): over the tokens of the head's OWN
 * admitted blocks plus every tail token T_i - NB*b,
 *   S_s  = s <q, k_s>,   S~_s = gate(S_s),   w_s = exp(S~_s)
 *   out  = sum_s w_s v_s / sum_s w_s .
 * Z (nullable, [B,Hq]) receives log(sum_s w_s); n_tok (nullable) the number
 * of attended tokens.  A head never attends a block fetched only for a
 * sibling head of its GQA group.
 * ungate_last: the newest token s = T_i - 1 (the query's own position) keeps
 * its raw logit, S~ = S (Eq. mult_attn, M_ts = 1 for s = t; the "restore token
 * diagonal" line of Algorithm 2).  Off, every token is gated (Algorithm 3 as
 * printed).
 */
void eta_oracle_gated_block_attention(
    const uint16_t* q,
    const uint16_t* K, int64_t k_stride_b, int64_t k_stride_h, int64_t k_stride_t,
    const uint16_t* V, int64_t v_stride_b, int64_t v_stride_h, int64_t v_stride_t,
    const uint8_t* sel, const float* tau, const float* head_const,
    int B, int Hq, int Hkv, int d, int b, int NBcap, const int32_t* seq_lens,
    double a, double beta, double s, int ungate_last,
    double* out, double* logZ, int64_t* n_tok)
{
    int G = Hq / Hkv;
    #pragma omp parallel for collapse(2) schedule(dynamic)
    for (int i = 0; i < B; ++i) {
        for (int h = 0; h < Hq; ++h) {
            int hk = h / G, g = h % G;
            int T = seq_lens[i];
            int NB = T / b;
            if (NB > NBcap) NB = NBcap;
            double t = head_const ? (double)head_const[h] : (double)tau[i * Hq + h];
            double tau_eff = t - a;
            const uint16_t* qv = q + ((int64_t)i * Hq + h) * d;
            const uint16_t* Kh = K + i * k_stride_b + hk * k_stride_h;
            const uint16_t* Vh = V + i * v_stride_b + hk * v_stride_h;
            const uint8_t* row = sel + (int64_t)(i * Hkv + hk) * NBcap;
            double* St = (double*)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1));
            /* pass 1: gated logits of attended tokens, and their maximum */
            double mx = -INFINITY;
            int64_t cnt = 0;
            for (int p = 0; p < T; ++p) {
                int j = p / b;
                int attended = (j >= NB) ? 1 : ((row[j] >> g) & 1);
                if (!attended) { St[p] = NAN; continue; }
                double dot = 0.0;
                for (int c = 0; c < d; ++c)
                    dot += eta_oracle_bf16_to_double(qv[c]) * eta_oracle_bf16_to_double(Kh[p * k_stride_t + c]);
                double Sg = eta_oracle_gate(s * dot, tau_eff, beta);
                if (ungate_last && p == T - 1) Sg = s * dot;
                St[p] = Sg;
                if (Sg > mx) mx = Sg;
                cnt += 1;
            }
            /* pass 2: weights and weighted values */
            double* o = out + ((int64_t)i * Hq + h) * d;
            for (int c = 0; c < d; ++c) o[c] = 0.0;
            double Zs = 0.0;
            for (int p = 0; p < T; ++p) {
                if (St[p] != St[p]) continue;
                double w = exp(St[p] - mx);
                Zs += w;
                for (int c = 0; c < d; ++c)
                    o[c] += w * eta_oracle_bf16_to_double(Vh[p * v_stride_t + c]);
            }
            for (int c = 0; c < d; ++c) o[c] = (Zs > 0.0) ? o[c] / Zs : 0.0;
            if (logZ) logZ[i * Hq + h] = (Zs > 0.0) ? (mx + log(Zs)) : -INFINITY;
            if (n_tok) n_tok[i * Hq + h] = cnt;
            free(St);
        }
    }
}

/*
 * Section 2, dense attention: o = sum_s A_s v_s with
 * A_s = exp(<q,k_s>/sqrt(d)) / sum_j exp(<q,k_j>/sqrt(d)) over all T_i tokens.
 * Written on its own (no gate, no block structure) so that it can serve as
 * the textbook reference the gated routine is compared with at tau = -inf.
 */
void eta_oracle_dense_softmax_attention(
    const uint16_t* q,
    const uint16_t* K, int64_t k_stride_b, int64_t k_stride_h, int64_t k_stride_t,
    const uint16_t* V, int64_t v_stride_b, int64_t v_stride_h, int64_t v_stride_t,
    int B, int Hq, int Hkv, int d, const int32_t* seq_lens, double s,
    double* out)
{
    int G = Hq / Hkv;
    #pragma omp parallel for collapse(2) schedule(dynamic)
    for (int i = 0; i < B; ++i) {
        for (int h = 0; h < Hq; ++h) {
            int hk = h / G;
            int T = seq_lens[i];
            const uint16_t* qv = q + ((int64_t)i * Hq + h) * d;
            const uint16_t* Kh = K + i * k_stride_b + hk * k_stride_h;
            const uint16_t* Vh = V + i * v_stride_b + hk * v_stride_h;
            double* logit = (double*)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1));
            double mx = -INFINITY;
            for (int p = 0; p < T; ++p) {
                double dot = 0.0;
                for (int c = 0; c < d; ++c)
                    dot += eta_oracle_bf16_to_double(qv[c]) * eta_oracle_bf16_to_double(Kh[p * k_stride_t + c]);
                logit[p] = s * dot;
                if (logit[p] > mx) mx = logit[p];
            }
            double den = 0.0;
            for (int p = 0; p < T; ++p) den += exp(logit[p] - mx);
            double* o = out + ((int64_t)i * Hq + h) * d;
            for (int c = 0; c < d; ++c) {
                double acc = 0.0;
                for (int p = 0; p < T; ++p)
                    acc += (exp(logit[p] - mx) / den) * eta_oracle_bf16_to_double(Vh[p * v_stride_t + c]);
                o[c] = acc;
            }
            free(logit);
        }
    }
}

/*
 * Diagnostics (definitions of the index-quality table): the true largest
 * logit inside every full block, max_{s in B_j} s <q, k_s>, per query head.
 */
void eta_oracle_block_max_logit(
    const uint16_t* q,
    const uint16_t* K, int64_t k_stride_b, int64_t k_stride_h, int64_t k_stride_t,
    int B, int Hq, int Hkv, int d, int b, int NBcap, const int32_t* seq_lens,
    double s, double* maxlogit)
{
    int G = Hq / Hkv;
    #pragma omp parallel for collapse(2) schedule(dynamic)
    for (int i = 0; i < B; ++i) {
        for (int h = 0; h < Hq; ++h) {
            int hk = h / G;
            int NB = seq_lens[i] / b;
            if (NB > NBcap) NB = NBcap;
            const uint16_t* qv = q + ((int64_t)i * Hq + h) * d;
            const uint16_t* Kh = K + i * k_stride_b + hk * k_stride_h;
            for (int j = 0; j < NB; ++j) {
                double best = -INFINITY;
                for (int t = 0; t < b; ++t) {
                    int64_t p = (int64_t)j * b + t;
                    double dot = 0.0;
                    for (int c = 0; c < d; ++c)
                        dot += eta_oracle_bf16_to_double(qv[c]) * eta_oracle_bf16_to_double(Kh[p * k_stride_t + c]);
                    if (s * dot > best) best = s * dot;
                }
                maxlogit[((int64_t)i * Hq + h) * NBcap + j] = best;
            }
        }
    }
}

/* ------------------------------------------------------------------------ */
/* Offline threshold calibration (appendix "Offline Threshold Calibration via */
/* 1/t-Weighted Histograms", Algorithm "Density-Matched Offline Threshold     */
/* Calibration")                                                              */
/* ------------------------------------------------------------------------ */

static double oracle_sigmoid(double x) {
    if (x >= 0) return 1.0 / (1.0 + exp(-x));
    double e = exp(x);
    return e / (1.0 + e);
}

/* g(c) = sum_b H[b] sigmoid(beta (s_b - c)): the head's density under a static
 * threshold c, from the normalised 1/t-weighted score histogram. */
double eta_oracle_calibration_density(const double* hist, int n_bins, double s_min, double s_max,
                                      double beta, double c)
{
    double w = (s_max - s_min) / n_bins, g = 0.0;
    for (int b = 0; b < n_bins; ++b) g += hist[b] * oracle_sigmoid(beta * (s_min + (b + 0.5) * w - c));
    return g;
}

/*
 * The calibration pass over a split of n_seq sequences of T tokens, per query
 * head h (GQA: KV head h / G), with raw causal scores S_ts = s <q_t, k_s>,
 * s <= t, and the dynamic thresholds tau[x,h,t] of the predictor:
 *   target density   dbar_h = 1/(n_seq T) sum_x sum_t (1/t) sum_{s<=t} sigmoid(beta (S_ts - tau_t))
 *   histogram        H_h[bin(S_ts)] += 1/t    (t counted from 1), then H_h /= sum_b H_h[b]
 *   constant         c_h = root of g(c) = dbar_h by bisection (g decreases from 1 to 0)
 * Bins: n_bins equal bins on [s_min, s_max], centre s_b = s_min + (b + 1/2) w;
 * a score outside the range goes to the first / last bin (the paper fixes
 * neither range nor edge rule).  The bin of a score is decided on the score as
 * computed here, in double ("bin raw scores").
 * Bisection: `iters` halvings of [s_min - 40/beta, s_max + 40/beta].
 * hist [Hq, n_bins], dbar [Hq], head_const [Hq], residual [Hq] (= g(c) - dbar).
 */
void eta_oracle_calibrate(
    const uint16_t* Q, const uint16_t* K, const float* tau,
    int n_seq, int Hq, int Hkv, int T, int d, double beta, double s,
    int n_bins, double s_min, double s_max, int iters,
    double* hist, double* dbar, double* head_const, double* residual)
{
    int G = Hq / Hkv;
    double w = (s_max - s_min) / n_bins;
    #pragma omp parallel for schedule(dynamic)
    for (int h = 0; h < Hq; ++h) {
        double* H = hist + (int64_t)h * n_bins;
        for (int b = 0; b < n_bins; ++b) H[b] = 0.0;
        double dsum = 0.0;
        for (int x = 0; x < n_seq; ++x) {
            const uint16_t* Qh = Q + (((int64_t)x * Hq + h) * T) * d;
            const uint16_t* Kh = K + (((int64_t)x * Hkv + h / G) * T) * d;
            for (int t = 0; t < T; ++t) {
                double inv_t = 1.0 / (double)(t + 1);
                double th = (double)tau[((int64_t)x * Hq + h) * T + t];
                double rowsum = 0.0;
                for (int sidx = 0; sidx <= t; ++sidx) {
                    double dot = 0.0;
                    for (int c = 0; c < d; ++c)
                        dot += eta_oracle_bf16_to_double(Qh[(int64_t)t * d + c]) *
                               eta_oracle_bf16_to_double(Kh[(int64_t)sidx * d + c]);
                    double S = s * dot;
                    rowsum += oracle_sigmoid(beta * (S - th));
                    int b = (int)floor((S - s_min) / w);
                    if (b < 0) b = 0;
                    if (b >= n_bins) b = n_bins - 1;
                    H[b] += inv_t;
                }
                dsum += rowsum * inv_t;
            }
        }
        double tot = 0.0;
        for (int b = 0; b < n_bins; ++b) tot += H[b];
        for (int b = 0; b < n_bins; ++b) H[b] = tot > 0.0 ? H[b] / tot : 0.0;
        double target = dsum / ((double)n_seq * (double)T);
        double lo = s_min - 40.0 / beta, hi = s_max + 40.0 / beta;
        for (int it = 0; it < iters; ++it) {
            double mid = 0.5 * (lo + hi);
            if (eta_oracle_calibration_density(H, n_bins, s_min, s_max, beta, mid) > target) lo = mid; else hi = mid;
        }
        double c = 0.5 * (lo + hi);
        dbar[h] = target;
        head_const[h] = c;
        if (residual) residual[h] = eta_oracle_calibration_density(H, n_bins, s_min, s_max, beta, c) - target;
    }
}

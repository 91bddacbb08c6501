"""Shared test helpers: tensor <-> bit-pattern conversions and threshold calibration.

The calibration lives here (under tests/) because it calls the CPU oracle; the
product package never does.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import eta_oracle as orc


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 / fp16 torch tensor -> uint16 bit patterns (numpy, same shape)."""
    assert t.dtype in (torch.bfloat16, torch.float16)
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def bf16_bits_from_f64(x: np.ndarray) -> np.ndarray:
    """Round doubles to bf16 (via torch) and return the bit patterns."""
    return bits(torch.from_numpy(np.asarray(x, np.float64)).to(torch.float32).to(torch.bfloat16))


def bf16_values(b: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float64 values."""
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def fp16_values(b: np.ndarray) -> np.ndarray:
    return b.view(np.float16).astype(np.float64)


def random_cache(rng, B, Hkv, T, d, b, Tcap=None, scale=1.0):
    Tcap = Tcap or ((T + b - 1) // b) * b
    K = bf16_bits_from_f64(rng.standard_normal((B, Hkv, Tcap, d)) * scale)
    V = bf16_bits_from_f64(rng.standard_normal((B, Hkv, Tcap, d)))
    lens = np.full(B, T, np.int32)
    return orc.Cache(K, V, lens, b)


def cache_of(wl) -> orc.Cache:
    """Oracle view of a generated workload."""
    return orc.Cache(bits(wl.K), bits(wl.V), wl.seq_lens.numpy().astype(np.int32).copy(), wl.spec.block_size)


def union_density(bound, tau, seq_lens, b, G):
    """Fraction of full blocks admitted by at least one head of their GQA group (plain threshold, no rescue)."""
    B, Hq, NBcap = bound.shape
    adm = ~(bound < tau[:, :, None])                     # NaN (beyond NB) compares False -> masked below
    tot = 0
    hit = 0
    for i in range(B):
        NB = int(seq_lens[i]) // b
        u = adm[i, :, :NB].reshape(Hq // G, G, NB).any(axis=1)
        hit += int(u.sum())
        tot += u.size
    return hit / max(tot, 1)


def calibrate_bias(bound, tau_raw, seq_lens, b, G, target_union_sparsity):
    """Per-head predictor bias such that the union block sparsity hits a target.

    bound: oracle bounds [B,Hq,NBcap]; tau_raw: q̄W without bias [B,Hq].
    For a head-density level rho, bias_h(rho) = median_i(quantile_{1-rho}(bound[i,h]) - tau_raw[i,h]);
    rho is bisected until the union density is 1 - target.  Stand-in for a trained predictor.
    """
    B, Hq, _ = bound.shape
    srt = []
    for i in range(B):
        NB = int(seq_lens[i]) // b
        srt.append(np.sort(bound[i, :, :NB], axis=1))

    def bias_of(rho):
        qs = np.empty((B, Hq))
        for i in range(B):
            NB = srt[i].shape[1]
            k = min(NB - 1, max(1, int(np.floor((1.0 - rho) * NB))))
            qs[i] = 0.5 * (srt[i][:, k] + srt[i][:, k - 1])     # between two bounds, never exactly on one
        return np.median(qs - tau_raw, axis=0)

    lo, hi = 0.0, 1.0
    for _ in range(30):
        mid = 0.5 * (lo + hi)
        bias = bias_of(mid)
        u = union_density(bound, tau_raw + bias[None, :], seq_lens, b, G)
        if u > 1.0 - target_union_sparsity:
            hi = mid
        else:
            lo = mid
    return bias_of(0.5 * (lo + hi)).astype(np.float32)


def calibrate_head_const(bound, seq_lens, b, sparsity_levels):
    """Frozen per-head constants: c_h = median_i quantile_{level_h}(bound[i,h])."""
    B, Hq, _ = bound.shape
    qs = np.empty((B, Hq))
    for i in range(B):
        NB = int(seq_lens[i]) // b
        s = np.sort(bound[i, :, :NB], axis=1)
        for h in range(Hq):
            k = min(NB - 1, max(1, int(np.floor(sparsity_levels[h] * NB))))
            qs[i, h] = 0.5 * (s[h, k] + s[h, k - 1])
    return np.median(qs, axis=0).astype(np.float32)


# --------------------------------------------------------------------------
# GPU side (used by the -m gpu tests only)
# --------------------------------------------------------------------------

def gpu_decode(q_t, K_t, V_t, seq_lens, block_size, musig_bits, mnorm, tau=None, head_const=None, **params):
    """Run eta_decode on cuda:0 with the given (oracle-built) summaries.

    q_t, K_t, V_t: bf16 CPU tensors; musig_bits uint16 numpy; mnorm float32 numpy; tau/head_const float32 numpy.
    -> out float32 numpy [B,Hq,d], sel uint8 numpy, stats, status
    """
    from paper_2609_20888_b200 import binding as eb
    dev = torch.device("cuda:0")
    K, V, q = K_t.to(dev), V_t.to(dev), q_t.to(dev)
    st = eb.DecodeState(K, V, q_t.shape[1], block_size)
    st.musig.copy_(torch.from_numpy(musig_bits.view(np.int16)).view(torch.float16).to(dev))
    st.mnorm.copy_(torch.from_numpy(mnorm).to(dev))
    lens = torch.from_numpy(np.asarray(seq_lens, np.int32)).to(dev)
    tau_d = None if tau is None else torch.from_numpy(np.ascontiguousarray(tau, np.float32)).to(dev)
    hc_d = None if head_const is None else torch.from_numpy(np.ascontiguousarray(head_const, np.float32)).to(dev)
    p = eb.DecodeParams(**params)
    st.out.fill_(float("nan"))
    eb.eta_decode(st.desc, p, q, K, V, lens, st.musig, st.mnorm, tau_d, hc_d, st.out, st.sel_mask, st.workspace,
                  stats=st.stats, status=st.status)
    torch.cuda.synchronize()
    return st.out.cpu().numpy(), st.sel_mask.cpu().numpy(), st.stats.cpu().numpy(), int(st.status.item())


def compare_masks(sel_gpu, sel_ref, bound, tau_eff, seq_lens, b, G, band=1e-5, rescued=None):
    """Selected-block sets must agree bit for bit except (head, block) pairs whose oracle bound lies within
    `band` (absolute: 1e-5 unless a test states another) of tau_eff, which are returned (logged), and rescue
    choices made among bounds tied within `band`.

    bound [B,Hq,NBcap] float64, tau_eff [B,Hq] float64.  -> list of near-tie mismatches (i, h, j, bound - tau_eff)
    """
    B, Hkv, NBcap = sel_ref.shape
    near = []
    diff = sel_gpu ^ sel_ref
    for i, hk, j in zip(*np.nonzero(diff)):
        NB = int(seq_lens[i]) // b
        assert j < NB, f"mask bit set past the last full block: seq {i} kv head {hk} block {j}"
        for g in range(G):
            if (diff[i, hk, j] >> g) & 1:
                h = hk * G + g
                gap = float(bound[i, h, j] - tau_eff[i, h])
                is_rescue_tie = False
                if rescued is not None and rescued[i, h] >= 0:
                    # the oracle rescued some block for this head: a different argmax is fine if the bounds tie
                    is_rescue_tie = abs(float(bound[i, h, j] - bound[i, h, rescued[i, h]])) <= band
                assert abs(gap) <= band or is_rescue_tie, \
                    f"selection differs away from the threshold: seq {i} head {h} block {j} bound-tau={gap:.3e}"
                near.append((int(i), int(h), int(j), gap))
    return near


def heads_without_near_tie(near, batch, n_q_heads):
    """Boolean [batch, n_q_heads]: heads whose selection had no logged near tie.  A head with one attends a
    different block set on the two sides, so only that head is left out of the output comparison."""
    keep = np.ones((batch, n_q_heads), bool)
    for (i, h, _, _) in near:
        keep[i, h] = False
    return keep


def fp16_ulp_distance(a_bits, b_bits):
    """Distance in units in the last place between fp16 bit patterns (sign-magnitude aware)."""
    def key(x):
        x = x.astype(np.int32)
        return np.where(x & 0x8000, -(x & 0x7fff), x & 0x7fff)
    return np.abs(key(a_bits) - key(b_bits))


def output_errors(out_gpu, out_ref):
    err = np.abs(out_gpu.astype(np.float64) - out_ref)
    return float(err.max()), float(err.mean())

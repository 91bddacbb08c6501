"""Seeded synthetic decode workloads (inputs only).

This module holds no arithmetic of the method (no summaries, bounds, gates or
attention): it only draws K/V caches, queries and predictor weights with the
shapes and value structure of long-context decode, so that the CUDA library
and the CPU checker can be fed the same bytes.  Everything is generated on the
host with counter-based numpy streams keyed by (seed, tensor, sequence, head),
so a tensor does not depend on the order or the number of threads used.

All tensors are rounded to their storage type here (bf16 for q/K/V, fp32 for
the predictor) before anybody sees them.
"""
from __future__ import annotations

import math
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field, replace

import numpy as np
import torch

SEED_BASE = 20888 * 10

_TENSOR_IDS = {"K": 1, "V": 2, "q": 3, "W": 4, "plant": 5, "lens": 6, "mean": 7, "cent": 8, "newkv": 9,
               "const": 10}


def _rng(seed: int, tensor: str, *key: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed << 8) + _TENSOR_IDS[tensor],
                                                     sum((int(k) + 1) << (16 * n) for n, k in enumerate(key))]))


@dataclass(frozen=True)
class Spec:
    """Shape and structure of one workload (one of the five decode configurations)."""
    name: str
    config_id: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    block_size: int
    context: int                    # tokens in the cache at step 0 (max over the batch)
    decode_steps: int               # tokens appended after step 0
    structure: str                  # "planted_keys" | "rope_planted_blocks" | "clustered" | "needle_blocks"
    min_context: int = 0            # >0: per-sequence lengths uniform in [min_context, context]
    z: float = 1.0
    beta: float = 5.0
    lwb: int = 0
    rescue_window: int = 128
    target_sparsity: tuple = (0.85,)   # union block sparsity targets the thresholds are calibrated to
    frozen: bool = False

    @property
    def gqa(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def t_cap(self) -> int:
        b = self.block_size
        return ((self.context + self.decode_steps + b - 1) // b) * b

    @property
    def seed(self) -> int:
        return SEED_BASE + self.config_id

    def scaled(self, context: int, batch: int | None = None, min_context: int | None = None) -> "Spec":
        """Same structure at a smaller context (for tests the CPU checker can finish quickly)."""
        mc = self.min_context if min_context is None else min_context
        return replace(self, context=context, batch=self.batch if batch is None else batch,
                       min_context=min(mc, context))


CONFIGS = {
    # tiny decode step; correctness configuration (cache is L2-resident)
    "c1_tiny": Spec("c1_tiny", 1, 1, 8, 2, 64, 32, 2048, 16, "planted_keys", target_sparsity=(0.80,)),
    # batch 8, 32K context, RoPE-rotated keys with a per-head mean and 1% planted relevant blocks
    "c2_32k": Spec("c2_32k", 2, 8, 32, 8, 128, 64, 32768, 128, "rope_planted_blocks", target_sparsity=(0.85,)),
    # batch 4, 128K context, clustered keys; sparsity sweep through the threshold bias
    "c3_128k": Spec("c3_128k", 3, 4, 32, 8, 128, 64, 131072, 0, "clustered", target_sparsity=(0.50, 0.90, 0.97)),
    # batch 1, 512K context, block size 128, needle blocks at random depths
    "c4_512k": Spec("c4_512k", 4, 1, 16, 4, 128, 128, 524288 - 64, 64, "needle_blocks", target_sparsity=(0.90,)),
    # frozen per-head constants, mixed context lengths 8K..64K
    "c5_frozen": Spec("c5_frozen", 5, 16, 32, 8, 128, 64, 65536, 0, "needle_blocks", min_context=8192,
                      target_sparsity=(0.70,), frozen=True),
}


def _to_bf16(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(x).to(torch.bfloat16)


def _rope_inplace(x: np.ndarray, first_pos: int, theta: float = 5e5) -> None:
    """Rotate rows of x [T, d] as rotary position embedding does, row t at position first_pos + t.

    Pairs are (c, c + d/2), frequency theta^(-2c/d)."""
    T, d = x.shape
    half = d // 2
    inv = theta ** (-np.arange(half, dtype=np.float64) * 2.0 / d)
    ang = (first_pos + np.arange(T, dtype=np.float64))[:, None] * inv[None, :]
    cs, sn = np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)
    a, b = x[:, :half].copy(), x[:, half:].copy()
    x[:, :half] = a * cs - b * sn
    x[:, half:] = a * sn + b * cs


@dataclass
class Workload:
    spec: Spec
    K: torch.Tensor                 # bf16 [B, Hkv, Tcap, d]
    V: torch.Tensor                 # bf16 [B, Hkv, Tcap, d]
    seq_lens: torch.Tensor          # int32 [B], tokens valid at step 0
    W: torch.Tensor                 # fp32 [Hq*d, Hq]
    bias: torch.Tensor              # fp32 [Hq], zero until a calibration sets it
    q_shared0: np.ndarray           # fp32 [B, Hkv, d], the group direction of the step-0 queries
    meta: dict = field(default_factory=dict)

    def queries(self, step: int) -> torch.Tensor:
        """bf16 [B, Hq, d] post-RoPE-like queries of decode step `step`.

        The G heads of a KV group share a common direction (weight 0.95) plus
        head noise (0.05); steps > 0 stay correlated with step 0 (weight 0.5)
        so planted keys keep their relevance while every step reads a
        different set of blocks."""
        sp = self.spec
        B, Hq, Hkv, d, G = sp.batch, sp.n_q_heads, sp.n_kv_heads, sp.head_dim, sp.gqa
        shared = self.q_shared0
        if step > 0:
            fresh = _rng(sp.seed, "q", 2 * step).standard_normal((B, Hkv, d), dtype=np.float32)
            shared = math.sqrt(0.5) * shared + math.sqrt(0.5) * fresh
        noise = _rng(sp.seed, "q", 2 * step + 1).standard_normal((B, Hkv, G, d), dtype=np.float32)
        q = math.sqrt(0.95) * shared[:, :, None, :] + math.sqrt(0.05) * noise
        return _to_bf16(q.reshape(B, Hq, d))

    def new_kv(self, step: int):
        """bf16 k_t, v_t [B, Hkv, d] appended to the cache before decode step `step` (step >= 1)."""
        sp = self.spec
        r = _rng(sp.seed, "newkv", step)
        k = r.standard_normal((sp.batch, sp.n_kv_heads, sp.head_dim), dtype=np.float32)
        v = r.standard_normal((sp.batch, sp.n_kv_heads, sp.head_dim), dtype=np.float32)
        return _to_bf16(k), _to_bf16(v)


def _fill_head(sp: Spec, i: int, h: int, T: int, qdir: np.ndarray, K: torch.Tensor, V: torch.Tensor) -> dict:
    """Draw K[i,h,:T] and V[i,h,:T] for one (sequence, KV head)."""
    d, b = sp.head_dim, sp.block_size
    rk = _rng(sp.seed, "K", i, h)
    k = rk.standard_normal((T, d), dtype=np.float32)
    v = _rng(sp.seed, "V", i, h).standard_normal((T, d), dtype=np.float32)
    NB = T // b
    rp = _rng(sp.seed, "plant", i, h)
    info = {}
    qhat = qdir / np.linalg.norm(qdir)
    if sp.structure == "planted_keys":
        # 16 single keys aligned with the group's query direction, strong enough to move a block's summary
        pos = rp.choice(T, size=min(16, T), replace=False)
        k[pos] = 24.0 * qhat[None, :] + 0.1 * k[pos]
        info["planted_tokens"] = np.sort(pos)
    elif sp.structure == "rope_planted_blocks":
        mean = _rng(sp.seed, "mean", h).standard_normal(d, dtype=np.float32)
        k += mean[None, :]
        _rope_inplace(k, 0)
        n_pl = max(1, NB // 100)
        blocks = rp.choice(NB, size=n_pl, replace=False) if NB > 0 else np.zeros(0, np.int64)
        alpha = rp.uniform(2.0, 8.0, size=n_pl).astype(np.float32)
        for j, al in zip(blocks, alpha):
            k[j * b:(j + 1) * b] = al * qhat[None, :] + 0.3 * k[j * b:(j + 1) * b]
        info["planted_blocks"] = np.sort(blocks)
    elif sp.structure == "clustered":
        cent = _rng(sp.seed, "cent", h).standard_normal((64, d), dtype=np.float32)
        which = rp.integers(0, 64, size=NB + 1)
        k = 0.3 * k + np.repeat(cent[which], b, axis=0)[:T]
    elif sp.structure == "needle_blocks":
        n_pl = max(1, NB // 200)
        blocks = rp.choice(NB, size=n_pl, replace=False) if NB > 0 else np.zeros(0, np.int64)
        alpha = rp.uniform(3.0, 9.0, size=n_pl).astype(np.float32)
        # a slowly drifting context mean gives non-needle blocks a spread of scores
        drift = np.cumsum(rp.standard_normal((NB + 1, d), dtype=np.float32), axis=0) * (1.0 / math.sqrt(64.0))
        k += np.repeat(drift, b, axis=0)[:T] * 0.5
        for j, al in zip(blocks, alpha):
            k[j * b:(j + 1) * b] = al * qhat[None, :] + 0.3 * k[j * b:(j + 1) * b]
        info["planted_blocks"] = np.sort(blocks)
    else:
        raise ValueError(sp.structure)
    K[i, h, :T] = _to_bf16(k)
    V[i, h, :T] = _to_bf16(v)
    return info


def make_workload(sp: Spec, threads: int = 8) -> Workload:
    B, Hq, Hkv, d = sp.batch, sp.n_q_heads, sp.n_kv_heads, sp.head_dim
    if sp.min_context > 0:
        lens = _rng(sp.seed, "lens").integers(sp.min_context, sp.context + 1, size=B).astype(np.int32)
        lens[0] = sp.context
    else:
        lens = np.full(B, sp.context, np.int32)
    # capacity beyond seq_len is zero-filled: those bytes are never meant to be read
    K = torch.zeros((B, Hkv, sp.t_cap, d), dtype=torch.bfloat16)
    V = torch.zeros((B, Hkv, sp.t_cap, d), dtype=torch.bfloat16)
    q_shared0 = _rng(sp.seed, "q", 0).standard_normal((B, Hkv, d), dtype=np.float32)
    jobs = [(i, h) for i in range(B) for h in range(Hkv)]
    meta = {}

    def run(job):
        i, h = job
        return job, _fill_head(sp, i, h, int(lens[i]), q_shared0[i, h], K, V)

    with ThreadPoolExecutor(max_workers=threads) as ex:
        for job, info in ex.map(run, jobs):
            meta[job] = info
    # fan-in scaled init: std 0.02 at the tiny configuration's fan-in of 512
    fan_in = Hq * d
    w_std = 0.02 * math.sqrt(512.0 / fan_in)
    W = torch.from_numpy(_rng(sp.seed, "W").standard_normal((fan_in, Hq), dtype=np.float32) * np.float32(w_std))
    bias = torch.zeros(Hq, dtype=torch.float32)
    return Workload(sp, K, V, torch.from_numpy(lens), W, bias, q_shared0, meta)


def frozen_sparsity_levels(sp: Spec) -> np.ndarray:
    """Per-query-head block sparsity levels in [0.30, 0.95] for the frozen-constant mode."""
    return _rng(sp.seed, "const").uniform(0.30, 0.95, size=sp.n_q_heads)

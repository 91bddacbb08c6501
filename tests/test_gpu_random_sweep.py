"""Seeded sweep over random shapes and parameters: the CUDA decode step against the CPU oracle.

Every case draws its own head_dim, block size, group size, batch, ragged lengths (tails, sequences shorter than
a block, several 64-record segments), key scale, threshold quantile, offset a, z, beta, lwb, rescue window and
flags (newest token ungated, dense), and whether the thresholds are predicted per sequence or frozen per head.
The comparison is the one of the fixed parity cases: masks bit for bit outside the 1e-5 near-tie band, outputs of
heads without a near tie within 1e-2 (max) / 1e-3 (mean), union counts equal to the mask's.
"""
import warnings

import numpy as np
import pytest
import torch

from oracle import eta_oracle as orc
from tests.helpers import bits, compare_masks, gpu_decode, heads_without_near_tie, output_errors

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 1e-2, 1e-3


def _build():
    from paper_2609_20888_b200 import binding as eb
    from paper_2609_20888_b200 import build as ebuild
    ebuild.build()
    eb.load()
    return eb


def _draw(seed):
    rng = np.random.default_rng(1000 + seed)
    d = int(rng.choice([64, 128]))
    b = int(rng.choice([32, 64, 128]))
    G = int(rng.choice([1, 2, 4, 8]))
    Hkv = int(rng.choice([1, 2, 3, 5]))
    B = int(rng.integers(1, 6))
    # lengths: mostly a few thousand tokens (several segments at b = 32), some shorter than a block, any tail
    lens = []
    for _ in range(B):
        kind = rng.integers(0, 10)
        if kind == 0:
            lens.append(int(rng.integers(1, b)))                       # tail only
        elif kind == 1:
            lens.append(int(rng.integers(1, 4)) * b)                    # a few whole blocks, no tail
        else:
            lens.append(int(rng.integers(b, 96 * b if b == 32 else 40 * b)))
    return dict(rng=rng, d=d, b=b, G=G, Hkv=Hkv, B=B, lens=lens,
                scale=float(rng.choice([0.3, 1.0, 3.0])),
                quantile=float(rng.choice([0.0, 0.3, 0.6, 0.9, 0.98])),
                a=float(rng.choice([0.0, 0.0, 0.25, -0.5])),
                z=float(rng.choice([0.0, 0.5, 1.0, 2.5])),
                beta=float(rng.choice([0.0, 1.0, 5.0, 20.0])),
                lwb=int(rng.choice([0, 0, 1, 3])),
                rescue_window=int(rng.choice([1, 2, 128, 1 << 20])),
                ungate_last=bool(rng.integers(0, 2)),
                frozen=bool(rng.integers(0, 3) == 0))


@pytest.mark.parametrize("seed", range(40))
def test_random_configuration_matches_the_oracle(seed):
    eb = _build()
    cfg = _draw(seed)
    rng, d, b, G, Hkv, B, lens = (cfg[k] for k in ("rng", "d", "b", "G", "Hkv", "B", "lens"))
    t_cap = ((max(lens) + b - 1) // b) * b
    K = torch.from_numpy(rng.standard_normal((B, Hkv, t_cap, d)) * cfg["scale"]).to(torch.bfloat16)
    V = torch.from_numpy(rng.standard_normal((B, Hkv, t_cap, d))).to(torch.bfloat16)
    q = torch.from_numpy(rng.standard_normal((B, Hkv * G, d))).to(torch.bfloat16)
    lens = np.asarray(lens, np.int32)
    c = orc.Cache(bits(K), bits(V), lens, b)
    musig, mnorm = orc.block_summaries(c)
    z = cfg["z"]
    bound = orc.score_dual(bits(q), musig, mnorm, lens, b, z)
    # thresholds between two bounds (never on one): per (sequence, head) a quantile of its own bounds, or one value
    # per head over the batch in the frozen mode; sequences without a whole block get 0
    with np.errstate(all="ignore"), warnings.catch_warnings():
        warnings.simplefilter("ignore")
        qt = np.nan_to_num(np.nanquantile(bound, cfg["quantile"], axis=2), nan=0.0)
    qt = qt + cfg["a"] + 3e-4
    kw = dict(z=z, a=cfg["a"], beta=cfg["beta"], lwb=cfg["lwb"], rescue_window=cfg["rescue_window"])
    if cfg["frozen"]:
        head_const = np.median(qt, axis=0).astype(np.float32)
        tau, t_used = None, np.broadcast_to(head_const, (B, Hkv * G))
    else:
        head_const, tau = None, qt.astype(np.float32)
        t_used = tau
    ref = orc.decode_step(bits(q), c, musig, mnorm, tau=tau, head_const=head_const, ungate_last=cfg["ungate_last"], **kw)
    flags = eb.ETA_FLAG_UNGATE_LAST if cfg["ungate_last"] else 0
    out, sel, stats, status = gpu_decode(q, K, V, lens, b, musig, mnorm, tau=tau, head_const=head_const, flags=flags, **kw)
    assert status == 0
    assert not np.isnan(out).any()
    tau_eff = t_used.astype(np.float64) - cfg["a"]
    near = compare_masks(sel, ref["sel"], ref["bound"], tau_eff, lens, b, G, rescued=ref["rescued"])
    keep = heads_without_near_tie(near, B, Hkv * G)
    assert keep.mean() >= 0.75, (len(near), cfg)
    mx, mean = output_errors(out[keep], ref["out"][keep])
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean, {k: v for k, v in cfg.items() if k != "rng"})
    union = np.array([[int((sel[i, hk, :int(lens[i]) // b] != 0).sum()) for hk in range(Hkv)] for i in range(B)])
    assert np.array_equal(stats, union)
    # the dense flag on the same inputs is plain softmax attention over the whole sequence, gate off
    if seed % 4 == 0:
        dense = orc.dense_softmax_attention(bits(q), c)
        out_d, _, _, status = gpu_decode(q, K, V, lens, b, musig, mnorm, tau=tau, head_const=head_const,
                                         flags=eb.ETA_FLAG_DENSE, **kw)
        assert status == 0
        mx, mean = output_errors(out_d, dense)
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)


@pytest.mark.parametrize("B,Hkv,G,d,b,longest", [(1024, 1, 4, 128, 64, 600), (256, 4, 2, 64, 32, 3000),
                                                  (512, 2, 8, 128, 128, 1000)])
def test_many_short_sequences_up_to_the_row_limit(B, Hkv, G, d, b, longest):
    """Up to 1024 (sequence, KV head) rows of 1 .. `longest` tokens: far more rows than streaming CTAs, most pieces a
    tile or two, many rows with a tail only."""
    _build()
    rng = np.random.default_rng(B)
    lens = rng.integers(1, longest, size=B).astype(np.int32)
    t_cap = ((int(lens.max()) + b - 1) // b) * b
    K = torch.from_numpy(rng.standard_normal((B, Hkv, t_cap, d), dtype=np.float32)).to(torch.bfloat16)
    V = torch.from_numpy(rng.standard_normal((B, Hkv, t_cap, d), dtype=np.float32)).to(torch.bfloat16)
    q = torch.from_numpy(rng.standard_normal((B, Hkv * G, d), dtype=np.float32)).to(torch.bfloat16)
    c = orc.Cache(bits(K), bits(V), lens, b)
    musig, mnorm = orc.block_summaries(c)
    bound = orc.score_dual(bits(q), musig, mnorm, lens, b, 1.0)
    with np.errstate(all="ignore"), warnings.catch_warnings():
        warnings.simplefilter("ignore")
        tau = (np.nan_to_num(np.nanquantile(bound, 0.7, axis=2), nan=0.0) + 3e-4).astype(np.float32)
    ref = orc.decode_step(bits(q), c, musig, mnorm, tau=tau, lwb=1, rescue_window=4)
    out, sel, stats, status = gpu_decode(q, K, V, lens, b, musig, mnorm, tau=tau, lwb=1, rescue_window=4)
    assert status == 0 and not np.isnan(out).any()
    near = compare_masks(sel, ref["sel"], ref["bound"], tau.astype(np.float64), lens, b, G, rescued=ref["rescued"])
    keep = heads_without_near_tie(near, B, Hkv * G)
    assert keep.mean() > 0.95
    mx, mean = output_errors(out[keep], ref["out"][keep])
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)
    union = np.array([[int((sel[i, hk, :int(lens[i]) // b] != 0).sum()) for hk in range(Hkv)] for i in range(B)])
    assert np.array_equal(stats, union)

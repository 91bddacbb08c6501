"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element.

Tolerances (bf16 K/V, fp32 accumulation):
  - block summaries: mu, sigma within 1 fp16 ulp, M within 4 fp32 ulp of the fp64 oracle;
  - predicted thresholds: 1e-4 absolute;
  - selected-block masks: bit-exact, except (head, block) pairs whose oracle bound lies within
    1e-5 (absolute) of tau_eff (logged) and rescue choices among bounds tied that closely;
  - outputs: max abs error <= 1e-2 and mean abs error <= 1e-3.
Decode parity feeds the ORACLE's summary bytes and the same fp32 tau array to both sides, so rounding of the
summaries cannot masquerade as a selection bug; the chained path (GPU summaries -> GPU decode) is checked too.
"""
import warnings

import numpy as np
import pytest
import torch

from oracle import eta_oracle as orc
from paper_2609_20888_b200 import workloads as wl
from tests.helpers import (bits, cache_of, calibrate_bias, calibrate_head_const, compare_masks, fp16_ulp_distance,
                           gpu_decode, heads_without_near_tie, output_errors)

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 1e-2, 1e-3


def _eb():
    from paper_2609_20888_b200 import binding as eb
    from paper_2609_20888_b200 import build as ebuild
    ebuild.build()
    eb.load()
    return eb


def _rand_cache_t(seed, B, Hkv, T_list, d, b, t_cap=None, scale=1.0):
    rng = np.random.default_rng(seed)
    t_cap = t_cap or ((max(T_list) + b - 1) // b) * b
    K = torch.from_numpy(rng.standard_normal((B, Hkv, t_cap, d)) * scale).to(torch.bfloat16)
    V = torch.from_numpy(rng.standard_normal((B, Hkv, t_cap, d))).to(torch.bfloat16)
    lens = np.asarray(T_list, np.int32)
    return rng, K, V, lens


# ---------------------------------------------------------------------------------------------------
# summaries
# ---------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("d,b", [(128, 64), (128, 128), (128, 32), (64, 32), (64, 64), (64, 128)])
@pytest.mark.parametrize("envelope", [False, True])
def test_build_block_summaries(d, b, envelope):
    eb = _eb()
    B, Hkv = 3, 2
    lens = [7 * b + 5, 3 * b, b - 1]
    rng, K, V, lens = _rand_cache_t(100 + d + b, B, Hkv, lens, d, b, scale=1.7)
    K[0, 0, :b] *= 30.0                       # wide dynamic range in one block
    K[1, 1, b:2 * b] = K[1, 1, b].clone()     # a block of identical keys: sigma exactly 0
    ref_ms, ref_mn = orc.block_summaries(orc.Cache(bits(K), bits(V), lens, b), envelope=envelope)
    dev = torch.device("cuda:0")
    Kd = K.to(dev)
    desc = eb.cache_desc(Kd, Kd, Hkv * 4, b)
    musig, mnorm = eb.alloc_summaries(desc, dev)
    musig.fill_(-3.0)
    mnorm.fill_(-3.0)
    eb.eta_build_block_summaries(desc, Kd, torch.from_numpy(lens).to(dev), musig, mnorm,
                                 flags=eb.ETA_BUILD_SIGMA_ENVELOPE if envelope else 0)
    torch.cuda.synchronize()
    got_ms = bits(musig.cpu())
    got_mn = mnorm.cpu().numpy()
    for i in range(B):
        NB = int(lens[i]) // b
        assert fp16_ulp_distance(got_ms[i, :, :NB], ref_ms[i, :, :NB]).max(initial=0) <= 1
        a, r = got_mn[i, :, :NB], ref_mn[i, :, :NB]
        assert np.all(np.abs(a.view(np.int32) - r.view(np.int32)) <= 4)
        # records of blocks that are not full stay untouched
        assert np.all(got_mn[i, :, NB:] == -3.0)
        assert np.all(musig[i, :, NB:].cpu().numpy() == -3.0)
    if not envelope:
        assert np.all(got_ms[1, 1, 1, 1] == 0)    # identical keys: sigma is exactly zero


def test_append_equals_rebuild_byte_for_byte():
    eb = _eb()
    d, b, B, Hkv = 128, 64, 4, 2
    rng, K, V, lens = _rand_cache_t(7, B, Hkv, [5 * b - 1, 3 * b - 1, 2 * b + 10, b - 1], d, b, t_cap=8 * b)
    dev = torch.device("cuda:0")
    Kd = K.to(dev)
    desc = eb.cache_desc(Kd, Kd, 8, b)
    musig, mnorm = eb.alloc_summaries(desc, dev)
    lens_d = torch.from_numpy(lens).to(dev)
    eb.eta_build_block_summaries(desc, Kd, lens_d, musig, mnorm)
    before = musig.clone()
    # one more token per sequence: sequences 0, 1, 3 complete a block, sequence 2 does not
    lens_d += 1
    eb.eta_append_summary(desc, Kd, lens_d, musig, mnorm)
    m2, n2 = eb.alloc_summaries(desc, dev)
    eb.eta_build_block_summaries(desc, Kd, lens_d, m2, n2)
    torch.cuda.synchronize()
    assert torch.equal(musig.view(torch.int16), m2.view(torch.int16))
    assert torch.equal(mnorm.view(torch.int32), n2.view(torch.int32))
    assert not torch.equal(before.view(torch.int16), musig.view(torch.int16))
    # idempotent
    eb.eta_append_summary(desc, Kd, lens_d, musig, mnorm)
    torch.cuda.synchronize()
    assert torch.equal(musig.view(torch.int16), m2.view(torch.int16))


# ---------------------------------------------------------------------------------------------------
# predictor and bound
# ---------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("B,Hq,d", [(1, 8, 64), (8, 32, 128), (3, 16, 128)])
def test_predict_threshold(B, Hq, d):
    eb = _eb()
    rng = np.random.default_rng(B + Hq)
    q = torch.from_numpy(rng.standard_normal((B, Hq, d))).to(torch.bfloat16)
    W = (rng.standard_normal((Hq * d, Hq)) * 0.02).astype(np.float32)
    bias = rng.standard_normal(Hq).astype(np.float32)
    ref = orc.predict_threshold(bits(q), W, bias)
    dev = torch.device("cuda:0")
    tau = torch.empty((B, Hq), dtype=torch.float32, device=dev)
    eb.eta_predict_threshold(q.to(dev), torch.from_numpy(W).to(dev), torch.from_numpy(bias).to(dev), tau)
    torch.cuda.synchronize()
    assert np.abs(tau.cpu().numpy() - ref).max() <= 1e-4
    # start-dense initialisation: W = 0, bias = -8
    eb.eta_predict_threshold(q.to(dev), torch.zeros_like(torch.from_numpy(W)).to(dev),
                             torch.full((Hq,), -8.0, device=dev), tau)
    assert torch.all(tau == -8.0)


def test_score_dual_matches_oracle():
    eb = _eb()
    sp = wl.CONFIGS["c2_32k"].scaled(2048 + 37, batch=2)
    w = wl.make_workload(sp)
    c = cache_of(w)
    musig, mnorm = orc.block_summaries(c)
    q = w.queries(0)
    for z in (1.0, 2.5):
        ref = orc.score_dual(bits(q), musig, mnorm, c.seq_lens, sp.block_size, z)
        dev = torch.device("cuda:0")
        Kd = w.K.to(dev)
        desc = eb.cache_desc(Kd, Kd, sp.n_q_heads, sp.block_size)
        bound = torch.full((sp.batch, sp.n_q_heads, desc.nb_cap), float("nan"), device=dev)
        eb.eta_score_dual(desc, eb.DecodeParams(z=z), q.to(dev), torch.from_numpy(c.seq_lens).to(dev),
                          torch.from_numpy(musig.view(np.int16)).view(torch.float16).to(dev),
                          torch.from_numpy(mnorm).to(dev), bound)
        got = bound.cpu().numpy()
        NB = int(c.seq_lens[0]) // sp.block_size
        assert np.abs(got[:, :, :NB] - ref[:, :, :NB]).max() <= 1e-5 * max(1.0, np.abs(ref[:, :, :NB]).max())
        assert np.all(np.isnan(got[:, :, NB:]))


# ---------------------------------------------------------------------------------------------------
# decode: oracle summaries + the same tau on both sides
# ---------------------------------------------------------------------------------------------------

def _decode_case(w, q, tau=None, head_const=None, **params):
    """Run both sides; -> (errors, near-ties, selection stats)."""
    sp = w.spec
    c = cache_of(w)
    musig, mnorm = orc.block_summaries(c)
    params = dict(params)
    ungate = params.pop("ungate_last", False)
    ref = orc.decode_step(bits(q), c, musig, mnorm, tau=tau, head_const=head_const, z=params.get("z", 1.0),
                          a=params.get("a", 0.0), beta=params.get("beta", 5.0), lwb=params.get("lwb", 0),
                          rescue_window=params.get("rescue_window", 128), ungate_last=ungate)
    if ungate:
        params["flags"] = params.get("flags", 0) | _eb().ETA_FLAG_UNGATE_LAST
    out, sel, stats, status = gpu_decode(q, w.K, w.V, c.seq_lens, sp.block_size, musig, mnorm, tau=tau,
                                         head_const=head_const, **params)
    assert status == 0
    assert not np.isnan(out).any()
    t = np.broadcast_to(head_const, (sp.batch, sp.n_q_heads)) if tau is None else tau
    tau_eff = t.astype(np.float64) - params.get("a", 0.0)
    near = compare_masks(sel, ref["sel"], ref["bound"], tau_eff, c.seq_lens, sp.block_size, sp.gqa,
                         rescued=ref["rescued"])
    # heads with a logged near-tie attend a different block set: leave them out of the output comparison
    keep = heads_without_near_tie(near, sp.batch, sp.n_q_heads)
    assert keep.mean() > 0.9
    mx, mean = output_errors(out[keep], ref["out"][keep])
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)
    # union blocks per KV head as reported by the library
    union = np.array([[int((sel[i, hk, :int(c.seq_lens[i]) // sp.block_size] != 0).sum())
                       for hk in range(sp.n_kv_heads)] for i in range(sp.batch)])
    assert np.array_equal(stats, union)
    return (mx, mean), near, ref


def _calibrated_tau(w, q, target):
    sp = w.spec
    c = cache_of(w)
    musig, mnorm = orc.block_summaries(c)
    bound = orc.score_dual(bits(q), musig, mnorm, c.seq_lens, sp.block_size, sp.z)
    tau_raw = orc.predict_threshold(bits(q), w.W.numpy(), np.zeros(sp.n_q_heads, np.float32))
    bias = calibrate_bias(bound, tau_raw, c.seq_lens, sp.block_size, sp.gqa, target)
    return orc.predict_threshold(bits(q), w.W.numpy(), bias).astype(np.float32), bound


CASES = [
    ("c1_tiny", 2048 + 16, 1, dict()),                       # tail of 16 tokens, d=64, b=32
    ("c1_tiny", 2048, 1, dict(lwb=2)),
    ("c2_32k", 4096 + 77, 3, dict(lwb=2)),                   # ragged tail, several segments
    ("c2_32k", 2048, 2, dict(a=0.4, z=1.5)),
    ("c3_128k", 8192, 2, dict()),
    ("c4_512k", 16384 + 100, 1, dict(lwb=1)),                # b=128: two tiles per block, 100-token tail
    ("c5_frozen", 8192, 4, dict()),                          # mixed lengths
]


@pytest.mark.parametrize("name,ctx,batch,params", CASES)
def test_decode_matches_oracle_on_scaled_configs(name, ctx, batch, params):
    _eb()
    base = wl.CONFIGS[name]
    sp = base.scaled(ctx, batch=batch, min_context=ctx // 4 if base.min_context else None)
    w = wl.make_workload(sp)
    q = w.queries(0)
    for target in sp.target_sparsity:
        tau, _ = _calibrated_tau(w, q, target)
        kw = dict(z=sp.z, beta=sp.beta)
        kw.update(params)
        (mx, mean), near, ref = _decode_case(w, q, tau=tau, **kw)
        print(f"{name} ctx={ctx} target={target}: max {mx:.2e} mean {mean:.2e} near-ties {len(near)}")


@pytest.mark.parametrize("name,ctx,batch", [("c2_32k", 4096, 2), ("c2_32k", 4096 + 77, 2), ("c4_512k", 16384, 1),
                                            ("c4_512k", 16384 + 100, 1), ("c1_tiny", 2048 + 16, 1), ("c1_tiny", 2048, 1)])
def test_ungated_newest_token(name, ctx, batch):
    """ETA_FLAG_UNGATE_LAST: the newest token keeps its raw logit; when it closes a block the block is admitted.
    Contexts that end on a block boundary and in a tail, one and two tiles per block."""
    _eb()
    sp = wl.CONFIGS[name].scaled(ctx, batch=batch)
    w = wl.make_workload(sp)
    q = w.queries(0)
    tau, _ = _calibrated_tau(w, q, 0.9)
    (mx, mean), near, ref = _decode_case(w, q, tau=tau, z=sp.z, beta=sp.beta, ungate_last=True)
    if ctx % sp.block_size == 0:
        NB = ctx // sp.block_size
        assert np.all(ref["sel"][:, :, NB - 1] == (1 << sp.gqa) - 1)
    # an infinite threshold closes every other gate: the newest token then dominates in closed form (oracle pin);
    # here: both sides agree on it
    inf = np.full_like(tau, np.inf)
    (_, _), _, r1 = _decode_case(w, q, tau=inf, z=sp.z, beta=sp.beta, ungate_last=True)
    (_, _), _, r0 = _decode_case(w, q, tau=inf, z=sp.z, beta=sp.beta)
    assert np.abs(r1["out"] - r0["out"]).max() > 1e-6            # here the flag does change the result


def test_frozen_constants_against_predicted_mode_on_the_same_cache():
    _eb()
    sp = wl.CONFIGS["c5_frozen"].scaled(8192, batch=4, min_context=2048)
    w = wl.make_workload(sp)
    q = w.queries(0)
    c = cache_of(w)
    musig, mnorm = orc.block_summaries(c)
    bound = orc.score_dual(bits(q), musig, mnorm, c.seq_lens, sp.block_size, sp.z)
    consts = calibrate_head_const(bound, c.seq_lens, sp.block_size, wl.frozen_sparsity_levels(sp))
    (_, _), near, ref = _decode_case(w, q, head_const=consts)
    dens = np.array([[(ref["sel"][i, h // sp.gqa, :int(c.seq_lens[i]) // sp.block_size] >> (h % sp.gqa) & 1).mean()
                      for h in range(sp.n_q_heads)] for i in range(sp.batch)]).mean(axis=0)
    assert dens.min() < 0.2 and dens.max() > 0.5          # heads span a wide range of sparsity
    tau, _ = _calibrated_tau(w, q, 0.7)
    _decode_case(w, q, tau=tau)


def test_minus_infinite_threshold_and_dense_flag_are_softmax_attention():
    eb = _eb()
    sp = wl.CONFIGS["c2_32k"].scaled(1024 + 13, batch=2)
    w = wl.make_workload(sp)
    q = w.queries(0)
    c = cache_of(w)
    dense = orc.dense_softmax_attention(bits(q), c)
    tau = np.full((sp.batch, sp.n_q_heads), -np.inf, np.float32)
    (mx, mean), near, ref = _decode_case(w, q, tau=tau)
    assert not near and np.all(ref["sel"][:, :, :16] == 0x0f)
    musig, mnorm = orc.block_summaries(c)
    for flags, t in ((0, tau), (eb.ETA_FLAG_DENSE, np.zeros_like(tau))):
        out, sel, _, status = gpu_decode(q, w.K, w.V, c.seq_lens, sp.block_size, musig, mnorm, tau=t, flags=flags)
        assert status == 0
        mx, mean = output_errors(out, dense)
        assert mx <= MAX_ABS and mean <= MEAN_ABS
        assert np.all(sel[:, :, :16] == 0x0f) and np.all(sel[:, :, 16:] == 0)


def test_plus_infinite_threshold_attends_rescue_pins_and_tail_only():
    _eb()
    sp = wl.CONFIGS["c3_128k"].scaled(4096 + 5, batch=2)
    w = wl.make_workload(sp)
    q = w.queries(0)
    tau = np.full((sp.batch, sp.n_q_heads), np.inf, np.float32)
    for rw, lwb in ((128, 0), (16, 2), (1 << 30, 0), (1 << 30, 1)):
        (_, _), near, ref = _decode_case(w, q, tau=tau, rescue_window=rw, lwb=lwb)
        cnt = np.array([bin(int(x)).count("1") for x in ref["sel"].ravel()]).sum()
        expect_rescues = 0 if (lwb and rw > 64) else sp.batch * sp.n_q_heads
        assert cnt == sp.batch * sp.n_q_heads * lwb + expect_rescues


def test_rescue_window_longer_than_four_segments_and_many_segment_counts():
    """Two loops of the streaming kernel's set-up that ordinary shapes do not enter: a rescue window of more than
    4 x 64 blocks (its statistics are then combined in rounds of four segments), and more segment counts than one
    pass of the set-up loads (8 per thread x 416 threads = 3328; here 64 rows x 56 segments = 3584)."""
    _eb()
    d, b, B, Hkv, G = 64, 32, 8, 8, 1
    T = 32 * 64 * 56
    rng, K, V, lens = _rand_cache_t(77, B, Hkv, [T] * B, d, b)
    lens = lens.copy()
    lens[1] = T - 5 * b - 3                     # a shorter row with a tail, so that rows differ
    q = torch.from_numpy(rng.standard_normal((B, Hkv * G, d))).to(torch.bfloat16)
    c = orc.Cache(bits(K), bits(V), lens, b)
    musig, mnorm = orc.block_summaries(c)
    bound = orc.score_dual(bits(q), musig, mnorm, lens, b, 1.0)
    # (a) a threshold nothing passes, the whole sequence as rescue window: the global argmax of 3584 bounds per head
    inf = np.full((B, Hkv * G), np.inf, np.float32)
    ref = orc.decode_step(bits(q), c, musig, mnorm, tau=inf, rescue_window=1 << 30)
    out, sel, stats, status = gpu_decode(q, K, V, lens, b, musig, mnorm, tau=inf, rescue_window=1 << 30)
    assert status == 0
    assert np.array_equal(sel, ref["sel"])
    first = np.array([[int(np.nanargmax(bound[i, h, :int(lens[i]) // b])) for h in range(Hkv * G)] for i in range(B)])
    assert np.array_equal(ref["rescued"], first) and (first >= 4 * 64).any()
    mx, mean = output_errors(out, ref["out"])
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)
    # (b) an ordinary sparse step on the same shape
    tau = (np.nanquantile(bound, 0.95, axis=2) + 1e-4).astype(np.float32)
    ref = orc.decode_step(bits(q), c, musig, mnorm, tau=tau, rescue_window=1000)
    out, sel, stats, status = gpu_decode(q, K, V, lens, b, musig, mnorm, tau=tau, rescue_window=1000)
    assert status == 0
    near = compare_masks(sel, ref["sel"], ref["bound"], tau.astype(np.float64), lens, b, G, rescued=ref["rescued"])
    keep = heads_without_near_tie(near, B, Hkv * G)
    assert keep.mean() > 0.9
    mx, mean = output_errors(out[keep], ref["out"][keep])
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)
    union = np.array([[int((sel[i, hk, :int(lens[i]) // b] != 0).sum()) for hk in range(Hkv)] for i in range(B)])
    assert np.array_equal(stats, union)


EDGE = [
    dict(d=128, b=64, lens=[1]),                    # a single token: tail only
    dict(d=128, b=64, lens=[63, 64, 65]),           # just below / at / above one block
    dict(d=64, b=32, lens=[31, 32, 33, 95]),
    dict(d=128, b=128, lens=[127, 128, 129, 300]),
    dict(d=128, b=64, lens=[64 * 70]),              # exact multiple, more than one segment, no tail
    dict(d=64, b=64, lens=[64 * 3 + 1, 5]),
]


@pytest.mark.parametrize("case", EDGE)
@pytest.mark.parametrize("G", [1, 2, 4, 8])
def test_edge_shapes_and_group_sizes(case, G):
    _eb()
    d, b, lens = case["d"], case["b"], case["lens"]
    B, Hkv = len(lens), 2
    rng, K, V, lens = _rand_cache_t(hash((d, b, G)) % 1000, B, Hkv, lens, d, b)
    q = torch.from_numpy(rng.standard_normal((B, Hkv * G, d))).to(torch.bfloat16)
    c = orc.Cache(bits(K), bits(V), lens, b)
    musig, mnorm = orc.block_summaries(c)
    bound = orc.score_dual(bits(q), musig, mnorm, lens, b, 1.0)
    with np.errstate(all="ignore"), warnings.catch_warnings():
        warnings.simplefilter("ignore")
        tau = np.nan_to_num(np.nanmedian(bound, axis=2), nan=0.0).astype(np.float32)
    for params in (dict(), dict(lwb=1, rescue_window=2)):
        ref = orc.decode_step(bits(q), c, musig, mnorm, tau=tau, **params)
        out, sel, stats, status = gpu_decode(q, K, V, lens, b, musig, mnorm, tau=tau, **params)
        assert status == 0
        near = compare_masks(sel, ref["sel"], ref["bound"], tau.astype(np.float64), lens, b, G, rescued=ref["rescued"])
        # (the median of a few bounds IS one of them, rounded to fp32: these thresholds sit within an fp32 rounding of a
        # bound on purpose, so several heads may log a near tie; their outputs are left out, the others compared)
        keep = heads_without_near_tie(near, B, Hkv * G)
        assert keep.mean() >= 0.5
        mx, mean = output_errors(out[keep], ref["out"][keep])
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)


@pytest.mark.parametrize("d,b,G", [(64, 32, 4), (128, 64, 4), (128, 64, 8), (64, 64, 2)])
def test_threshold_equal_to_a_bound_admits_the_block_on_the_device(d, b, G):
    """Algorithm 3 admits a block when its bound is >= tau_eff: equality admits.  Here the bounds are exactly
    representable on both sides, so thresholds can be SET EQUAL to bounds: every key of a block is the same
    small-integer vector (sigma = 0, centroid = the key, so the moment term is the centroid logit), the queries are
    small integers, and the scale is 1/8 (a power of two); the sphere term never binds (<q,k> <= |q||k|).  Then
    bound = <q,k>/8 with no rounding anywhere, in fp64, in fp32 and through the fp16 tensor-core product alike.
    The masks must agree bit for bit with no near tie to excuse anything; the next fp32 number above the threshold
    must drop exactly the blocks that sat on it; and with tau = +inf the rescue must take the FIRST of the many
    blocks tied at the largest bound."""
    _eb()
    B, Hkv, NB, tail = 2, 2, 75, 5
    rng = np.random.default_rng(d * 7 + b + G)
    T = NB * b + tail
    kvec = rng.integers(-3, 4, size=(B, Hkv, NB + 1, d)).astype(np.float64)
    K = torch.from_numpy(np.repeat(kvec, b, axis=2)[:, :, :((T + b - 1) // b) * b]).to(torch.bfloat16)
    V = torch.from_numpy(rng.standard_normal(K.shape)).to(torch.bfloat16)
    q = torch.from_numpy(rng.integers(-2, 3, size=(B, Hkv * G, d)).astype(np.float64)).to(torch.bfloat16)
    lens = np.full(B, T, np.int32)
    c = orc.Cache(bits(K), bits(V), lens, b)
    musig, mnorm = orc.block_summaries(c)
    assert not musig[:, :, :NB, 1].any()                      # sigma is exactly zero
    bound = orc.score_dual(bits(q), musig, mnorm, lens, b, 1.0, scale=0.125)
    # the bound is the integer dot product over 8, exactly
    for i in range(B):
        for h in range(Hkv * G):
            dots = kvec[i, h // G, :NB] @ q[i, h].double().numpy()
            assert np.array_equal(bound[i, h, :NB], dots / 8.0)
    # thresholds ON a bound: the 60th-percentile block's value (shared by several blocks: integers tie often)
    tau = np.sort(bound[:, :, :NB], axis=2)[:, :, int(0.6 * NB)].astype(np.float32)
    assert np.array_equal(tau.astype(np.float64), np.sort(bound[:, :, :NB], axis=2)[:, :, int(0.6 * NB)])
    on_tau = bound[:, :, :NB] == tau[:, :, None]
    assert on_tau.any(axis=2).all() and on_tau.sum() > B * Hkv * G
    above = np.nextafter(tau, np.float32(np.inf))
    for t, admits_equal in ((tau, True), (above, False), (np.full_like(tau, np.inf), None)):
        ref = orc.decode_step(bits(q), c, musig, mnorm, tau=t, scale=0.125)
        out, sel, stats, status = gpu_decode(q, K, V, lens, b, musig, mnorm, tau=t, scale=0.125)
        assert status == 0
        assert np.array_equal(sel, ref["sel"]), "masks differ although every bound is exact"
        if admits_equal is not None:
            for i in range(B):
                for h in range(Hkv * G):
                    bits_h = (sel[i, h // G, :NB] >> (h % G)) & 1
                    assert np.all(bits_h[on_tau[i, h]] == (1 if admits_equal else 0))
                    assert np.all(bits_h[bound[i, h, :NB] > t[i, h]] == 1)
        else:
            # rescue: the first block attaining the largest bound of the window, per head
            first = np.argmax(bound[:, :, :NB], axis=2)
            assert np.array_equal(ref["rescued"], first)
            for i in range(B):
                for h in range(Hkv * G):
                    assert (sel[i, h // G, first[i, h]] >> (h % G)) & 1
        mx, mean = output_errors(out, ref["out"])
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)


@pytest.mark.parametrize("d,G", [(128, 4), (64, 4)])
def test_query_magnitudes_outside_the_fp16_range_screen_like_their_scaled_twins(d, G):
    """Score_dual is positively homogeneous: scaling a head's query and its threshold by 2^k scales every bound by
    2^k, exactly, in any binary floating-point format.  At head_dim 128 with four heads per group the centroid term
    runs on the tensor cores with fp16 operands, which hold neither bf16 values above 65504 nor tiny ones: the
    kernel normalises each head's query by a power of two first, so the selection must not depend on k.  Heads are
    scaled by 2^17 (components beyond fp16's largest number), 2^-40 (far below its smallest), 1 and 2^9; the
    masks must equal those of the unscaled call bit for bit, and agree with the oracle run on the scaled inputs
    (near-tie band scaled with the head, as every bound is)."""
    _eb()
    b, B, Hkv = 64, 2, 2
    rng, K, V, lens = _rand_cache_t(31 + d, B, Hkv, [64 * 70 + 9, 64 * 33], d, b)
    q = torch.from_numpy(rng.standard_normal((B, Hkv * G, d))).to(torch.bfloat16)
    c = orc.Cache(bits(K), bits(V), lens, b)
    musig, mnorm = orc.block_summaries(c)
    bound = orc.score_dual(bits(q), musig, mnorm, lens, b, 1.0)
    tau = (np.nanquantile(bound, 0.8, axis=2) + 1e-4).astype(np.float32)
    ks = np.array([17, -40, 0, 9] * (Hkv * G // 4))
    scale = np.ldexp(1.0, ks)
    q_s = (q.float() * torch.from_numpy(scale).float()[None, :, None]).to(torch.bfloat16)
    assert torch.equal(q_s.float(), q.float() * torch.from_numpy(scale).float()[None, :, None])     # exact in bf16
    assert float(q_s.float().abs().max()) > 65504.0
    tau_s = (tau.astype(np.float64) * scale[None, :]).astype(np.float32)
    _, sel0, _, status0 = gpu_decode(q, K, V, lens, b, musig, mnorm, tau=tau)
    out1, sel1, _, status1 = gpu_decode(q_s, K, V, lens, b, musig, mnorm, tau=tau_s)
    assert status0 == 0 and status1 == 0 and np.isfinite(out1).all()
    assert np.array_equal(sel0, sel1), "the selection depends on the magnitude of the query"
    ref = orc.decode_step(bits(q_s), c, musig, mnorm, tau=tau_s)
    diff = sel1 ^ ref["sel"]
    for i, hk, j in zip(*np.nonzero(diff)):
        for g in range(G):
            if (diff[i, hk, j] >> g) & 1:
                h = hk * G + g
                assert abs(ref["bound"][i, h, j] - float(tau_s[i, h])) <= 1e-5 * scale[h], (i, h, j)
    assert 0.05 < float((sel1 != 0).mean()) < 0.9


def test_sphere_term_binds_and_large_logits_stay_finite():
    _eb()
    # a z-score above sqrt(d): the moment term exceeds the Cauchy-Schwarz ceiling, so the sphere term decides
    d, b, B, Hkv, G = 128, 64, 1, 2, 4
    rng, K, V, lens = _rand_cache_t(5, B, Hkv, [64 * 40 + 9], d, b, scale=4.0)
    q = torch.from_numpy(rng.standard_normal((B, Hkv * G, d)) * 3.0).to(torch.bfloat16)
    c = orc.Cache(bits(K), bits(V), lens, b)
    musig, mnorm = orc.block_summaries(c)
    bound, g, s = orc.score_dual(bits(q), musig, mnorm, lens, b, 20.0, parts=True)
    assert (s[:, :, :40] < g[:, :, :40]).mean() > 0.5
    tau = np.quantile(bound[:, :, :40], 0.7, axis=2).astype(np.float32)
    ref = orc.decode_step(bits(q), c, musig, mnorm, tau=tau, z=20.0)
    out, sel, _, status = gpu_decode(q, K, V, lens, b, musig, mnorm, tau=tau, z=20.0)
    assert status == 0
    near = compare_masks(sel, ref["sel"], ref["bound"], tau.astype(np.float64), lens, b, G, rescued=ref["rescued"])
    keep = heads_without_near_tie(near, B, Hkv * G)
    mx, mean = output_errors(out[keep], ref["out"][keep])
    assert mx <= MAX_ABS and mean <= MEAN_ABS


def test_strided_cache_layout_bthd():
    """K/V stored [batch, t, kv_head, d] (token-major): only the strides in the descriptor change."""
    eb = _eb()
    d, b, B, Hkv, G, T = 128, 64, 2, 2, 4, 64 * 9 + 20
    rng, K, V, lens = _rand_cache_t(11, B, Hkv, [T, T - 70], d, b)
    q = torch.from_numpy(rng.standard_normal((B, Hkv * G, d))).to(torch.bfloat16)
    c = orc.Cache(bits(K), bits(V), lens, b)
    musig, mnorm = orc.block_summaries(c)
    bound = orc.score_dual(bits(q), musig, mnorm, lens, b, 1.0)
    tau = np.nanquantile(bound, 0.6, axis=2).astype(np.float32)
    ref = orc.decode_step(bits(q), c, musig, mnorm, tau=tau)
    dev = torch.device("cuda:0")
    Kd = K.permute(0, 2, 1, 3).contiguous().to(dev).permute(0, 2, 1, 3)     # logical [B,Hkv,T,d], memory [B,T,Hkv,d]
    Vd = V.permute(0, 2, 1, 3).contiguous().to(dev).permute(0, 2, 1, 3)
    assert Kd.stride(2) == Hkv * d and Kd.stride(1) == d
    st = eb.DecodeState(Kd, Vd, Hkv * G, b)
    lens_d = torch.from_numpy(lens).to(dev)
    eb.eta_build_block_summaries(st.desc, Kd, lens_d, st.musig, st.mnorm)
    torch.cuda.synchronize()
    NBs = [int(x) // b for x in lens]
    got = bits(st.musig.cpu())
    for i in range(B):
        assert fp16_ulp_distance(got[i, :, :NBs[i]], musig[i, :, :NBs[i]]).max() <= 1
    st.musig.copy_(torch.from_numpy(musig.view(np.int16)).view(torch.float16).to(dev))
    st.mnorm.copy_(torch.from_numpy(mnorm).to(dev))
    eb.eta_decode(st.desc, eb.DecodeParams(), q.to(dev), Kd, Vd, lens_d, st.musig, st.mnorm,
                  torch.from_numpy(tau).to(dev), None, st.out, st.sel_mask, st.workspace, status=st.status)
    torch.cuda.synchronize()
    assert int(st.status.item()) == 0
    near = compare_masks(st.sel_mask.cpu().numpy(), ref["sel"], ref["bound"], tau.astype(np.float64), lens, b, G,
                         rescued=ref["rescued"])
    keep = heads_without_near_tie(near, B, Hkv * G)
    assert keep.mean() > 0.7
    mx, mean = output_errors(st.out.cpu().numpy()[keep], ref["out"][keep])
    assert mx <= MAX_ABS and mean <= MEAN_ABS


def test_chained_gpu_path_and_multi_step_append():
    """Prefill build -> 16+ decode steps appending to the cache (crossing a block boundary), everything on the GPU,
    against the oracle run on the same growing cache.  Summary rounding may flip a selection only at a near-tie."""
    eb = _eb()
    sp = wl.CONFIGS["c1_tiny"]
    w = wl.make_workload(sp)
    dev = torch.device("cuda:0")
    K, V = w.K.clone(), w.V.clone()
    Kd, Vd = K.to(dev), V.to(dev)
    st = eb.DecodeState(Kd, Vd, sp.n_q_heads, sp.block_size)
    lens = w.seq_lens.numpy().astype(np.int32).copy()
    lens_d = torch.from_numpy(lens).to(dev)
    eb.eta_build_block_summaries(st.desc, Kd, lens_d, st.musig, st.mnorm)
    Wd = w.W.to(dev)
    q0 = w.queries(0)
    tau0, _ = _calibrated_tau(w, q0, sp.target_sparsity[0])
    bias = (tau0 - orc.predict_threshold(bits(q0), w.W.numpy(), np.zeros(sp.n_q_heads, np.float32)))[0].astype(np.float32)
    bias_d = torch.from_numpy(bias).to(dev)
    total_near = 0
    for step in range(0, 33):
        if step > 0:
            k_t, v_t = w.new_kv(step)
            for i in range(sp.batch):
                K[i, :, lens[i]] = k_t[i]
                V[i, :, lens[i]] = v_t[i]
                Kd[i, :, lens[i]] = k_t[i].to(dev)
                Vd[i, :, lens[i]] = v_t[i].to(dev)
            lens += 1
            lens_d += 1
            eb.eta_append_summary(st.desc, Kd, lens_d, st.musig, st.mnorm)
        q = w.queries(step)
        qd = q.to(dev)
        eb.eta_predict_threshold(qd, Wd, bias_d, st.tau)
        eb.eta_decode(st.desc, eb.DecodeParams(z=sp.z, beta=sp.beta), qd, Kd, Vd, lens_d, st.musig, st.mnorm, st.tau,
                      None, st.out, st.sel_mask, st.workspace, status=st.status)
        torch.cuda.synchronize()
        assert int(st.status.item()) == 0
        c = orc.Cache(bits(K), bits(V), lens.copy(), sp.block_size)
        musig, mnorm = orc.block_summaries(c)
        tau_ref = orc.predict_threshold(bits(q), w.W.numpy(), bias)
        assert np.abs(st.tau.cpu().numpy() - tau_ref).max() <= 1e-4
        # the oracle takes the same fp32 thresholds the kernels used? No: it takes ITS OWN prediction, rounded
        ref = orc.decode_step(bits(q), c, musig, mnorm, tau=tau_ref.astype(np.float32), z=sp.z, beta=sp.beta)
        near = compare_masks(st.sel_mask.cpu().numpy(), ref["sel"], ref["bound"], tau_ref, lens, sp.block_size, sp.gqa,
                             band=2e-3, rescued=ref["rescued"])   # wider band: fp16 summary ulp and fp32 tau differ
        total_near += len(near)
        keep = heads_without_near_tie(near, sp.batch, sp.n_q_heads)
        mx, mean = output_errors(st.out.cpu().numpy()[keep], ref["out"][keep])
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (step, mx, mean)
    assert lens[0] == 2048 + 32 and total_near <= 8


def test_run_to_run_determinism():
    _eb()
    sp = wl.CONFIGS["c3_128k"].scaled(16384, batch=2)
    w = wl.make_workload(sp)
    q = w.queries(0)
    tau, _ = _calibrated_tau(w, q, 0.9)
    c = cache_of(w)
    musig, mnorm = orc.block_summaries(c)
    outs = [gpu_decode(q, w.K, w.V, c.seq_lens, sp.block_size, musig, mnorm, tau=tau) for _ in range(3)]
    for o in outs[1:]:
        assert np.array_equal(o[0].view(np.int32), outs[0][0].view(np.int32))
        assert np.array_equal(o[1], outs[0][1])


def test_query_staged_from_pinned_memory_and_output_written_to_it():
    """The host-facing variant of a step: the query is fetched from page-locked host memory by eta_stage_query and
    the merge kernel stores the output into page-locked host memory.  Same bits as the device-resident step, and the
    same agreement with the oracle."""
    eb = _eb()
    dev = torch.device("cuda:0")
    sp = wl.CONFIGS["c2_32k"].scaled(4096 + 33, batch=2)
    w = wl.make_workload(sp)
    q = w.queries(0)
    tau, _ = _calibrated_tau(w, q, 0.85)
    c = cache_of(w)
    musig, mnorm = orc.block_summaries(c)
    ref_out, ref_sel, _, status = gpu_decode(q, w.K, w.V, c.seq_lens, sp.block_size, musig, mnorm, tau=tau)
    assert status == 0

    K, V = w.K.to(dev), w.V.to(dev)
    st = eb.DecodeState(K, V, sp.n_q_heads, sp.block_size)
    st.musig.copy_(torch.from_numpy(musig.view(np.int16)).view(torch.float16).to(dev))
    st.mnorm.copy_(torch.from_numpy(mnorm).to(dev))
    lens = torch.from_numpy(np.asarray(c.seq_lens, np.int32)).to(dev)
    tau_d = torch.from_numpy(np.ascontiguousarray(tau, np.float32)).to(dev)
    q_host = q.contiguous().pin_memory()
    q_dev = torch.zeros_like(q_host, device=dev)
    out_host = torch.full((sp.batch, sp.n_q_heads, sp.head_dim), float("nan"), dtype=torch.float32).pin_memory()
    eb.eta_stage_query(q_host, q_dev)
    eb.eta_decode(st.desc, eb.DecodeParams(), q_dev, K, V, lens, st.musig, st.mnorm, tau_d, None, out_host,
                  st.sel_mask, st.workspace, stats=st.stats, status=st.status)
    torch.cuda.synchronize()
    assert int(st.status.item()) == 0
    assert torch.equal(q_dev.cpu().view(torch.int16), q_host.view(torch.int16))
    assert np.array_equal(out_host.numpy().view(np.int32), ref_out.view(np.int32))
    assert np.array_equal(st.sel_mask.cpu().numpy(), ref_sel)
    # and the unaligned / wrong-kind arguments are refused
    with pytest.raises(eb.EtaError):
        eb.eta_stage_query(q.contiguous(), q_dev)           # pageable host memory

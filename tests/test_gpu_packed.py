"""Packed block summaries (format sigma8: centroid fp16, sigma rounded up to e4m3; the paper's outlook names "FP8
metadata") on the GPU against the CPU oracle.

Tolerances: the centroid within 1 fp16 ulp; sigma's code within one e4m3 code, and different in under 2 % of the
coordinates (the kernel rounds up the sigma it computed in fp32, the oracle the one it computed in double: the codes
differ only where a representable value lies between the two); M within 4 fp32 ulp.  Decode parity feeds the
ORACLE's packed bytes and the same fp32 thresholds to both sides: masks bit-exact outside the 1e-5 near-tie band,
block counts exact, outputs within 1e-2 max / 1e-3 mean.
"""
import numpy as np
import pytest
import torch

from oracle import eta_oracle as orc
from paper_2609_20888_b200 import workloads as wl
from tests.helpers import bits, cache_of, compare_masks, fp16_ulp_distance, heads_without_near_tie, output_errors

pytestmark = pytest.mark.gpu


def _eb():
    from paper_2609_20888_b200 import binding as eb
    from paper_2609_20888_b200 import build as ebuild
    ebuild.build()
    eb.load()
    return eb


def _rand_cache_t(seed, B, Hkv, T_list, d, b, scale=1.0):
    rng = np.random.default_rng(seed)
    t_cap = ((max(T_list) + b - 1) // b) * b
    K = torch.from_numpy(rng.standard_normal((B, Hkv, t_cap, d)) * scale).to(torch.bfloat16)
    V = torch.from_numpy(rng.standard_normal((B, Hkv, t_cap, d))).to(torch.bfloat16)
    return rng, K, V, np.asarray(T_list, np.int32)


@pytest.mark.parametrize("d,b", [(128, 64), (64, 32), (128, 128), (64, 64)])
@pytest.mark.parametrize("envelope", [False, True])
def test_packed_build_and_append_against_the_oracle(d, b, envelope):
    eb = _eb()
    B, Hkv = 3, 2
    rng, K, V, lens = _rand_cache_t(300 + d + b, B, Hkv, [6 * b + 5, 3 * b, b - 1], d, b, scale=1.3)
    K[0, 0, :b] *= 25.0                       # a block with a wide dynamic range (sigma far above 1)
    K[0, 1, b:2 * b] *= 1e-3                  # and one with a tiny spread
    K[1, 1, b:2 * b] = K[1, 1, b].clone()     # identical keys: sigma exactly 0, code 0
    c = orc.Cache(bits(K), bits(V), lens, b)
    ref8, ref_mn = orc.block_summaries_sigma8(c, envelope=envelope)
    dev = torch.device("cuda:0")
    Kd = K.to(dev)
    desc = eb.cache_desc(Kd, Kd, Hkv * 4, b)
    musig, mnorm = eb.alloc_summaries(desc, dev, packed=True)
    musig.fill_(0xee)
    flags = eb.ETA_BUILD_PACKED_SIGMA | (eb.ETA_BUILD_SIGMA_ENVELOPE if envelope else 0)
    lens_d = torch.from_numpy(lens).to(dev)
    eb.eta_build_block_summaries(desc, Kd, lens_d, musig, mnorm, flags=flags)
    torch.cuda.synchronize()
    got, got_mn = musig.cpu().numpy(), mnorm.cpu().numpy()
    for i in range(B):
        NB = int(lens[i]) // b
        mu_g = got[i, :, :NB, :2 * d].copy().view(np.uint16)
        mu_r = ref8[i, :, :NB, :2 * d].copy().view(np.uint16)
        assert fp16_ulp_distance(mu_g, mu_r).max(initial=0) <= 1
        dc = got[i, :, :NB, 2 * d:].astype(np.int32) - ref8[i, :, :NB, 2 * d:].astype(np.int32)
        assert np.abs(dc).max(initial=0) <= 1, "sigma codes differ by more than one e4m3 step"
        assert (dc != 0).mean() < 0.02 if dc.size else True
        assert np.abs(got_mn[i, :, :NB].view(np.int32) - ref_mn[i, :, :NB].view(np.int32)).max(initial=0) <= 4
        assert np.all(got[i, :, NB:] == 0xee)                    # records of blocks that are not full stay untouched
    if not envelope:
        assert not got[1, 1, 1, 2 * d:].any()                    # identical keys: sigma code 0
    # append == rebuild, byte for byte, in the packed layout too
    K2 = K.clone()
    lens2 = lens.copy()
    for i in range(B):                                           # grow every sequence to its next block boundary
        lens2[i] = ((int(lens[i]) // b) + 1) * b if int(lens[i]) % b else int(lens[i]) + b
    t_cap2 = int(lens2.max())
    if t_cap2 > K.shape[2]:
        pad = torch.from_numpy(rng.standard_normal((B, Hkv, t_cap2 - K.shape[2], d))).to(torch.bfloat16)
        K2 = torch.cat([K, pad], dim=2)
    Kd2 = K2.to(dev)
    desc2 = eb.cache_desc(Kd2, Kd2, Hkv * 4, b)
    m_a, n_a = eb.alloc_summaries(desc2, dev, packed=True)
    m_b, n_b = eb.alloc_summaries(desc2, dev, packed=True)
    lens2_d = torch.from_numpy(lens2).to(dev)
    eb.eta_build_block_summaries(desc2, Kd2, lens2_d, m_b, n_b, flags=flags)
    before = lens2 - b
    eb.eta_build_block_summaries(desc2, Kd2, torch.from_numpy(before.astype(np.int32)).to(dev), m_a, n_a, flags=flags)
    eb.eta_append_summary(desc2, Kd2, lens2_d, m_a, n_a, flags=flags)
    torch.cuda.synchronize()
    assert torch.equal(m_a, m_b) and torch.equal(n_a.view(torch.int32), n_b.view(torch.int32))


def _packed_decode(eb, q, K, V, lens, b, ms8, mnorm, tau, **params):
    dev = torch.device("cuda:0")
    Kd, Vd, qd = K.to(dev), V.to(dev), q.to(dev)
    st = eb.DecodeState(Kd, Vd, q.shape[1], b)
    musig = torch.from_numpy(ms8).to(dev)
    mn = torch.from_numpy(mnorm).to(dev)
    p = eb.DecodeParams(flags=eb.ETA_FLAG_PACKED_SIGMA | params.pop("flags", 0), **params)
    st.out.fill_(float("nan"))
    eb.eta_decode(st.desc, p, qd, Kd, Vd, torch.from_numpy(np.asarray(lens, np.int32)).to(dev), musig, mn,
                  torch.from_numpy(np.ascontiguousarray(tau, np.float32)).to(dev), None, st.out, st.sel_mask,
                  st.workspace, stats=st.stats, status=st.status)
    torch.cuda.synchronize()
    return st.out.cpu().numpy(), st.sel_mask.cpu().numpy(), st.stats.cpu().numpy(), int(st.status.item())


CASES = [("c2_32k", 4096 + 77, 3, dict(lwb=2)),           # head_dim 128, 4 heads per group: tensor-core centroid term
         ("c1_tiny", 2048 + 16, 1, dict()),               # head_dim 64, block 32
         ("c4_512k", 16384 + 100, 1, dict(lwb=1)),        # block 128
         ("c5_frozen", 8192, 4, dict(z=1.5, a=0.2))]      # mixed lengths


@pytest.mark.parametrize("name,ctx,batch,params", CASES)
def test_decode_on_packed_summaries_matches_the_oracle(name, ctx, batch, params):
    eb = _eb()
    base = wl.CONFIGS[name]
    sp = base.scaled(ctx, batch=batch, min_context=ctx // 4 if base.min_context else None)
    w = wl.make_workload(sp)
    q = w.queries(0)
    c = cache_of(w)
    ms8, mnorm = orc.block_summaries_sigma8(c)
    exp = orc.unpack_sigma8(ms8)
    z = params.get("z", sp.z)
    bound = orc.score_dual(bits(q), exp, mnorm, c.seq_lens, sp.block_size, z)
    with np.errstate(all="ignore"):
        tau = (np.nanquantile(bound, 0.85, axis=2) + 2e-4).astype(np.float32)
    kw = dict(z=sp.z, beta=sp.beta)
    kw.update(params)
    ref = orc.decode_step(bits(q), c, exp, mnorm, tau=tau, **kw)
    out, sel, stats, status = _packed_decode(eb, q, w.K, w.V, c.seq_lens, sp.block_size, ms8, mnorm, tau, **kw)
    assert status == 0 and not np.isnan(out).any()
    tau_eff = tau.astype(np.float64) - kw.get("a", 0.0)
    near = compare_masks(sel, ref["sel"], ref["bound"], tau_eff, c.seq_lens, sp.block_size, sp.gqa, rescued=ref["rescued"])
    keep = heads_without_near_tie(near, sp.batch, sp.n_q_heads)
    assert keep.mean() > 0.9
    mx, mean = output_errors(out[keep], ref["out"][keep])
    assert mx <= 1e-2 and mean <= 1e-3, (mx, mean)
    union = np.array([[int((sel[i, hk, :int(c.seq_lens[i]) // sp.block_size] != 0).sum()) for hk in range(sp.n_kv_heads)]
                      for i in range(sp.batch)])
    assert np.array_equal(stats, union)
    # at the same thresholds the packed index admits a superset of what the 4 d-byte records admit (oracle, fp16 records):
    # no new false negative
    ms16, _ = orc.block_summaries(c)
    ref16 = orc.decode_step(bits(q), c, ms16, mnorm, tau=tau, **kw)
    no_rescue = (ref16["rescued"] < 0) & (ref["rescued"] < 0)
    for i in range(sp.batch):
        for h in range(sp.n_q_heads):
            if no_rescue[i, h]:
                b16 = (ref16["sel"][i, h // sp.gqa] >> (h % sp.gqa)) & 1
                b8 = (ref["sel"][i, h // sp.gqa] >> (h % sp.gqa)) & 1
                assert np.all(b8 >= b16)
    print(f"{name}: union density packed {float((ref['sel'] != 0).mean()):.4f} vs compact {float((ref16['sel'] != 0).mean()):.4f},"
          f" near ties {len(near)}, max err {mx:.2e}")


@pytest.mark.parametrize("G", [1, 2, 8])
def test_packed_screen_for_other_group_sizes_and_the_bound_diagnostic(G):
    eb = _eb()
    d, b, B, Hkv = 64 if G == 8 else 128, 64, 2, 2
    rng, K, V, lens = _rand_cache_t(40 + G, B, Hkv, [64 * 70 + 9, 64 * 33 + 1], d, b)
    q = torch.from_numpy(rng.standard_normal((B, Hkv * G, d))).to(torch.bfloat16)
    c = orc.Cache(bits(K), bits(V), lens, b)
    ms8, mnorm = orc.block_summaries_sigma8(c)
    exp = orc.unpack_sigma8(ms8)
    bound = orc.score_dual(bits(q), exp, mnorm, lens, b, 1.0)
    # the bound diagnostic on packed records
    dev = torch.device("cuda:0")
    Kd = K.to(dev)
    desc = eb.cache_desc(Kd, Kd, Hkv * G, b)
    got = torch.full((B, Hkv * G, desc.nb_cap), float("nan"), device=dev)
    eb.eta_score_dual(desc, eb.DecodeParams(flags=eb.ETA_FLAG_PACKED_SIGMA), q.to(dev), torch.from_numpy(lens).to(dev),
                      torch.from_numpy(ms8).to(dev), torch.from_numpy(mnorm).to(dev), got)
    g = got.cpu().numpy()
    for i in range(B):
        NB = int(lens[i]) // b
        assert np.abs(g[i, :, :NB] - bound[i, :, :NB]).max() <= 1e-5 * max(1.0, np.abs(bound[i, :, :NB]).max())
    tau = (np.nanquantile(bound, 0.75, axis=2) + 2e-4).astype(np.float32)
    ref = orc.decode_step(bits(q), c, exp, mnorm, tau=tau)
    out, sel, stats, status = _packed_decode(eb, q, K, V, lens, b, ms8, mnorm, tau)
    assert status == 0
    near = compare_masks(sel, ref["sel"], ref["bound"], tau.astype(np.float64), lens, b, G, rescued=ref["rescued"])
    keep = heads_without_near_tie(near, B, Hkv * G)
    assert keep.mean() > 0.8
    mx, mean = output_errors(out[keep], ref["out"][keep])
    assert mx <= 1e-2 and mean <= 1e-3, (mx, mean)

"""The five decode configurations at FULL size, in the launch configuration the benchmark times, against the CPU
oracle.  The C oracle is fast enough (seconds per configuration on the host cores) to check every element rather
than a sample: block summaries, thresholds, the selected-block masks and all outputs.

Tolerances are those of tests/test_gpu_parity.py.  Thresholds come from the stored calibration
(tests/golden/workload_calibration.json, written from the oracle) that the benchmark uses too.
"""
import json
import os

import numpy as np
import pytest
import torch

from oracle import eta_oracle as orc
from paper_2609_20888_b200 import workloads as wl
from tests.helpers import bits, cache_of, compare_masks, fp16_ulp_distance, heads_without_near_tie, output_errors

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 1e-2, 1e-3
CALIB = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "workload_calibration.json")))


def _eb():
    from paper_2609_20888_b200 import binding as eb
    from paper_2609_20888_b200 import build as ebuild
    ebuild.build()
    eb.load()
    return eb


class Session:
    """A workload resident on the GPU with its decode state, plus the oracle's view of the same bytes."""

    def __init__(self, name):
        self.eb = _eb()
        self.sp = wl.CONFIGS[name]
        self.w = wl.make_workload(self.sp, threads=16)
        self.dev = torch.device("cuda:0")
        self.K, self.V = self.w.K, self.w.V                      # host copies the oracle reads (and we append to)
        self.Kd, self.Vd = self.K.to(self.dev), self.V.to(self.dev)
        self.st = self.eb.DecodeState(self.Kd, self.Vd, self.sp.n_q_heads, self.sp.block_size)
        self.lens = self.w.seq_lens.numpy().astype(np.int32).copy()
        self.lens_d = torch.from_numpy(self.lens).to(self.dev)
        self.Wd = self.w.W.to(self.dev)

    def cache(self):
        return orc.Cache(bits(self.K), bits(self.V), self.lens.copy(), self.sp.block_size)

    def check_summaries(self):
        eb, st, sp = self.eb, self.st, self.sp
        eb.eta_build_block_summaries(st.desc, self.Kd, self.lens_d, st.musig, st.mnorm)
        torch.cuda.synchronize()
        musig, mnorm = orc.block_summaries(self.cache())
        got_ms, got_mn = bits(st.musig.cpu()), st.mnorm.cpu().numpy()
        for i in range(sp.batch):
            NB = int(self.lens[i]) // sp.block_size
            assert fp16_ulp_distance(got_ms[i, :, :NB], musig[i, :, :NB]).max() <= 1
            assert np.abs(got_mn[i, :, :NB].view(np.int32) - mnorm[i, :, :NB].view(np.int32)).max() <= 4
        return musig, mnorm

    def append(self, step):
        """One decode step's worth of cache growth: a token per sequence, then the tail-block metadata update."""
        k_t, v_t = self.w.new_kv(step)
        for i in range(self.sp.batch):
            t = int(self.lens[i])
            self.K[i, :, t] = k_t[i]
            self.V[i, :, t] = v_t[i]
            self.Kd[i, :, t] = k_t[i].to(self.dev)
            self.Vd[i, :, t] = v_t[i].to(self.dev)
        self.lens += 1
        self.lens_d += 1
        self.eb.eta_append_summary(self.st.desc, self.Kd, self.lens_d, self.st.musig, self.st.mnorm)

    def decode_and_check(self, step, musig, mnorm, bias=None, head_const=None, flags=0):
        """GPU decode on the oracle's summaries and thresholds vs the oracle's decode step; -> stats for logging."""
        eb, st, sp = self.eb, self.st, self.sp
        q = self.w.queries(step)
        c = self.cache()
        tau = None
        if bias is not None:
            tau = orc.predict_threshold(bits(q), self.w.W.numpy(), bias).astype(np.float32)
            # the predictor kernel, on the same inputs
            eb.eta_predict_threshold(q.to(self.dev), self.Wd, torch.from_numpy(bias).to(self.dev), st.tau)
            assert np.abs(st.tau.cpu().numpy() - tau).max() <= 1e-4
        ref = orc.decode_step(bits(q), c, musig, mnorm, tau=tau, head_const=head_const, z=sp.z, beta=sp.beta,
                              lwb=sp.lwb, rescue_window=sp.rescue_window)
        st.musig.copy_(torch.from_numpy(musig.view(np.int16)).view(torch.float16).to(self.dev))
        st.mnorm.copy_(torch.from_numpy(mnorm).to(self.dev))
        p = eb.DecodeParams(z=sp.z, beta=sp.beta, lwb=sp.lwb, rescue_window=sp.rescue_window, flags=flags)
        st.out.fill_(float("nan"))
        eb.eta_decode(st.desc, p, q.to(self.dev), self.Kd, self.Vd, self.lens_d, st.musig, st.mnorm,
                      None if tau is None else torch.from_numpy(tau).to(self.dev),
                      None if head_const is None else torch.from_numpy(head_const).to(self.dev),
                      st.out, st.sel_mask, st.workspace, stats=st.stats, status=st.status)
        torch.cuda.synchronize()
        assert int(st.status.item()) == 0
        out, sel = st.out.cpu().numpy(), st.sel_mask.cpu().numpy()
        assert not np.isnan(out).any()
        t = np.broadcast_to(head_const, (sp.batch, sp.n_q_heads)) if tau is None else tau
        near = compare_masks(sel, ref["sel"], ref["bound"], t.astype(np.float64), self.lens, sp.block_size, sp.gqa,
                             rescued=ref["rescued"])
        keep = heads_without_near_tie(near, sp.batch, sp.n_q_heads)
        assert keep.mean() > 0.9
        mx, mean = output_errors(out[keep], ref["out"][keep])
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)
        nb = sum(int(x) // sp.block_size for x in self.lens) * sp.n_kv_heads
        union = sum(int((ref["sel"][i, :, :int(self.lens[i]) // sp.block_size] != 0).sum()) for i in range(sp.batch))
        assert int(st.stats.sum().item()) == sum(
            int((sel[i, :, :int(self.lens[i]) // sp.block_size] != 0).sum()) for i in range(sp.batch))
        return {"sparsity": 1 - union / nb, "near_ties": len(near), "max_err": mx, "mean_err": mean,
                "rescued": int((ref["rescued"] >= 0).sum())}


def _bias(name, target):
    return np.asarray(CALIB[name]["targets"][f"{target:.2f}"]["bias"], np.float32)


def test_c1_tiny_16_decode_steps():
    s = Session("c1_tiny")
    s.check_summaries()
    bias = _bias("c1_tiny", 0.80)
    for step in range(0, 17):
        if step > 0:
            s.append(step)
        musig, mnorm = orc.block_summaries(s.cache())
        r = s.decode_and_check(step, musig, mnorm, bias=bias)
    assert s.lens[0] == 2048 + 16
    print("c1", r)


def test_c2_32k_batch8_with_appends_across_block_boundaries():
    s = Session("c2_32k")
    musig, mnorm = s.check_summaries()
    bias = _bias("c2_32k", 0.85)
    r0 = s.decode_and_check(0, musig, mnorm, bias=bias)
    assert 0.6 < r0["sparsity"] < 0.97
    for step in range(1, 129):                  # 128 appended tokens: two blocks complete on the way
        s.append(step)
    torch.cuda.synchronize()
    musig, mnorm = orc.block_summaries(s.cache())
    NB = int(s.lens[0]) // s.sp.block_size
    assert NB == 32768 // 64 + 2
    # the summaries the per-step append left behind equal the oracle's for the grown cache
    assert fp16_ulp_distance(bits(s.st.musig.cpu())[:, :, :NB], musig[:, :, :NB]).max() <= 1
    r1 = s.decode_and_check(128, musig, mnorm, bias=bias)
    print("c2", r0, r1)


@pytest.mark.parametrize("target", [0.50, 0.90, 0.97])
def test_c3_128k_sparsity_sweep(target):
    s = Session("c3_128k")
    musig, mnorm = s.check_summaries()
    r = s.decode_and_check(0, musig, mnorm, bias=_bias("c3_128k", target))
    assert abs(r["sparsity"] - target) < 0.05
    print("c3", target, r)


def test_c3_128k_dense_flag_is_softmax_attention_on_a_sampled_head_set():
    """Full-size dense baseline: every block, gate off.  The oracle's dense routine recomputes exp per output
    coordinate, so it is run on sequence 0 only."""
    s = Session("c3_128k")
    eb, st, sp = s.eb, s.st, s.sp
    q = s.w.queries(0)
    p = eb.DecodeParams(flags=eb.ETA_FLAG_DENSE)
    tau = torch.zeros((sp.batch, sp.n_q_heads), dtype=torch.float32, device=s.dev)
    eb.eta_decode(st.desc, p, q.to(s.dev), s.Kd, s.Vd, s.lens_d, st.musig, st.mnorm, tau, None, st.out, st.sel_mask,
                  st.workspace, stats=st.stats, status=st.status)
    torch.cuda.synchronize()
    assert int(st.status.item()) == 0
    c = orc.Cache(bits(s.K[:1]), bits(s.V[:1]), s.lens[:1].copy(), sp.block_size)
    full = np.full((1, sp.n_kv_heads, c.NBcap), (1 << sp.gqa) - 1, np.uint8)
    ref = orc.gated_block_attention(bits(q[:1]), c, full, tau=np.full((1, sp.n_q_heads), -np.inf, np.float32))
    mx, mean = output_errors(st.out.cpu().numpy()[:1], ref)
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)
    assert int(st.stats.sum().item()) == sp.batch * sp.n_kv_heads * (sp.context // sp.block_size)


def test_c4_512k_batch1_block128_with_the_append_that_ends_on_a_block_boundary():
    s = Session("c4_512k")
    musig, mnorm = s.check_summaries()
    bias = _bias("c4_512k", 0.90)
    r0 = s.decode_and_check(0, musig, mnorm, bias=bias)           # 64-token tail
    for step in range(1, 65):
        s.append(step)
    torch.cuda.synchronize()
    assert s.lens[0] == 524288
    musig, mnorm = orc.block_summaries(s.cache())
    assert fp16_ulp_distance(bits(s.st.musig.cpu()), musig).max() <= 1    # the completed block was summarised
    r1 = s.decode_and_check(64, musig, mnorm, bias=bias)          # no tail
    print("c4", r0, r1)


def test_c5_frozen_constants_vs_predicted_thresholds_mixed_lengths():
    s = Session("c5_frozen")
    musig, mnorm = s.check_summaries()
    assert s.lens.min() < 0.6 * s.lens.max()
    consts = np.asarray(CALIB["c5_frozen"]["head_const"], np.float32)
    rf = s.decode_and_check(0, musig, mnorm, head_const=consts)
    rp = s.decode_and_check(0, musig, mnorm, bias=_bias("c5_frozen", 0.70))
    print("c5 frozen", rf, "predicted", rp)


def test_one_sequence_of_seventeen_million_tokens():
    """A single KV head of 17.8 M tokens (4.6 GB per tensor, 139 264 blocks of 128 tokens, 2177 segments): element
    offsets inside K and V pass 2^31, a row's block lists are far longer than any other test's.  Full comparison with
    the oracle: the summary build, the masks, the block count and all eight heads' outputs."""
    eb = _eb()
    dev = torch.device("cuda:0")
    B, Hkv, G, d, b = 1, 1, 8, 128, 128
    T = 17 * (1 << 20) + 77
    t_cap = ((T + b - 1) // b) * b
    gen = torch.Generator().manual_seed(20888)
    K = torch.empty((B, Hkv, t_cap, d), dtype=torch.bfloat16)
    V = torch.empty((B, Hkv, t_cap, d), dtype=torch.bfloat16)
    step = 1 << 20
    for t0 in range(0, t_cap, step):                          # drawn in chunks: the fp32 draws never exist all at once
        n = min(step, t_cap - t0)
        K[0, 0, t0:t0 + n] = torch.randn((n, d), generator=gen).to(torch.bfloat16)
        V[0, 0, t0:t0 + n] = torch.randn((n, d), generator=gen).to(torch.bfloat16)
    q = torch.randn((B, Hkv * G, d), generator=gen).to(torch.bfloat16)
    lens = np.asarray([T], np.int32)
    c = orc.Cache(bits(K), bits(V), lens, b)
    musig, mnorm = orc.block_summaries(c)
    NB = T // b
    # summary build on the device
    Kd, Vd = K.to(dev), V.to(dev)
    st = eb.DecodeState(Kd, Vd, Hkv * G, b)
    lens_d = torch.from_numpy(lens).to(dev)
    eb.eta_build_block_summaries(st.desc, Kd, lens_d, st.musig, st.mnorm)
    torch.cuda.synchronize()
    assert fp16_ulp_distance(bits(st.musig.cpu())[0, :, :NB], musig[0, :, :NB]).max() <= 1
    assert np.abs(st.mnorm.cpu().numpy()[0, :, :NB].view(np.int32) - mnorm[0, :, :NB].view(np.int32)).max() <= 4
    # decode on the oracle's summary bytes, thresholds that keep about one block in 200 per head
    bound = orc.score_dual(bits(q), musig, mnorm, lens, b, 1.0)
    tau = (np.nanquantile(bound, 0.995, axis=2) + 3e-4).astype(np.float32)
    ref = orc.decode_step(bits(q), c, musig, mnorm, tau=tau, lwb=2, rescue_window=128)
    st.musig.copy_(torch.from_numpy(musig.view(np.int16)).view(torch.float16).to(dev))
    st.mnorm.copy_(torch.from_numpy(mnorm).to(dev))
    st.out.fill_(float("nan"))
    eb.eta_decode(st.desc, eb.DecodeParams(lwb=2, rescue_window=128), q.to(dev), Kd, Vd, lens_d, st.musig, st.mnorm,
                  torch.from_numpy(tau).to(dev), None, st.out, st.sel_mask, st.workspace, stats=st.stats, status=st.status)
    torch.cuda.synchronize()
    assert int(st.status.item()) == 0
    sel, out = st.sel_mask.cpu().numpy(), st.out.cpu().numpy()
    near = compare_masks(sel, ref["sel"], ref["bound"], tau.astype(np.float64), lens, b, G, rescued=ref["rescued"])
    keep = heads_without_near_tie(near, B, Hkv * G)
    assert keep.mean() >= 0.75
    mx, mean = output_errors(out[keep], ref["out"][keep])
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)
    assert int(st.stats.sum().item()) == int((sel[0, 0, :NB] != 0).sum())
    assert 0.005 < st.stats.sum().item() / NB < 0.10

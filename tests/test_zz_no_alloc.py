"""eta_decode_static: the variant of eta_decode whose scratch is an array built into the library, for callers
that cannot hand it device memory (a server whose HBM all belongs to its KV-cache pool, a plug-in with no
allocator, a decode loop that must keep out of cudaMalloc).

Checked through the C ABI against the ordinary entry point on two calls in a row: the second call runs on the
scratch the first one left behind, with a different query and different thresholds, so anything that wrongly
survived from call one would show.  The two entry points run the same kernels with the same launch geometry and a
fixed merge order, so their results must be identical bit for bit; the static variant is also compared with the
CPU oracle (masks bit-exact outside the 1e-5 near-tie band, outputs within 1e-2 max / 1e-3 mean).  A second test
dirties the scratch on purpose first.  The file name makes pytest collect it last.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import eta_oracle as orc
from paper_2609_20888_b200 import workloads as wl
from tests.helpers import bits, cache_of, compare_masks, heads_without_near_tie, output_errors

pytestmark = pytest.mark.gpu


def test_static_scratch_variant_matches_eta_decode_twice_in_a_row():
    from paper_2609_20888_b200 import binding as eb
    from paper_2609_20888_b200 import build as ebuild
    ebuild.build()
    lib = eb.load()
    dev = torch.device("cuda:0")
    sp = wl.CONFIGS["c2_32k"].scaled(6144 + 45, batch=2)
    w = wl.make_workload(sp)
    Kd, Vd = w.K.to(dev), w.V.to(dev)
    st = eb.DecodeState(Kd, Vd, sp.n_q_heads, sp.block_size)
    lens_d = w.seq_lens.to(dev)
    eb.eta_build_block_summaries(st.desc, Kd, lens_d, st.musig, st.mnorm)
    assert eb.eta_workspace_bytes(st.desc) <= eb.eta_static_scratch_bytes() == 8 << 20

    out2 = torch.empty_like(st.out)
    sel2 = torch.empty_like(st.sel_mask)
    stats2 = torch.empty_like(st.stats)
    status2 = torch.zeros_like(st.status)
    for call, (bias, lwb) in enumerate([(1.4, 0), (2.2, 2)]):
        q = w.queries(call).to(dev)
        tau = torch.empty((sp.batch, sp.n_q_heads), dtype=torch.float32, device=dev)
        eb.eta_predict_threshold(q, w.W.to(dev), torch.full((sp.n_q_heads,), bias, device=dev), tau)
        params = eb.DecodeParams(z=sp.z, beta=sp.beta, lwb=lwb)
        eb.eta_decode(st.desc, params, q, Kd, Vd, lens_d, st.musig, st.mnorm, tau, None, st.out, st.sel_mask,
                      st.workspace, stats=st.stats, status=st.status)
        out2.fill_(float("nan"))
        sel2.fill_(0xff)
        eb.eta_decode_static(st.desc, params, q, Kd, Vd, lens_d, st.musig, st.mnorm, tau, None, out2, sel2,
                             stats=stats2, status=status2)
        torch.cuda.synchronize()
        assert int(st.status.item()) == 0 and int(status2.item()) == 0
        assert torch.equal(sel2, st.sel_mask), f"call {call}: selected-block masks differ"
        assert torch.equal(stats2, st.stats)
        assert torch.equal(out2.view(torch.int32), st.out.view(torch.int32)), f"call {call}: outputs differ"
        assert 0.02 < float((st.sel_mask != 0).float().mean()) < 0.98      # a genuinely sparse selection
        # and against the oracle, from the bytes the GPU call read (its own summaries and thresholds)
        c = cache_of(w)
        tau_np = tau.cpu().numpy()
        ref = orc.decode_step(bits(q.cpu()), c, bits(st.musig.cpu()), st.mnorm.cpu().numpy(), tau=tau_np, z=sp.z,
                              beta=sp.beta, lwb=lwb)
        near = compare_masks(sel2.cpu().numpy(), ref["sel"], ref["bound"], tau_np.astype(np.float64), c.seq_lens,
                             sp.block_size, sp.gqa, rescued=ref["rescued"])
        keep = heads_without_near_tie(near, sp.batch, sp.n_q_heads)
        assert keep.mean() > 0.9
        mx, mean = output_errors(out2.cpu().numpy()[keep], ref["out"][keep])
        assert mx <= 1e-2 and mean <= 1e-3, (call, mx, mean)


def test_scratch_left_by_a_different_call_is_never_consumed():
    """Both the caller's workspace and the built-in scratch keep the last call's contents, and the library
    promises that every word is written before it is read.  First a call that leaves plausible, in-range but
    wrong contents everywhere: every block of long sequences admitted (ETA_FLAG_DENSE), so every list is full,
    every count is 64 and every partial slot is used.  Then, on the same scratch, a highly sparse call on
    shorter, mixed lengths (fewer segments, other rows' spans, other rescue windows): its result must match the
    oracle, on the caller's workspace and on the built-in array alike."""
    from paper_2609_20888_b200 import binding as eb
    from paper_2609_20888_b200 import build as ebuild
    ebuild.build()
    eb.load()
    dev = torch.device("cuda:0")
    sp = wl.CONFIGS["c5_frozen"].scaled(12288 + 50, batch=3, min_context=0)
    w = wl.make_workload(sp)
    Kd, Vd = w.K.to(dev), w.V.to(dev)
    st = eb.DecodeState(Kd, Vd, sp.n_q_heads, sp.block_size)
    long_lens = w.seq_lens.to(dev)
    eb.eta_build_block_summaries(st.desc, Kd, long_lens, st.musig, st.mnorm)
    short = torch.tensor([3000, 12288 + 50, 700], dtype=torch.int32)
    q0, q1 = w.queries(0).to(dev), w.queries(1)
    c = orc.Cache(bits(w.K), bits(w.V), short.numpy().copy(), sp.block_size)
    musig, mnorm = bits(st.musig.cpu()), st.mnorm.cpu().numpy()
    bound = orc.score_dual(bits(q1), musig, mnorm, c.seq_lens, sp.block_size, sp.z)
    with np.errstate(all="ignore"):
        tau = (np.nanquantile(bound, 0.93, axis=2) + 1e-4).astype(np.float32)       # ~7 % of the blocks per head
    ref = orc.decode_step(bits(q1), c, musig, mnorm, tau=tau, z=sp.z, beta=sp.beta, lwb=1, rescue_window=16)
    dense = eb.DecodeParams(flags=eb.ETA_FLAG_DENSE)
    sparse = eb.DecodeParams(z=sp.z, beta=sp.beta, lwb=1, rescue_window=16)
    tau_d = torch.from_numpy(tau).to(dev)
    zero_tau = torch.zeros_like(tau_d)
    for static in (False, True):
        status = torch.zeros_like(st.status)
        out = torch.full_like(st.out, float("nan"))
        sel = torch.full_like(st.sel_mask, 0xff)
        stats = torch.zeros_like(st.stats)
        if static:
            eb.eta_decode_static(st.desc, dense, q0, Kd, Vd, long_lens, st.musig, st.mnorm, zero_tau, None, out, sel,
                                 stats=stats, status=status)
            eb.eta_decode_static(st.desc, sparse, q1.to(dev), Kd, Vd, short.to(dev), st.musig, st.mnorm, tau_d, None,
                                 out, sel, stats=stats, status=status)
        else:
            st.workspace.fill_(0xa5)         # not even zeros to start from
            eb.eta_decode(st.desc, dense, q0, Kd, Vd, long_lens, st.musig, st.mnorm, zero_tau, None, out, sel,
                          st.workspace, stats=stats, status=status)
            eb.eta_decode(st.desc, sparse, q1.to(dev), Kd, Vd, short.to(dev), st.musig, st.mnorm, tau_d, None,
                          out, sel, st.workspace, stats=stats, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        sel_np = sel.cpu().numpy()
        near = compare_masks(sel_np, ref["sel"], ref["bound"], tau.astype(np.float64), c.seq_lens, sp.block_size,
                             sp.gqa, rescued=ref["rescued"])
        keep = heads_without_near_tie(near, sp.batch, sp.n_q_heads)
        assert keep.mean() > 0.9
        mx, mean = output_errors(out.cpu().numpy()[keep], ref["out"][keep])
        assert mx <= 1e-2 and mean <= 1e-3, (static, mx, mean)
        union = np.array([[int((sel_np[i, hk, :int(short[i]) // sp.block_size] != 0).sum())
                           for hk in range(sp.n_kv_heads)] for i in range(sp.batch)])
        assert np.array_equal(stats.cpu().numpy(), union)
        assert union.sum() < 0.4 * sum(int(t) // sp.block_size for t in short) * sp.n_kv_heads


def test_static_scratch_variant_refuses_shapes_beyond_its_limit():
    from paper_2609_20888_b200 import binding as eb
    lib = eb.load()
    # 64 sequences x 8 KV heads x 512K tokens: needs far more than 8 MiB of scratch; refused before any launch
    T = 512 * 1024
    d = eb.CacheDesc(64, 32, 8, 128, 64, T, T // 64, 8 * T * 128, T * 128, 128, 8 * T * 128, T * 128, 128)
    assert eb.eta_workspace_bytes(d) > eb.eta_static_scratch_bytes()
    p = eb.DecodeParams().c()
    one, null = ctypes.c_void_p(256), ctypes.c_void_p(None)
    rc = lib.eta_decode_static(ctypes.byref(d), ctypes.byref(p), one, one, one, one, one, one, one, null, one, one,
                               null, null, null)
    assert rc == -3

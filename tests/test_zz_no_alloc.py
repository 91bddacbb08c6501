"""eta_decode_static: the variant of eta_decode whose scratch is an array built into the library, for callers
that cannot hand it device memory (a server whose HBM all belongs to its KV-cache pool, a plug-in with no
allocator, a decode loop that must keep out of cudaMalloc).

Checked through the C ABI against the ordinary entry point on two calls in a row: the second call runs on the
scratch the first one left behind, with a different query and different thresholds, so anything that wrongly
survived from call one would show.  The file name makes pytest collect it last.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2609_20888_b200 import workloads as wl

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
        err = (out2 - st.out).abs()
        assert float(err.max()) <= 1e-2 and float(err.mean()) <= 1e-3, (call, float(err.max()))
        assert 0.02 < float((st.sel_mask != 0).float().mean()) < 0.98      # a genuinely sparse selection


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

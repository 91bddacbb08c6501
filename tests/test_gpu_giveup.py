"""A bounded wait that runs out, on purpose, without faulting or hanging anything.

Every wait inside the kernels (on an mbarrier, on a flag) gives up after a fixed number of polls, reports
ETA_DEV_TIMEOUT through `status_dev`, and lets the CTA leave in order: copies already issued are given time to land
before the shared memory is released.  None of that runs in a healthy call.  Here it is made to run: a second build of
the same sources (`libeta_b200_test_giveup.so`: -DETA_TEST_SKIP_FLUSH_ARRIVE -DETA_WAIT_LIMIT=65536) in which one
consumer warp of the streaming kernel's first CTA never arrives at its group's barrier, with waits of 2^16 polls (a few
milliseconds: far longer than any copy takes, so no wait on a copy gives up by accident).  The group's wait runs
out, the group leaves, the producer finds no free stage and leaves after its copies have landed, the other groups find
no more tiles and leave.  Checked: the call returns, the status word has ETA_DEV_TIMEOUT, and an ordinary call of the
product library on the same workspace right afterwards agrees with the oracle.
"""
import numpy as np
import pytest
import torch

from oracle import eta_oracle as orc
from paper_2609_20888_b200 import workloads as wl
from tests.helpers import bits, cache_of, compare_masks, heads_without_near_tie, output_errors

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_reports_timeout_and_leaves_the_workspace_usable():
    from paper_2609_20888_b200 import binding as eb
    from paper_2609_20888_b200 import build as ebuild
    ebuild.build()
    eb.load()
    variant = eb.load(ebuild.build_giveup_variant())
    dev = torch.device("cuda:0")
    sp = wl.CONFIGS["c2_32k"].scaled(8192 + 21, batch=2)
    w = wl.make_workload(sp)
    q = w.queries(0)
    c = cache_of(w)
    musig, mnorm = orc.block_summaries(c)
    bound = orc.score_dual(bits(q), musig, mnorm, c.seq_lens, sp.block_size, sp.z)
    tau = (np.nanquantile(bound, 0.8, axis=2) + 2e-4).astype(np.float32)
    ref = orc.decode_step(bits(q), c, musig, mnorm, tau=tau, z=sp.z, beta=sp.beta)

    Kd, Vd, qd = w.K.to(dev), w.V.to(dev), q.to(dev)
    st = eb.DecodeState(Kd, Vd, sp.n_q_heads, sp.block_size)
    st.musig.copy_(torch.from_numpy(musig.view(np.int16)).view(torch.float16).to(dev))
    st.mnorm.copy_(torch.from_numpy(mnorm).to(dev))
    lens_d = w.seq_lens.to(dev)
    tau_d = torch.from_numpy(tau).to(dev)
    params = eb.DecodeParams(z=sp.z, beta=sp.beta)

    # the call with the warp that never arrives: it must come back, flagged
    eb.eta_decode(st.desc, params, qd, Kd, Vd, lens_d, st.musig, st.mnorm, tau_d, None, st.out, st.sel_mask,
                  st.workspace, stats=st.stats, status=st.status, lib=variant)
    torch.cuda.synchronize()
    assert int(st.status.item()) & eb.ETA_DEV_TIMEOUT, "the wait did not run out, or did not report it"
    # an ordinary call on the same workspace and buffers right afterwards
    st.status.zero_()
    st.out.fill_(float("nan"))
    eb.eta_decode(st.desc, params, qd, Kd, Vd, lens_d, st.musig, st.mnorm, tau_d, None, st.out, st.sel_mask,
                  st.workspace, stats=st.stats, status=st.status)
    torch.cuda.synchronize()
    assert int(st.status.item()) == 0
    near = compare_masks(st.sel_mask.cpu().numpy(), ref["sel"], ref["bound"], tau.astype(np.float64), c.seq_lens,
                         sp.block_size, sp.gqa, rescued=ref["rescued"])
    keep = heads_without_near_tie(near, sp.batch, sp.n_q_heads)
    assert keep.mean() > 0.9
    mx, mean = output_errors(st.out.cpu().numpy()[keep], ref["out"][keep])
    assert mx <= 1e-2 and mean <= 1e-3, (mx, mean)

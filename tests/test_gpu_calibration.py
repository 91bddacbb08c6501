"""Offline threshold calibration on the GPU against the CPU oracle (same split, same thresholds).

Tolerances: the histogram is an integer count of 1/t weights on both sides; a score within a few fp32 ulp of a bin
edge may fall on either side of it (the oracle bins the score it computed in double, the kernel the score its tensor
core accumulated in fp32, off by up to ~2e-6 for these O(1) dot products), which moves that score's weight to the
neighbouring bin: a fraction <= 2 * 2e-6 / w of the weight, w the bin width, so the normalised histograms agree to
2 * that in L1.  The target density (fp32 sigmoid on the GPU) agrees to 1e-6; the calibrated constant reproduces
the oracle's target density on the oracle's histogram to 5e-6 and, on splits of at least 64 tokens, equals the
oracle's constant to 1e-4.
"""
import math

import numpy as np
import pytest
import torch

from oracle import eta_oracle as orc
from tests.helpers import bits

pytestmark = pytest.mark.gpu


def _eb():
    from paper_2609_20888_b200 import binding as eb
    from paper_2609_20888_b200 import build as ebuild
    ebuild.build()
    eb.load()
    return eb


def _split(seed, n_seq, Hq, Hkv, T, d, qscale=1.0):
    g = torch.Generator().manual_seed(seed)
    Q = (torch.randn((n_seq, Hq, T, d), generator=g) * qscale).to(torch.bfloat16)
    K = torch.randn((n_seq, Hkv, T, d), generator=g).to(torch.bfloat16)
    tau = (0.3 + 0.6 * torch.randn((n_seq, Hq, T), generator=g)).to(torch.float32)
    return Q, K, tau


@pytest.mark.parametrize("n_seq,Hq,Hkv,T,d,n_bins", [(2, 4, 2, 200, 64, 512), (3, 8, 2, 333, 128, 2048),
                                                     (1, 2, 1, 64, 128, 64), (2, 4, 4, 1, 64, 16),
                                                     (4, 8, 2, 1024, 128, 4096)])
def test_calibration_matches_the_oracle(n_seq, Hq, Hkv, T, d, n_bins):
    eb = _eb()
    dev = torch.device("cuda:0")
    Q, K, tau = _split(100 + T, n_seq, Hq, Hkv, T, d, qscale=1.5)
    beta, s_min, s_max = 5.0, -7.0, 7.0
    ref = orc.calibrate(bits(Q), bits(K), tau.numpy(), beta=beta, n_bins=n_bins, s_min=s_min, s_max=s_max)
    hc = torch.full((Hq,), float("nan"), device=dev)
    dbar = torch.full((Hq,), float("nan"), device=dev)
    ws = eb.eta_calibrate_head_const(Q.to(dev), K.to(dev), tau.to(dev), hc, dbar, beta=beta, n_bins=n_bins,
                                     s_min=s_min, s_max=s_max)
    torch.cuda.synchronize()
    np.testing.assert_allclose(dbar.cpu().numpy(), ref["dbar"], rtol=0, atol=1e-6)
    # the constant is defined by the density it yields: on the oracle's histogram, the GPU's constant must give the
    # oracle's target density (how far the constant itself may move for that depends on the slope of g at the root)
    for h in range(Hq):
        g = orc.calibration_density(ref["hist"][h], s_min, s_max, beta, float(hc[h].item()))
        assert abs(g - ref["dbar"][h]) <= 5e-6, (h, g, ref["dbar"][h])
    if T >= 64:
        np.testing.assert_allclose(hc.cpu().numpy(), ref["head_const"], rtol=0, atol=1e-4)
    # the integer histogram the kernels left in the scratch, normalised, against the oracle's
    H = ws[:Hq * n_bins * 8].view(torch.int64).cpu().numpy().reshape(Hq, n_bins).astype(np.float64)
    Hn = H / H.sum(axis=1, keepdims=True)
    assert np.abs(Hn - ref["hist"]).sum(axis=1).max() <= 8e-6 * n_bins / (s_max - s_min) + 1e-9
    # a second call on the same scratch gives the same bits (nothing depends on the order of the atomics)
    hc2 = torch.empty_like(hc)
    eb.eta_calibrate_head_const(Q.to(dev), K.to(dev), tau.to(dev), hc2, None, beta=beta, n_bins=n_bins, s_min=s_min,
                                s_max=s_max, workspace=ws)
    torch.cuda.synchronize()
    assert torch.equal(hc, hc2)


def test_calibrated_constants_reproduce_the_predictor_density_in_decode_terms():
    """A constant threshold calibrates to itself (up to the bin width), on the GPU as in the oracle."""
    eb = _eb()
    dev = torch.device("cuda:0")
    Q, K, _ = _split(7, 2, 8, 2, 512, 128)
    tau = torch.full((2, 8, 512), 0.4)
    hc = torch.empty(8, device=dev)
    eb.eta_calibrate_head_const(Q.to(dev), K.to(dev), tau.to(dev), hc, None, beta=5.0, n_bins=4096, s_min=-8, s_max=8)
    torch.cuda.synchronize()
    assert float((hc - 0.4).abs().max()) < 16.0 / 4096


def test_calibration_argument_checks():
    eb = _eb()
    lib = eb.load()
    import ctypes
    n = ctypes.c_size_t(0)
    assert lib.eta_calibration_workspace_bytes(2, 128, 8, 1, ctypes.byref(n)) == -1
    assert lib.eta_calibration_workspace_bytes(2, 128, 8, 256, ctypes.byref(n)) == 0 and n.value > 0
    one = ctypes.c_void_p(256)
    f = ctypes.cast(one, ctypes.POINTER(ctypes.c_float))
    args = lambda d, bins: (2, 128, 8, 2, d, one, one, f, 5.0, 0.0, bins, -8.0, 8.0, f, f, one, n.value, None)
    assert lib.eta_calibrate_head_const(*args(96, 256)) == -2          # head_dim
    assert lib.eta_calibrate_head_const(*args(128, 8192)) == -2        # too many bins

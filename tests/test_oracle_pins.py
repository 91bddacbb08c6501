"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests obtains its expectation from the oracle function under
test: they use closed forms, numpy / scipy / torch library routines, brute
force over tiny inputs, and invariants, chosen so that a dropped term, a wrong
sign or index or a transposed operand fails at least one of them.
"""
import math

import numpy as np
import pytest
import torch
from scipy.special import lambertw

from oracle import eta_oracle as orc
from tests.helpers import bf16_bits_from_f64, bf16_values, fp16_values, random_cache


# --------------------------------------------------------------------------
# storage formats
# --------------------------------------------------------------------------

def test_fp16_decode_matches_numpy_for_every_bit_pattern():
    allbits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    ref = allbits.view(np.float16).astype(np.float64)
    got = np.array([orc.fp16_to_double(int(b)) for b in allbits])
    assert np.array_equal(np.isnan(ref), np.isnan(got))
    m = ~np.isnan(ref)
    assert np.array_equal(ref[m], got[m])


def test_fp16_encode_is_single_round_to_nearest_even():
    rng = np.random.default_rng(1)
    xs = np.concatenate([
        rng.standard_normal(4000) * 10.0 ** rng.integers(-9, 5, 4000),
        np.array([0.0, -0.0, 65504.0, 65519.999, 65520.0, 1e9, -1e9, 2.0 ** -24, 2.0 ** -25, 2.0 ** -25 * 1.0001,
                  2.0 ** -14, 2.0 ** -14 * (1 - 2.0 ** -12), np.inf, -np.inf]),
    ])
    # midpoints between neighbouring fp16 values must go to the even neighbour
    h = rng.integers(0x0001, 0x7bfe, 500).astype(np.uint16)
    lo = h.view(np.float16).astype(np.float64)
    hi = (h + 1).astype(np.uint16).view(np.float16).astype(np.float64)
    xs = np.concatenate([xs, 0.5 * (lo + hi)])
    with np.errstate(over="ignore"):
        ref = xs.astype(np.float16).view(np.uint16)      # numpy rounds float64 -> float16 directly, RNE
    got = np.array([orc.double_to_fp16(float(x)) for x in xs], dtype=np.uint16)
    assert np.array_equal(ref, got)


def test_double_rounding_case_differs_from_rounding_through_float32():
    # 1 + 2^-11 + 2^-30 lies just above the midpoint of two fp16 values: direct rounding goes up,
    # rounding through binary32 first lands on the midpoint and then (ties-to-even) goes down.
    x = 1.0 + 2.0 ** -11 + 2.0 ** -30
    assert orc.double_to_fp16(x) == 0x3c01
    assert np.float32(x).astype(np.float16).view(np.uint16) == 0x3c00


def test_bf16_decode_matches_torch():
    allbits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    ref = torch.from_numpy(allbits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    got = np.array([orc.bf16_to_double(int(b)) for b in allbits])
    m = ~np.isnan(ref)
    assert np.array_equal(np.isnan(ref), np.isnan(got))
    assert np.array_equal(ref[m], got[m])


# --------------------------------------------------------------------------
# block summaries (Section 3: centroid, coordinate-wise population variance, max norm)
# --------------------------------------------------------------------------

def test_summaries_match_numpy_mean_std_norm():
    rng = np.random.default_rng(2)
    c = random_cache(rng, B=2, Hkv=3, T=5 * 32 + 7, d=16, b=32)
    musig, mnorm, mu, sg, M = orc.block_summaries(c, raw=True)
    Kv = bf16_values(c.K)
    NB = c.seq_lens[0] // 32
    assert NB == 5
    blocks = Kv[:, :, :NB * 32].reshape(2, 3, NB, 32, 16)
    np.testing.assert_allclose(mu[:, :, :NB], blocks.mean(axis=3), rtol=0, atol=1e-14)
    np.testing.assert_allclose(sg[:, :, :NB], blocks.std(axis=3), rtol=1e-13, atol=1e-14)   # ddof=0: population
    np.testing.assert_allclose(M[:, :, :NB], np.linalg.norm(blocks, axis=4).max(axis=3), rtol=1e-14)
    # storage rounding: fp16 for mu and sigma (sigma, not the variance), fp32 for M
    assert np.array_equal(musig[:, :, :NB, 0].view(np.float16), mu[:, :, :NB].astype(np.float16))
    assert np.array_equal(musig[:, :, :NB, 1].view(np.float16), sg[:, :, :NB].astype(np.float16))
    assert np.array_equal(mnorm[:, :, :NB], M[:, :, :NB].astype(np.float32))
    # the partial block past NB is not summarised
    assert not musig[:, :, NB:].any() and not mnorm[:, :, NB:].any()


def test_summaries_of_identical_keys():
    d, b = 16, 8
    k = np.linspace(-1.5, 2.0, d)
    K = bf16_bits_from_f64(np.broadcast_to(k, (1, 1, b, d)).copy())
    c = orc.Cache(K, K.copy(), np.array([b], np.int32), b)
    _, _, mu, sg, M = orc.block_summaries(c, raw=True)
    kv = bf16_values(K)[0, 0, 0]
    np.testing.assert_allclose(mu[0, 0, 0], kv, atol=1e-15)
    assert np.all(sg[0, 0, 0] == 0.0)
    assert M[0, 0, 0] == pytest.approx(np.linalg.norm(kv), rel=1e-15)


def test_summaries_of_axis_pairs_have_closed_form():
    # keys mu0 +- s_c e_c (b = 2d): centroid mu0, variance_c = 2 s_c^2 / b, exactly diagonal covariance
    d = 8
    b = 2 * d
    mu0 = np.array([0.5, -1.0, 0.25, 2.0, -0.75, 1.5, 0.0, -2.0])
    s = np.array([0.5, 1.0, 0.25, 2.0, 0.125, 1.0, 0.5, 4.0])
    keys = np.concatenate([mu0 + np.diag(s), mu0 - np.diag(s)])       # all exactly representable in bf16
    K = bf16_bits_from_f64(keys.reshape(1, 1, b, d))
    assert np.array_equal(bf16_values(K)[0, 0], keys)
    c = orc.Cache(K, K.copy(), np.array([b], np.int32), b)
    _, _, mu, sg, M = orc.block_summaries(c, raw=True)
    np.testing.assert_allclose(mu[0, 0, 0], mu0, atol=1e-15)
    np.testing.assert_allclose(sg[0, 0, 0] ** 2, 2 * s ** 2 / b, rtol=1e-14)
    assert M[0, 0, 0] == pytest.approx(max(np.linalg.norm(keys, axis=1)), rel=1e-15)


def test_summary_invariants_and_permutation():
    rng = np.random.default_rng(3)
    c = random_cache(rng, B=1, Hkv=2, T=4 * 64, d=32, b=64, scale=2.0)
    _, _, mu, sg, M = orc.block_summaries(c, raw=True)
    Kv = bf16_values(c.K).reshape(1, 2, 4, 64, 32)
    # second formula for the variance: E[k^2] - mu^2
    np.testing.assert_allclose(sg ** 2, (Kv ** 2).mean(axis=3) - mu ** 2, rtol=1e-10, atol=1e-12)
    # the largest norm dominates the root mean square norm: M^2 >= |mu|^2 + sum sigma^2
    assert np.all(M ** 2 >= (mu ** 2).sum(-1) + (sg ** 2).sum(-1) - 1e-12)
    # permuting the tokens inside a block changes nothing
    perm = rng.permutation(64)
    Kp = c.K.reshape(1, 2, 4, 64, 32)[:, :, :, perm].reshape(c.K.shape).copy()
    _, _, mu2, sg2, M2 = orc.block_summaries(orc.Cache(Kp, c.V, c.seq_lens, 64), raw=True)
    np.testing.assert_allclose(mu2, mu, atol=1e-14)
    np.testing.assert_allclose(sg2, sg, atol=1e-13)
    np.testing.assert_array_equal(M2, M)


def test_record_size_is_the_stated_overhead():
    # compact layout: fp16[d] + fp16[d] + fp32 per block per KV head; 1.6% of the K,V bytes at b = 64
    for d in (64, 128):
        rec = 2 * d + 2 * d + 4
        kv = 2 * 64 * d * 2
        assert rec == 4 * d + 4
        assert round(100.0 * rec / kv, 1) == 1.6


def test_envelope_bounds_flat_sigma():
    # sub-block envelope: sigma <= sigma~ <= sqrt(b/4) sigma, and equality with numpy's definition
    rng = np.random.default_rng(4)
    c = random_cache(rng, B=1, Hkv=1, T=3 * 64, d=16, b=64)
    _, _, mu, sg, _ = orc.block_summaries(c, raw=True)
    _, _, mu_e, sg_e, _ = orc.block_summaries(c, envelope=True, raw=True)
    np.testing.assert_array_equal(mu, mu_e)
    assert np.all(sg_e >= sg - 1e-14) and np.all(sg_e <= math.sqrt(64 / 4) * sg + 1e-14)
    Kv = bf16_values(c.K).reshape(1, 1, 3, 16, 4, 16)
    ref = np.sqrt(((Kv - mu[:, :, :, None, None, :]) ** 2).mean(axis=4)).max(axis=3)
    np.testing.assert_allclose(sg_e, ref, rtol=1e-13)


# --------------------------------------------------------------------------
# threshold predictor (Eq. tau_pred)
# --------------------------------------------------------------------------

def test_predictor_is_head_major_concat_times_W_plus_bias():
    rng = np.random.default_rng(5)
    B, Hq, d = 3, 4, 8
    q = bf16_bits_from_f64(rng.standard_normal((B, Hq, d)))
    W = rng.standard_normal((Hq * d, Hq)).astype(np.float32)
    bias = rng.standard_normal(Hq).astype(np.float32)
    ref = bf16_values(q).reshape(B, Hq * d) @ W.astype(np.float64) + bias.astype(np.float64)
    np.testing.assert_allclose(orc.predict_threshold(q, W, bias), ref, rtol=1e-13, atol=1e-13)
    # start-dense initialisation: W = 0 gives tau = bias = -8 for every query
    tau0 = orc.predict_threshold(q, np.zeros_like(W), np.full(Hq, -8.0, np.float32))
    assert np.all(tau0 == -8.0)


# --------------------------------------------------------------------------
# Score_dual (Eq. dual_bound_eq)
# --------------------------------------------------------------------------

def _setup_bound(seed=6, B=2, Hq=4, Hkv=2, T=6 * 16, d=16, b=16, scale=1.0):
    rng = np.random.default_rng(seed)
    c = random_cache(rng, B, Hkv, T, d, b, scale=scale)
    q = bf16_bits_from_f64(rng.standard_normal((B, Hq, d)))
    musig, mnorm = orc.block_summaries(c)
    return rng, c, q, musig, mnorm


def test_bound_matches_formula_written_with_numpy():
    _, c, q, musig, mnorm = _setup_bound()
    z, s = 1.5, 1 / math.sqrt(16)
    bound, g, sp = orc.score_dual(q, musig, mnorm, c.seq_lens, 16, z, parts=True)
    qv = bf16_values(q)                                     # [B,Hq,d]
    mu = fp16_values(musig[:, :, :, 0])                     # [B,Hkv,NB,d]
    sg = fp16_values(musig[:, :, :, 1])
    G = 2
    for h in range(4):
        hk = h // G
        dot = np.einsum("bd,bjd->bj", qv[:, h], mu[:, hk])
        var = np.einsum("bd,bjd->bj", qv[:, h] ** 2, sg[:, hk] ** 2)
        gg = s * (dot + z * np.sqrt(var))
        ss = s * np.linalg.norm(qv[:, h], axis=-1)[:, None] * mnorm[:, hk].astype(np.float64)
        np.testing.assert_allclose(g[:, h], gg, rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(sp[:, h], ss, rtol=1e-12)
        np.testing.assert_allclose(bound[:, h], np.minimum(gg, ss), rtol=1e-12, atol=1e-13)


def test_bound_homogeneity_monotone_in_z_and_centroid_logit_at_z0():
    _, c, q, musig, mnorm = _setup_bound(seed=7)
    b1 = orc.score_dual(q, musig, mnorm, c.seq_lens, 16, 1.0)
    # positive homogeneity: Score(2q) = 2 Score(q)  (2q is exact in bf16)
    q2 = bf16_bits_from_f64(2.0 * bf16_values(q))
    np.testing.assert_allclose(orc.score_dual(q2, musig, mnorm, c.seq_lens, 16, 1.0), 2 * b1, rtol=1e-13)
    # monotone in z
    b2 = orc.score_dual(q, musig, mnorm, c.seq_lens, 16, 2.0)
    assert np.all(b2 >= b1 - 1e-15)
    # z = 0: the moment term is the centroid logit
    _, g0, _ = orc.score_dual(q, musig, mnorm, c.seq_lens, 16, 0.0, parts=True)
    mu = fp16_values(musig[:, :, :, 0])
    for h in range(4):
        ref = np.einsum("bd,bjd->bj", bf16_values(q)[:, h], mu[:, h // 2]) / 4.0
        np.testing.assert_allclose(g0[:, h], ref, rtol=1e-12, atol=1e-14)


def test_sphere_term_is_sound_by_brute_force_and_identical_keys_are_tight():
    _, c, q, musig, mnorm = _setup_bound(seed=8, scale=3.0)
    _, _, sp = orc.score_dual(q, musig, mnorm, c.seq_lens, 16, 1.0, parts=True)
    true_max = orc.block_max_logit(q, c)
    # Cauchy-Schwarz: s |q| M_B >= every logit of the block (fp32 rounding of M allowed for)
    assert np.all(sp * (1 + 1e-6) >= true_max)
    # brute-force cross-check of block_max_logit itself with numpy
    Kv = bf16_values(c.K).reshape(2, 2, 6, 16, 16)
    for h in range(4):
        ref = np.einsum("bd,bjtd->bjt", bf16_values(q)[:, h], Kv[:, h // 2]).max(-1) / 4.0
        np.testing.assert_allclose(true_max[:, h], ref, rtol=1e-12, atol=1e-13)
    # a block of identical keys: both terms equal the true logit when q is parallel to k; moment term always
    d, b = 16, 8
    k = np.linspace(-1, 1, d)
    K = bf16_bits_from_f64(np.broadcast_to(k, (1, 1, b, d)).copy())
    kv = bf16_values(K)[0, 0, 0]
    cc = orc.Cache(K, K.copy(), np.array([b], np.int32), b)
    ms, mn = orc.block_summaries(cc)
    assert np.array_equal(fp16_values(ms[0, 0, 0, 0]), kv)      # bf16 linspace values happen to be fp16-exact
    qq = bf16_bits_from_f64(np.random.default_rng(0).standard_normal((1, 1, d)))
    bound, g, sp2 = orc.score_dual(qq, ms, mn, cc.seq_lens, b, 3.0, parts=True)
    logit = float(bf16_values(qq)[0, 0] @ kv) / 4.0
    assert g[0, 0, 0] == pytest.approx(logit, rel=1e-12, abs=1e-14)
    assert bound[0, 0, 0] == pytest.approx(logit, rel=1e-12, abs=1e-14)
    assert sp2[0, 0, 0] >= logit


def test_cantelli_count_and_diagonal_case():
    # Finite-population Cantelli: #{k: <q,k> >= <q,mu> + z sqrt(q' Sigma q)} <= floor(b/(1+z^2)) with the
    # FULL directional variance.  With exactly diagonal covariance the stored (diagonal) form is that bound,
    # so for z > sqrt(b-1) the oracle's moment term is a certified maximum.
    rng = np.random.default_rng(9)
    d, b = 8, 16
    for z in (0.5, 1.0, 2.0, 4.0):
        for _ in range(50):
            keys = rng.standard_normal((b, d)) @ rng.standard_normal((d, d))
            q = rng.standard_normal(d)
            mu = keys.mean(0)
            Sigma = (keys - mu).T @ (keys - mu) / b
            thr = q @ mu + z * math.sqrt(q @ Sigma @ q)
            assert int((keys @ q >= thr).sum()) <= math.floor(b / (1 + z * z))
    mu0 = np.array([0.5, -1.0, 0.25, 2.0, -0.75, 1.5, 0.0, -2.0])
    s = np.array([0.5, 1.0, 0.25, 2.0, 0.125, 1.0, 0.5, 4.0])
    keys = np.concatenate([mu0 + np.diag(s), mu0 - np.diag(s)])
    K = bf16_bits_from_f64(keys.reshape(1, 1, b, d))
    c = orc.Cache(K, K.copy(), np.array([b], np.int32), b)
    ms, mn = orc.block_summaries(c)
    zc = math.sqrt(b - 1) * 1.001
    for _ in range(20):
        q = bf16_bits_from_f64(rng.standard_normal((1, 1, d)))
        _, g, _ = orc.score_dual(q, ms, mn, c.seq_lens, b, zc, parts=True)
        assert g[0, 0, 0] * (1 + 1e-3) + 1e-6 >= orc.block_max_logit(q, c)[0, 0, 0]


# --------------------------------------------------------------------------
# packed summaries (format "sigma8": mu fp16, sigma rounded up to e4m3)
# --------------------------------------------------------------------------

def _e4m3_value(code: int) -> float:
    """The e4m3 value of a code, from the format's definition: (-1)^s 2^(e-7) (1 + m/8), subnormals m/8 2^-6."""
    sgn = -1.0 if code & 0x80 else 1.0
    e, m = (code >> 3) & 0xf, code & 7
    if e == 15 and m == 7:
        return float("nan")
    return sgn * (m / 8.0 * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7))


def test_e4m3_decode_and_round_up_over_every_code():
    vals = [_e4m3_value(c) for c in range(256)]
    for c in range(256):
        got = orc.e4m3_to_double(c)
        assert (math.isnan(got) and math.isnan(vals[c])) or got == vals[c]
    assert vals[0x7e] == 448.0 and vals[0x01] == 2.0 ** -9 and vals[0x08] == 2.0 ** -6
    # every e4m3 value is an fp16 value (what lets the packed record be read as an fp16 record)
    assert all(orc.fp16_to_double(orc.double_to_fp16(v)) == v for v in vals[:0x7f])
    # rounding toward +infinity: a representable value maps to itself, anything just above it to the next code
    for c in range(0x7f):
        assert orc.double_to_e4m3_up(vals[c]) == c
        assert orc.double_to_e4m3_up(np.nextafter(vals[c], np.inf)) == c + 1        # 0x7e + 1 = the NaN code
    assert orc.double_to_e4m3_up(1e9) == 0x7f and orc.double_to_e4m3_up(float("nan")) == 0x7f
    rng = np.random.default_rng(3)
    xs = np.abs(rng.standard_normal(3000)) * 10.0 ** rng.integers(-4, 3, 3000)
    up = np.array([vals[orc.double_to_e4m3_up(x)] for x in xs])
    ok = xs <= 448
    assert np.all(up[ok] >= xs[ok])
    normal = ok & (xs >= 2.0 ** -6)
    assert np.all(up[normal] <= xs[normal] * (1 + 1 / 8.0))        # at most one part in eight above
    assert np.all(np.isnan(up[~ok]))


def test_packed_record_layout_size_and_exact_expansion():
    rng = np.random.default_rng(12)
    d, b = 64, 64
    c = random_cache(rng, 2, 2, 5 * b + 3, d, b, scale=0.7)
    musig, mnorm, _, sg_raw, _ = orc.block_summaries(c, raw=True)
    ms8, mn8 = orc.block_summaries_sigma8(c)
    assert ms8.shape[-1] == 3 * d and np.array_equal(mn8, mnorm)          # M (the sphere term's input) is untouched
    # 3 d + 4 bytes per block and KV head against 4 b d bytes of K and V: 1.2 % at b = 64 (1.6 % unpacked)
    assert (3 * d + 4) / (4 * b * d) == pytest.approx(0.0120, abs=2e-4)
    NB = 5
    # mu bytes are the fp16 centroid, byte for byte
    assert np.array_equal(ms8[:, :, :NB, :2 * d].copy().view(np.uint16), musig[:, :, :NB, 0])
    # sigma^ is the smallest e4m3 value that is >= sigma (numpy restatement over the table of values)
    table = np.array([_e4m3_value(k) for k in range(0x7f)])
    want = np.searchsorted(table, sg_raw[:, :, :NB], side="left").astype(np.uint8)
    assert np.array_equal(ms8[:, :, :NB, 2 * d:], want)
    # expansion to the fp16 layout is exact and never below the fp16 sigma
    exp = orc.unpack_sigma8(ms8)
    assert np.array_equal(exp[:, :, :NB, 0], musig[:, :, :NB, 0])
    assert np.array_equal(fp16_values(exp[:, :, :NB, 1]), table[want])
    assert np.all(fp16_values(exp[:, :, :NB, 1]) >= fp16_values(musig[:, :, :NB, 1]))


def test_packed_bound_never_falls_below_the_fp16_bound_and_keeps_the_sphere_term():
    rng = np.random.default_rng(13)
    for scale in (0.05, 1.0, 30.0):
        c = random_cache(rng, 2, 2, 12 * 16, 16, 16, scale=scale)
        q = bf16_bits_from_f64(rng.standard_normal((2, 4, 16)) * 2.0)
        musig, mnorm = orc.block_summaries(c)
        ms8, _ = orc.block_summaries_sigma8(c)
        exp = orc.unpack_sigma8(ms8)
        for z in (0.0, 1.0, 2.5):
            b16, g16, s16 = orc.score_dual(q, musig, mnorm, c.seq_lens, 16, z, parts=True)
            b8, g8, s8 = orc.score_dual(q, exp, mnorm, c.seq_lens, 16, z, parts=True)
            assert np.all(b8 >= b16) and np.all(g8 >= g16)              # every (query head, block): no new false negative
            assert np.array_equal(s8, s16)                              # the Cauchy-Schwarz ceiling is bit-identical
            if z == 0.0:
                assert np.array_equal(g8, g16)                          # without the variance term nothing changes
            else:
                # and it is not much looser: the variance term grows by at most one part in eight
                var16 = (g16 - orc.score_dual(q, musig, mnorm, c.seq_lens, 16, 0.0, parts=True)[1])
                assert np.all(g8 - g16 <= var16 / 8.0 + 1e-12)
    # selection on packed summaries is a superset of the selection on fp16 summaries at the same thresholds
    # (thresholds that admit about a third of the blocks of every head, so that no rescue interferes)
    tau = np.nanquantile(b16, 0.7, axis=2).astype(np.float32)
    sel16, r16 = orc.select(b16, c.seq_lens, 16, 2, tau=tau, rescue_window=1 << 30)
    sel8, r8 = orc.select(b8, c.seq_lens, 16, 2, tau=tau, rescue_window=1 << 30)
    assert np.all(r16 < 0) and np.all(r8 < 0)
    assert np.all((sel16 & ~sel8) == 0) and sel8.sum() >= sel16.sum() > 0


def test_packed_identical_keys_stay_tight_and_huge_sigma_admits():
    d, b = 16, 8
    k = np.linspace(-1, 1, d)
    K = bf16_bits_from_f64(np.broadcast_to(k, (1, 1, b, d)).copy())
    cc = orc.Cache(K, K.copy(), np.array([b], np.int32), b)
    ms8, mn = orc.block_summaries_sigma8(cc)
    assert not ms8[0, 0, 0, 2 * d:].any()                               # sigma = 0 stays 0
    qq = bf16_bits_from_f64(np.random.default_rng(0).standard_normal((1, 1, d)))
    bound, g, _ = orc.score_dual(qq, orc.unpack_sigma8(ms8), mn, cc.seq_lens, b, 3.0, parts=True)
    logit = float(bf16_values(qq)[0, 0] @ bf16_values(K)[0, 0, 0]) / 4.0
    assert g[0, 0, 0] == pytest.approx(logit, rel=1e-12, abs=1e-14)
    # a coordinate whose spread exceeds e4m3's range: NaN code, NaN bound, block admitted whatever the threshold
    Kbig = bf16_values(K).copy()
    Kbig[0, 0, ::2, 3] = 3000.0
    Kbig[0, 0, 1::2, 3] = -3000.0
    cb = orc.Cache(bf16_bits_from_f64(Kbig), K.copy(), np.array([b], np.int32), b)
    ms8b, mnb = orc.block_summaries_sigma8(cb)
    assert ms8b[0, 0, 0, 2 * d + 3] == 0x7f
    bb = orc.score_dual(qq, orc.unpack_sigma8(ms8b), mnb, cb.seq_lens, b, 1.0)
    assert np.isnan(bb[0, 0, 0])
    sel, _ = orc.select(bb, cb.seq_lens, b, 1, tau=np.full((1, 1), 1e30, np.float32))
    assert sel[0, 0, 0] == 1


# --------------------------------------------------------------------------
# selection (Algorithm 3: threshold, rescue; lwb pinning)
# --------------------------------------------------------------------------

def test_selection_extremes_nesting_offset_and_start_dense():
    rng, c, q, musig, mnorm = _setup_bound(seed=10, B=2, Hq=4, Hkv=2, T=40 * 16 + 5, d=16, b=16)
    NB = 40
    bound = orc.score_dual(q, musig, mnorm, c.seq_lens, 16, 1.0)
    full = np.zeros((2, 2, c.NBcap), np.uint8)
    full[:, :, :NB] = 0b11
    # tau = -inf: every full block, every head
    sel, resc = orc.select(bound, c.seq_lens, 16, 2, tau=np.full((2, 4), -np.inf))
    assert np.array_equal(sel, full) and np.all(resc == -1)
    # start-dense initialisation tau = -8 on N(0,1) data: 100% of blocks pass
    sel8, _ = orc.select(bound, c.seq_lens, 16, 2, tau=np.full((2, 4), -8.0))
    assert np.array_equal(sel8, full)
    # tau = +inf: only the rescue block (first argmax of the window) and the lwb pinned blocks
    sel, resc = orc.select(bound, c.seq_lens, 16, 2, tau=np.full((2, 4), np.inf), lwb=2, rescue_window=16)
    for i in range(2):
        for h in range(4):
            expect = np.zeros(c.NBcap, bool)
            expect[NB - 2:NB] = True
            r = int(np.argmax(bound[i, h, :16]))            # np.argmax returns the first maximiser
            expect[r] = True
            assert resc[i, h] == r
            assert np.array_equal(((sel[i, h // 2] >> (h % 2)) & 1).astype(bool), expect)
    # a pinned block inside the window counts as attended: no rescue then
    sel, resc = orc.select(bound, c.seq_lens, 16, 2, tau=np.full((2, 4), np.inf), lwb=2, rescue_window=1 << 30)
    assert np.all(resc == -1)
    assert np.all(sel[:, :, :NB - 2] == 0) and np.all(sel[:, :, NB - 2:NB] == 0b11)
    # nesting: a higher threshold admits a subset (rescue aside)
    t1 = rng.standard_normal((2, 4)).astype(np.float32) * 0.3 + 1.0
    s1, _ = orc.select(bound, c.seq_lens, 16, 2, tau=t1, rescue_window=1)
    s2, _ = orc.select(bound, c.seq_lens, 16, 2, tau=t1 + 0.5, rescue_window=1)
    assert np.all((s2[:, :, 1:] & ~s1[:, :, 1:]) == 0)
    assert 0 < (s2 != 0).sum() < (s1 != 0).sum() < full.astype(bool).sum()
    # plain definition with numpy for the thresholded part
    for h in range(4):
        ref = ~(bound[:, h, 1:NB] < t1[:, h:h + 1].astype(np.float64))
        assert np.array_equal(((s1[:, h // 2, 1:NB] >> (h % 2)) & 1).astype(bool), ref)
    # operating offset: sel(tau, a) = sel(tau - a, 0)   (0.25 keeps the float32 subtraction exact enough)
    ta = np.round(t1 * 4) / 4
    sa, _ = orc.select(bound, c.seq_lens, 16, 2, tau=ta, a=0.25)
    sb, _ = orc.select(bound, c.seq_lens, 16, 2, tau=ta - 0.25, a=0.0)
    assert np.array_equal(sa, sb)
    # frozen constants are per query head and independent of the sequence
    cst = np.array([0.5, 1.0, 1.5, 2.0], np.float32)
    sc, _ = orc.select(bound, c.seq_lens, 16, 2, head_const=cst)
    st, _ = orc.select(bound, c.seq_lens, 16, 2, tau=np.broadcast_to(cst, (2, 4)).copy())
    assert np.array_equal(sc, st)


def test_rescue_tie_goes_to_lowest_index_and_equal_bound_is_admitted():
    bound = np.array([[[1.0, 3.0, 3.0, 2.0]]])
    lens = np.array([4 * 8], np.int32)
    sel, resc = orc.select(bound, lens, 8, 1, tau=np.array([[5.0]]))
    assert resc[0, 0] == 1 and sel[0, 0].tolist() == [0, 1, 0, 0]
    # bound == tau_eff is admitted ("bypassed" needs a strict <)
    sel, resc = orc.select(bound, lens, 8, 1, tau=np.array([[3.0]]))
    assert sel[0, 0].tolist() == [0, 1, 1, 0] and resc[0, 0] == -1
    # a NaN bound is admitted (not below the threshold)
    bn = np.array([[[1.0, np.nan, 0.0, 0.0]]])
    sel, _ = orc.select(bn, lens, 8, 1, tau=np.array([[5.0]]))
    assert sel[0, 0].tolist() == [0, 1, 0, 0]
    # rescue looks only inside its window
    sel, resc = orc.select(bound, lens, 8, 1, tau=np.array([[5.0]]), rescue_window=1)
    assert resc[0, 0] == 0 and sel[0, 0].tolist() == [1, 0, 0, 0]


# --------------------------------------------------------------------------
# the shifted-SiLU gate (Section 2.2 closed forms)
# --------------------------------------------------------------------------

def test_gate_closed_forms():
    beta, tau = 5.0, 2.81
    f = lambda S: orc.gate(S, tau, beta)
    # value at the threshold is tau/2 and the slope there is (1 + beta tau / 2) / 2
    assert f(tau) == pytest.approx(tau / 2, rel=1e-15)
    h = 1e-6
    assert (f(tau + h) - f(tau - h)) / (2 * h) == pytest.approx(0.5 * (1 + beta * tau / 2), rel=1e-8)
    # unique minimiser S* = -(1 + W0(e^{-1-beta tau}))/beta with value -W0(.)/beta, and -1.28/beta < S* < -1/beta
    w = float(lambertw(math.exp(-1 - beta * tau)).real)
    s_star = -(1 + w) / beta
    grid = np.linspace(-3, 3, 600001)
    vals = np.array([f(x) for x in grid[::50]])
    assert abs(grid[::50][vals.argmin()] - s_star) < 1e-3
    assert f(s_star) == pytest.approx(-w / beta, rel=1e-9)
    assert -1.28 / beta < s_star < -1 / beta
    assert (f(s_star + h) - f(s_star - h)) / (2 * h) == pytest.approx(0.0, abs=1e-8)
    # regime 1 (tau << -2/beta): the gate is the identity on the support of the scores
    assert orc.gate(1.3, -8.0, 1.0) == pytest.approx(1.3 / (1 + math.exp(-9.3)), rel=1e-15)
    # sigma'(8) = 3.35e-4: the low-gradient regime of the start-dense initialisation
    sg8 = orc.gate(1.0, 1.0 - 8.0, 1.0)                  # = sigmoid(8)
    assert sg8 * (1 - sg8) == pytest.approx(3.35e-4, rel=2e-3)
    # limits
    assert orc.gate(0.7, -math.inf, 5.0) == 0.7
    assert orc.gate(0.7, math.inf, 5.0) == 0.0
    assert orc.gate(-3.0, math.inf, 5.0) == 0.0
    assert orc.gate(0.7, 123.0, 0.0) == 0.35


# --------------------------------------------------------------------------
# gated attention over admitted blocks
# --------------------------------------------------------------------------

def _attn_case(seed=11, B=2, Hq=4, Hkv=2, T=5 * 16 + 9, d=16, b=16):
    rng = np.random.default_rng(seed)
    c = random_cache(rng, B, Hkv, T, d, b)
    q = bf16_bits_from_f64(rng.standard_normal((B, Hq, d)) * 1.5)
    return rng, c, q


def test_minus_infinite_threshold_is_textbook_softmax_attention():
    _, c, q = _attn_case()
    B, Hq, d, T = 2, 4, 16, int(c.seq_lens[0])
    full = np.full((B, 2, c.NBcap), 0b11, np.uint8)
    out = orc.gated_block_attention(q, c, full, tau=np.full((B, Hq), -np.inf), beta=5.0)
    # library routine: torch scaled_dot_product_attention in float64 with GQA heads expanded
    qt = torch.from_numpy(bf16_values(q))[:, :, None, :]
    Kt = torch.from_numpy(bf16_values(c.K))[:, :, :T].repeat_interleave(2, dim=1)
    Vt = torch.from_numpy(bf16_values(c.V))[:, :, :T].repeat_interleave(2, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(qt, Kt, Vt)[:, :, 0].numpy()
    np.testing.assert_allclose(out, ref, rtol=1e-11, atol=1e-13)
    # and the oracle's own, separately written, dense routine agrees with the library too
    np.testing.assert_allclose(orc.dense_softmax_attention(q, c), ref, rtol=1e-11, atol=1e-13)


def test_plus_infinite_threshold_is_the_mean_of_loaded_values_and_beta0_is_half_scale():
    _, c, q = _attn_case(seed=12)
    B, Hq, T = 2, 4, int(c.seq_lens[0])
    sel = np.zeros((B, 2, c.NBcap), np.uint8)
    sel[:, :, 1] = 0b01                                    # head 0 of each group: block 1
    sel[:, :, 3] = 0b11                                    # both heads: block 3
    out, logZ, ntok = orc.gated_block_attention(q, c, sel, tau=np.full((B, Hq), np.inf), extras=True)
    Vv = bf16_values(c.V)
    tail = list(range(5 * 16, T))
    for h in range(Hq):
        toks = (list(range(16, 32)) if h % 2 == 0 else []) + list(range(48, 64)) + tail
        np.testing.assert_allclose(out[:, h], Vv[:, h // 2][:, toks].mean(axis=1), rtol=1e-12, atol=1e-14)
        assert np.all(ntok[:, h] == len(toks))
        np.testing.assert_allclose(logZ[:, h], math.log(len(toks)), rtol=1e-13)
    # beta = 0: S~ = S/2, i.e. softmax attention at half the scale, for any finite tau
    full = np.full((B, 2, c.NBcap), 0b11, np.uint8)
    o0 = orc.gated_block_attention(q, c, full, tau=np.full((B, Hq), 0.37), beta=0.0)
    np.testing.assert_allclose(o0, orc.dense_softmax_attention(q, c, scale=0.5 / 4.0), rtol=1e-11, atol=1e-13)


def test_general_case_against_per_token_brute_force_and_sibling_blocks_are_not_attended():
    rng, c, q = _attn_case(seed=13)
    B, Hq, d, b, T = 2, 4, 16, 16, int(c.seq_lens[0])
    NB = T // b
    sel = rng.integers(0, 4, size=(B, 2, c.NBcap)).astype(np.uint8)
    sel[:, :, 0] |= 1
    tau = rng.standard_normal((B, Hq)).astype(np.float32)
    a, beta = 0.25, 3.0
    out, logZ, ntok = orc.gated_block_attention(q, c, sel, tau=tau, a=a, beta=beta, extras=True)
    qv, Kv, Vv = bf16_values(q), bf16_values(c.K), bf16_values(c.V)
    for i in range(B):
        for h in range(Hq):
            te = float(tau[i, h]) - a
            num = np.zeros(d)
            den = 0.0
            n = 0
            for p in range(T):
                j = p // b
                if j < NB and not (sel[i, h // 2, j] >> (h % 2)) & 1:
                    continue
                S = float(qv[i, h] @ Kv[i, h // 2, p]) / math.sqrt(d)
                St = S / (1.0 + math.exp(-beta * (S - te)))
                w = math.exp(St)
                num += w * Vv[i, h // 2, p]
                den += w
                n += 1
            np.testing.assert_allclose(out[i, h], num / den, rtol=1e-11, atol=1e-13)
            assert logZ[i, h] == pytest.approx(math.log(den), rel=1e-12)
            assert ntok[i, h] == n


def test_exact_output_decomposition_and_skipped_mass_bound():
    # Z_all o_train = Z_load o_block + Z_D v_D  (exact), hence
    # |o_train - o_block| <= (Z_D / Z_all) max_{s in D} |v_s - o_block|.
    rng, c, q = _attn_case(seed=14, T=8 * 16 + 3)
    B, Hq, b, T = 2, 4, 16, int(c.seq_lens[0])
    NB = T // b
    musig, mnorm = orc.block_summaries(c)
    tau = np.full((B, Hq), 0.9, np.float32)
    res = orc.decode_step(q, c, musig, mnorm, tau=tau, z=1.0, beta=5.0, rescue_window=4)
    sel = res["sel"]
    assert 0 < sum(bin(int(x)).count("1") for x in sel.ravel()) < B * Hq * NB   # genuinely sparse
    full = np.full_like(sel, 0b11)
    o_train, lz_all, _ = orc.gated_block_attention(q, c, full, tau=tau, extras=True)
    o_block, lz_load, _ = orc.gated_block_attention(q, c, sel, tau=tau, extras=True)
    # the dropped set alone: complement of the mask; its tail tokens must not be counted twice, so
    # compute Z_D and v_D directly
    qv, Kv, Vv = bf16_values(q), bf16_values(c.K), bf16_values(c.V)
    for i in range(B):
        for h in range(Hq):
            ZD, vD, worst = 0.0, np.zeros(16), 0.0
            for p in range(NB * b):
                if (sel[i, h // 2, p // b] >> (h % 2)) & 1:
                    continue
                S = float(qv[i, h] @ Kv[i, h // 2, p]) / 4.0
                w = math.exp(orc.gate(S, float(np.float32(0.9)), 5.0))   # tau travels as float32
                ZD += w
                vD += w * Vv[i, h // 2, p]
                worst = max(worst, float(np.linalg.norm(Vv[i, h // 2, p] - o_block[i, h])))
            Zall, Zload = math.exp(lz_all[i, h]), math.exp(lz_load[i, h])
            assert Zall == pytest.approx(Zload + ZD, rel=1e-12)
            np.testing.assert_allclose(Zall * o_train[i, h], Zload * o_block[i, h] + vD, rtol=1e-10, atol=1e-12)
            assert np.linalg.norm(o_train[i, h] - o_block[i, h]) <= (ZD / Zall) * worst + 1e-12


def test_screening_soundness_where_the_paper_certifies_it():
    # With z huge the bound is the sphere term alone (exact Cauchy-Schwarz): every skipped block's true
    # maximum logit lies below tau_eff, by brute force; and then each skipped key weighs at most
    # max(1, exp(tau_eff/2)), so Z_D <= |D| max(1, exp(tau_eff/2)).
    rng = np.random.default_rng(15)
    c = random_cache(rng, 1, 2, 24 * 8, 8, 8)
    # spread the key norms so that the sphere term separates blocks
    Kv = bf16_values(c.K) * np.repeat(rng.uniform(0.2, 2.0, (1, 2, 24)), 8, axis=2)[..., None]
    c = orc.Cache(bf16_bits_from_f64(Kv), c.V, c.seq_lens, 8)
    q = bf16_bits_from_f64(rng.standard_normal((1, 4, 8)))
    musig, mnorm = orc.block_summaries(c)
    bound, g, sp = orc.score_dual(q, musig, mnorm, c.seq_lens, 8, 1e6, parts=True)
    np.testing.assert_array_equal(bound, sp)
    tau = np.quantile(bound[0], 0.6, axis=1)[None, :].astype(np.float32)
    sel, _ = orc.select(bound, c.seq_lens, 8, 2, tau=tau, rescue_window=1)
    true_max = orc.block_max_logit(q, c)
    skipped = 0
    for h in range(4):
        for j in range(24):
            if not (sel[0, h // 2, j] >> (h % 2)) & 1:
                skipped += 1
                assert true_max[0, h, j] < float(tau[0, h])
    assert skipped > 20
    o_all, lz_all, _ = orc.gated_block_attention(q, c, np.full_like(sel, 3), tau=tau, extras=True)
    o_blk, lz_blk, n_blk = orc.gated_block_attention(q, c, sel, tau=tau, extras=True)
    for h in range(4):
        ZD = math.exp(lz_all[0, h]) - math.exp(lz_blk[0, h])
        nD = 24 * 8 - int(n_blk[0, h])
        assert ZD <= nD * max(1.0, math.exp(float(tau[0, h]) / 2)) * (1 + 1e-9)


def test_decode_step_composes_the_three_stages():
    rng, c, q = _attn_case(seed=16, T=12 * 16 + 4)
    musig, mnorm = orc.block_summaries(c)
    tau = np.full((2, 4), 0.8, np.float32)
    res = orc.decode_step(q, c, musig, mnorm, tau=tau, z=1.0, lwb=2, rescue_window=8)
    bound = orc.score_dual(q, musig, mnorm, c.seq_lens, 16, 1.0)
    sel, _ = orc.select(bound, c.seq_lens, 16, 2, tau=tau, lwb=2, rescue_window=8)
    assert np.array_equal(res["sel"], sel)
    np.testing.assert_array_equal(res["out"], orc.gated_block_attention(q, c, sel, tau=tau))


def test_ungated_newest_token_closed_forms():
    """Eq. mult_attn leaves the diagonal s = t ungated; at decode time that is the newest token."""
    _, c, q = _attn_case(seed=21)
    B, Hq, d, T = 2, 4, 16, int(c.seq_lens[0])
    Kv, Vv, qv = bf16_values(c.K), bf16_values(c.V), bf16_values(q)
    full = np.full((B, 2, c.NBcap), 0b11, np.uint8)
    # tau = -inf: every gate is open already, the flag changes nothing (textbook softmax either way)
    a0 = orc.gated_block_attention(q, c, full, tau=np.full((B, Hq), -np.inf), ungate_last=False)
    a1 = orc.gated_block_attention(q, c, full, tau=np.full((B, Hq), -np.inf), ungate_last=True)
    np.testing.assert_array_equal(a0, a1)
    # tau = +inf: every gated logit is 0 (weight 1); the newest token keeps its raw logit S, so
    #   out = (sum of the other values + e^S v_last) / (T - 1 + e^S)
    out = orc.gated_block_attention(q, c, full, tau=np.full((B, Hq), np.inf), ungate_last=True)
    for i in range(B):
        for h in range(Hq):
            S = (qv[i, h] @ Kv[i, h // 2, T - 1]) / math.sqrt(d)
            num = Vv[i, h // 2, :T - 1].sum(axis=0) + math.exp(S) * Vv[i, h // 2, T - 1]
            np.testing.assert_allclose(out[i, h], num / (T - 1 + math.exp(S)), rtol=1e-12, atol=1e-14)
    # beta = 0: the others sit at half scale, the newest token at full scale
    out = orc.gated_block_attention(q, c, full, tau=np.full((B, Hq), 0.3), beta=0.0, ungate_last=True)
    for i in range(B):
        for h in range(Hq):
            S = (Kv[i, h // 2, :T] @ qv[i, h]) / math.sqrt(d)
            w = np.exp(np.concatenate([0.5 * S[:-1], S[-1:]]))
            np.testing.assert_allclose(out[i, h], (w[:, None] * Vv[i, h // 2, :T]).sum(0) / w.sum(), rtol=1e-11, atol=1e-13)


def test_ungated_newest_token_forces_its_block_when_it_closes_one():
    rng = np.random.default_rng(5)
    B, Hq, Hkv, b, NB = 2, 4, 2, 16, 6
    bound = rng.standard_normal((B, Hq, NB))
    tau = np.full((B, Hq), 10.0, np.float32)                 # nothing passes the screen
    lens = np.array([NB * b, NB * b - 3], np.int32)          # sequence 0 ends on a block boundary, sequence 1 in a tail
    sel0, _ = orc.select(bound, lens, b, Hkv, tau=tau, rescue_window=2)
    sel1, _ = orc.select(bound, lens, b, Hkv, tau=tau, rescue_window=2, ungate_last=True)
    assert np.all(sel1[0, :, NB - 1] == 0b11)                # the block holding token T-1, for every head
    sel1_rest = sel1.copy(); sel1_rest[0, :, NB - 1] = sel0[0, :, NB - 1]
    np.testing.assert_array_equal(sel1_rest, sel0)           # nothing else changes
    np.testing.assert_array_equal(sel1[1], sel0[1])          # newest token in the tail: already attended


# ---------------------------------------------------------------------------------------------------
# offline threshold calibration (1/t-weighted histogram + bisection)
# ---------------------------------------------------------------------------------------------------

def _calib_case(seed=3, n_seq=2, Hq=4, Hkv=2, T=40, d=16):
    rng = np.random.default_rng(seed)
    Q = bf16_bits_from_f64(rng.standard_normal((n_seq, Hq, T, d)))
    K = bf16_bits_from_f64(rng.standard_normal((n_seq, Hkv, T, d)))
    return rng, Q, K


def test_calibration_hand_example_of_the_causal_row_weights():
    # one sequence, one head, T = 2, d = 1: scores S11 = 1*1, S21 = 2*1, S22 = 2*3 (scale 1)
    Q = bf16_bits_from_f64(np.array([1.0, 2.0]).reshape(1, 1, 2, 1))
    K = bf16_bits_from_f64(np.array([1.0, 3.0]).reshape(1, 1, 2, 1))
    tau = np.array([0.5, 4.0], np.float32).reshape(1, 1, 2)
    r = orc.calibrate(Q, K, tau, beta=2.0, scale=1.0, n_bins=8, s_min=0.0, s_max=8.0)
    # bins of width 1: S11 = 1 -> bin 1 (weight 1), S21 = 2 -> bin 2 (1/2), S22 = 6 -> bin 6 (1/2); total 2
    expect = np.zeros(8); expect[1], expect[2], expect[6] = 0.5, 0.25, 0.25
    np.testing.assert_allclose(r["hist"][0], expect, rtol=0, atol=1e-15)
    sig = lambda x: 1.0 / (1.0 + math.exp(-x))
    dbar = 0.5 * (sig(2.0 * (1 - 0.5)) + 0.5 * (sig(2.0 * (2 - 4.0)) + sig(2.0 * (6 - 4.0))))
    np.testing.assert_allclose(r["dbar"][0], dbar, rtol=1e-14)
    # the root solves 0.5 s(1.5-c) + 0.25 s(2.5-c) + 0.25 s(6.5-c) = dbar (bin centres), to the stated residual
    g = 0.5 * sig(2 * (1.5 - r["head_const"][0])) + 0.25 * sig(2 * (2.5 - r["head_const"][0])) + 0.25 * sig(2 * (6.5 - r["head_const"][0]))
    assert abs(g - dbar) < 5e-16 and abs(r["residual"][0]) < 5e-16          # machine precision, as the paper states


def test_calibration_constant_scores_give_a_closed_form_constant():
    n_seq, Hq, T, d = 2, 2, 24, 8
    Q = bf16_bits_from_f64(np.tile(np.eye(1, d) * 1.5, (n_seq, Hq, T, 1)))
    K = bf16_bits_from_f64(np.tile(np.eye(1, d) * 2.0, (n_seq, Hq, T, 1)))
    S0, tau0, beta = 3.0 * 0.5, 0.9, 4.0                      # scale 0.5
    r = orc.calibrate(Q, K, np.full((n_seq, Hq, T), tau0, np.float32), beta=beta, scale=0.5, n_bins=64, s_min=-4, s_max=4)
    w = 8.0 / 64
    s_b = -4 + (math.floor((S0 + 4) / w) + 0.5) * w          # centre of the bin that holds every score
    tau0f = float(np.float32(tau0))
    np.testing.assert_allclose(r["dbar"], 1.0 / (1.0 + math.exp(-beta * (S0 - tau0f))), rtol=1e-13)
    np.testing.assert_allclose(r["head_const"], s_b - (S0 - tau0f), rtol=0, atol=1e-12)


def test_calibration_reproduces_a_static_threshold_and_matches_brute_force_density():
    rng, Q, K = _calib_case()
    n_seq, Hq, T, d = Q.shape
    beta, n_bins, s_min, s_max = 5.0, 1024, -6.0, 6.0
    w = (s_max - s_min) / n_bins
    tau = np.full((n_seq, Hq, T), 0.25, np.float32)
    r = orc.calibrate(Q, K, tau, beta=beta, n_bins=n_bins, s_min=s_min, s_max=s_max)
    assert np.all(np.abs(r["residual"]) < 5e-16)                        # machine precision (the paper: < 2e-16)
    assert np.all(np.abs(r["head_const"] - 0.25) < w)                   # a constant predictor calibrates to itself
    np.testing.assert_allclose(r["hist"].sum(axis=1), 1.0, rtol=1e-13)
    # g(c) from the histogram against g(c) from the raw scores: sigmoid is beta/4-Lipschitz, scores move <= w/2
    Qv, Kv = bf16_values(Q), bf16_values(K)
    for h in range(Hq):
        for c in (-1.0, 0.1, 0.25, 2.0):
            tot = 0.0
            for x in range(n_seq):
                S = (Qv[x, h] @ Kv[x, h // 2].T) / math.sqrt(d)
                for t in range(T):
                    tot += (1.0 / (1.0 + np.exp(-beta * (S[t, :t + 1] - c)))).sum() / (t + 1)
            g_raw = tot / (n_seq * T)
            g_hist = orc.calibration_density(r["hist"][h], s_min, s_max, beta, c)
            assert abs(g_raw - g_hist) <= beta * w / 8 + 1e-12
    # g decreases in c
    gs = [orc.calibration_density(r["hist"][0], s_min, s_max, beta, c) for c in np.linspace(-8, 8, 33)]
    assert all(a > b for a, b in zip(gs, gs[1:])) and gs[0] > 0.999 and gs[-1] < 1e-3


def test_calibration_matches_a_dynamic_predictor_in_density():
    rng, Q, K = _calib_case(seed=8)
    n_seq, Hq, T, d = Q.shape
    tau = (0.2 + 0.5 * rng.standard_normal((n_seq, Hq, T))).astype(np.float32)     # token-dependent thresholds
    r = orc.calibrate(Q, K, tau, beta=5.0, n_bins=2048, s_min=-6, s_max=6)
    # the static constant yields the dynamic predictor's density on the split (that is its definition)
    for h in range(Hq):
        assert abs(orc.calibration_density(r["hist"][h], -6, 6, 5.0, r["head_const"][h]) - r["dbar"][h]) < 5e-16
    assert np.all((r["dbar"] > 0.05) & (r["dbar"] < 0.95))

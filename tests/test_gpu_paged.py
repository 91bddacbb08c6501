"""Paged KV cache (Section 3: summaries in a held-out table beside a paged cache): the paged entry points are checked
against the CPU oracle run on the gathered cache (summaries within 1 fp16 ulp / 4 fp32 ulp; with the oracle's summary
bytes and the same thresholds on both sides, masks bit-exact outside the 1e-5 near-tie band, block counts exact,
outputs within 1e-2 max / 1e-3 mean), and must also give, bit for bit, what the contiguous entry points give.  Pages
are scattered by a seeded permutation; unused pages and the unused part of every tail page hold large finite garbage
that must not leak into any result."""
import numpy as np
import pytest
import torch

from oracle import eta_oracle as orc
from paper_2609_20888_b200 import workloads as wl
from tests.helpers import bits, cache_of, compare_masks, fp16_ulp_distance, heads_without_near_tie, output_errors

pytestmark = pytest.mark.gpu


def _eb():
    if not torch.cuda.is_available():
        pytest.skip("needs a GPU")
    from paper_2609_20888_b200 import binding as eb
    eb.load()
    return eb


def _scatter(K, V, lens, b, seed, layout):
    """-> K_pool, V_pool (bf16 CUDA), block_table (int32 CUDA [B, stride]), n_pages"""
    B, Hkv, Tcap, d = K.shape
    per_seq = (Tcap + b - 1) // b
    n_pages = B * per_seq + 7
    g = torch.Generator().manual_seed(seed)
    perm = torch.randperm(n_pages, generator=g)[:B * per_seq].view(B, per_seq)
    shape = (n_pages, Hkv, b, d) if layout == "phbd" else (n_pages, b, Hkv, d)
    Kp = torch.full(shape, 1.0e4, dtype=torch.bfloat16)
    Vp = torch.full(shape, -1.0e4, dtype=torch.bfloat16)
    if layout != "phbd":
        Kp, Vp = Kp.permute(0, 2, 1, 3), Vp.permute(0, 2, 1, 3)      # logical [page, head, token, dim], other strides
    for i in range(B):
        T = int(lens[i])
        for j in range((T + b - 1) // b):
            n = min(b, T - j * b)
            Kp[perm[i, j], :, :n] = K[i, :, j * b:j * b + n]
            Vp[perm[i, j], :, :n] = V[i, :, j * b:j * b + n]
    table = torch.full((B, per_seq + 3), -12345, dtype=torch.int32)      # entries past the sequence are never read
    table[:, :per_seq] = perm.to(torch.int32)
    dev = torch.device("cuda:0")
    return Kp.to(dev), Vp.to(dev), table.to(dev), n_pages


@pytest.mark.parametrize("name,ctx,batch,layout", [("c2_32k", 4096 + 77, 2, "phbd"), ("c5_frozen", 8192, 4, "pbhd"),
                                                   ("c4_512k", 16384 + 5, 1, "phbd"), ("c1_tiny", 2048 + 16, 1, "pbhd")])
def test_paged_cache_equals_contiguous_bit_for_bit(name, ctx, batch, layout):
    eb = _eb()
    dev = torch.device("cuda:0")
    sp = wl.CONFIGS[name].scaled(ctx, batch=batch)
    w = wl.make_workload(sp)
    b = sp.block_size
    lens = w.seq_lens.clone()
    K, V = w.K.to(dev), w.V.to(dev)
    lens_d = lens.to(dev)
    q = w.queries(0).to(dev)
    params = eb.DecodeParams(z=sp.z, beta=sp.beta, lwb=sp.lwb, rescue_window=sp.rescue_window)

    # contiguous reference run
    st = eb.DecodeState(K, V, sp.n_q_heads, b)
    eb.eta_build_block_summaries(st.desc, K, lens_d, st.musig, st.mnorm)
    # thresholds at each head's median bound: about half of the blocks are pruned
    bound = torch.full((sp.batch, sp.n_q_heads, st.desc.nb_cap), float("nan"), dtype=torch.float32, device=dev)
    eb.eta_score_dual(st.desc, params, q, lens_d, st.musig, st.mnorm, bound)
    # (a little above the median element, so that the threshold does not sit on a bound: the oracle comparison below
    # then has no built-in near tie)
    tau = (torch.nanmedian(bound, dim=2).values + 3e-4).contiguous()
    eb.eta_decode(st.desc, params, q, K, V, lens_d, st.musig, st.mnorm, tau, None, st.out, st.sel_mask, st.workspace,
                  stats=st.stats, status=st.status)
    torch.cuda.synchronize()
    assert int(st.status.item()) == 0
    frac = float(st.stats.sum().item()) / max(1, sum(int(t) // b for t in lens) * sp.n_kv_heads)
    assert 0.02 < frac < 0.98, "the case must prune some blocks and keep some"

    # paged run on the scattered pools
    Kp, Vp, table, n_pages = _scatter(w.K, w.V, lens, b, seed=sp.seed + 1, layout=layout)
    pdesc = eb.paged_cache_desc(Kp, Vp, sp.batch, sp.n_q_heads, t_cap=w.K.shape[2], nb_cap=st.desc.nb_cap)
    pages = eb.page_table(table, n_pages)
    musig, mnorm = eb.alloc_summaries(pdesc, dev)
    eb.eta_build_block_summaries_paged(pdesc, pages, Kp, lens_d, musig, mnorm)
    torch.cuda.synchronize()
    assert torch.equal(musig.view(torch.int16), st.musig.view(torch.int16))
    assert torch.equal(mnorm.view(torch.int32), st.mnorm.view(torch.int32))
    out = torch.full_like(st.out, float("nan"))
    sel = torch.zeros_like(st.sel_mask)
    stats = torch.zeros_like(st.stats)
    status = torch.zeros_like(st.status)
    ws = torch.zeros_like(st.workspace)
    eb.eta_decode_paged(pdesc, pages, params, q, Kp, Vp, lens_d, musig, mnorm, tau, None, out, sel, ws,
                        stats=stats, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(sel, st.sel_mask)
    assert torch.equal(stats, st.stats)
    assert torch.equal(out.view(torch.int32), st.out.view(torch.int32))

    # the paged path against the oracle on the gathered cache: first the paged summary build ...
    c = cache_of(w)
    o_musig, o_mnorm = orc.block_summaries(c)
    got_ms, got_mn = bits(musig.cpu()), mnorm.cpu().numpy()
    for i in range(sp.batch):
        NB = int(lens[i]) // b
        assert fp16_ulp_distance(got_ms[i, :, :NB], o_musig[i, :, :NB]).max(initial=0) <= 1
        assert np.abs(got_mn[i, :, :NB].view(np.int32) - o_mnorm[i, :, :NB].view(np.int32)).max(initial=0) <= 4
    # ... then the paged decode on the oracle's summary bytes and the same fp32 thresholds
    tau_np = tau.cpu().numpy()
    ref = orc.decode_step(bits(w.queries(0)), c, o_musig, o_mnorm, tau=tau_np, z=sp.z, beta=sp.beta, lwb=sp.lwb,
                          rescue_window=sp.rescue_window)
    musig.copy_(torch.from_numpy(o_musig.view(np.int16)).view(torch.float16).to(dev))
    mnorm.copy_(torch.from_numpy(o_mnorm).to(dev))
    out.fill_(float("nan"))
    eb.eta_decode_paged(pdesc, pages, params, q, Kp, Vp, lens_d, musig, mnorm, tau, None, out, sel, ws,
                        stats=stats, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    sel_np, out_np = sel.cpu().numpy(), out.cpu().numpy()
    near = compare_masks(sel_np, ref["sel"], ref["bound"], tau_np.astype(np.float64), c.seq_lens, b, sp.gqa,
                         rescued=ref["rescued"])
    keep = heads_without_near_tie(near, sp.batch, sp.n_q_heads)
    assert keep.mean() > 0.9
    mx, mean = output_errors(out_np[keep], ref["out"][keep])
    assert mx <= 1e-2 and mean <= 1e-3, (mx, mean)
    union = np.array([[int((sel_np[i, hk, :int(lens[i]) // b] != 0).sum()) for hk in range(sp.n_kv_heads)]
                      for i in range(sp.batch)])
    assert np.array_equal(stats.cpu().numpy(), union)
    if not near:
        assert np.array_equal(sel_np, ref["sel"])


def test_paged_append_equals_paged_rebuild():
    """Appending tokens until a block fills up: the paged append writes the record the paged build writes."""
    eb = _eb()
    dev = torch.device("cuda:0")
    sp = wl.CONFIGS["c2_32k"].scaled(2048, batch=3)
    w = wl.make_workload(sp)
    b = sp.block_size
    lens = torch.tensor([2048 - b, 2048 - 2 * b, 2048 - b - 5], dtype=torch.int32)
    Kp, Vp, table, n_pages = _scatter(w.K, w.V, torch.full((3,), 2048), b, seed=7, layout="phbd")
    pdesc = eb.paged_cache_desc(Kp, Vp, sp.batch, sp.n_q_heads, t_cap=2048)
    pages = eb.page_table(table, n_pages)
    musig, mnorm = eb.alloc_summaries(pdesc, dev)
    eb.eta_build_block_summaries_paged(pdesc, pages, Kp, lens.to(dev), musig, mnorm)
    after = lens + torch.tensor([b, b, 5], dtype=torch.int32)          # all three now end on a block boundary
    eb.eta_append_summary_paged(pdesc, pages, Kp, after.to(dev), musig, mnorm)
    ref_musig, ref_mnorm = eb.alloc_summaries(pdesc, dev)
    eb.eta_build_block_summaries_paged(pdesc, pages, Kp, after.to(dev), ref_musig, ref_mnorm)
    torch.cuda.synchronize()
    assert torch.equal(musig.view(torch.int16), ref_musig.view(torch.int16))
    assert torch.equal(mnorm.view(torch.int32), ref_mnorm.view(torch.int32))


def test_paged_arguments_are_validated():
    eb = _eb()
    dev = torch.device("cuda:0")
    Kp = torch.zeros((8, 2, 32, 64), dtype=torch.bfloat16, device=dev)
    pdesc = eb.paged_cache_desc(Kp, Kp, 1, 4, t_cap=128)
    lens = torch.tensor([64], dtype=torch.int32, device=dev)
    musig, mnorm = eb.alloc_summaries(pdesc, dev)
    short = torch.zeros((1, 3), dtype=torch.int32, device=dev)           # 3 * 32 < t_cap
    with pytest.raises(eb.EtaError):
        eb.eta_build_block_summaries_paged(pdesc, eb.page_table(short, 8), Kp, lens, musig, mnorm)
    ok = torch.zeros((1, 4), dtype=torch.int32, device=dev)
    with pytest.raises(eb.EtaError):
        eb.eta_build_block_summaries_paged(pdesc, eb.page_table(ok, 0), Kp, lens, musig, mnorm)


def test_shared_prefix_batch_whose_counts_do_not_fit_the_set_up_buffer():
    """128 sequences that share one 311 K-token prefix through their page tables (1024 rows of 153 segments): the
    streaming kernel's set-up cannot keep the per-segment counts of all rows in shared memory and reads them from
    global memory window by window, and its row search runs over more than 32 rows.  The oracle is run on three
    sampled sequences (each gathered into a contiguous cache of its own); every row is checked for the properties
    that hold at any size (status, finite outputs, block counts equal to the mask's)."""
    eb = _eb()
    dev = torch.device("cuda:0")
    B, Hkv, G, d, b = 128, 8, 1, 64, 32
    nb_full = 152 * 64
    t_cap = nb_full * b + b
    rng = np.random.default_rng(4242)
    K = torch.from_numpy(rng.standard_normal((1, Hkv, t_cap, d), dtype=np.float32)).to(torch.bfloat16)
    V = torch.from_numpy(rng.standard_normal((1, Hkv, t_cap, d), dtype=np.float32)).to(torch.bfloat16)
    q = torch.from_numpy(rng.standard_normal((B, Hkv * G, d), dtype=np.float32)).to(torch.bfloat16)
    lens = np.full(B, nb_full * b + 7, np.int32)
    lens[77] = 5000 * b                        # a shorter sharer that ends on a block boundary
    lens[127] = 9000 * b + 31
    lens[3] = 11                               # and one that holds a tail only
    Kp, Vp, table1, n_pages = _scatter(K, V, [t_cap], b, seed=5, layout="phbd")
    table = table1.expand(B, -1).contiguous()
    pdesc = eb.paged_cache_desc(Kp, Vp, B, Hkv * G, t_cap=t_cap)
    pages = eb.page_table(table, n_pages)
    # the oracle's summaries of the shared prefix, the same bytes for every sharer
    c1 = orc.Cache(bits(K), bits(V), np.asarray([t_cap], np.int32), b)
    o_musig, o_mnorm = orc.block_summaries(c1)
    musig, mnorm = eb.alloc_summaries(pdesc, dev)
    musig.copy_(torch.from_numpy(o_musig.view(np.int16)).view(torch.float16).to(dev).expand_as(musig))
    mnorm.copy_(torch.from_numpy(o_mnorm).to(dev).expand_as(mnorm))
    lens_d = torch.from_numpy(lens).to(dev)
    qd = q.to(dev)
    params = eb.DecodeParams(z=1.0, beta=5.0, lwb=1, rescue_window=128)
    bound = torch.full((B, Hkv * G, pdesc.nb_cap), float("nan"), dtype=torch.float32, device=dev)
    eb.eta_score_dual(pdesc, params, qd, lens_d, musig, mnorm, bound)
    tau = torch.nan_to_num(torch.nanquantile(bound, 0.97, dim=2), nan=0.0).add_(3e-4).contiguous()
    del bound
    out = torch.full((B, Hkv * G, d), float("nan"), dtype=torch.float32, device=dev)
    sel = torch.zeros((B, Hkv, pdesc.nb_cap), dtype=torch.uint8, device=dev)
    stats = torch.zeros((B, Hkv), dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    nws = eb.eta_workspace_bytes(pdesc)
    ws = torch.zeros(nws + 256, dtype=torch.uint8, device=dev)
    off = (-ws.data_ptr()) % 256
    ws = ws[off:off + nws]
    eb.eta_decode_paged(pdesc, pages, params, qd, Kp, Vp, lens_d, musig, mnorm, tau, None, out, sel, ws,
                        stats=stats, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    out_np, sel_np, stats_np, tau_np = out.cpu().numpy(), sel.cpu().numpy(), stats.cpu().numpy(), tau.cpu().numpy()
    assert np.isfinite(out_np).all()
    for i in range(B):
        NB = int(lens[i]) // b
        assert np.array_equal(stats_np[i], (sel_np[i, :, :NB] != 0).sum(axis=1))
        assert not sel_np[i, :, NB:].any()
    assert 0.01 < stats_np.sum() / ((lens // b).sum() * Hkv) < 0.10
    for i in (0, 77, 127, 3):
        T = int(lens[i])
        ci = orc.Cache(bits(K), bits(V), np.asarray([T], np.int32), b)
        ref = orc.decode_step(bits(q[i:i + 1]), ci, o_musig, o_mnorm, tau=tau_np[i:i + 1], z=1.0, beta=5.0, lwb=1,
                              rescue_window=128)
        near = compare_masks(sel_np[i:i + 1], ref["sel"], ref["bound"], tau_np[i:i + 1].astype(np.float64),
                             np.asarray([T], np.int32), b, G, rescued=ref["rescued"])
        keep = heads_without_near_tie(near, 1, Hkv * G)
        assert keep.mean() >= 0.75
        mx, mean = output_errors(out_np[i:i + 1][keep], ref["out"][keep])
        assert mx <= 1e-2 and mean <= 1e-3, (i, mx, mean)

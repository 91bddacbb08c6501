#!/usr/bin/env python
"""Benchmark of the ETA block-sparse decode path on B200.

One "step" = one decode step of one layer for a whole batch: tail-block summary update, threshold prediction,
screening, streaming of the surviving K/V blocks, merge - six kernels of the library, all through the C ABI.
Workload at N=1: the 128K-context configuration (batch 4, 32 query / 8 KV heads, head_dim 128, block 64,
clustered keys), thresholds calibrated to 90% union block sparsity; the 50% / 97% points of the sweep and the
dense baseline (same kernels, every block, gate off) are reported beside it.  Metric: decode queries per second.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (launched under torchrun) every rank runs an independent replica of the workload: the path is fixed
to one GPU and has no exchange step, so scaling is weak by construction.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2609_20888_b200 import workloads as wl

METRIC = "eta_decode_queries_per_s"
UNIT = "queries/s"
DEFAULT_WORKLOAD = "c3_128k"
DEFAULT_TARGET = 0.90
CALIB = os.path.join(ROOT, "tests", "golden", "workload_calibration.json")
PEAKS = os.path.join(ROOT, "MEASURED_PEAKS.json")
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes (read + write) per launch of the streaming kernel as ncu counted them, keyed by
# "workload@target sparsity": a small data file kept beside the ncu summaries it was taken from.
NCU_TRAFFIC = os.path.join(ROOT, "profiles", "decode_kernel_dram_traffic.json")


def ncu_traffic(name: str, target: float, algorithmic_bytes: float):
    """DRAM traffic per launch of the streaming kernel for this run: what ncu counted on a captured run of the same
    workload, scaled by the algorithmic bytes (the union of surviving blocks, hence the bytes, changes with the
    step's query; traffic grows in proportion)."""
    try:
        e = json.load(open(NCU_TRAFFIC))[f"{name}@{target:.2f}"]
        return float(e["dram_bytes_per_launch"]) * algorithmic_bytes / float(e["algorithmic_bytes_of_captured_run"])
    except Exception:
        return None


def load_bias(name: str, target: float) -> np.ndarray:
    data = json.load(open(CALIB))
    return np.asarray(data[name]["targets"][f"{target:.2f}"]["bias"], np.float32)


def hbm_peak():
    try:
        return float(json.load(open(PEAKS))["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clocks and throttle reasons while the timed region runs: through NVML (read-only queries, a
    sample every few milliseconds), or, where the NVML module is missing, by calling nvidia-smi (about ten a second)."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self._halt = index, [], threading.Event()
        self.nvml = None
        try:
            import pynvml
            pynvml.nvmlInit()
            # CUDA_VISIBLE_DEVICES may renumber the devices: find the NVML handle of torch's device by its UUID
            uuid = str(torch.cuda.get_device_properties(index).uuid)
            handle = None
            for k in range(pynvml.nvmlDeviceGetCount()):
                h = pynvml.nvmlDeviceGetHandleByIndex(k)
                u = pynvml.nvmlDeviceGetUUID(h)
                u = u.decode() if isinstance(u, bytes) else u
                if uuid in u or u.replace("GPU-", "") == uuid:
                    handle = h
            if handle is not None:
                self.nvml, self.handle = pynvml, handle
                self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nvml = None

    def _sample_nvml(self):
        n = self.nvml
        mhz = float(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM))
        r = int(n.nvmlDeviceGetCurrentClocksEventReasons(self.handle)) if hasattr(n, "nvmlDeviceGetCurrentClocksEventReasons") \
            else int(n.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
        bits = [getattr(n, "nvmlClocksEventReasonHwSlowdown", 0x8), getattr(n, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                getattr(n, "nvmlClocksEventReasonSwThermalSlowdown", 0x20), getattr(n, "nvmlClocksEventReasonSwPowerCap", 0x4)]
        return [mhz, self.sm_max] + ["Active" if (r & b) else "Not Active" for b in bits]

    def run(self):
        while not self._halt.is_set():
            try:
                if self.nvml is not None:
                    self.samples.append(self._sample_nvml())
                    self._halt.wait(0.002)
                    continue
                out = subprocess.run(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=5).stdout
                parts = [p.strip() for p in out.strip().split(",")]
                if len(parts) >= 6:
                    self.samples.append(parts)
            except Exception:
                pass
            self._halt.wait(0.005)

    def stop(self) -> dict:
        self._halt.set()
        self.join(timeout=6)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unsampled"]}
        mhz = sorted(float(s[0]) for s in self.samples)
        reasons = [n for k, n in enumerate(self.NAMES) if any(str(s[2 + k]).lower().startswith("active") for s in self.samples)]
        return {"sm_mhz": mhz[len(mhz) // 2], "sm_max_mhz": float(self.samples[0][1]), "reasons": reasons,
                "samples": len(self.samples), "source": "nvml" if self.nvml is not None else "nvidia-smi"}


def algorithmic_bytes(sp, lens, union_blocks: float):
    """Algorithmic bytes of one step, i.e. what the method must move: summaries of every full block, K and V of the
    union of surviving blocks and of the tails, queries, thresholds, mask, output.  Split by kernel."""
    d, b, G = sp.head_dim, sp.block_size, sp.gqa
    nb = sum(int(t) // b for t in lens) * sp.n_kv_heads
    tails = sum(int(t) % b for t in lens) * sp.n_kv_heads
    screen = nb * (4 * d + 4) + nb + sp.batch * sp.n_q_heads * (2 * d + 4)
    decode = union_blocks * 4 * b * d + tails * 4 * d + sp.batch * sp.n_q_heads * 2 * d
    other = sp.batch * sp.n_q_heads * (2 * d + 4 * d) + sp.n_q_heads * d * sp.n_q_heads * 4
    return {"screen": float(screen), "decode": float(decode), "total": float(screen + decode + other)}


def max_over_ranks(x: float, dist, dev) -> float:
    """Device-timed numbers are reported as the maximum over ranks."""
    if dist is None:
        return x
    t = torch.tensor([x], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, batch: int, ms_step: float) -> float:
    """Replicas only: every rank decodes its own batch, so the job answers world * batch queries per step."""
    return world * batch / (ms_step * 1e-3)


def run_dry(args):
    """Host-side logic of the multi-rank run without a GPU (gloo): rendezvous, barrier, max over ranks, one JSON
    line from rank 0.  Each rank pretends to have measured 1.0 + 0.5 * rank ms per step."""
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    sp = wl.CONFIGS[args.workload]
    ms = max_over_ranks(1.0 + 0.5 * rank, dist if world > 1 else None, torch.device("cpu"))
    if world > 1:
        dist.barrier()
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": whole_job_value(world, sp.batch, ms), "unit": UNIT,
                          "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
                          "higher_is_better": True, "scaling": "weak", "dry_run": True,
                          "config": {"workload": sp.name, "replicas": world}}))
    if world > 1:
        dist.destroy_process_group()


def run_ours(args):
    from paper_2609_20888_b200 import binding as eb
    from paper_2609_20888_b200 import build as ebuild

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        ebuild.build()
    if world > 1:
        dist.barrier()
    eb.load()
    eb.eta_set_pdl(args.pdl)

    sp = wl.CONFIGS[args.workload]
    t0 = time.time()
    w = wl.make_workload(sp, threads=min(16, len(os.sched_getaffinity(0))))
    gen_s = time.time() - t0
    Kd, Vd = w.K.to(dev), w.V.to(dev)
    st = eb.DecodeState(Kd, Vd, sp.n_q_heads, sp.block_size)
    lens = w.seq_lens.numpy().astype(np.int32)
    lens_d = w.seq_lens.to(dev)
    Wd = w.W.to(dev)

    # --paged: the same cache scattered over a pool of pages of one block each by a seeded permutation; the step
    # then runs through the paged entry points (same results bit for bit; tests/test_gpu_paged.py)
    pdesc = pages = Kp = Vp = None
    if args.paged:
        B_, H_, T_, d_ = Kd.shape
        b_ = sp.block_size
        assert T_ % b_ == 0, "--paged needs a token capacity that is a multiple of the block size"
        nbp = T_ // b_
        gperm = torch.Generator(device=dev).manual_seed(sp.seed + 99)
        perm = torch.randperm(B_ * nbp, generator=gperm, device=dev)
        Kp, Vp = torch.empty((B_ * nbp, H_, b_, d_), dtype=Kd.dtype, device=dev), None
        Kp[perm] = Kd.view(B_, H_, nbp, b_, d_).permute(0, 2, 1, 3, 4).reshape(B_ * nbp, H_, b_, d_)
        Vp = torch.empty_like(Kp)
        Vp[perm] = Vd.view(B_, H_, nbp, b_, d_).permute(0, 2, 1, 3, 4).reshape(B_ * nbp, H_, b_, d_)
        table = perm.view(B_, nbp).to(torch.int32).contiguous()
        pdesc = eb.paged_cache_desc(Kp, Vp, sp.batch, sp.n_q_heads, t_cap=T_, nb_cap=st.desc.nb_cap)
        pages = eb.page_table(table, B_ * nbp)

    # prefill-side index build (once per sequence; timed on its own, not part of a decode step)
    # (three warm-up launches, then the median of seven; K is far larger than the L2, so nothing of a launch's input
    # is left in the cache for the next)
    build_times = []
    for k in range(10):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        eb.eta_build_block_summaries(st.desc, Kd, lens_d, st.musig, st.mnorm)
        ev1.record()
        torch.cuda.synchronize()
        if k >= 3:
            build_times.append(ev0.elapsed_time(ev1))
    build_ms = sorted(build_times)[len(build_times) // 2]
    k_bytes = sum(int(t) // sp.block_size for t in lens) * sp.n_kv_heads * sp.block_size * sp.head_dim * 2
    # the packed index (centroid fp16, sigma rounded up to e4m3: 3 d bytes per record instead of 4 d), for the sweep
    musig8, mnorm8 = eb.alloc_summaries(st.desc, dev, packed=True)
    eb.eta_build_block_summaries(st.desc, Kd, lens_d, musig8, mnorm8, flags=eb.ETA_BUILD_PACKED_SIGMA)
    torch.cuda.synchronize()

    # offline calibration (prefill-side tool, timed on its own): 16 sequences of 1024 tokens at this head geometry
    cal = None
    if rank == 0 and world == 1:
        gcal = torch.Generator(device=dev).manual_seed(208880)
        cq = torch.randn((16, sp.n_q_heads, 1024, sp.head_dim), generator=gcal, device=dev).to(torch.bfloat16)
        ck = torch.randn((16, sp.n_kv_heads, 1024, sp.head_dim), generator=gcal, device=dev).to(torch.bfloat16)
        ctau = torch.full((16, sp.n_q_heads, 1024), 0.5, device=dev)
        chc = torch.empty(sp.n_q_heads, device=dev)
        cws = eb.eta_calibrate_head_const(cq, ck, ctau, chc, None, beta=sp.beta, n_bins=2048)
        torch.cuda.synchronize()
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record()
        for _ in range(5):
            eb.eta_calibrate_head_const(cq, ck, ctau, chc, None, beta=sp.beta, n_bins=2048, workspace=cws)
        c1.record()
        torch.cuda.synchronize()
        cal_ms = c0.elapsed_time(c1) / 5
        pairs = 16 * sp.n_q_heads * (1024 * 1025 // 2)
        cal = {"ms": cal_ms, "n_seq": 16, "seq_len": 1024, "n_bins": 2048,
               "causal_pairs_per_s": pairs / (cal_ms * 1e-3), "max_abs_dev_from_0.5": float((chc - 0.5).abs().max())}
        del cq, ck, ctau, cws

    n_q = args.steps + args.warmup
    q_host = [w.queries(s).pin_memory() for s in range(n_q)]
    q_dev = [q.to(dev) for q in q_host]
    out_host = torch.empty((sp.batch, sp.n_q_heads, sp.head_dim), dtype=torch.float32).pin_memory()
    flush = torch.empty(384 << 20, dtype=torch.uint8, device=dev)     # > 126 MB of L2
    flush_rd = torch.zeros(96 << 20, dtype=torch.int32, device=dev)   # 384 MiB read after the write (see l2_flush)

    flush_mode = [args.flush]

    def l2_flush(k):
        """Evicts the step's data from L2 between timed steps: a 384 MiB write, then (unless the mode is "write") a
        384 MiB read.  After the write alone the L2 is full of dirty lines, and the next ~126 MB the step reads each
        push one of them out to memory: the step is then charged for the write-back of the flush (c3 at 90 %: 87
        against 76 us per step; the streaming kernel 66.6 against 55.7 us).  The read leaves clean lines behind."""
        flush.fill_(k & 0xff)
        if flush_mode[0] == "write+read":
            torch.sum(flush_rd)

    static_q = torch.empty_like(q_dev[0])

    q_stage = torch.empty_like(q_host[0]).pin_memory()      # fixed page-locked buffer the end-to-end step reads its query from

    def make_step(bias_np, flags=0, profiled=False, host_io=False, host_q=None, host_out=None, packed=False):
        """One decode step on the query in `static_q`.  With --graph (default) the launches are captured once
        into a CUDA graph and replayed, so the host costs one graph launch per step instead of several kernel
        launches through ctypes; the library calls are the same either way.  With host_io the step starts by
        fetching the query from the page-locked buffer `q_stage` (eta_stage_query) and the merge kernel writes the
        output straight into the page-locked `out_host`."""
        bias_d = torch.from_numpy(bias_np).to(dev)
        if packed:
            flags |= eb.ETA_FLAG_PACKED_SIGMA
        params = eb.DecodeParams(z=sp.z, beta=sp.beta, lwb=sp.lwb, rescue_window=sp.rescue_window, flags=flags)
        ms_t, mn_t = (musig8, mnorm8) if packed else (st.musig, st.mnorm)
        bflags = eb.ETA_BUILD_PACKED_SIGMA if packed else 0

        host_q = host_io if host_q is None else host_q
        host_out = host_io if host_out is None else host_out

        def launch():
            if host_q:
                eb.eta_stage_query(q_stage, static_q)
            o = out_host if host_out else st.out
            if pages is not None:
                eb.eta_append_summary_paged(pdesc, pages, Kp, lens_d, ms_t, mn_t, flags=bflags)
                eb.eta_predict_threshold(static_q, Wd, bias_d, st.tau)
                eb.eta_decode_paged(pdesc, pages, params, static_q, Kp, Vp, lens_d, ms_t, mn_t, st.tau, None,
                                    o, st.sel_mask, st.workspace, stats=st.stats, status=st.status)
                return
            eb.eta_append_summary(st.desc, Kd, lens_d, ms_t, mn_t, flags=bflags)
            eb.eta_predict_threshold(static_q, Wd, bias_d, st.tau)
            eb.eta_decode(st.desc, params, static_q, Kd, Vd, lens_d, ms_t, mn_t, st.tau, None,
                          o, st.sel_mask, st.workspace, stats=st.stats, status=st.status)

        graph = None
        if args.graph or profiled:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                static_q.copy_(q_dev[0])
                for _ in range(2):
                    launch()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            eb.eta_profile_enable(profiled)     # timing events are captured as nodes of the graph
            with torch.cuda.graph(graph):
                launch()
            eb.eta_profile_enable(False)

        def step(qd=None):
            """One step on the query in `static_q`; with a query given, it is first copied there (device to device)."""
            if qd is not None:
                static_q.copy_(qd, non_blocking=True)
            if graph is not None:
                graph.replay()
            else:
                launch()
        return step

    def timed(step):
        """W warm-up steps, then K steps each bracketed by CUDA events with an L2 flush in between."""
        for s in range(args.warmup):
            step(q_dev[s])
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        union = 0
        wall0 = time.perf_counter()
        for k in range(args.steps):
            l2_flush(k)
            # the step's query is put where the kernels read it before the timed region starts (inputs resident in
            # HBM; the 32 KB it leaves in L2 after the flush are a fraction of a percent of what the step reads)
            static_q.copy_(q_dev[args.warmup + k], non_blocking=True)
            evs[k][0].record()
            step()
            evs[k][1].record()
            union += 0        # stats are read after the region
        torch.cuda.synchronize()
        wall = time.perf_counter() - wall0
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        ms = [a.elapsed_time(b) for a, b in evs]
        assert int(st.status.item()) == 0, "device status flagged a problem"
        return ms, wall

    def union_blocks_of(step):
        tot = 0
        for k in range(args.steps):
            step(q_dev[args.warmup + k])
            tot += int(st.stats.sum().item())
        return tot / args.steps

    def kernel_times(bias_np, flags=0, packed=False):
        """Device time from each launch to the next, averaged over the steps, from events captured in the graph."""
        stp = make_step(bias_np, flags, profiled=True, packed=packed)
        acc = {}
        for k in range(args.steps):
            l2_flush(k)
            stp(q_dev[args.warmup + k])
            for name, v in eb.eta_profile_read().items():
                acc[name] = acc.get(name, 0.0) + v
        return {k: v / args.steps for k, v in acc.items()}

    targets = list(sp.target_sparsity)
    main_target = DEFAULT_TARGET if DEFAULT_TARGET in targets else targets[0]
    # clocks are sampled while the main workload runs: its timed region, the per-kernel pass and the end-to-end pass
    sampler = ClockSampler(local)
    sampler.start()
    step_main = make_step(load_bias(sp.name, main_target))
    ms_main, wall_main = timed(step_main)
    ms_step = max_over_ranks(sum(ms_main) / len(ms_main), dist if world > 1 else None, dev)
    # the same K steps with the write-only flush, reported beside the headline
    ms_step_wo = None
    if args.flush == "write+read":
        flush_mode[0] = "write"
        ms_wo, _ = timed(step_main)
        flush_mode[0] = args.flush
        ms_step_wo = max_over_ranks(sum(ms_wo) / len(ms_wo), dist if world > 1 else None, dev)
    union_main = union_blocks_of(step_main)
    kt = kernel_times(load_bias(sp.name, main_target))
    nb_total = sum(int(t) // sp.block_size for t in lens) * sp.n_kv_heads
    ab = algorithmic_bytes(sp, lens, union_main)
    peak, peak_kind = hbm_peak()
    dec_s = kt["decode_kernel"] * 1e-3
    achieved = ab["decode"] / dec_s / 1e9

    # end to end: the query comes from pinned host memory and the output goes back to it, every step.  The step's
    # first kernel reads the query over the interconnect (eta_stage_query) and the merge kernel stores the output
    # into pinned host memory, which costs less than two copy-engine transfers of a few tens of kilobytes.  Each
    # step is bracketed by events on the launching stream and followed by a host synchronise.
    io_q = args.e2e_io in ("kernel", "stage")
    io_out = args.e2e_io in ("kernel", "hostout")
    step_e2e = make_step(load_bias(sp.name, main_target), host_q=io_q, host_out=io_out) if (io_q or io_out) else step_main
    e2e_ms = 0.0
    for k in range(args.steps):
        l2_flush(k)
        a_ev, b_ev = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a_ev.record()
        if io_q:
            # this step's query, host to host, into the buffer the graph reads (a plain memmove: a tensor copy of
            # more than 32 K elements would wake a thread pool)
            ctypes.memmove(q_stage.data_ptr(), q_host[args.warmup + k].data_ptr(), q_stage.numel() * 2)
        else:
            static_q.copy_(q_host[args.warmup + k], non_blocking=True)
        step_e2e()
        if not io_out:
            out_host.copy_(st.out, non_blocking=True)
        b_ev.record()
        torch.cuda.synchronize()
        e2e_ms += a_ev.elapsed_time(b_ev)
    # the host-resident result of the last step equals what the device-resident step computes for the same query
    step_main(q_dev[args.warmup + args.steps - 1])
    torch.cuda.synchronize()
    assert torch.equal(out_host, st.out.cpu()), "end-to-end output differs from the device-resident step"
    e2e_s = max_over_ranks(e2e_ms * 1e-3 / args.steps, dist if world > 1 else None, dev)

    clocks = sampler.stop()

    sweep = {}
    if rank == 0 and world == 1 and not args.no_sweep:
        for tgt in targets:
            if tgt == main_target:
                continue
            stp = make_step(load_bias(sp.name, tgt))
            ms, _ = timed(stp)
            ub = union_blocks_of(stp)
            abt = algorithmic_bytes(sp, lens, ub)
            m = sum(ms) / len(ms)
            ktt = kernel_times(load_bias(sp.name, tgt))
            sweep[f"{tgt:.2f}"] = {"ms_per_step": m, "union_sparsity": 1 - ub / nb_total,
                                   "gbs_on_algorithmic_bytes": abt["total"] / (m * 1e-3) / 1e9, "kernel_ms": ktt,
                                   "decode_kernel_gbs": abt["decode"] / (ktt["decode_kernel"] * 1e-3) / 1e9}
        # the packed index at the same thresholds: a quarter less screening traffic, a few more blocks admitted
        for tgt in targets:
            stp = make_step(load_bias(sp.name, tgt), packed=True)
            ms, _ = timed(stp)
            ub = union_blocks_of(stp)
            m = sum(ms) / len(ms)
            ktt = kernel_times(load_bias(sp.name, tgt), packed=True)
            sweep[f"{tgt:.2f}_packed_sigma"] = {"ms_per_step": m, "union_sparsity": 1 - ub / nb_total, "kernel_ms": ktt,
                                                "summary_bytes_per_record": 3 * sp.head_dim + 4}
        stp = make_step(np.zeros(sp.n_q_heads, np.float32), flags=eb.ETA_FLAG_DENSE)
        ms, _ = timed(stp)
        m = sum(ms) / len(ms)
        abt = algorithmic_bytes(sp, lens, nb_total)
        ktt = kernel_times(np.zeros(sp.n_q_heads, np.float32), flags=eb.ETA_FLAG_DENSE)
        sweep["dense_baseline"] = {"ms_per_step": m, "gbs_on_algorithmic_bytes": (abt["decode"]) / (m * 1e-3) / 1e9,
                                   "speedup_of_main": m / ms_step, "kernel_ms": ktt,
                                   "decode_kernel_gbs": abt["decode"] / (ktt["decode_kernel"] * 1e-3) / 1e9}
        sweep["sdpa_outside_baseline"] = sdpa_outside(sp, Kd, Vd, q_dev, lens, args, l2_flush, dev)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu = cpu_baseline(sp, w, load_bias(sp.name, main_target), budget_s=20.0)

    if rank == 0:
        line = {
            "metric": METRIC, "value": whole_job_value(world, sp.batch, ms_step), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": sp.name, "batch": sp.batch, "n_q_heads": sp.n_q_heads, "n_kv_heads": sp.n_kv_heads,
                       "head_dim": sp.head_dim, "context": sp.context, "block_size": sp.block_size,
                       "target_union_sparsity": main_target, "measured_union_sparsity": 1 - union_main / nb_total,
                       "z": sp.z, "beta": sp.beta,
                       "l2": "flushed between timed steps (384 MiB write" + (", then 384 MiB read so that the step is not charged for the write-back of the flush's dirty lines)" if args.flush == "write+read" else ")"),
                       "fresh_query_every_step": True, "replicas": world, "cuda_graph": bool(args.graph), "pdl": bool(args.pdl),
                       "paged_cache": bool(args.paged), "e2e_io": args.e2e_io},
            "attention_us_per_token": ms_step * 1e3,
            "write_only_l2_flush": (None if ms_step_wo is None else
                                    {"ms_per_step": ms_step_wo, "value": world * sp.batch / (ms_step_wo * 1e-3), "unit": UNIT}),
            "achieved_gbs_all_kernels": ab["total"] / (ms_step * 1e-3) / 1e9,
            "frac_of_8tbs_nominal": ab["total"] / (ms_step * 1e-3) / 8e12,
            "kernel_ms": kt,
            "clocks": clocks,
            "e2e": {"value": world * sp.batch / e2e_s, "unit": UNIT, "h2d_bytes_per_step": q_host[0].numel() * 2,
                    "d2h_bytes_per_step": out_host.numel() * 4},
            "gpu_launches": args.steps * (2 + eb.eta_decode_kernel_count()),
            "roofline": {"bound": "hbm", "kernel": "decode_kernel", "achieved": achieved, "peak": peak,
                         "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": ncu_traffic(sp.name, main_target, ab["decode"]),
                         "traffic_unit": "bytes per launch (ncu capture of this workload, scaled by the algorithmic bytes of this run)",
                         "algorithmic_bytes_per_launch": ab["decode"]},
            "prefill_build": {"ms": build_ms, "gbs": k_bytes / (build_ms * 1e-3) / 1e9},
            "calibration": cal,
            "sweep": sweep,
            "sweep_regime": "every figure of `sweep`, `kernel_ms`, `e2e` and `value` was taken with the L2 flush named in config.l2 (" + args.flush + "), CUDA-graph replay " + ("on" if args.graph else "off") + ", a fresh query every step",
            "cpu_baseline": cpu,
            "setup_s": {"generate": round(gen_s, 1)},
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def sdpa_outside(sp, Kd, Vd, q_dev, lens, args, l2_flush, dev):
    """An outside sanity number for the dense baseline (Section 2's dense attention): torch's
    scaled_dot_product_attention on the same shapes, bf16, the G query heads of a group as the query length of their KV
    head (one decode query per sequence).  Library code, timed for context beside `dense_baseline`; never a product
    path, and only meaningful when all sequences have the same length."""
    import torch.nn.functional as F
    if len(set(int(t) for t in lens)) != 1:
        return {"unavailable": "sequences of different lengths"}
    T = int(lens[0])
    B, Hkv, G, d = sp.batch, sp.n_kv_heads, sp.gqa, sp.head_dim
    Kt, Vt = Kd[:, :, :T], Vd[:, :, :T]

    def run(q):
        return F.scaled_dot_product_attention(q.view(B, Hkv, G, d), Kt, Vt)

    for s in range(args.warmup):
        run(q_dev[s])
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for k in range(args.steps):
        l2_flush(k)
        evs[k][0].record()
        run(q_dev[args.warmup + k])
        evs[k][1].record()
    torch.cuda.synchronize()
    ms = sum(a.elapsed_time(b) for a, b in evs) / len(evs)
    kv_bytes = 2 * B * Hkv * T * d * 2
    return {"ms_per_step": ms, "gbs_on_kv_bytes": kv_bytes / (ms * 1e-3) / 1e9,
            "what": "torch.nn.functional.scaled_dot_product_attention, bf16, q as [batch, kv_heads, G, d] (library code; context only)"}


def cpu_baseline(sp, w, bias, budget_s: float, steps: int | None = None):
    """The oracle, as it stands, on this machine's host cores: whole decode steps (threshold prediction, bounds,
    selection, gated attention over the admitted blocks) on the whole batch of the workload, a bounded number of
    steps."""
    from oracle import eta_oracle as orc
    from tests.helpers import bits
    orc.build()
    nseq = sp.batch
    K, V = bits(w.K[:nseq]), bits(w.V[:nseq])
    lens = w.seq_lens.numpy().astype(np.int32)[:nseq].copy()
    c = orc.Cache(K, V, lens, sp.block_size)
    musig, mnorm = orc.block_summaries(c)           # prefill-side, not timed (as on the GPU side)
    times = []
    t_all = time.perf_counter()
    s = 0
    while True:
        q = bits(w.queries(s))[:nseq].copy()
        t0 = time.perf_counter()
        tau = orc.predict_threshold(q, w.W.numpy(), bias)
        orc.decode_step(q, c, musig, mnorm, tau=tau.astype(np.float32), z=sp.z, beta=sp.beta, lwb=sp.lwb,
                        rescue_window=sp.rescue_window)
        times.append(time.perf_counter() - t0)
        s += 1
        if steps is not None:
            if s >= steps:
                break
        elif time.perf_counter() - t_all > budget_s or s >= 128:
            break
    per = sum(times) / len(times)
    return {"value": nseq / per, "unit": UNIT, "cores": orc.n_threads(), "kind": "oracle",
            "sample": f"{len(times)} decode steps of {sp.name} (all {sp.batch} sequences, all {sp.n_q_heads} heads, "
                      f"full context), {sum(times):.1f} s of CPU work", "s_per_step": per}


def run_reference(args):
    """Reference arm: the CPU oracle on the host cores, same metric and configuration."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sp = wl.CONFIGS[args.workload]
    w = wl.make_workload(sp, threads=min(16, len(os.sched_getaffinity(0))))
    targets = list(sp.target_sparsity)
    main_target = DEFAULT_TARGET if DEFAULT_TARGET in targets else targets[0]
    bias = load_bias(sp.name, main_target)
    cpu_baseline(sp, w, bias, 0.0, steps=max(1, args.warmup))
    cpu = cpu_baseline(sp, w, bias, 0.0, steps=args.steps)
    line = {"impl": "reference", "metric": METRIC, "value": cpu["value"], "unit": UNIT,
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": cpu["s_per_step"] * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": sp.name, "batch": sp.batch, "n_q_heads": sp.n_q_heads, "n_kv_heads": sp.n_kv_heads,
                       "head_dim": sp.head_dim, "context": sp.context, "block_size": sp.block_size,
                       "target_union_sparsity": main_target},
            "cpu_baseline": {k: cpu[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": cpu["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=list(wl.CONFIGS))
    ap.add_argument("--no-graph", dest="graph", action="store_false", help="launch the kernels directly every step")
    ap.add_argument("--no-pdl", dest="pdl", action="store_false", help="fully serialise the kernel launches")
    ap.add_argument("--e2e-io", default="kernel", choices=["kernel", "copy", "stage", "hostout"],
                    help="end-to-end leg: the step's kernels read the query from / write the output to pinned host "
                         "memory themselves (kernel), or two copy-engine transfers bracket the device-resident step (copy)")
    ap.add_argument("--paged", action="store_true", help="run the step on a paged copy of the cache (pages scattered by a seeded permutation)")
    ap.add_argument("--flush", default="write+read", choices=["write", "write+read"],
                    help="L2 flush between timed steps: a 384 MiB write, optionally followed by a 384 MiB read")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--dry-run", action="store_true", help="exercise the multi-rank host logic on CPU (gloo)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    elif args.dry_run:
        run_dry(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

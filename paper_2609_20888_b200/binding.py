"""Thin ctypes binding of the C-ABI library (`include/eta.h`).

Argument marshalling only: torch tensors provide device memory and the current
CUDA stream; every step of the path runs in the library's kernels.  There is no
CPU fallback: a missing library or a CPU tensor raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libeta_b200.so")

ETA_FLAG_DENSE = 1
ETA_FLAG_UNGATE_LAST = 2
ETA_FLAG_PACKED_SIGMA = 4
ETA_BUILD_SIGMA_ENVELOPE = 1
ETA_BUILD_PACKED_SIGMA = 2
ETA_DEV_TIMEOUT, ETA_DEV_LEN_CLAMPED, ETA_DEV_EMPTY_ROW = 1, 2, 4

EXPORTS = ("eta_workspace_bytes", "eta_build_block_summaries", "eta_append_summary", "eta_build_block_summaries_paged",
           "eta_append_summary_paged", "eta_decode_paged", "eta_stage_query", "eta_predict_threshold",
           "eta_score_dual", "eta_calibration_workspace_bytes", "eta_calibrate_head_const", "eta_decode", "eta_decode_static", "eta_static_scratch_bytes", "eta_decode_kernel_count", "eta_profile_enable", "eta_profile_read",
           "eta_profile_kernel_name", "eta_set_pdl", "eta_strerror", "eta_last_cuda_error")


class CacheDesc(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("block_size", ctypes.c_int32), ("t_cap", ctypes.c_int32),
                ("nb_cap", ctypes.c_int32),
                ("k_stride_b", ctypes.c_int64), ("k_stride_h", ctypes.c_int64), ("k_stride_t", ctypes.c_int64),
                ("v_stride_b", ctypes.c_int64), ("v_stride_h", ctypes.c_int64), ("v_stride_t", ctypes.c_int64)]


class Params(ctypes.Structure):
    _fields_ = [("z", ctypes.c_float), ("a", ctypes.c_float), ("beta", ctypes.c_float), ("scale", ctypes.c_float),
                ("lwb", ctypes.c_int32), ("rescue_window", ctypes.c_int32), ("flags", ctypes.c_uint32)]


class PageTable(ctypes.Structure):
    _fields_ = [("block_table", ctypes.c_void_p), ("table_stride", ctypes.c_int32), ("n_pages", ctypes.c_int32)]


class EtaError(RuntimeError):
    pass


_lib = None


def load(path: str | None = None) -> ctypes.CDLL:
    """Load the in-tree library; fails loudly when it has not been built.  With a path: another build of the same
    sources (a test variant), loaded beside the product library and not remembered."""
    global _lib
    if _lib is None or path is not None:
        lib_path = path or LIB_PATH
        if not os.path.exists(lib_path):
            raise EtaError(f"{lib_path} is missing: build it with `python -m paper_2609_20888_b200.build` "
                           "(there is no fallback path)")
        lib = ctypes.CDLL(lib_path)
        vp, i32p, f32p = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p
        D, P = ctypes.POINTER(CacheDesc), ctypes.POINTER(Params)
        lib.eta_workspace_bytes.argtypes = [D, ctypes.POINTER(ctypes.c_size_t)]
        lib.eta_build_block_summaries.argtypes = [D, vp, i32p, vp, f32p, ctypes.c_uint32, vp]
        lib.eta_append_summary.argtypes = [D, vp, i32p, vp, f32p, ctypes.c_uint32, vp]
        PT = ctypes.POINTER(PageTable)
        lib.eta_build_block_summaries_paged.argtypes = [D, PT, vp, i32p, vp, f32p, ctypes.c_uint32, vp]
        lib.eta_append_summary_paged.argtypes = [D, PT, vp, i32p, vp, f32p, ctypes.c_uint32, vp]
        lib.eta_decode_paged.argtypes = [D, PT, P, vp, vp, vp, i32p, vp, f32p, f32p, f32p, f32p, vp, i32p, vp, vp,
                                         ctypes.c_size_t, vp]
        lib.eta_predict_threshold.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp, f32p, f32p, f32p, vp]
        lib.eta_stage_query.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp, vp, vp]
        lib.eta_score_dual.argtypes = [D, P, vp, i32p, vp, f32p, f32p, vp]
        i32 = ctypes.c_int32
        lib.eta_calibration_workspace_bytes.argtypes = [i32, i32, i32, i32, ctypes.POINTER(ctypes.c_size_t)]
        lib.eta_calibrate_head_const.argtypes = [i32, i32, i32, i32, i32, vp, vp, f32p, ctypes.c_float, ctypes.c_float,
                                                 i32, ctypes.c_float, ctypes.c_float, f32p, f32p, vp, ctypes.c_size_t, vp]
        lib.eta_decode.argtypes = [D, P, vp, vp, vp, i32p, vp, f32p, f32p, f32p, f32p, vp, i32p, vp, vp,
                                   ctypes.c_size_t, vp]
        lib.eta_decode_static.argtypes = [D, P, vp, vp, vp, i32p, vp, f32p, f32p, f32p, f32p, vp, i32p, vp, vp]
        lib.eta_static_scratch_bytes.restype = ctypes.c_size_t
        lib.eta_decode_kernel_count.restype = ctypes.c_int
        lib.eta_strerror.restype = ctypes.c_char_p
        lib.eta_strerror.argtypes = [ctypes.c_int]
        lib.eta_last_cuda_error.restype = ctypes.c_char_p
        lib.eta_profile_enable.argtypes = [ctypes.c_int]
        lib.eta_set_pdl.argtypes = [ctypes.c_int]
        lib.eta_profile_read.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.c_int]
        lib.eta_profile_kernel_name.restype = ctypes.c_char_p
        lib.eta_profile_kernel_name.argtypes = [ctypes.c_int]
        for name in EXPORTS:
            if name not in ("eta_strerror", "eta_last_cuda_error", "eta_decode_kernel_count",
                            "eta_profile_kernel_name", "eta_static_scratch_bytes"):
                getattr(lib, name).restype = ctypes.c_int
        if path is not None:
            return lib
        _lib = lib
    return _lib


def _check(rc: int, what: str) -> None:
    if rc != 0:
        lib = load()
        raise EtaError(f"{what}: {lib.eta_strerror(rc).decode()} ({rc}) {lib.eta_last_cuda_error().decode()}")


def _dev(t: torch.Tensor | None, dtype=None, name="tensor"):
    if t is None:
        return None
    if not t.is_cuda:
        raise EtaError(f"{name} must be a CUDA tensor (no CPU path exists)")
    if dtype is not None and t.dtype != dtype:
        raise EtaError(f"{name} must be {dtype}, got {t.dtype}")
    return ctypes.c_void_p(t.data_ptr())


def _dev_or_pinned(t: torch.Tensor, dtype=None, name="tensor"):
    """Device pointer of a CUDA tensor, or of a page-locked host tensor (addressable by the device as it is)."""
    if t is not None and not t.is_cuda and t.is_pinned():
        if dtype is not None and t.dtype != dtype:
            raise EtaError(f"{name} must be {dtype}, got {t.dtype}")
        return ctypes.c_void_p(t.data_ptr())
    return _dev(t, dtype, name)


def _dev_musig(t: torch.Tensor):
    """Summary records: fp16 (compact layout) or uint8 (packed layout)."""
    if t is not None and t.dtype not in (torch.float16, torch.uint8):
        raise EtaError(f"musig must be float16 (compact records) or uint8 (packed records), got {t.dtype}")
    return _dev(t, None, "musig")


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


@dataclass
class DecodeParams:
    z: float = 1.0
    a: float = 0.0
    beta: float = 5.0
    scale: float = 0.0
    lwb: int = 0
    rescue_window: int = 128
    flags: int = 0

    def c(self) -> Params:
        return Params(self.z, self.a, self.beta, self.scale, self.lwb, self.rescue_window, self.flags)


def cache_desc(K: torch.Tensor, V: torch.Tensor, n_q_heads: int, block_size: int, nb_cap: int | None = None) -> CacheDesc:
    """Describe a cache K, V of logical shape [batch, n_kv_heads, t_cap, head_dim] (any strides with unit
    stride along head_dim)."""
    B, Hkv, Tcap, d = K.shape
    if K.stride(3) != 1 or V.stride(3) != 1 or V.shape != K.shape:
        raise EtaError("K and V must have the same shape and unit stride along head_dim")
    nb = nb_cap if nb_cap is not None else (Tcap + block_size - 1) // block_size
    return CacheDesc(B, n_q_heads, Hkv, d, block_size, Tcap, nb, K.stride(0), K.stride(1), K.stride(2),
                     V.stride(0), V.stride(1), V.stride(2))


def paged_cache_desc(K_pool: torch.Tensor, V_pool: torch.Tensor, batch: int, n_q_heads: int, t_cap: int,
                     nb_cap: int | None = None) -> CacheDesc:
    """Describe a paged cache: pools of logical shape [n_pages, n_kv_heads, block_size, head_dim] (any strides with
    unit stride along head_dim); the page size is the block size, the stride of the first axis the page stride."""
    n_pages, Hkv, b, d = K_pool.shape
    if K_pool.stride(3) != 1 or V_pool.stride(3) != 1 or V_pool.shape != K_pool.shape:
        raise EtaError("K_pool and V_pool must have the same shape and unit stride along head_dim")
    nb = nb_cap if nb_cap is not None else (t_cap + b - 1) // b
    return CacheDesc(batch, n_q_heads, Hkv, d, b, t_cap, nb, K_pool.stride(0), K_pool.stride(1), K_pool.stride(2),
                     V_pool.stride(0), V_pool.stride(1), V_pool.stride(2))


def page_table(block_table: torch.Tensor, n_pages: int) -> PageTable:
    """block_table: int32 CUDA tensor [batch, table_stride], page of every block of tokens of every sequence."""
    if block_table.dim() != 2 or block_table.stride(1) != 1:
        raise EtaError("block_table must be a 2-D tensor with unit stride along its second axis")
    return PageTable(_dev(block_table, torch.int32, "block_table"), block_table.stride(0), n_pages)


def eta_workspace_bytes(desc: CacheDesc) -> int:
    n = ctypes.c_size_t(0)
    _check(load().eta_workspace_bytes(ctypes.byref(desc), ctypes.byref(n)), "eta_workspace_bytes")
    return n.value


def alloc_summaries(desc: CacheDesc, device, packed: bool = False):
    """musig, mnorm for the compact layout (fp16 [.., 2, d]) or, with `packed`, the packed one (bytes [.., 3 d]: the
    centroid as fp16, then sigma rounded up to e4m3)."""
    if packed:
        musig = torch.zeros((desc.batch, desc.n_kv_heads, desc.nb_cap, 3 * desc.head_dim), dtype=torch.uint8, device=device)
        mnorm = torch.zeros((desc.batch, desc.n_kv_heads, desc.nb_cap), dtype=torch.float32, device=device)
        return musig, mnorm
    musig = torch.zeros((desc.batch, desc.n_kv_heads, desc.nb_cap, 2, desc.head_dim), dtype=torch.float16, device=device)
    mnorm = torch.zeros((desc.batch, desc.n_kv_heads, desc.nb_cap), dtype=torch.float32, device=device)
    return musig, mnorm


def eta_build_block_summaries(desc, K, seq_lens, musig, mnorm, flags: int = 0) -> None:
    _check(load().eta_build_block_summaries(ctypes.byref(desc), _dev(K, torch.bfloat16, "K"),
                                            _dev(seq_lens, torch.int32, "seq_lens"), _dev_musig(musig),
                                            _dev(mnorm, torch.float32, "mnorm"), flags, _stream()),
           "eta_build_block_summaries")


def eta_append_summary(desc, K, seq_lens_after, musig, mnorm, flags: int = 0) -> None:
    _check(load().eta_append_summary(ctypes.byref(desc), _dev(K, torch.bfloat16, "K"),
                                     _dev(seq_lens_after, torch.int32, "seq_lens"), _dev_musig(musig),
                                     _dev(mnorm, torch.float32, "mnorm"), flags, _stream()),
           "eta_append_summary")


def eta_build_block_summaries_paged(desc, pages: PageTable, K_pool, seq_lens, musig, mnorm, flags: int = 0) -> None:
    _check(load().eta_build_block_summaries_paged(ctypes.byref(desc), ctypes.byref(pages), _dev(K_pool, torch.bfloat16, "K_pool"),
                                                  _dev(seq_lens, torch.int32, "seq_lens"),
                                                  _dev_musig(musig), _dev(mnorm, torch.float32, "mnorm"),
                                                  flags, _stream()),
           "eta_build_block_summaries_paged")


def eta_append_summary_paged(desc, pages: PageTable, K_pool, seq_lens_after, musig, mnorm, flags: int = 0) -> None:
    _check(load().eta_append_summary_paged(ctypes.byref(desc), ctypes.byref(pages), _dev(K_pool, torch.bfloat16, "K_pool"),
                                           _dev(seq_lens_after, torch.int32, "seq_lens"),
                                           _dev_musig(musig), _dev(mnorm, torch.float32, "mnorm"),
                                           flags, _stream()),
           "eta_append_summary_paged")


def eta_stage_query(q_host, q_dev) -> None:
    """Copies a step's queries from a page-locked host tensor into `q_dev` with a kernel on the current stream."""
    if q_host.is_cuda or not q_host.is_pinned():
        raise EtaError("q_host must be a page-locked host tensor")
    if q_host.shape != q_dev.shape or q_host.dtype != torch.bfloat16 or not q_host.is_contiguous() or not q_dev.is_contiguous():
        raise EtaError("q_host and q_dev must be contiguous bf16 tensors of the same shape")
    B, Hq, d = q_host.shape
    _check(load().eta_stage_query(B, Hq, d, ctypes.c_void_p(q_host.data_ptr()), _dev(q_dev, torch.bfloat16, "q_dev"),
                                  _stream()), "eta_stage_query")


def eta_predict_threshold(q, W, bias, tau) -> None:
    B, Hq, d = q.shape
    _check(load().eta_predict_threshold(B, Hq, d, _dev(q, torch.bfloat16, "q"), _dev(W, torch.float32, "W"),
                                        _dev(bias, torch.float32, "bias"), _dev(tau, torch.float32, "tau"), _stream()),
           "eta_predict_threshold")


def eta_score_dual(desc, params: DecodeParams, q, seq_lens, musig, mnorm, bound) -> None:
    p = params.c()
    _check(load().eta_score_dual(ctypes.byref(desc), ctypes.byref(p), _dev(q, torch.bfloat16, "q"),
                                 _dev(seq_lens, torch.int32, "seq_lens"), _dev_musig(musig),
                                 _dev(mnorm, torch.float32, "mnorm"), _dev(bound, torch.float32, "bound"), _stream()),
           "eta_score_dual")


def eta_calibrate_head_const(Q, K, tau, head_const, dbar=None, beta=5.0, scale=0.0, n_bins=2048, s_min=-8.0,
                             s_max=8.0, workspace=None):
    """Q bf16 [n_seq, Hq, T, d], K bf16 [n_seq, Hkv, T, d], tau fp32 [n_seq, Hq, T] -> head_const fp32 [Hq]
    (and dbar fp32 [Hq]).  Allocates the scratch with torch when none is given; returns it for reuse."""
    n_seq, Hq, T, d = Q.shape
    Hkv = K.shape[1]
    need = ctypes.c_size_t(0)
    _check(load().eta_calibration_workspace_bytes(n_seq, T, Hq, n_bins, ctypes.byref(need)),
           "eta_calibration_workspace_bytes")
    if workspace is None:
        workspace = torch.empty(need.value + 256, dtype=torch.uint8, device=Q.device)
        off = (-workspace.data_ptr()) % 256
        workspace = workspace[off:off + need.value]
    _check(load().eta_calibrate_head_const(n_seq, T, Hq, Hkv, d, _dev(Q, torch.bfloat16, "Q"),
                                           _dev(K, torch.bfloat16, "K"), _dev(tau, torch.float32, "tau"), beta, scale,
                                           n_bins, s_min, s_max, _dev(head_const, torch.float32, "head_const"),
                                           _dev(dbar, torch.float32, "dbar"), _dev(workspace, torch.uint8, "workspace"),
                                           workspace.numel(), _stream()),
           "eta_calibrate_head_const")
    return workspace


def eta_decode(desc, params: DecodeParams, q, K, V, seq_lens, musig, mnorm, tau, head_const, out, sel_mask,
               workspace, stats=None, status=None, lib=None) -> None:
    p = params.c()
    _check((lib or load()).eta_decode(ctypes.byref(desc), ctypes.byref(p), _dev(q, torch.bfloat16, "q"),
                             _dev(K, torch.bfloat16, "K"), _dev(V, torch.bfloat16, "V"),
                             _dev(seq_lens, torch.int32, "seq_lens"), _dev_musig(musig),
                             _dev(mnorm, torch.float32, "mnorm"), _dev(tau, torch.float32, "tau"),
                             _dev(head_const, torch.float32, "head_const"), _dev_or_pinned(out, torch.float32, "out"),
                             _dev(sel_mask, torch.uint8, "sel_mask"), _dev(stats, torch.int32, "stats"),
                             _dev(status, torch.int32, "status"), _dev(workspace, torch.uint8, "workspace"),
                             workspace.numel(), _stream()),
           "eta_decode")


def eta_decode_paged(desc, pages: PageTable, params: DecodeParams, q, K_pool, V_pool, seq_lens, musig, mnorm, tau,
                     head_const, out, sel_mask, workspace, stats=None, status=None) -> None:
    p = params.c()
    _check(load().eta_decode_paged(ctypes.byref(desc), ctypes.byref(pages), ctypes.byref(p), _dev(q, torch.bfloat16, "q"),
                                   _dev(K_pool, torch.bfloat16, "K_pool"), _dev(V_pool, torch.bfloat16, "V_pool"),
                                   _dev(seq_lens, torch.int32, "seq_lens"), _dev_musig(musig),
                                   _dev(mnorm, torch.float32, "mnorm"), _dev(tau, torch.float32, "tau"),
                                   _dev(head_const, torch.float32, "head_const"), _dev_or_pinned(out, torch.float32, "out"),
                                   _dev(sel_mask, torch.uint8, "sel_mask"), _dev(stats, torch.int32, "stats"),
                                   _dev(status, torch.int32, "status"), _dev(workspace, torch.uint8, "workspace"),
                                   workspace.numel(), _stream()),
           "eta_decode_paged")


def eta_decode_static(desc, params: DecodeParams, q, K, V, seq_lens, musig, mnorm, tau, head_const, out, sel_mask,
                      stats=None, status=None) -> None:
    """eta_decode without a workspace argument, for callers that have no device memory to give: the scratch is
    an 8 MiB array built into the library (see include/eta.h for its limit and sharing rules)."""
    p = params.c()
    _check(load().eta_decode_static(ctypes.byref(desc), ctypes.byref(p), _dev(q, torch.bfloat16, "q"),
                                    _dev(K, torch.bfloat16, "K"), _dev(V, torch.bfloat16, "V"),
                                    _dev(seq_lens, torch.int32, "seq_lens"), _dev_musig(musig),
                                    _dev(mnorm, torch.float32, "mnorm"), _dev(tau, torch.float32, "tau"),
                                    _dev(head_const, torch.float32, "head_const"), _dev_or_pinned(out, torch.float32, "out"),
                                    _dev(sel_mask, torch.uint8, "sel_mask"), _dev(stats, torch.int32, "stats"),
                                    _dev(status, torch.int32, "status"), _stream()),
           "eta_decode_static")


def eta_static_scratch_bytes() -> int:
    return int(load().eta_static_scratch_bytes())


def eta_decode_kernel_count() -> int:
    return load().eta_decode_kernel_count()


def eta_set_pdl(on: bool) -> None:
    _check(load().eta_set_pdl(1 if on else 0), "eta_set_pdl")


def eta_profile_enable(on: bool) -> None:
    _check(load().eta_profile_enable(1 if on else 0), "eta_profile_enable")


def eta_profile_read() -> dict:
    """Device time (ms) of each kernel of the most recent profiled eta_decode call, by kernel name."""
    lib = load()
    ms = (ctypes.c_float * 8)()
    n = lib.eta_profile_read(ms, 8)
    if n < 0:
        _check(n, "eta_profile_read")
    return {lib.eta_profile_kernel_name(k).decode(): float(ms[k]) for k in range(n)}


class DecodeState:
    """Device buffers one decode loop needs (allocated once with torch; the library allocates nothing)."""

    def __init__(self, K: torch.Tensor, V: torch.Tensor, n_q_heads: int, block_size: int):
        dev = K.device
        self.desc = cache_desc(K, V, n_q_heads, block_size)
        self.K, self.V = K, V
        self.musig, self.mnorm = alloc_summaries(self.desc, dev)
        self.workspace = torch.zeros(eta_workspace_bytes(self.desc) + 256, dtype=torch.uint8, device=dev)
        off = (-self.workspace.data_ptr()) % 256
        self.workspace = self.workspace[off:off + eta_workspace_bytes(self.desc)]
        B, Hkv, d = self.desc.batch, self.desc.n_kv_heads, self.desc.head_dim
        self.out = torch.empty((B, n_q_heads, d), dtype=torch.float32, device=dev)
        self.sel_mask = torch.zeros((B, Hkv, self.desc.nb_cap), dtype=torch.uint8, device=dev)
        self.tau = torch.empty((B, n_q_heads), dtype=torch.float32, device=dev)
        self.stats = torch.zeros((B, Hkv), dtype=torch.int32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)

"""ctypes front end of the CPU oracle (`eta_oracle.c`).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by
the benchmark's CPU-baseline leg; never by the product path.  Arguments are
numpy arrays; bf16 / fp16 tensors travel as uint16 bit patterns.  Nothing in
here does arithmetic of the method: it marshals arguments and calls C.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "eta_oracle.c")
_LIB = os.path.join(_HERE, "liboracle_eta.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP for the outer, independent loops)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.eta_oracle_bf16_to_double.restype = ctypes.c_double
        _lib.eta_oracle_bf16_to_double.argtypes = [ctypes.c_uint16]
        _lib.eta_oracle_fp16_to_double.restype = ctypes.c_double
        _lib.eta_oracle_fp16_to_double.argtypes = [ctypes.c_uint16]
        _lib.eta_oracle_double_to_fp16.restype = ctypes.c_uint16
        _lib.eta_oracle_double_to_fp16.argtypes = [ctypes.c_double]
        _lib.eta_oracle_gate.restype = ctypes.c_double
        _lib.eta_oracle_gate.argtypes = [ctypes.c_double] * 3
    return _lib


def n_threads() -> int:
    """Threads the OpenMP loops of the oracle will use in this process."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    return len(os.sched_getaffinity(0))


def _p(a, ctype):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"], "oracle arrays must be C-contiguous"
    return a.ctypes.data_as(ctypes.POINTER(ctype))


_u16 = ctypes.c_uint16
_f32 = ctypes.c_float
_f64 = ctypes.c_double
_i32 = ctypes.c_int32
_i64 = ctypes.c_int64
_u8 = ctypes.c_uint8
_I = ctypes.c_int
_L = ctypes.c_int64
_D = ctypes.c_double


@dataclass
class Cache:
    """A KV cache as the oracle sees it: bf16 bit patterns with capacity.

    K, V: uint16 arrays [B, Hkv, Tcap, d]; seq_lens: int32 [B].
    """
    K: np.ndarray
    V: np.ndarray
    seq_lens: np.ndarray
    block_size: int

    @property
    def B(self): return self.K.shape[0]
    @property
    def Hkv(self): return self.K.shape[1]
    @property
    def Tcap(self): return self.K.shape[2]
    @property
    def d(self): return self.K.shape[3]
    @property
    def NBcap(self): return self.Tcap // self.block_size

    def strides(self, which="K"):
        a = self.K if which == "K" else self.V
        it = a.itemsize
        return a.strides[0] // it, a.strides[1] // it, a.strides[2] // it


def bf16_to_double(bits: int) -> float:
    return lib().eta_oracle_bf16_to_double(int(bits))


def fp16_to_double(bits: int) -> float:
    return lib().eta_oracle_fp16_to_double(int(bits))


def double_to_fp16(x: float) -> int:
    return lib().eta_oracle_double_to_fp16(float(x))


def gate(S: float, tau_eff: float, beta: float) -> float:
    return lib().eta_oracle_gate(float(S), float(tau_eff), float(beta))


def block_summaries(cache: Cache, envelope: bool = False, raw: bool = False):
    """-> musig uint16 [B,Hkv,NBcap,2,d], mnorm float32 [B,Hkv,NBcap] (+ raw doubles)."""
    B, Hkv, d, NBcap = cache.B, cache.Hkv, cache.d, cache.NBcap
    musig = np.zeros((B, Hkv, NBcap, 2, d), np.uint16)
    mnorm = np.zeros((B, Hkv, NBcap), np.float32)
    mu_raw = np.zeros((B, Hkv, NBcap, d), np.float64) if raw else None
    sg_raw = np.zeros((B, Hkv, NBcap, d), np.float64) if raw else None
    m_raw = np.zeros((B, Hkv, NBcap), np.float64) if raw else None
    sb, sh, st = cache.strides("K")
    lib().eta_oracle_block_summaries(
        _p(cache.K, _u16), _L(sb), _L(sh), _L(st), _I(B), _I(Hkv), _I(d), _I(cache.block_size), _I(NBcap),
        _p(cache.seq_lens, _i32), _I(1 if envelope else 0),
        _p(musig, _u16), _p(mnorm, _f32), _p(mu_raw, _f64), _p(sg_raw, _f64), _p(m_raw, _f64))
    if raw:
        return musig, mnorm, mu_raw, sg_raw, m_raw
    return musig, mnorm


def e4m3_to_double(bits: int) -> float:
    f = lib().eta_oracle_e4m3_to_double
    f.restype, f.argtypes = ctypes.c_double, [ctypes.c_uint8]
    return f(int(bits))


def double_to_e4m3_up(x: float) -> int:
    f = lib().eta_oracle_double_to_e4m3_up
    f.restype, f.argtypes = ctypes.c_uint8, [ctypes.c_double]
    return int(f(float(x)))


def block_summaries_sigma8(cache: Cache, envelope: bool = False):
    """Packed index: -> musig8 uint8 [B,Hkv,NBcap,3d] (mu fp16, then sigma rounded up to e4m3), mnorm float32."""
    musig, mnorm, _, sg_raw, _ = block_summaries(cache, envelope=envelope, raw=True)
    B, Hkv, NBcap, d = cache.B, cache.Hkv, cache.NBcap, cache.d
    musig8 = np.zeros((B, Hkv, NBcap, 3 * d), np.uint8)
    lib().eta_oracle_pack_sigma8(_p(musig, _u16), _p(sg_raw, _f64), _I(B), _I(Hkv), _I(d), _I(cache.block_size), _I(NBcap),
                                 _p(cache.seq_lens, _i32), _p(musig8, _u8))
    return musig8, mnorm


def unpack_sigma8(musig8: np.ndarray) -> np.ndarray:
    """Packed records -> the fp16 record layout [.., 2, d] with the rounded-up sigma (exact: e4m3 is a subset of fp16)."""
    *lead, d3 = musig8.shape
    d = d3 // 3
    n_rec = int(np.prod(lead))
    musig = np.zeros((*lead, 2, d), np.uint16)
    lib().eta_oracle_unpack_sigma8(_p(np.ascontiguousarray(musig8), _u8), _L(n_rec), _I(d), _p(musig, _u16))
    return musig


def predict_threshold(q: np.ndarray, W: np.ndarray, bias: np.ndarray) -> np.ndarray:
    """q uint16 [B,Hq,d], W float32 [Hq*d,Hq], bias float32 [Hq] -> tau float64 [B,Hq]."""
    B, Hq, d = q.shape
    assert W.shape == (Hq * d, Hq) and bias.shape == (Hq,)
    tau = np.zeros((B, Hq), np.float64)
    lib().eta_oracle_predict_threshold(_p(q, _u16), _p(W, _f32), _p(bias, _f32), _I(B), _I(Hq), _I(d), _p(tau, _f64))
    return tau


def score_dual(q, musig, mnorm, seq_lens, block_size, z, scale=None, parts=False):
    """-> bound float64 [B,Hq,NBcap] (NaN where j >= number of full blocks)."""
    B, Hq, d = q.shape
    _, Hkv, NBcap, _, _ = musig.shape
    s = (1.0 / np.sqrt(d)) if scale is None else scale
    bound = np.full((B, Hq, NBcap), np.nan, np.float64)
    g = np.full_like(bound, np.nan) if parts else None
    sp = np.full_like(bound, np.nan) if parts else None
    lib().eta_oracle_score_dual(
        _p(q, _u16), _p(musig, _u16), _p(mnorm, _f32), _I(B), _I(Hq), _I(Hkv), _I(d), _I(block_size), _I(NBcap),
        _p(seq_lens, _i32), _D(z), _D(s), _p(bound, _f64), _p(g, _f64), _p(sp, _f64))
    if parts:
        return bound, g, sp
    return bound


def select(bound, seq_lens, block_size, Hkv, tau=None, head_const=None, a=0.0, lwb=0, rescue_window=128,
           ungate_last=False):
    """-> sel uint8 [B,Hkv,NBcap] (bit g = query head hk*G+g), rescued int32 [B,Hq]."""
    B, Hq, NBcap = bound.shape
    assert (tau is None) != (head_const is None)
    sel = np.zeros((B, Hkv, NBcap), np.uint8)
    rescued = np.zeros((B, Hq), np.int32)
    tau32 = None if tau is None else np.ascontiguousarray(tau, np.float32)
    hc32 = None if head_const is None else np.ascontiguousarray(head_const, np.float32)
    lib().eta_oracle_select(
        _p(np.ascontiguousarray(bound), _f64), _p(tau32, _f32), _p(hc32, _f32), _I(B), _I(Hq), _I(Hkv),
        _I(block_size), _I(NBcap), _p(seq_lens, _i32), _D(a), _I(lwb), _I(rescue_window), _I(int(ungate_last)),
        _p(sel, _u8), _p(rescued, _i32))
    return sel, rescued


def gated_block_attention(q, cache: Cache, sel, tau=None, head_const=None, a=0.0, beta=5.0, scale=None,
                          extras=False, ungate_last=False):
    """-> out float64 [B,Hq,d] (+ logZ [B,Hq], n_tok [B,Hq] when extras)."""
    B, Hq, d = q.shape
    s = (1.0 / np.sqrt(d)) if scale is None else scale
    assert (tau is None) != (head_const is None)
    tau32 = None if tau is None else np.ascontiguousarray(tau, np.float32)
    hc32 = None if head_const is None else np.ascontiguousarray(head_const, np.float32)
    out = np.zeros((B, Hq, d), np.float64)
    logZ = np.zeros((B, Hq), np.float64)
    ntok = np.zeros((B, Hq), np.int64)
    ks, vs = cache.strides("K"), cache.strides("V")
    lib().eta_oracle_gated_block_attention(
        _p(q, _u16), _p(cache.K, _u16), _L(ks[0]), _L(ks[1]), _L(ks[2]),
        _p(cache.V, _u16), _L(vs[0]), _L(vs[1]), _L(vs[2]),
        _p(np.ascontiguousarray(sel), _u8), _p(tau32, _f32), _p(hc32, _f32),
        _I(B), _I(Hq), _I(cache.Hkv), _I(d), _I(cache.block_size), _I(cache.NBcap), _p(cache.seq_lens, _i32),
        _D(a), _D(beta), _D(s), _I(int(ungate_last)), _p(out, _f64), _p(logZ, _f64), _p(ntok, _i64))
    if extras:
        return out, logZ, ntok
    return out


def dense_softmax_attention(q, cache: Cache, scale=None):
    B, Hq, d = q.shape
    s = (1.0 / np.sqrt(d)) if scale is None else scale
    out = np.zeros((B, Hq, d), np.float64)
    ks, vs = cache.strides("K"), cache.strides("V")
    lib().eta_oracle_dense_softmax_attention(
        _p(q, _u16), _p(cache.K, _u16), _L(ks[0]), _L(ks[1]), _L(ks[2]),
        _p(cache.V, _u16), _L(vs[0]), _L(vs[1]), _L(vs[2]),
        _I(B), _I(Hq), _I(cache.Hkv), _I(d), _p(cache.seq_lens, _i32), _D(s), _p(out, _f64))
    return out


def block_max_logit(q, cache: Cache, scale=None):
    B, Hq, d = q.shape
    s = (1.0 / np.sqrt(d)) if scale is None else scale
    out = np.full((B, Hq, cache.NBcap), np.nan, np.float64)
    ks = cache.strides("K")
    lib().eta_oracle_block_max_logit(
        _p(q, _u16), _p(cache.K, _u16), _L(ks[0]), _L(ks[1]), _L(ks[2]),
        _I(B), _I(Hq), _I(cache.Hkv), _I(d), _I(cache.block_size), _I(cache.NBcap), _p(cache.seq_lens, _i32),
        _D(s), _p(out, _f64))
    return out


def calibration_density(hist, s_min, s_max, beta, c):
    """g(c) of the calibration appendix for one head's normalised histogram."""
    h = np.ascontiguousarray(hist, np.float64)
    f = lib().eta_oracle_calibration_density
    f.restype = ctypes.c_double
    return f(_p(h, _f64), _I(h.shape[0]), _D(s_min), _D(s_max), _D(beta), _D(c))


def calibrate(Q, K, tau, beta=5.0, scale=None, n_bins=2048, s_min=-8.0, s_max=8.0, iters=80):
    """Density-matched static thresholds.  Q uint16 (bf16 bits) [n_seq, Hq, T, d], K [n_seq, Hkv, T, d],
    tau float32 [n_seq, Hq, T]  ->  dict(hist [Hq, n_bins], dbar [Hq], head_const [Hq], residual [Hq])."""
    n_seq, Hq, T, d = Q.shape
    Hkv = K.shape[1]
    s = (1.0 / np.sqrt(d)) if scale is None else scale
    hist = np.zeros((Hq, n_bins), np.float64)
    dbar = np.zeros(Hq, np.float64)
    hc = np.zeros(Hq, np.float64)
    res = np.zeros(Hq, np.float64)
    lib().eta_oracle_calibrate(
        _p(np.ascontiguousarray(Q), _u16), _p(np.ascontiguousarray(K), _u16),
        _p(np.ascontiguousarray(tau, np.float32), _f32), _I(n_seq), _I(Hq), _I(Hkv), _I(T), _I(d), _D(beta), _D(s),
        _I(n_bins), _D(s_min), _D(s_max), _I(iters), _p(hist, _f64), _p(dbar, _f64), _p(hc, _f64), _p(res, _f64))
    return {"hist": hist, "dbar": dbar, "head_const": hc, "residual": res}


def decode_step(q, cache: Cache, musig, mnorm, tau=None, head_const=None, z=1.0, a=0.0, beta=5.0, lwb=0,
                rescue_window=128, scale=None, ungate_last=False):
    """The whole inference rule in the paper's order: bound -> select -> attend.

    -> dict(out, sel, bound, rescued).  `tau` / `head_const` are float32 inputs.
    """
    bound = score_dual(q, musig, mnorm, cache.seq_lens, cache.block_size, z, scale)
    sel, rescued = select(bound, cache.seq_lens, cache.block_size, cache.Hkv, tau=tau, head_const=head_const,
                          a=a, lwb=lwb, rescue_window=rescue_window, ungate_last=ungate_last)
    out = gated_block_attention(q, cache, sel, tau=tau, head_const=head_const, a=a, beta=beta, scale=scale,
                                ungate_last=ungate_last)
    return {"out": out, "sel": sel, "bound": bound, "rescued": rescued}

"""CPU checks of the C-ABI boundary: the library builds, loads, exports every declared symbol, and its host-side
argument validation answers without touching a device."""
import ctypes
import os
import re

import pytest

from paper_2609_20888_b200 import binding as eb
from paper_2609_20888_b200 import build as ebuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    ebuild.build()
    return eb.load()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "eta.h")).read()
    declared = set(re.findall(r"^(?:int|size_t|const char\*)\s+(eta_\w+)\s*\(", header, flags=re.M))
    assert declared, "no declarations found in include/eta.h"
    assert declared == set(eb.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in eta.h but not exported"


def _desc(**kw):
    base = dict(batch=2, n_q_heads=8, n_kv_heads=2, head_dim=128, block_size=64, t_cap=4096, nb_cap=64,
                k_stride_b=2 * 4096 * 128, k_stride_h=4096 * 128, k_stride_t=128,
                v_stride_b=2 * 4096 * 128, v_stride_h=4096 * 128, v_stride_t=128)
    base.update(kw)
    return eb.CacheDesc(**base)


def test_workspace_bytes_and_validation(lib):
    n = eb.eta_workspace_bytes(_desc())
    assert n > 0 and n % 256 == 0
    # grows with the block capacity, not with anything else
    assert eb.eta_workspace_bytes(_desc(t_cap=8192, nb_cap=128)) > n
    sz = ctypes.c_size_t(0)
    for bad, code in [(_desc(head_dim=96), -2), (_desc(block_size=48), -2), (_desc(n_q_heads=6), -2),
                      (_desc(n_q_heads=7), -1), (_desc(batch=0), -1), (_desc(k_stride_t=100), -2),
                      (_desc(nb_cap=8), -1)]:
        assert lib.eta_workspace_bytes(ctypes.byref(bad), ctypes.byref(sz)) == code
    assert lib.eta_workspace_bytes(None, ctypes.byref(sz)) == -1
    assert lib.eta_workspace_bytes(ctypes.byref(_desc()), None) == -1


def test_null_and_inconsistent_arguments_are_rejected_before_any_launch(lib):
    d, p = _desc(), eb.DecodeParams().c()
    null = ctypes.c_void_p(None)
    one = ctypes.c_void_p(256)          # never dereferenced on the host
    assert lib.eta_build_block_summaries(ctypes.byref(d), null, one, one, one, 0, null) == -1
    assert lib.eta_append_summary(ctypes.byref(d), one, null, one, one, 0, null) == -1
    assert lib.eta_predict_threshold(1, 8, 128, null, one, one, one, null) == -1
    assert lib.eta_predict_threshold(0, 8, 128, one, one, one, one, null) == -1
    assert lib.eta_score_dual(ctypes.byref(d), None, one, one, one, one, one, null) == -1
    # both tau and head_const, then neither
    args = [ctypes.byref(d), ctypes.byref(p), one, one, one, one, one, one]
    tail = [one, one, null, null, one, 1 << 30, null]
    assert lib.eta_decode(*args, one, one, *tail) == -1
    assert lib.eta_decode(*args, null, null, *tail) == -1
    # misaligned workspace, too-small workspace
    assert lib.eta_decode(*args, one, null, one, one, null, null, ctypes.c_void_p(264), 1 << 30, null) == -3
    assert lib.eta_decode(*args, one, null, one, one, null, null, one, 16, null) == -3
    # misaligned K
    args_bad = list(args)
    args_bad[3] = ctypes.c_void_p(260)
    assert lib.eta_decode(*args_bad, one, null, *tail) == -2
    bad = eb.DecodeParams(rescue_window=0).c()
    args2 = [ctypes.byref(d), ctypes.byref(bad)] + args[2:]
    assert lib.eta_decode(*args2, one, null, *tail) == -1


def test_kernel_attributes_are_remembered_per_device(lib):
    """cudaFuncSetAttribute results hold per (device, kernel): the library's bookkeeping must ask again on a second
    device, ask again for more shared memory, not ask twice for the same, and never remember a failure.  Host-only
    self-check with made-up device ordinals and a recording setter; 0 = every expectation held."""
    lib.eta_selftest_kernel_attr_table.restype = ctypes.c_int
    assert lib.eta_selftest_kernel_attr_table() == 0


def test_status_text(lib):
    assert lib.eta_strerror(0) == b"ok"
    assert b"workspace" in lib.eta_strerror(-3)
    assert lib.eta_decode_kernel_count() >= 1


def test_binding_refuses_cpu_tensors(lib):
    import torch
    K = torch.zeros((1, 2, 128, 128), dtype=torch.bfloat16)
    d = eb.cache_desc(K, K, 8, 64)
    ms = torch.zeros((1, 2, 2, 2, 128), dtype=torch.float16)
    mn = torch.zeros((1, 2, 2), dtype=torch.float32)
    with pytest.raises(eb.EtaError):
        eb.eta_build_block_summaries(d, K, torch.zeros(1, dtype=torch.int32), ms, mn)

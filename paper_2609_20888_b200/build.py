"""Build the C-ABI library `libeta_b200.so` in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libeta_b200.so")
HEADER = os.path.join(os.path.dirname(HERE), "include", "eta.h")


# A second copy of the library for one test: a consumer warp of the streaming kernel skips a barrier arrival, and the
# bounded waits are short (2^16 polls, a few milliseconds), so that a give-up path runs and can be checked.
GIVEUP_LIB = os.path.join(HERE, "libeta_b200_test_giveup.so")
GIVEUP_FLAGS = ["-DETA_TEST_SKIP_FLUSH_ARRIVE", "-DETA_WAIT_LIMIT=65536"]


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + [HEADER]
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False, lib: str = LIB, extra_flags: tuple = ()) -> str:
    if not force and not needs_build(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-o", lib] + list(extra_flags) + sources()
    cmd[1:1] = os.environ.get("ETA_NVCC_FLAGS", "").split()     # e.g. -DETA_WAIT_LIMIT=65536 while debugging
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.run(cmd, check=True)
    return lib


def build_giveup_variant(force: bool = False) -> str:
    return build(force=force, lib=GIVEUP_LIB, extra_flags=tuple(GIVEUP_FLAGS))


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))

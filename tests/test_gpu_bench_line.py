"""bench.py on a GPU, short run: the JSON line carries every key of the measurement contract and sane values."""
import json
import os
import subprocess
import sys

import pytest
import torch

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*extra):
    if not torch.cuda.is_available():
        pytest.skip("needs a GPU")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "4", "--warmup", "3", "--no-cpu",
                          "--no-sweep", *extra], cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    return json.loads(out.stdout.strip().splitlines()[-1])


@pytest.mark.parametrize("extra", [(), ("--paged",), ("--e2e-io", "copy"), ("--no-graph",)])
def test_bench_line_has_the_contract_keys(extra):
    d = _run(*extra)
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline"):
        assert key in d, key
    assert d["metric"] == "eta_decode_queries_per_s" and d["unit"] == "queries/s" and d["higher_is_better"] is True
    assert d["n_gpus"] == 1 and d["steps"] == 4 and d["warmup"] == 3 and d["vs_baseline"] is None
    assert d["config"]["workload"] == "c3_128k" and d["data"] == "synthetic" and d["scaling"] == "weak"
    assert d["value"] > 0 and abs(d["value"] * d["ms_per_step"] * 1e-3 - d["config"]["batch"]) < 1e-6 * d["config"]["batch"]
    assert d["gpu_launches"] == 4 * 5
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and 0.0 < r["frac"] < 1.2
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    e = d["e2e"]
    # (with four steps, and direct launches in particular, the two passes are too noisy to be ordered strictly)
    assert 0 < e["value"] < d["value"] * 1.5 and e["h2d_bytes_per_step"] == 4 * 32 * 128 * 2 and e["d2h_bytes_per_step"] == 4 * 32 * 128 * 4
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}

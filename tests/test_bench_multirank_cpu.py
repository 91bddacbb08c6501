"""Host-side logic of the N > 1 benchmark run, exercised on CPU with the gloo backend and two ranks: the path has
no exchange step, so a multi-GPU run is N independent replicas whose step time is the maximum over ranks and whose
value is the whole job's queries per second; rank 0 alone prints the JSON line."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _torchrun(extra, port):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"), "--gpus", "2"]
    env = dict(os.environ, OMP_NUM_THREADS="2")
    return subprocess.run(cmd + extra, cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)


def _json_lines(out):
    return [json.loads(l) for l in out.splitlines() if l.startswith("{")]


def test_two_gloo_ranks_report_the_slowest_rank_and_the_whole_job_value():
    r = _torchrun(["--dry-run", "--steps", "4", "--warmup", "3"], 29731)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = _json_lines(r.stdout)
    assert len(lines) == 1, "rank 0 alone prints"
    line = lines[0]
    assert line["n_gpus"] == 2 and line["scaling"] == "weak"
    assert line["ms_per_step"] == 1.5                      # ranks "measured" 1.0 and 1.5 ms: the maximum is reported
    assert abs(line["value"] - 2 * 4 / 1.5e-3) < 1e-6      # two replicas of the batch-4 workload per step


def test_reference_arm_under_two_ranks_prints_once():
    r = _torchrun(["--impl", "reference", "--workload", "c1_tiny", "--steps", "2", "--warmup", "1"], 29732)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = _json_lines(r.stdout)
    assert len(lines) == 1 and lines[0]["impl"] == "reference"
    assert lines[0]["cpu_baseline"]["kind"] == "oracle" and lines[0]["value"] > 0
    assert lines[0]["e2e"]["h2d_bytes_per_step"] == 0

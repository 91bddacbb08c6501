"""Writes tests/golden/workload_calibration.json: the predictor biases (and frozen per-head constants) that make
the seeded synthetic workloads hit their target union block sparsity.

Stand-in for a trained threshold predictor.  Calls only the CPU oracle and the input generators; run on the
host:  python tests/golden/make_workload_calibration.py [config ...]
The benchmark reads the stored biases; tests recompute theirs for scaled-down configurations.
"""
import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import eta_oracle as orc                                  # noqa: E402
from paper_2609_20888_b200 import workloads as wl                     # noqa: E402
from tests.helpers import bits, cache_of, calibrate_bias, calibrate_head_const, union_density  # noqa: E402

OUT = os.path.join(ROOT, "tests", "golden", "workload_calibration.json")
N_QUERY_DRAWS = 4


def calibrate(name: str) -> dict:
    sp = wl.CONFIGS[name]
    t0 = time.time()
    w = wl.make_workload(sp)
    c = cache_of(w)
    musig, mnorm = orc.block_summaries(c)
    bounds, taus = [], []
    for step in range(N_QUERY_DRAWS):
        q = bits(w.queries(step))
        bounds.append(orc.score_dual(q, musig, mnorm, c.seq_lens, sp.block_size, sp.z))
        taus.append(orc.predict_threshold(q, w.W.numpy(), np.zeros(sp.n_q_heads, np.float32)))
    bound = np.concatenate(bounds, axis=0)
    tau_raw = np.concatenate(taus, axis=0)
    lens = np.tile(c.seq_lens, N_QUERY_DRAWS)
    entry = {"seed": sp.seed, "z": sp.z, "query_draws": N_QUERY_DRAWS, "targets": {}}
    for tgt in sp.target_sparsity:
        bias = calibrate_bias(bound, tau_raw, lens, sp.block_size, sp.gqa, tgt)
        u = union_density(bound, tau_raw + bias[None, :], lens, sp.block_size, sp.gqa)
        entry["targets"][f"{tgt:.2f}"] = {"bias": [float(x) for x in bias], "union_sparsity": 1.0 - u}
        print(f"{name}: target {tgt:.2f} -> union sparsity {1 - u:.4f}", flush=True)
    if sp.frozen:
        consts = calibrate_head_const(bound, lens, sp.block_size, wl.frozen_sparsity_levels(sp))
        u = union_density(bound, np.broadcast_to(consts, tau_raw.shape), lens, sp.block_size, sp.gqa)
        entry["head_const"] = [float(x) for x in consts]
        entry["head_const_union_sparsity"] = 1.0 - u
    entry["seconds"] = round(time.time() - t0, 1)
    return entry


def main():
    names = sys.argv[1:] or list(wl.CONFIGS)
    data = json.load(open(OUT)) if os.path.exists(OUT) else {}
    for name in names:
        data[name] = calibrate(name)
        json.dump(data, open(OUT, "w"), indent=1, sort_keys=True)
    print("wrote", OUT)


if __name__ == "__main__":
    main()

"""Writes tests/golden/config_golden.json: what the CPU oracle gives on the five seeded workload
configurations at full size (baseline makespan and energy, selection per latency budget with its
margin, digests of the per-policy integer results, sampled per-policy values).

The script calls only the input generators and oracle/ - never the CUDA library.  Run it from the
repository root:  python tests/golden/make_config_golden.py [config ...]
"""
from __future__ import annotations

import hashlib
import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2607_12324_b200 import workloads as W  # noqa: E402

OUT = os.path.join(ROOT, "tests", "golden", "config_golden.json")


def digest(a: np.ndarray) -> str:
    return hashlib.sha256(np.ascontiguousarray(a).tobytes()).hexdigest()


def one(name: str, threads: int) -> dict:
    t0 = time.time()
    g = W.make_graph(name)
    B = g.meta["B"]
    lv = W.policies_for(g, ldb=B).numpy()
    r = oracle.batch(g, lv, B=B, want_slack=True, threads=threads)
    allmax = np.full((g.n, 1), g.L - 1, dtype=np.uint8)
    base = oracle.batch(g, allmax, want_slack=True)
    T0, E0 = int(base["makespan"][0]), float(base["energy"][0])
    rec = {"n": g.n, "m": g.m, "L": g.L, "B": B, "n_levels": g.n_levels, "T0": T0, "E0": E0,
           "n_critical_allmax": int(base["n_critical"][0]), "slack_sum_allmax": int(base["slack_sum"][0]),
           "makespan_sha256": digest(r["makespan"]), "slack_sum_sha256": digest(r["slack_sum"]),
           "n_critical_sha256": digest(r["n_critical"]),
           "energy_fsum": float(np.sum(r["energy"].astype(np.longdouble))),
           "sample_idx": [], "sample_makespan": [], "sample_energy": [], "select": []}
    idx = sorted(set(np.linspace(0, B - 1, 48).astype(int).tolist()))
    rec["sample_idx"] = idx
    rec["sample_makespan"] = [int(r["makespan"][i]) for i in idx]
    rec["sample_energy"] = [float(r["energy"][i]) for i in idx]
    for ppm in g.meta["delta_ppm"]:
        tgt = oracle.target_from_delta(T0, ppm)
        feas = r["makespan"] <= tgt
        i = oracle.select(r["makespan"], r["energy"], tgt)
        e_sorted = np.sort(r["energy"][feas])
        margin = float((e_sorted[1] - e_sorted[0]) / e_sorted[0]) if e_sorted.size > 1 else None
        rec["select"].append({"delta_ppm": ppm, "target": int(tgt), "index": int(i),
                              "T": int(r["makespan"][i]) if i >= 0 else None,
                              "E": float(r["energy"][i]) if i >= 0 else None,
                              "n_feasible": int(feas.sum()), "margin_rel": margin,
                              "energy_saving": float(1 - r["energy"][i] / E0) if i >= 0 else None,
                              "perf_loss": float(r["makespan"][i] / T0 - 1) if i >= 0 else None})
    rec["seconds"] = round(time.time() - t0, 1)
    return rec


def main():
    names = sys.argv[1:] or list(W.CONFIGS)
    threads = os.cpu_count() or 1
    data = {}
    if os.path.exists(OUT):
        with open(OUT) as f:
            data = json.load(f)
    for name in names:
        data[name] = one(name, threads)
        print(name, json.dumps(data[name]["select"]), data[name]["seconds"], "s", flush=True)
        with open(OUT, "w") as f:
            json.dump(data, f, indent=1, sort_keys=True)
            f.write("\n")


if __name__ == "__main__":
    main()

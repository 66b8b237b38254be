"""Writes tests/golden/config_seeds.json: the graph seeds of the two random-DAG workloads.

Rule (mechanical, uses only the oracle): starting at BASE_SEED + k (k = 3 for the elementwise
DAG, 5 for the row-reduction DAG) take the smallest seed whose graph, evaluated on a reduced
tensor size, has
  * every fp64 intermediate finite and below 1e30 in magnitude, and
  * "fp32 floor" <= 0.25: the same interpreter run in float32 on the CPU stays within a quarter
    of the 1e-5*(1+|ref|) tolerance of the fp64 result for every fetched tensor,
so that the tolerance is spent on the GPU kernels and not on the conditioning of the graph.
Rejected seeds are recorded with their floors.  Run from the repository root:
    python tests/golden/select_seeds.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle import interp, prune  # noqa: E402
from paper_1707_08265_b200 import workloads as wl  # noqa: E402

TOL = 1e-5


def floor_of(desc, inputs, outputs, feeds):
    ref, val, gval = interp.run_function(desc, inputs, outputs, feeds, return_all=True)
    for v in list(val.values()) + [x for gv in gval for x in gv.values()]:
        a = np.asarray(v, dtype=np.float64)
        if not np.all(np.isfinite(a)) or np.max(np.abs(a), initial=0.0) >= 1e30:
            return float("inf")
    low = interp.run_function(desc, inputs, outputs, feeds, dtype=np.float32)
    worst = 0.0
    for r, l in zip(ref, low):
        worst = max(worst, float(np.max(np.abs(l.astype(np.float64) - r) / (TOL * (1 + np.abs(r))))))
    return worst


def elementwise(seed):
    n = 1 << 16
    g, inputs, fetch = wl.random_dag(n, seed)
    feeds = wl.normal_feeds([[n]] * 4, seed)
    return floor_of(g.desc, inputs, fetch, feeds)


def row_dag(seed):
    rows, cols = 32, 4096
    g, inputs, fetch = wl.random_row_dag(rows, cols, seed)
    G = prune.backward_marks(g.desc, fetch, inputs)
    wrts = [i for i in inputs if i in G]
    grads = g.grad(fetch, wrts)
    feeds = wl.normal_feeds([g.shape(i) for i in inputs], seed)
    return floor_of(g.desc, inputs, fetch + grads, feeds)


def search(fn, start):
    rejected = []
    seed = start
    while True:
        f = fn(seed)
        if f <= 0.25:
            return seed, f, rejected
        rejected.append([seed, None if not np.isfinite(f) else round(f, 3)])
        seed += 1
        if seed - start > 500:
            raise RuntimeError("no well-conditioned seed in 500 tries")


if __name__ == "__main__":
    out = {}
    for name, fn, k in (("random_dag", elementwise, 3), ("random_row_dag", row_dag, 5)):
        seed, f, rej = search(fn, wl.BASE_SEED + k)
        out[name] = {"seed": seed, "floor": round(f, 4), "rejected": rej}
        print(name, out[name])
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "config_seeds.json"), "w") as fh:
        json.dump(out, fh, indent=1)

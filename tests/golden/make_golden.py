"""Writes tests/golden/tiny_cascade.json from the CPU oracle alone.

    python tests/golden/make_golden.py

The values are the oracle's results on the tiny fp32 workload (4 layers, 4 heads, N = 512): per layer
H, V, P, the final budgets, and for every (layer, head) the number of retained positions, their sum
and the sum of their squares.  Nothing here comes from the CUDA path.
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import cake_oracle as O                      # noqa: E402
from paper_2503_12491_b200 import synth                  # noqa: E402  (seeded inputs only)


def compute():
    w = synth.workload(1)
    qs, ks = [], []
    for l in range(w.n_layers):
        q, k, _ = synth.layer_inputs(w, l, "cpu")
        qs.append(q[0].double().numpy())
        ks.append(k.double().numpy())
    res = O.run_request(qs, ks, gamma=w.gamma, pool_kernel=w.pool_kernel,
                        total_budget=w.total_budget, tau1=w.tau1, tau2=w.tau2)
    c = res["cascade"]
    out = {"workload": w.name,
           "H": [float(s["H"]) for s in res["scored"]],
           "V": [float(s["V"]) for s in res["scored"]],
           "P": [float(s["P"]) for s in res["scored"]],
           "budgets": [int(b) for b in c.budgets],
           "positions": []}
    for l in range(w.n_layers):
        for g in range(w.n_kv_heads):
            p = np.asarray(c.positions[l][g], dtype=np.int64)
            out["positions"].append([l, g, int(p.size), int(p.sum()), int((p * p).sum())])
    return out


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_cascade.json")
    with open(path, "w") as f:
        json.dump(compute(), f, indent=1)
        f.write("\n")
    print("wrote", path)

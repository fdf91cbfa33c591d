"""Writes the stored per-step traces under tests/golden/ by running the CPU
reference checker (and nothing else) on the small seeded configurations.

    python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402
from paper_2605_06113_b200 import workload as wlm  # noqa: E402


def run(name, steps):
    cfg = wlm.get_config(name)
    wl = wlm.make_workload(cfg)
    o = oracle.instance_from_workload(wl, 0)
    rows = []
    for k in range(steps):
        probs = wlm.term_probs_np(wl, k)[0] if cfg.H > 0 else None
        assign, load, trace, _ = o.step(probs)
        adm = np.nonzero(assign >= 0)[0]
        rows.append((k, int(trace[0]), int(trace[1]), int(trace[2]), len(adm),
                     int(assign[adm].sum()) if len(adm) else 0))
    return rows


if __name__ == "__main__":
    for name, steps in (("c0", 300), ("c2", 200)):
        path = os.path.join(HERE, f"{name}_trace.txt")
        with open(path, "w") as f:
            f.write(f"# configuration {name}, instance 0: per decode step k the load trace after admissions\n"
                    "# (max_g L_g, min_g L_g, sum_g L_g), the number of admissions and the sum of the\n"
                    "# admitted slot indices.  Written by tests/golden/make_golden.py from the CPU checker.\n")
            for r in run(name, steps):
                f.write(" ".join(str(x) for x in r) + "\n")
        print("wrote", path)

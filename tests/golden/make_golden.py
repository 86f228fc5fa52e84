"""Writes tests/golden/oracle_cfg_tiny.txt from the CPU oracle alone (never from the CUDA path).

Run from the repository root:  python tests/golden/make_golden.py
The file is a regression pin: it freezes the oracle's answers on the tiny forms of the five
configurations, so an accidental change to the oracle's arithmetic shows up as a diff."""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import oracle  # noqa: E402
import workloads  # noqa: E402


def main():
    lines = ["# oracle outputs on workloads.make(cfg, tiny=True): sum, sum of squares, first bag's first 4 values"]
    for cfg in (1, 2, 3, 4, 5):
        wl = workloads.make(cfg, tiny=True)
        out = oracle.forward_workload(wl)
        vals = [out.sum(), (out ** 2).sum(), *out[0, :4]]
        lines.append(f"cfg{cfg} " + " ".join(f"{v:.17e}" for v in vals))
        if wl.grad_out is not None:
            grads = oracle.backward_workload(wl)
            g = [sum(float(c.sum()) for c in tg) for tg in grads]
            lines.append(f"cfg{cfg}_grad_sums " + " ".join(f"{v:.17e}" for v in g))
    with open(os.path.join(os.path.dirname(__file__), "oracle_cfg_tiny.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()

"""Writes tau_calibration.txt: for each synthetic workload, the CPU oracle's interval scores U of
the two token classes (interior / boundary) on a bounded number of rows, and where the workload's
frozen threshold tau sits between them.  Calls only the oracle and the input generator.

    python tests/golden/make_tau_calibration.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2603_25463_b200 import synth  # noqa: E402

LIMITS = {"llamagen256": 256, "llamagen384": 2304, "anole": 1024, "largevocab": 64, "decode": 1024}


def main():
    lines = ["# workload rows max_U_interior min_U_boundary geometric_middle tau flagged_fraction",
             "# written by tests/golden/make_tau_calibration.py from the CPU oracle (no GPU involved)"]
    for name, limit in LIMITS.items():
        wl = synth.WORKLOADS[name]
        inp = synth.make_inputs(wl, row_limit=limit)
        prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=inp.radius_row, tau=wl.tau)
        q = oracle.quantify(inp.draft, prm, wl.valid_begin, wl.n_valid)
        b = inp.boundary.numpy()
        hi_int, lo_bnd = float(q.score[~b].max()), float(q.score[b].min())
        assert hi_int < wl.tau < lo_bnd, (name, hi_int, wl.tau, lo_bnd)
        lines.append("%s %d %.6e %.6e %.6e %.1e %.4f" % (name, inp.draft.shape[0], hi_int, lo_bnd,
                                                          float(np.sqrt(hi_int * lo_bnd)), wl.tau, float(q.flag.mean())))
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "tau_calibration.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")
    print("\n".join(lines))


if __name__ == "__main__":
    main()

"""Writes tests/golden/c1_trajectory.txt: the float64 oracle's trajectory on workload C1 (64x32, bilateral,
S = 2nd, tau = 2, refresh every 5 updates, 20 calls), as a few sampled entries and norms per call.

Calls only `oracle/` and the seeded input generators of `workloads/`.  The stored values are not the
paper's (it prints no worked example of a step): they guard the oracle against accidental changes of its
arithmetic -- a later edit that moves any of them needs a reason that names the passage of the paper.

    python tests/golden/make_c1_trajectory.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import br_oracle as O  # noqa: E402
from workloads import GradientStream, get_workload, initial_weight  # noqa: E402

SAMPLES = [(0, 0), (3, 7), (17, 30), (63, 31), (40, 5)]


def rows():
    w = get_workload("c1")
    orc = O.make_oracle(w, [initial_weight(w, 0)])
    gs = GradientStream(w, 0)
    lay = orc.layers[0]
    for c in range(1, w.calls + 1):
        st = orc.step([gs(c)], w.tau)
        vals = [lay.W[i, j] for i, j in SAMPLES] + [np.linalg.norm(lay.W), np.linalg.norm(lay.M), np.linalg.norm(lay.V2),
                                                   np.linalg.norm(lay.L), np.linalg.norm(lay.R), lay.U[0, 0], lay.V[1, 0]]
        yield c, st, lay.t, lay.refresh_count, vals


if __name__ == "__main__":
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "c1_trajectory.txt")
    with open(out, "w") as f:
        f.write("# oracle trajectory on C1; written by tests/golden/make_c1_trajectory.py (calls only oracle/ and workloads/)\n")
        f.write("# call status t refresh_count W[0,0] W[3,7] W[17,30] W[63,31] W[40,5] |W| |M| |V~| |L| |R| U[0,0] V[1,0]\n")
        for c, st, t, rc, vals in rows():
            f.write(f"{c} {st} {t} {rc} " + " ".join(f"{v:.17e}" for v in vals) + "\n")
    print(out)

"""Writes tests/golden/config0_bruteforce.txt.

Every stored value comes from the oracle's exhaustive enumerator
(orc_brute_force: the plain definition of the search problem) run on the
seeded tiny workload; the dynamic program is *not* used, so the file can pin it.

    python tests/golden/make_golden.py
"""
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import oracle                                   # noqa: E402
from paper_2504_03662_b200 import inputs                    # noqa: E402


def main():
    w = inputs.config0()
    t, m, x = w.time_q[0], w.mem_q[0], w.trans_q[0]
    lines = ["# Tiny workload (L=4, S=6, M=64, seed 0): optimum per budget by exhaustive enumeration of all 6^4 plans.",
             "# The paper prints no worked example; these follow its problem statement (Section 3, Dynamic Strategy Selector).",
             "# budget opt_cost mem_used n_feasible plan[0..3]"]
    for budget in range(w.M + 1):
        opt, plan, used, n = oracle.brute_force(t, m, x, budget)
        lines.append(f"{budget} {opt} {used} {n} " + " ".join(str(int(p)) for p in plan))
    with open(os.path.join(HERE, "config0_bruteforce.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()

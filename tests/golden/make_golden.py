"""Writes tests/golden/config1_oracle.txt from the CPU oracle alone (no CUDA code is imported).

The paper prints no worked numeric example, so there is no published value to store; this file
freezes the oracle's own results on the first instances of the tiny configuration (V=16, n=2,
full-support draft; the seeded generator of paper_2511_15898_b200/workloads.py), after they have
been checked against subset enumeration by tests/test_oracle_pins.py, to catch later drift of the
oracle's arithmetic.  Run:  python tests/golden/make_golden.py
"""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import gr_oracle as O                       # noqa: E402
from paper_2511_15898_b200 import workloads as W        # noqa: E402


def main():
    wl = W.config1(batch=8)
    tl = W.logits_to_f64(wl.q_logits); dl = W.logits_to_f64(wl.p_logits)
    lines = ["# instance alpha_star jstar nblocks  (Eq. subset-select; Sec. 6.1) -- oracle values, config 1 seed 1000"]
    for b in range(8):
        sol = O.solve(tl[b], dl[b], wl.n, wl.topk, tol=1e-12)
        lines.append(f"{b} {sol.alpha_star:.15f} {sol.jstar} {sol.nblocks}")
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "config1_oracle.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()

"""Writes tests/golden/cfg1_oracle_rows.txt from the CPU oracle alone.

The paper prints no numeric example of an attention result, so this fixture is not a paper value: it freezes what the
pinned oracle (oracle/psa_oracle.c, see tests/test_oracle_pins.py) computes for 16 rows of configuration 1, so that
later changes to the oracle, to the input generator or to the seeds are noticed.  Run from the repository root:

    python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
import psa_workloads as wl  # noqa: E402

ROWS = [0, 3, 7, 8, 13, 21, 26, 31, 32, 38, 45, 47, 52, 55, 60, 63]


def main():
    w = wl.make_workload(wl.CONFIGS["cfg1"])
    out, lse, _ = oracle.attend(w, rows=np.array(ROWS))
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "cfg1_oracle_rows.txt")
    with open(path, "w") as f:
        f.write("# cfg1 (1 prompt, 8 samples, 8 q / 2 kv heads, D 64, prefix 512, suffix U[1,128], seed 0), fp64 oracle\n")
        f.write("# operator: softmax(S).V with S = QK^T (paper, appendix 'Benchmark details', group attn); not a value the paper prints\n")
        f.write(f"# input checksum {wl.checksum(w)}\n")
        f.write("# row  lse  out[0]  out[1]  out[31]  out[63]  sum(out)\n")
        for i, r in enumerate(ROWS):
            o = out[i]
            f.write(f"{r} {lse[i]:.17g} {o[0]:.17g} {o[1]:.17g} {o[31]:.17g} {o[63]:.17g} {o.sum():.17g}\n")
    print("wrote", path)


if __name__ == "__main__":
    main()

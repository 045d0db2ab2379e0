"""The stored oracle rows of configuration 1 (tests/golden/, written by make_golden.py from the oracle alone)."""
import os

import numpy as np
import pytest

import psa_workloads as wl

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "cfg1_oracle_rows.txt")


def load():
    rows, vals, checksum = [], [], None
    for line in open(GOLDEN):
        if line.startswith("# input checksum"):
            checksum = int(line.split()[-1])
        if line.startswith("#") or not line.strip():
            continue
        parts = line.split()
        rows.append(int(parts[0])); vals.append([float(x) for x in parts[1:]])
    return np.array(rows), np.array(vals), checksum


def test_generator_and_oracle_still_reproduce_the_stored_rows():
    import oracle
    rows, vals, checksum = load()
    w = wl.make_workload(wl.CONFIGS["cfg1"])
    assert wl.checksum(w) == checksum, "the seeded inputs of cfg1 changed"
    out, lse, _ = oracle.attend(w, rows=rows)
    got = np.column_stack([lse, out[:, 0], out[:, 1], out[:, 31], out[:, 63], out.sum(axis=1)])
    assert np.max(np.abs(got - vals)) < 1e-12


@pytest.mark.gpu
def test_gpu_matches_the_stored_rows():
    from psa_testlib import LSE_TOL, OUT_TOL, run_gpu
    rows, vals, _ = load()
    w = wl.make_workload(wl.CONFIGS["cfg1"], poison=True)
    out, lse, _ = run_gpu(w, "f32")
    assert np.max(np.abs(lse[rows] - vals[:, 0])) <= LSE_TOL
    got = np.column_stack([out[rows, 0], out[rows, 1], out[rows, 31], out[rows, 63]])
    assert np.max(np.abs(got - vals[:, 1:5])) <= OUT_TOL

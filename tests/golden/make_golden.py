"""Writes tests/golden/worked_example.txt by calling only the CPU oracle.

The paper prints no numeric worked example for the Newton-Schulz iteration (Eq. 1), so
the fixture is generated: inputs are given by the integer formula
    g(m, n, k)[i, j] = ((3 i + 5 j + k) mod 7) - 3 + 0.25 i
and the stored numbers are the oracle's float64 results.  The test that reads the
fixture also checks the same numbers against an SVD closed form, so the file is a
regression pin, not the only pin.

Run:  python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle import muon_oracle as orc  # noqa: E402

QUINTIC = (3.4445, -4.7750, 2.0315)


def g(m, n, k=0):
    i = np.arange(m)[:, None]
    j = np.arange(n)[None, :]
    return (((3 * i + 5 * j + k) % 7) - 3 + 0.25 * i).astype(np.float64)


def main():
    lines = ["# Eq. 1 worked example, quintic (3.4445, -4.7750, 2.0315) x 5, eps 1e-7, float64",
             "# written by tests/golden/make_golden.py from oracle/muon_oracle.py only"]

    def put(name, arr):
        arr = np.asarray(arr, dtype=np.float64)
        lines.append(f"{name} {arr.shape[0]} {arr.shape[1]} " + " ".join(repr(float(v)) for v in arr.reshape(-1)))

    put("NS5_g350", orc.newton_schulz(g(3, 5, 0), 5, QUINTIC, 1e-7, "fp64"))
    put("NS5_g530", orc.newton_schulz(g(5, 3, 0), 5, QUINTIC, 1e-7, "fp64"))
    lr, mu, wd = 0.02, 0.95, 0.01
    W = 0.01 * g(3, 5, 2)
    M = np.zeros((3, 5))
    for t in (1, 2):
        W, M, O = orc.muon_step(W, 1e-3 * g(3, 5, 3 + t), M, lr, mu, wd, 5, QUINTIC, 1e-7, True, "fp64")
        put(f"W_after_step{t}", W)
        put(f"M_after_step{t}", M)
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "worked_example.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()

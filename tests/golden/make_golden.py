"""Writes tests/golden/oracle_small_cases.json: what the CPU oracle returns on small inputs given by a formula.

The paper prints no worked example, so there are no values of the paper's to store; this file is a regression
anchor for the oracle itself (a later change to its arithmetic shows up as a diff here and has to be justified).
It calls only ``oracle/``.  Run from the repository root:  python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import oracle  # noqa: E402


def inputs(m: int, n: int):
    """theta[k][i], g[k][i] from integer formulas (exactly representable in fp32, no random numbers)."""
    k = np.arange(m, dtype=np.float64)[:, None]
    i = np.arange(n, dtype=np.float64)[None, :]
    theta = ((7 * k + 3 * i) % 11 - 5) / 8.0 + i / 16.0
    d = 1.0 + (i % 5)                       # a diagonal quadratic: g = d * theta - b + a small cross term
    b = ((5 * i) % 7 - 3) / 4.0
    g = d * theta - b + ((k * k + 2 * i) % 5 - 2) / 64.0
    return theta.astype(np.float32), g.astype(np.float32)


CASES = [(2, 5, 1.0, 0.5), (4, 9, 0.5, 0.01), (6, 12, 1.0, 0.1), (8, 40, 0.25, 0.001)]


def main():
    oracle.build()
    out = []
    for m, n, tau, lam in CASES:
        theta, g = inputs(m, n)
        r = oracle.update(theta, g, tau, lam)
        out.append({"m": m, "n": n, "tau": tau, "lam": lam, "j": int(r.j),
                    "sigma": [float.hex(float(x)) for x in r.sigma],
                    "theta_new": [float.hex(float(x)) for x in r.theta_new]})
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_small_cases.json")
    with open(path, "w") as f:
        json.dump({"written_by": "tests/golden/make_golden.py (oracle only)", "cases": out}, f, indent=1)
    print("wrote", path, "cases", len(out), "max j", max(c["j"] for c in out))


if __name__ == "__main__":
    main()

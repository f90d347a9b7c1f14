"""Writes tests/golden/tiny_oracle_samples.txt: sampled fp64 oracle values for the
"tiny" configuration (B=1, T=256, H=2, d=64, fp32 inputs, seed 0).

The paper prints no worked example for the chunked scan, so this fixture does not
carry paper values: it is a drift guard.  It is produced by the sequential fp64
oracle alone (this script imports only ``oracle`` and the input generator) and lets
the tests notice any later change to the oracle's arithmetic or to the generator.
Run from the repository root:  python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from workloads import get_config, make_inputs, widen  # noqa: E402

SAMPLES = [(0, 0, 0), (1, 0, 5), (63, 1, 63), (64, 0, 17), (130, 1, 2), (255, 0, 0), (255, 1, 63)]
STATE_SAMPLES = [(0, 0, 0), (0, 63, 63), (1, 10, 20), (1, 31, 7)]


def main():
    x = make_inputs(get_config("tiny"))
    out, fin = oracle.sequential(widen(x.q), widen(x.k), widen(x.v), x.log_alpha, x.beta, None)
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_oracle_samples.txt")
    with open(path, "w") as f:
        f.write("# sequential fp64 oracle, config 'tiny' (seed 0); written by make_golden.py\n")
        f.write("# kind index... value(hex float)\n")
        for t, h, j in SAMPLES:
            f.write(f"out {t} {h} {j} {float(out[0, t, h, j]).hex()}\n")
        for h, m, j in STATE_SAMPLES:
            f.write(f"state {h} {m} {j} {float(fin[0, h, m, j]).hex()}\n")
        f.write(f"norm_out 0 0 0 {float(np.linalg.norm(out)).hex()}\n")
        f.write(f"norm_state 0 0 0 {float(np.linalg.norm(fin)).hex()}\n")
    print("wrote", path)


if __name__ == "__main__":
    main()

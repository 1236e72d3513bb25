"""Writes the stored oracle outputs under tests/golden/.  Calls only the CPU oracle."""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import ngc_inputs                      # noqa: E402
from oracle import ngc_oracle as orc   # noqa: E402


def main():
    w = ngc_inputs.WORKLOADS["tiny"]
    pl = orc.plan(w.n, list(w.levels), w.seed)
    vals = np.concatenate([B.reshape(-1) for B in pl["B"]])
    with open(os.path.join(HERE, "B_tiny_oracle.txt"), "w") as f:
        for v in vals:
            f.write(float(v).hex() + "\n")


if __name__ == "__main__":
    main()

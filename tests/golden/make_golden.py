"""Writes the stored expected values under tests/golden/ from the CPU oracle
alone (never from the CUDA path).  Run from the repository root:

    python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402
from paper_2604_09244_b200 import workloads as W  # noqa: E402


def main():
    wl = W.config1_tiny()
    st = oracle.State(wl.samples[0].n_vis)
    r = oracle.run_workload_step(wl, 0, [st])[0]
    np.savetxt(os.path.join(HERE, "config1_kept_idx.txt"), r.kept_idx, fmt="%d",
               header="kept positions of the tiny reference workload (seed 0), adaptive keep 50 %,\n"
                      "written by tests/golden/make_golden.py from the fp64 oracle")
    print("k_2d, k_3d =", r.k_2d, r.k_3d, "indicators", r.x)


if __name__ == "__main__":
    main()

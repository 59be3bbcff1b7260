"""Writes tests/golden/sampled_subspaces.txt: index lists of the random subspace rules for fixed seeds.

Calls nothing but the CPU checker under oracle/ (and numpy for the seeded norms).  Run from the repository
root:  python tests/golden/make_sampled_subspaces.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle import pvt_oracle as oracle  # noqa: E402

CASES = [  # (name, groups, k, mode, seed)
    ("uniform_g1000_k25_seed7", 1000, 25, oracle.SAMPLE_UNIFORM, 7),
    ("uniform_g4099_k40_seed2pow40", 4099, 40, oracle.SAMPLE_UNIFORM, 1 << 40),
    ("proportional_g1000_k25_seed7", 1000, 25, oracle.SAMPLE_PROPORTIONAL, 7),
    ("proportional_g4099_k40_seed123456789", 4099, 40, oracle.SAMPLE_PROPORTIONAL, 123456789),
]


def norms_for(groups):
    """Squared update norms of a seeded gradient (8 weights per group, eta = 1), by the checker."""
    g = np.random.default_rng(4242).normal(0.0, 1e-3, size=(groups, 8)).astype(np.float32)
    return oracle.group_norms(g, 1.0, 8)


def main():
    lines = ["# Index lists of the random subspace rules (CPU checker, fixed seeds); norms: squared update norms of",
             "# numpy.random.default_rng(4242).normal(0, 1e-3, (groups, 8)) as binary32, eta = 1.",
             "# Written by tests/golden/make_sampled_subspaces.py"]
    for name, groups, k, mode, seed in CASES:
        norms = norms_for(groups) if mode == oracle.SAMPLE_PROPORTIONAL else None
        idx = oracle.sample_subspace(groups, k, mode, seed, norms)
        lines.append(f"{name}: " + " ".join(str(int(i)) for i in idx))
    with open(os.path.join(ROOT, "tests", "golden", "sampled_subspaces.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()

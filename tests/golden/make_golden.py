"""Writes the stored known-answer files in this folder. Calls only the CPU oracle.

    python tests/golden/make_golden.py
"""
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import numpy as np  # noqa: E402

import oracle  # noqa: E402


def main():
    n, K, seed = 10, 3, 0
    owner, off, members = oracle.partition(n, K, seed)
    with open(os.path.join(HERE, "partition_n10_K3_seed0.txt"), "w") as f:
        f.write("# partition(n=10, K=3, seed=0) and the visiting orders of round 2, local epoch 1.\n")
        f.write("# Integer spec: SplitMix64 mixer; ids sorted by mix64(mix64(seed) ^ id); blocks of 4,3,3.\n")
        f.write("owner: " + " ".join(map(str, owner.tolist())) + "\n")
        f.write("part_off: " + " ".join(map(str, off.tolist())) + "\n")
        f.write("members: " + " ".join(map(str, members.tolist())) + "\n")
        for k in range(K):
            p = oracle.permutation(members[off[k]:off[k + 1]], seed, 2, 1)
            f.write("perm_r2_e1_k%d: " % k + " ".join(map(str, p.tolist())) + "\n")


if __name__ == "__main__":
    main()

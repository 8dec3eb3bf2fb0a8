"""Writes tests/golden/config1_oracle.txt: the seeded tiny config (config 1) as the generator draws it and
what the fp64 oracle computes for it.  Calls only the input generator and the oracle (never the CUDA path).

    python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import dyspec_oracle as orc                      # noqa: E402
from paper_2410_11744_b200 import workloads as wl            # noqa: E402


def main():
    w = wl.make_config(1)
    bits, depths = orc.build_tree_mask(w.parents[0], 4)
    out = orc.tree_attention(w.q, w.k, w.v, int(w.prefix_len[0]), w.parents[0])
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "config1_oracle.txt")
    with open(path, "w") as f:
        f.write("# config 1 (1 request, 4/4 heads, D 64, prefix 128, 16-node greedy tree, seed 241011745):\n")
        f.write("# generator output and fp64 oracle results; written by tests/golden/make_golden.py\n")
        f.write("parents " + " ".join(str(int(x)) for x in w.parents[0]) + "\n")
        f.write("depths " + " ".join(str(int(x)) for x in depths) + "\n")
        f.write("mask_word0 " + " ".join(f"0x{int(x):04x}" for x in bits[:, 0]) + "\n")
        f.write("q_bits_first8 " + " ".join(f"0x{int(x):04x}" for x in w.q.reshape(-1)[:8]) + "\n")
        f.write("k_bits_sum " + str(int(w.k.astype(np.uint64).sum())) + "\n")
        f.write("v_bits_sum " + str(int(w.v.astype(np.uint64).sum())) + "\n")
        for (i, h) in ((0, 0), (7, 3), (15, 1)):
            f.write(f"out {i} {h} " + " ".join(f"{x:.15e}" for x in out[i, h, :6]) + "\n")
        f.write(f"out_abs_sum {np.abs(out).sum():.12e}\n")
    print("wrote", path)


if __name__ == "__main__":
    main()

"""Writes tests/golden/tiny_expected.txt: the float64 oracle's output for the `tiny` workload
(batch 4, lengths {1, 7, 64, 300}, 4 query heads / 1 KV head, head_dim 64, seed 0).

The paper prints no number for decode attention, so this file is not a paper value: it is a
regression pin of the oracle itself, written by this script, which calls nothing but the seeded
input generators and `oracle/`.  Run from the repository root:

    python tests/golden/make_tiny_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import attention_oracle as O  # noqa: E402
from paper_2606_03077_b200 import workloads as W  # noqa: E402


def main():
    lay, q, k, v = W.make_host_inputs("tiny")
    out, lse = O.paged_decode_attention(q, k, v, lay.block_table, lay.seq_lens)
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_expected.txt")
    with open(path, "w") as f:
        f.write("# oracle output for workload `tiny`, seed 0: per (sequence, head): lse, then out[0], out[21], out[42], out[63]\n")
        f.write("# written by tests/golden/make_tiny_golden.py (float64, 17 significant digits)\n")
        for b in range(out.shape[0]):
            for h in range(out.shape[1]):
                vals = [lse[b, h]] + [out[b, h, j] for j in (0, 21, 42, 63)]
                f.write(f"{b} {h} " + " ".join(f"{x:.17e}" for x in vals) + "\n")
    print("wrote", path)


if __name__ == "__main__":
    main()

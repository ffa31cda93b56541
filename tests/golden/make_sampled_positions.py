"""Writes tests/golden/sampled_positions.txt: literal sample positions of the sampled-threshold mode.

The position rule of the sampled-threshold mode (Section 4, fourth paragraph: the threshold is taken on
a 0.1 % sample) is part of that mode's definition and is frozen.  This script calls only the oracle and
stores, for a few (lo, hi, scope) triples, the sample size and the first, middle and last eight
positions, so that the pin compares the oracle with literal numbers instead of with a second copy of
its formula.  Run it only to add cases; a change in an existing line is a change of the definition.

    python tests/golden/make_sampled_positions.py
"""
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import graddrop_oracle as orc  # noqa: E402

CASES = [
    (1, 8201, 0),                        # 8200 elements from an odd start: 4096 samples, strata of 2 or 3 pairs
    (0, 1 << 20, 0),                     # the flat 2^20 workload
    (42_500_003, 85_000_003, 7),         # an embedding-sized scope at an odd offset, scope number 7
    (0, 1 << 30, 0),                     # the flat 2^30 workload
    (5, 1 << 32, 3),                     # the largest gradient the library takes
]


def main():
    lines = ["# lo hi scope m | first 8 | middle 8 (from m/2 - 4) | last 8   (written by make_sampled_positions.py from oracle/)"]
    for lo, hi, s in CASES:
        pos = orc.sampled_positions(lo, hi, s)
        m = pos.shape[0]
        mid = m // 2 - 4
        parts = [pos[:8], pos[mid:mid + 8], pos[-8:]]
        lines.append(f"{lo} {hi} {s} {m} | " + " | ".join(" ".join(str(int(x)) for x in p) for p in parts))
    with open(os.path.join(HERE, "sampled_positions.txt"), "w") as fh:
        fh.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()

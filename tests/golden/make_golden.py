"""Writes tests/golden/tiny_oracle.txt: oracle outputs for the seeded 'tiny' workload.

Calls only the oracle and the seeded input generator.  The paper prints no worked example for this
path, so these values are not the paper's: they freeze the oracle's own result (after it passed its
pins) so that a later, unintended change to the oracle or to the input recipe is noticed.

Run:  python tests/golden/make_golden.py
"""
import os
import sys
import zlib

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
from oracle import paged_decode_oracle as O  # noqa: E402
from paper_2606_07665_b200 import workloads as W  # noqa: E402


def summary():
    w = W.tiny()
    q_rot, k_after, v_after, out = O.oracle_decode_step(w)
    lines = [
        "# oracle result on workloads.tiny() (seed 1); written by tests/golden/make_golden.py",
        f"q_rot_crc32 {zlib.crc32(q_rot.tobytes()):08x}",
        f"k_cache_after_crc32 {zlib.crc32(k_after.tobytes()):08x}",
        f"v_cache_after_crc32 {zlib.crc32(v_after.tobytes()):08x}",
        f"block_table_crc32 {zlib.crc32(w.block_table.tobytes()):08x}",
    ]
    for h in range(w.Hq):
        vals = " ".join(f"{x:.17e}" for x in out[0, h, :4])
        lines.append(f"out_head{h}_first4 {vals}")
    return "\n".join(lines) + "\n"


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_oracle.txt")
    with open(path, "w") as f:
        f.write(summary())
    print(open(path).read())

"""Writes tests/golden/cfg1_decode_oracle.txt: outputs of the fp64 decode oracle on workload 1.

The paper prints no worked numerical example of attention, so this fixture is not a value
from the paper: it is what `oracle.pa_decode` (and nothing else) computes for the seeded tiny
workload, stored so that an accidental change of the oracle or of the input generator shows
up as a diff.  Run from the repository root:  python tests/golden/make_cfg1_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2602_07878_b200 import workloads as wl  # noqa: E402


def main():
    spec = wl.config_spec(1)
    q = wl.q_np(spec)
    k, v = wl.pools_np(spec)
    out = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "cfg1_decode_oracle.txt")
    with open(path, "w") as f:
        f.write("# oracle.pa_decode on workload 1 (4 sequences of 17/64/100/256 tokens, 8 heads,\n")
        f.write("# head_dim 64); written by tests/golden/make_cfg1_golden.py, not taken from the paper.\n")
        f.write("# columns: sequence head dim value(%.17g)\n")
        for b in range(spec.batch):
            for h in (0, 3, 7):
                for d in (0, 1, 31, 63):
                    f.write(f"{b} {h} {d} {out[b, h, d]:.17g}\n")
    print(path)


if __name__ == "__main__":
    main()

"""The stored oracle outputs for workload 1 still come out of the oracle and the generator."""
import os

import numpy as np

import oracle
from paper_2602_07878_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "cfg1_decode_oracle.txt")


def load_golden():
    rows = [ln.split() for ln in open(GOLDEN) if not ln.startswith("#")]
    return [(int(b), int(h), int(d), float(x)) for b, h, d, x in rows]


def test_oracle_reproduces_stored_cfg1_values():
    spec = wl.config_spec(1)
    out = oracle.pa_decode(wl.q_np(spec), *wl.pools_np(spec), spec.block_tables, spec.seq_lens,
                           spec.scale)
    rows = load_golden()
    assert len(rows) == 4 * 3 * 4
    for b, h, d, x in rows:
        assert abs(out[b, h, d] - x) <= 1e-15 * max(1.0, abs(x))

"""Writes tests/golden/cfg1_oracle_rows.json from the oracle alone (never from the CUDA path).

The paper prints no worked numerical example for attention, so there is no
paper-given fixture; this file is a drift guard for the oracle's arithmetic on
the single-request configuration (256 cached tokens, 128 new, 8/2 heads, d=64).
Run:  python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
import wpp_workloads as W  # noqa: E402


def main():
    w = W.cfg1()
    kp, vp = oracle.oracle_append(w.k_new(), w.v_new(), w.k_pool(), w.v_pool(), w.block_tables,
                                  w.prefix_lens, w.chunk_lens)
    units = [(0, 0, 0), (0, 1, 7), (0, 15, 3), (0, 16, 4), (0, 64, 1), (0, 127, 0), (0, 127, 7)]
    out, lse = oracle.oracle_attention_units(w.q(), kp, vp, w.block_tables, w.prefix_lens, w.chunk_lens,
                                             np.array(units, dtype=np.int32))
    doc = {
        "what": "fp64 oracle outputs for selected (request, chunk row, query head) of the single-request config",
        "units": units,
        "out_hex": [[float(x).hex() for x in row] for row in out],
        "lse_hex": [float(x).hex() for x in lse],
    }
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "cfg1_oracle_rows.json")
    with open(path, "w") as f:
        json.dump(doc, f, indent=1)
    print("wrote", path)


if __name__ == "__main__":
    main()

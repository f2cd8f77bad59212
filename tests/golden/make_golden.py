"""Writes tests/golden/oracle_tiny.json from the fp64 oracle alone.

Run from the repository root:  python tests/golden/make_golden.py
The file freezes what the oracle returns on one tiny seeded workload, so that a
later, accidental change to the oracle's arithmetic shows up as a diff.  It calls
nothing but `oracle/` and the seeded generator.  The paper prints no worked numeric
example (its one illustration of the ordering is a figure), so no fixture here
carries paper values; the closed-form cases of Eq. (5) live in the pin tests.
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle import cosa_oracle as O                      # noqa: E402
from synth.configs import tiny                           # noqa: E402
from synth.generator import bf16_bits_to_f64             # noqa: E402


def main():
    w = tiny(seed=7, hq=2, hkv=1, n=1024, needles=2)
    q, k, v, _ = w.make()
    q, k, v = (bf16_bits_to_f64(x) for x in (q, k, v))
    order, count = O.kap_select(q, k, s=8, budget=0.5)
    r = O.osk_attention(q, k, v, order, count, skip_scale=200.0, tightened_budget=0.3)
    doc = {
        "workload": {"seed": 7, "hq": 2, "hkv": 1, "n": 1024, "needles": 2, "band": 2,
                     "stride": 8, "kap_budget": 0.5, "skip_scale": 200.0, "osk_budget": 0.3},
        "order": order.tolist(), "count": count.tolist(),
        "visited": r["visited"].tolist(), "scored": r["scored"].tolist(),
        "out_sample": [float(x) for x in r["out"][1, 1000, :4]],
        "lse_sample": [float(x) for x in r["lse"][0, ::128]],
    }
    with open(os.path.join(os.path.dirname(__file__), "oracle_tiny.json"), "w") as f:
        json.dump(doc, f, indent=1)


if __name__ == "__main__":
    main()

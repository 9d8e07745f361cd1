"""Writes tests/golden/example_layer.json from the float64 oracle alone (run from the repository root:
`python -m tests.golden.make_golden`).  The file is a change detector for the oracle and a fixed target for
the CUDA path; the oracle's own pins against the paper and the mathematics are in tests/test_oracle_pins.py."""
import json
import os

import numpy as np

from oracle import shareprefill_oracle as orc
from tests.golden import inputs

SAMPLES = [(0, 5, 3), (0, 700, 127), (1, 129, 64), (1, 1023, 0), (2, 255, 17), (2, 640, 90), (3, 3, 3), (3, 1000, 101)]


def compute():
    q, k, v = inputs.make()
    Q, K, V = (t.double().numpy() for t in (q, k, v))
    res = orc.prefill_attn(Q, K, V, inputs.CLUSTER_MAP, inputs.PIVOT_HEADS, inputs.GAMMA, inputs.B)
    out, masks, imps = res["out"], res["mask"], res["importance"]
    nb = inputs.N // inputs.B
    doc = {
        "what": "Section 5.1 / Algorithm 'Construct Pivotal Pattern' (per row-block, gamma 0.9) / 'Share Pivotal Pattern' "
                "on the closed-form inputs of tests/golden/inputs.py, computed by oracle.shareprefill_oracle.prefill_attn",
        "shape": {"Hq": inputs.HQ, "Hkv": inputs.HKV, "N": inputs.N, "d": inputs.D, "B": inputs.B},
        "mask_rows_per_head": [["".join(str(int(x)) for x in masks[h][i]) for i in range(nb)] for h in range(inputs.HQ)],
        "importance_of_pivots": {str(p): [[float(x) for x in imps[t][i]] for i in range(nb)] for t, p in enumerate(inputs.PIVOT_HEADS)},
        "output_samples": [{"head": h, "row": r, "col": c, "value": float(out[h][r, c])} for h, r, c in SAMPLES],
    }
    return doc


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "example_layer.json")
    with open(path, "w") as f:
        json.dump(compute(), f, indent=1)
    print("wrote", path)

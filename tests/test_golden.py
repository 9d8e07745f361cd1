"""The stored example under tests/golden/: written by tests/golden/make_golden.py from the float64 oracle alone, on
closed-form inputs.  On the CPU it is a change detector for the oracle (whose pins against the paper and the
mathematics are in test_oracle_pins.py); on the GPU it is a fixed target for the CUDA path through the C ABI."""
import json
import os

import numpy as np
import pytest
import torch

from tests import _parity as par
from tests.golden import inputs

HERE = os.path.dirname(os.path.abspath(__file__))


def _golden():
    with open(os.path.join(HERE, "golden", "example_layer.json")) as f:
        d = json.load(f)
    nb = inputs.N // inputs.B
    mask = np.array([[[int(c) for c in row] for row in head] for head in d["mask_rows_per_head"]], np.uint8)
    assert mask.shape == (inputs.HQ, nb, nb)
    imp = {int(p): np.array(rows) for p, rows in d["importance_of_pivots"].items()}
    return d, mask, imp


def test_oracle_still_gives_the_stored_example():
    from tests.golden import make_golden
    d, mask, imp = _golden()
    now = make_golden.compute()
    assert now["mask_rows_per_head"] == d["mask_rows_per_head"]
    for p in inputs.PIVOT_HEADS:
        np.testing.assert_allclose(np.array(now["importance_of_pivots"][str(p)]), imp[p], rtol=0, atol=1e-13)
    for a, b in zip(now["output_samples"], d["output_samples"]):
        assert (a["head"], a["row"], a["col"]) == (b["head"], b["row"], b["col"])
        assert abs(a["value"] - b["value"]) <= 1e-12
    # what any such example must satisfy: rows of the importance map are distributions, the members carry their
    # pivot's mask, every row-block keeps at least one key-block and nothing above the diagonal
    for p in inputs.PIVOT_HEADS:
        np.testing.assert_allclose(imp[p].sum(axis=1), 1.0, atol=1e-12)
    for h in range(inputs.HQ):
        assert np.array_equal(mask[h], mask[inputs.PIVOT_HEADS[inputs.CLUSTER_MAP[h]]])
        assert (mask[h].sum(axis=1) >= 1).all() and np.array_equal(mask[h], np.tril(mask[h]))


@pytest.mark.gpu
def test_cuda_path_gives_the_stored_example():
    from paper_2505_19578_b200 import binding, build
    build.build()
    d, mask, imp = _golden()
    q, k, v = (t.cuda() for t in inputs.make())
    nb = inputs.N // inputs.B
    ctx = binding.Context()
    out = torch.full_like(q, float("nan"))
    got_mask = torch.full((inputs.HQ, nb, nb), 9, dtype=torch.uint8, device="cuda")
    ctx.sp_prefill_attn(q, k, v, inputs.CLUSTER_MAP, inputs.PIVOT_HEADS, inputs.GAMMA, inputs.B, out, mask_out=got_mask)
    torch.cuda.synchronize()
    assert ctx.status() == (0, 0)
    assert np.array_equal(got_mask.cpu().numpy(), mask)                       # bit-exact
    got_imp = torch.empty(len(inputs.PIVOT_HEADS), nb, nb, device="cuda")
    ctx.sp_dense_pivot_attn(q, k, v, inputs.PIVOT_HEADS, inputs.B, torch.empty_like(q), importance_out=got_imp)
    torch.cuda.synchronize()
    for t, p in enumerate(inputs.PIVOT_HEADS):
        np.testing.assert_allclose(got_imp[t].cpu().numpy(), imp[p], rtol=0, atol=par.IMP_ATOL)
    o = out.double().cpu().numpy()
    for s in d["output_samples"]:
        # bf16 output of values of order 1: half a unit in the last place is 2^-9 relative, plus the P rounding
        assert abs(o[s["head"], s["row"], s["col"]] - s["value"]) <= par.OUT_MAX_ABS, s

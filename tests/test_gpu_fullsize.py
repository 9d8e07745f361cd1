"""Parity at the benchmark's full sizes, in the launch configuration bench.py
times (sp_prefill_attn on the default kernel), on sampled row-blocks.

A row-block's mask and outputs depend only on that row-block's queries and the
keys before it, so the oracle can check any sample of row-blocks of a layer that
is far too large for it to compute in full.
"""
import numpy as np
import pytest
import torch

from paper_2505_19578_b200 import synth
from tests import _parity as par

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2505_19578_b200 import binding as b, build
    build.build()
    return b


def _sample(Nb, n_extra, seed):
    rng = np.random.default_rng(seed)
    return sorted({0, 1, Nb // 2, Nb - 1} | set(rng.choice(Nb, n_extra, replace=False).tolist()))


@pytest.mark.parametrize("name,gamma,n_extra", [("llama8b_128k", 0.9, 1), ("llama8b_32k", 0.9, 4),
                                                ("qwen7b_64k", 0.9, 2)])
def test_full_size_sampled_row_blocks(binding, name, gamma, n_extra):
    cfg = synth.CONFIGS[name]
    L = synth.make_layer(cfg, seed=0, device="cuda")          # the bench's workload (seed 0)
    out, mask = par.run_layer(binding, L, gamma, "tc")
    rows = _sample(cfg.seq // cfg.block, n_extra, 3)
    Lh = dict(L, q=L["q"].cpu(), k=L["k"].cpu(), v=L["v"].cpu())
    worst, exempt = par.check_layer(Lh, gamma, out, mask, row_blocks=rows)
    print(f"{name}: row-blocks {rows}: worst max_abs {worst[0]:.3e} rel_l2 {worst[1]:.3e}, "
          f"{exempt} row-blocks within {par.MASK_BAND} of the threshold flipped")
    # properties that hold at any size, over the whole mask
    m = mask.cpu().numpy()
    for p in L["pivot_heads"]:
        assert np.all(m[p].sum(axis=1) >= 1)
        assert np.all(np.triu(m[p], 1) == 0)
    assert torch.isfinite(out.float()).all()


def test_sweep_gamma_at_128k_mask_nesting(binding):
    # configs[2] sweeps gamma over 0.8 / 0.9 / 0.95: masks must be nested and density must grow
    cfg = synth.scaled(synth.CONFIGS["llama8b_128k"], 32768)
    L = synth.make_layer(cfg, seed=0, device="cuda")
    prev, dens = None, []
    for gamma in (0.8, 0.9, 0.95):
        out, mask = par.run_layer(binding, L, gamma, "tc")
        m = mask[L["pivot_heads"]].cpu().numpy()
        if prev is not None:
            assert np.all(prev <= m)
        prev = m
        dens.append(m.sum() / (len(L["pivot_heads"]) * cfg.seq // cfg.block * (cfg.seq // cfg.block + 1) / 2))
    assert dens[0] < dens[1] < dens[2] < 0.7

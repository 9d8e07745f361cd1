"""Parity at the benchmark's full sizes, in the launch configuration bench.py
times (sp_prefill_attn on the default kernel), on sampled row-blocks.

A row-block's mask and outputs depend only on that row-block's queries and the
keys before it, so the oracle can check any sample of row-blocks of a layer that
is far too large for it to compute in full.  Samples always hold row-blocks 0, 1,
Nb/2 and Nb-1; 16 row-blocks per head at 131072 tokens, 48 at 32768 and 65536.
"""
import dataclasses
import random

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


def _host(L):
    return dict(L, q=L["q"].cpu(), k=L["k"].cpu(), v=L["v"].cpu())


def _whole_mask_properties(L, mask, out):
    m = mask.cpu().numpy()
    for p in L["pivot_heads"]:
        assert np.all(m[p].sum(axis=1) >= 1)
        assert np.all(np.triu(m[p], 1) == 0)
    assert torch.isfinite(out.float()).all()


def _one_member_per_cluster(L):
    seen, pick = set(), []
    for h, c in enumerate(L["cluster_map"]):
        if h not in L["pivot_heads"] and c not in seen:
            seen.add(c)
            pick.append(h)
    return pick


def test_llama8b_128k_all_three_thresholds(binding):
    # the 131072-token workload at gamma 0.8 / 0.9 / 0.95 (the bench's seed): 16 row-blocks; every head at 0.9,
    # the pivots and one member of each cluster at 0.8 and 0.95; masks nested in gamma over the whole map
    cfg = synth.CONFIGS["llama8b_128k"]
    L = synth.make_layer(cfg, seed=0, device="cuda")
    runs = {}
    for gamma in (0.8, 0.9, 0.95):
        runs[gamma] = par.run_layer(binding, L, gamma, "tc")
        _whole_mask_properties(L, runs[gamma][1], runs[gamma][0])
    piv = L["pivot_heads"]
    m = {g: runs[g][1][piv].cpu().numpy() for g in runs}
    assert np.all(m[0.8] <= m[0.9]) and np.all(m[0.9] <= m[0.95])
    dens = [m[g].sum() for g in (0.8, 0.9, 0.95)]
    assert dens[0] < dens[1] < dens[2]
    rows = par.sample_rows(cfg.seq // cfg.block, 16, 3)
    few = _one_member_per_cluster(L)
    everyone = [h for h in range(cfg.n_q_heads) if h not in piv]
    st = par.check_layer_sampled(_host(L), runs, rows, members={0.8: few, 0.9: everyone, 0.95: few}, what="llama8b_128k")
    print(f"llama8b_128k gamma 0.8/0.9/0.95, row-blocks {rows}: worst max_abs {st['worst_max_abs']:.3e} "
          f"rel_l2 {st['worst_rel_l2']:.3e}; {st['exempt']} row-blocks within {par.MASK_BAND} of a threshold flipped; "
          f"{st['near_ties']} near-ties at a cut")


@pytest.mark.parametrize("name", ["llama8b_32k", "qwen7b_64k"])
def test_full_size_sampled_row_blocks(binding, name):
    cfg = synth.CONFIGS[name]
    gamma = 0.9
    L = synth.make_layer(cfg, seed=0, device="cuda")          # the bench's workload (seed 0)
    out, mask = par.run_layer(binding, L, gamma, "tc")
    _whole_mask_properties(L, mask, out)
    rows = par.sample_rows(cfg.seq // cfg.block, 48, 3)
    st = par.check_layer_sampled(_host(L), {gamma: (out, mask)}, rows, what=name)
    print(f"{name}: {len(rows)} row-blocks: worst max_abs {st['worst_max_abs']:.3e} rel_l2 {st['worst_rel_l2']:.3e}; "
          f"{st['exempt']} row-blocks within {par.MASK_BAND} of the threshold flipped; {st['near_ties']} near-ties at a cut")


def test_layer_stack_two_layers_at_128k(binding):
    # two layers of the 32-layer stack workload exactly as bench.py draws them (layer seeds 1 and 2, 3-6 clusters
    # each): 16 row-blocks, the pivots and one member of each cluster
    cfg = synth.CONFIGS["llama8b_128k"]
    rng = random.Random(0)
    for layer in range(2):
        lcfg = dataclasses.replace(cfg, n_clusters=rng.randint(3, 6))
        L = synth.make_layer(lcfg, seed=1 + layer, device="cuda")
        out, mask = par.run_layer(binding, L, 0.9, "tc")
        _whole_mask_properties(L, mask, out)
        rows = par.sample_rows(cfg.seq // cfg.block, 16, 11 + layer)
        st = par.check_layer_sampled(_host(L), {0.9: (out, mask)}, rows, members={0.9: _one_member_per_cluster(L)},
                                     what=f"stack layer {layer}")
        print(f"stack layer {layer} ({len(L['pivot_heads'])} pivots), row-blocks {rows}: worst max_abs "
              f"{st['worst_max_abs']:.3e} rel_l2 {st['worst_rel_l2']:.3e}; {st['exempt']} flipped in the band; "
              f"{st['near_ties']} near-ties")
        del L, out, mask
        torch.cuda.empty_cache()

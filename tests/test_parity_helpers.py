"""The sampled layer checker used by the full-size GPU tests, exercised on the CPU: fed with the oracle's own
full-layer result it must pass, and it must catch a planted mistake (a flipped mask bit, a perturbed output row)."""
import numpy as np
import pytest
import torch

from oracle import shareprefill_oracle as orc
from paper_2505_19578_b200 import synth
from tests import _parity as par


def _oracle_runs(L, gammas):
    cfg = L["cfg"]
    Q, K, V = par.f64(L["q"]), par.f64(L["k"]), par.f64(L["v"])
    runs = {}
    for g in gammas:
        ref = orc.prefill_attn(Q, K, V, L["cluster_map"], L["pivot_heads"], par.gamma32(g), cfg.block)
        runs[g] = (torch.from_numpy(ref["out"]).to(torch.bfloat16), torch.from_numpy(ref["mask"]))
    return runs


def test_sampled_checker_accepts_the_oracle_and_catches_planted_mistakes():
    cfg = synth.scaled(synth.CONFIGS["tiny"], 512)
    L = synth.make_layer(cfg, seed=5, device="cpu")
    Nb = cfg.seq // cfg.block
    runs = _oracle_runs(L, (0.8, 0.95))
    rows = par.sample_rows(Nb, 6, 1)
    assert {0, 1, Nb // 2, Nb - 1} <= set(rows) and len(rows) == 6
    st = par.check_layer_sampled(L, runs, rows)
    assert st["exempt"] == 0 and st["worst_max_abs"] <= 1e-2
    piv = L["pivot_heads"]
    member = next(h for h in range(cfg.n_q_heads) if h not in piv)
    # a mask bit flipped in a checked row-block of a pivot
    out, mask = runs[0.8]
    bad_mask = mask.clone()
    i = rows[-1]
    j = int(np.nonzero(bad_mask[piv[0], i].numpy() == 0)[0][0]) if (bad_mask[piv[0], i, :i + 1] == 0).any() else 0
    bad_mask[piv[0], i, j] ^= 1
    with pytest.raises(AssertionError):
        par.check_layer_sampled(L, {0.8: (out, bad_mask)}, rows)
    # an output row of a member perturbed
    bad_out = out.clone()
    bad_out[member, rows[2] * cfg.block + 3] += 0.25
    with pytest.raises(AssertionError):
        par.check_layer_sampled(L, {0.8: (bad_out, mask)}, rows)
    # restricting the members leaves that mistake unseen, as documented
    others = [h for h in range(cfg.n_q_heads) if h not in piv and h != member]
    par.check_layer_sampled(L, {0.8: (bad_out, mask)}, rows, members={0.8: others})


def test_vectorised_line_mask_equals_the_oracles_rule():
    # the full-size vertical-slash test rebuilds the block mask from the selected lines with a vectorised helper;
    # here that helper is held against the oracle's entry-by-entry rule
    from oracle import pooled_pattern_oracle as ppo
    from tests.test_gpu_pooled_pattern import _lines_mask
    rng = np.random.default_rng(0)
    for N, B, gamma in ((1024, 64, 0.5), (768, 128, 0.9), (512, 64, 0.05)):
        Q, K = rng.standard_normal((N, 32)), rng.standard_normal((N, 32))
        res = ppo.search_vertical_slash_pattern(Q, K, gamma, B)
        assert np.array_equal(_lines_mask(res["sel_v"], res["sel_s"], N // B, B, N), res["mask"])

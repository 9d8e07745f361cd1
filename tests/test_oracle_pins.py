"""Pins for the float64 oracle: things the paper's definitions and plain
mathematics fix, checked without the CUDA path.

Each pin is chosen so that a plausible mistake in the oracle (dropped 1/sqrt(d),
missing causal term, wrong GQA mapping, ascending sort, '>' for '>=', wrong
normalisation of the importance, transposed operand) fails at least one test.
"""
import itertools
import math

import numpy as np
import pytest
import torch

from oracle import shareprefill_oracle as orc
from tests import _brute


def _rand_qkv(rng, Hq, Hkv, N, d, scale=1.0):
    Q = rng.standard_normal((Hq, N, d)) * scale
    K = rng.standard_normal((Hkv, N, d)) * scale
    V = rng.standard_normal((Hkv, N, d))
    return Q, K, V


# ---------------------------------------------------------------- dense attention

@pytest.mark.parametrize("Hq,Hkv,N,d,B", [(2, 2, 48, 8, 16), (4, 2, 40, 4, 16), (6, 2, 33, 8, 8), (1, 1, 256, 4, 64)])
def test_dense_matches_bruteforce(Hq, Hkv, N, d, B):
    rng = np.random.default_rng(1)
    Q, K, V = _rand_qkv(rng, Hq, Hkv, N, d, scale=1.5)
    O = orc.dense_causal_attention(Q, K, V, B=B)
    for h in range(Hq):
        g = h // (Hq // Hkv)
        P = _brute.causal_probs(Q[h].tolist(), K[g].tolist())
        Ob = np.array(_brute.apply_probs(P, V[g].tolist()))
        np.testing.assert_allclose(O[h], Ob, rtol=0, atol=1e-12)


def test_dense_matches_torch_sdpa_float64():
    rng = np.random.default_rng(2)
    Hq, Hkv, N, d = 4, 2, 200, 16
    Q, K, V = _rand_qkv(rng, Hq, Hkv, N, d, scale=2.0)
    O = orc.dense_causal_attention(Q, K, V, B=32)
    tq = torch.from_numpy(Q)[None]
    tk = torch.from_numpy(K).repeat_interleave(Hq // Hkv, dim=0)[None]
    tv = torch.from_numpy(V).repeat_interleave(Hq // Hkv, dim=0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0].numpy()
    np.testing.assert_allclose(O, ref, rtol=0, atol=1e-12)


def test_result_independent_of_block_size():
    rng = np.random.default_rng(3)
    Q, K, V = _rand_qkv(rng, 2, 1, 96, 8)
    a = orc.dense_causal_attention(Q, K, V, B=16)
    b = orc.dense_causal_attention(Q, K, V, B=96)
    c = orc.dense_causal_attention(Q, K, V, B=7)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-13)
    np.testing.assert_allclose(a, c, rtol=0, atol=1e-13)


def test_probability_rows_sum_to_one_via_identity_values():
    # With V = identity (d = N) the output IS the probability matrix.
    rng = np.random.default_rng(4)
    N = 40
    Q = rng.standard_normal((1, N, N)) * 3
    K = rng.standard_normal((1, N, N)) * 3
    V = np.eye(N)[None]
    P = orc.dense_causal_attention(Q, K, V, B=16)[0]
    np.testing.assert_allclose(P.sum(axis=1), np.ones(N), rtol=0, atol=1e-12)
    assert np.all(np.triu(P, 1) == 0.0)            # causal: no mass on future keys
    assert np.all(P >= 0)
    Pb = np.array(_brute.causal_probs(Q[0].tolist(), K[0].tolist()))
    np.testing.assert_allclose(P, Pb, rtol=0, atol=1e-13)


def test_zero_queries_closed_form():
    # Q = 0: every admissible key gets 1/(r+1); O[r] = prefix mean of V;
    # I[i][j] = H(iB+B) - H(iB) for j < i; I[i][i] = (1/B) sum_t (t+1)/(iB+t+1).
    rng = np.random.default_rng(5)
    N, d, B = 128, 8, 16
    Q = np.zeros((1, N, d))
    K = rng.standard_normal((1, N, d))
    V = rng.standard_normal((1, N, d))
    I, O = orc.importance_map(Q, K, V, 0, B)
    prefix_mean = np.cumsum(V[0], axis=0) / np.arange(1, N + 1)[:, None]
    np.testing.assert_allclose(O, prefix_mean, rtol=0, atol=1e-13)
    H = np.concatenate([[0.0], np.cumsum(1.0 / np.arange(1, N + 1))])
    for i in range(N // B):
        for j in range(i):
            assert abs(I[i, j] - (H[i * B + B] - H[i * B])) < 1e-13
        diag = sum((t + 1) / (i * B + t + 1) for t in range(B)) / B
        assert abs(I[i, i] - diag) < 1e-13
        assert np.all(I[i, i + 1:] == 0)


def test_scale_is_one_over_sqrt_d():
    # Two keys, one query row r=1: p1/p0 = exp((q.k1 - q.k0)/sqrt(d)).
    d = 16
    Q = np.zeros((1, 2, d)); K = np.zeros((1, 2, d)); V = np.zeros((1, 2, d))
    Q[0, 1, 0] = 2.0
    K[0, 0, 0] = 1.0
    K[0, 1, 0] = 3.0
    V[0, 0, 0] = 1.0
    V[0, 1, 1] = 1.0
    O = orc.dense_causal_attention(Q, K, V, B=2)[0]
    ratio = O[1, 1] / O[1, 0]
    assert abs(ratio - math.exp((6.0 - 2.0) / math.sqrt(d))) < 1e-12
    assert O[0, 0] == 1.0 and O[0, 1] == 0.0      # row 0 sees only key 0


def test_gqa_equals_replicated_kv():
    rng = np.random.default_rng(6)
    Hq, Hkv, N, d = 6, 2, 64, 8
    Q, K, V = _rand_qkv(rng, Hq, Hkv, N, d)
    a = orc.dense_causal_attention(Q, K, V, B=16)
    Kr = np.repeat(K, Hq // Hkv, axis=0)
    Vr = np.repeat(V, Hq // Hkv, axis=0)
    b = orc.dense_causal_attention(Q, Kr, Vr, B=16)
    assert np.array_equal(a, b)
    # and the mapping is h // G, not h % Hkv
    assert orc.kv_head_of(2, 6, 2) == 0 and orc.kv_head_of(3, 6, 2) == 1


# ---------------------------------------------------------------- importance map

@pytest.mark.parametrize("N,d,B", [(64, 8, 16), (50, 4, 16), (256, 4, 64)])
def test_importance_matches_bruteforce_tile_sums(N, d, B):
    rng = np.random.default_rng(7)
    Q, K, V = _rand_qkv(rng, 1, 1, N, d, scale=2.0)
    I, _ = orc.importance_map(Q, K, V, 0, B)
    P = _brute.causal_probs(Q[0].tolist(), K[0].tolist())
    Ib = np.array(_brute.tile_mass(P, B))
    np.testing.assert_allclose(I, Ib, rtol=0, atol=1e-13)
    np.testing.assert_allclose(I.sum(axis=1), 1.0, rtol=0, atol=1e-12)


def test_importance_one_hot_key():
    # One key with a huge logit for every later query: its key-block takes ~all mass.
    rng = np.random.default_rng(8)
    N, d, B = 128, 8, 16
    Q, K, V = _rand_qkv(rng, 1, 1, N, d, scale=0.1)
    hot = 37
    Q[0, :, 0] = 10.0
    K[0, :, 0] = 0.0
    K[0, hot, 0] = 60.0 * math.sqrt(d) / 10.0      # logit +60 on that key
    I, _ = orc.importance_map(Q, K, V, 0, B)
    jb = hot // B
    for i in range(jb + 1, N // B):
        assert I[i, jb] > 1 - 1e-12


# ---------------------------------------------------------------- threshold rule

def test_threshold_ge_not_gt_and_descending():
    # exact binary fractions: 0.5 + 0.25 == 0.75 exactly
    x = np.array([0.25, 0.5, 0.25, 0.0])
    sel, info = orc.block_mask_row(x, 3, 0.75)
    assert info["K"] == 2                          # '>=': stops at exactly gamma
    assert sel.tolist() == [1, 1, 0, 0]            # tie 0.25/0.25 -> smaller index
    sel, info = orc.block_mask_row(x, 3, 0.76)
    assert info["K"] == 3 and sel.tolist() == [1, 1, 1, 0]
    sel, info = orc.block_mask_row(x, 3, 1e-9)
    assert sel.tolist() == [0, 1, 0, 0]            # gamma -> 0+: the arg-max tile only
    sel, info = orc.block_mask_row(x, 3, 2.0)
    assert sel.tolist() == [1, 1, 1, 1]            # unreachable gamma: everything causal
    sel, info = orc.block_mask_row(x, 1, 0.7)      # only entries 0..i are candidates
    assert sel.tolist() == [1, 1] and info["K"] == 2


def test_threshold_minimal_exhaustive_small():
    rng = np.random.default_rng(9)
    for trial in range(200):
        n = int(rng.integers(1, 9))
        x = rng.random(n) ** 3
        x /= x.sum()
        gamma = float(rng.uniform(0.05, 0.99))
        sel, info = orc.block_mask_row(x, n - 1, gamma)
        Kc = info["K"]
        assert sel.sum() == Kc
        assert x[sel == 1].sum() >= gamma - 1e-15
        # no subset with fewer tiles reaches gamma
        for k in range(1, Kc):
            best = max(sum(c) for c in itertools.combinations(x.tolist(), k))
            assert best < gamma
        # dropping the smallest selected tile falls below gamma
        if Kc > 1:
            assert x[sel == 1].sum() - x[sel == 1].min() < gamma


def test_masks_nested_in_gamma_and_invariants_on_attention():
    rng = np.random.default_rng(10)
    N, d, B = 256, 8, 16
    Q, K, V = _rand_qkv(rng, 1, 1, N, d, scale=3.0)
    I, _ = orc.importance_map(Q, K, V, 0, B)
    prev = None
    for gamma in (0.5, 0.8, 0.9, 0.95, 0.999):
        M, counts, lists, infos = orc.block_mask_from_importance(I, gamma)
        assert np.all(np.triu(M, 1) == 0)
        for i in range(N // B):
            assert counts[i] == M[i].sum() == len(lists[i]) >= 1
            assert np.all(np.diff(lists[i]) > 0)
            assert (I[i] * M[i]).sum() >= gamma - 1e-12
        if prev is not None:
            assert np.all(prev <= M)
        prev = M
    M, counts, _, _ = orc.block_mask_from_importance(I, 1.5)
    assert np.array_equal(M, np.tril(np.ones_like(M)))


# ---------------------------------------------------------------- masked attention

def test_all_ones_mask_is_dense_bit_for_bit():
    rng = np.random.default_rng(11)
    N, d, B = 96, 8, 16
    Q, K, V = _rand_qkv(rng, 2, 1, N, d)
    Nb = N // B
    dense = orc.dense_causal_attention(Q, K, V, B=B)
    for h in range(2):
        m = orc.masked_attention(Q, K, V, h, np.ones((Nb, Nb), np.uint8), B)
        assert np.array_equal(m, dense[h])
        m = orc.masked_attention(Q, K, V, h, np.tril(np.ones((Nb, Nb), np.uint8)), B)
        assert np.array_equal(m, dense[h])


def test_masked_matches_bruteforce_and_sdpa_boolean_mask():
    rng = np.random.default_rng(12)
    N, d, B = 80, 8, 16
    Q, K, V = _rand_qkv(rng, 1, 1, N, d, scale=2.0)
    Nb = N // B
    M = (rng.random((Nb, Nb)) < 0.5).astype(np.uint8)
    M[np.arange(Nb), np.arange(Nb)] = 1           # keep every row non-empty
    M = np.tril(M)
    O = orc.masked_attention(Q, K, V, 0, M, B)
    P = _brute.causal_probs(Q[0].tolist(), K[0].tolist(), allowed=lambda r, c: bool(M[r // B][c // B]))
    Ob = np.array(_brute.apply_probs(P, V[0].tolist()))
    np.testing.assert_allclose(O, Ob, rtol=0, atol=1e-12)
    np.testing.assert_allclose(np.array(P).sum(axis=1), 1.0, atol=1e-12)
    full = np.kron(M, np.ones((B, B), dtype=np.uint8)).astype(bool) & np.tril(np.ones((N, N), dtype=bool))
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None],
        attn_mask=torch.from_numpy(full)[None, None])[0, 0].numpy()
    np.testing.assert_allclose(O, ref, rtol=0, atol=1e-12)


def test_masked_attention_without_diagonal_tile():
    # A selected tile j < i alone is admissible for every row of block i.
    rng = np.random.default_rng(13)
    N, d, B = 48, 4, 16
    Q, K, V = _rand_qkv(rng, 1, 1, N, d)
    M = np.array([[1, 0, 0], [1, 0, 0], [0, 1, 0]], np.uint8)
    O = orc.masked_attention(Q, K, V, 0, M, B)
    P = _brute.causal_probs(Q[0].tolist(), K[0].tolist(), allowed=lambda r, c: bool(M[r // B][c // B]))
    np.testing.assert_allclose(O, np.array(_brute.apply_probs(P, V[0].tolist())), atol=1e-12)
    with pytest.raises(ValueError):
        orc.attention_rowblock(Q[0], K[0], V[0], 1, B, mask_row=np.array([0, 0, 0]))


def test_pivot_own_mask_error_bound():
    # With its own mask the pivot loses at most (1-gamma) mass per row-block on
    # average: mean over rows of ||o_sparse - o_dense||_inf <= 2 (1-gamma) max|V|.
    rng = np.random.default_rng(14)
    N, d, B = 256, 8, 32
    Q, K, V = _rand_qkv(rng, 1, 1, N, d, scale=3.0)
    gamma = 0.9
    I, Od = orc.importance_map(Q, K, V, 0, B)
    M, _, _, _ = orc.block_mask_from_importance(I, gamma)
    Os = orc.masked_attention(Q, K, V, 0, M, B)
    err = np.abs(Os - Od).max(axis=1).reshape(N // B, B).mean(axis=1)
    assert np.all(err <= 2 * (1 - gamma) * np.abs(V).max() + 1e-12)


# ---------------------------------------------------------------- sharing

def test_share_rule_first_pivot_of_cluster_and_dense_fallback():
    cluster_map = [0, 1, 0, 1, -1, 2, 0]
    src, mask_src = orc.share_masks(cluster_map, [2, 1, 0])
    # head 2 listed first for cluster 0 -> heads 6 share pivot index 0; head 0 is itself a pivot
    assert src == [-1, -1, -1, 1, -1, -1, 0]
    assert mask_src == [2, 1, 0, 1, -1, -1, 0]


def test_prefill_invariances():
    rng = np.random.default_rng(15)
    Hq, Hkv, N, d, B = 6, 2, 128, 8, 16
    base = rng.standard_normal((2, N, d))
    Q = np.stack([base[h % 2] + 0.2 * rng.standard_normal((N, d)) for h in range(Hq)]) * 2
    K = rng.standard_normal((Hkv, N, d)) * 2
    V = rng.standard_normal((Hkv, N, d))
    cm = [0, 1, 0, 1, 0, 1]
    r1 = orc.prefill_attn(Q, K, V, cm, [0, 1], 0.9, B)
    r2 = orc.prefill_attn(Q, K, V, [5, 3, 5, 3, 5, 3], [1, 0], 0.9, B)     # relabel clusters, reorder pivots
    assert np.array_equal(r1["out"], r2["out"]) and np.array_equal(r1["mask"], r2["mask"])
    dense = orc.dense_causal_attention(Q, K, V, B=B)
    assert np.array_equal(r1["out"][0], dense[0]) and np.array_equal(r1["out"][1], dense[1])
    assert np.array_equal(r1["mask"][2], r1["mask"][0]) and np.array_equal(r1["mask"][3], r1["mask"][1])
    # members differ from dense (tiles were skipped) yet stay close on average
    for h in (2, 3, 4, 5):
        diff = np.abs(r1["out"][h] - dense[h])
        assert diff.max() > 0 and diff.mean() < 0.1
    # no pivot for cluster 1 -> its heads run dense and report the causal mask
    r3 = orc.prefill_attn(Q, K, V, cm, [0], 0.9, B)
    Nb = N // B
    assert np.array_equal(r3["out"][3], dense[3])
    assert np.array_equal(r3["mask"][3], np.tril(np.ones((Nb, Nb), np.uint8)))
    # gamma above 1 -> everything dense
    r4 = orc.prefill_attn(Q, K, V, cm, [0, 1], 1.5, B)
    assert np.array_equal(r4["out"], dense)
    # sampled row-blocks agree with the full run
    r5 = orc.prefill_attn(Q, K, V, cm, [0, 1], 0.9, B, row_blocks=[0, 3, 7])
    for i in (0, 3, 7):
        assert np.array_equal(r5["out"][:, i * B:(i + 1) * B], r1["out"][:, i * B:(i + 1) * B])
        assert np.array_equal(r5["mask"][:, i], r1["mask"][:, i])

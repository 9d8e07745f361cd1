"""Pins of the paper-literal pattern oracle (oracle/pooled_pattern_oracle.py): brute force with
scalar arithmetic on tiny inputs, mathematical identities, closed forms, a library routine for
the Jensen-Shannon distance, exhaustive minimality of the selected set."""
import itertools
import math

import numpy as np
import pytest
from scipy.spatial.distance import jensenshannon

from oracle import pooled_pattern_oracle as ppo


def _rand(N, d, seed):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((N, d)), rng.standard_normal((N, d))


@pytest.mark.parametrize("N,d,B", [(64, 8, 16), (50, 4, 16), (16, 4, 16), (33, 8, 8)])
def test_pooled_logits_equal_scalar_brute_force(N, d, B):
    Q, K = _rand(N, d, 1)
    got = ppo.pooled_logits(Q, K, B)
    Nb = (N + B - 1) // B
    for i in range(Nb):
        for j in range(Nb):
            tot, cnt = 0.0, 0
            for r in range(i * B, min((i + 1) * B, N)):
                for c in range(j * B, min((j + 1) * B, N)):
                    if c <= r:
                        tot += sum(Q[r, t] * K[c, t] for t in range(d)) / math.sqrt(d)
                        cnt += 1
            if j > i:
                assert cnt == 0 and got[i, j] == -np.inf
            else:
                assert got[i, j] == pytest.approx(tot / cnt, abs=1e-12)


def test_off_diagonal_block_average_is_product_of_block_means():
    # mean over a full block of q_r . k_c = (mean of q rows) . (mean of k rows): an identity of the mathematics
    N, d, B = 96, 16, 32
    Q, K = _rand(N, d, 2)
    got = ppo.pooled_logits(Q, K, B)
    for i in range(3):
        for j in range(i):
            qm, km = Q[i * B:(i + 1) * B].mean(axis=0), K[j * B:(j + 1) * B].mean(axis=0)
            assert got[i, j] == pytest.approx(float(qm @ km) / math.sqrt(d), abs=1e-12)
    # the diagonal block is NOT that product (only the visible half is averaged)
    qm, km = Q[:B].mean(axis=0), K[:B].mean(axis=0)
    assert abs(got[0, 0] - float(qm @ km) / math.sqrt(d)) > 1e-6


def test_scale_is_one_over_sqrt_d():
    Q = np.ones((8, 4)); K = np.ones((8, 4))
    assert ppo.pooled_logits(Q, K, 8)[0, 0] == pytest.approx(4 / 2.0)


def test_zero_queries_closed_form():
    # Q = 0: every computed average is 0, each row is uniform over its i+1 blocks
    N, d, B, Nb = 64, 8, 16, 4
    Q = np.zeros((N, d)); K = np.random.default_rng(0).standard_normal((N, d))
    At = ppo.pooled_logits(Q, K, B)
    A = ppo.pooled_softmax(At)
    for i in range(Nb):
        np.testing.assert_allclose(A[i, :i + 1], 1.0 / (i + 1))
        assert np.all(A[i, i + 1:] == 0)
    # normalised scores 1/((i+1) Nb): rows 0 and 1 reach exactly 0.5 -> K = 3, rows 2, 3 get their diagonal
    res = ppo.construct_pivotal_pattern(At, 0.5)
    assert res["K"] == 3 and res["forced"] == [2, 3]
    expect = np.zeros((Nb, Nb), np.uint8)
    expect[0, 0] = expect[1, 0] = expect[1, 1] = 1
    expect[2, 2] = expect[3, 3] = 1
    assert np.array_equal(res["mask"], expect)
    np.testing.assert_allclose(res["a_last"], 0.25)
    # just above: one more entry, the first of row 2 (ties go to the smaller flattened index)
    res = ppo.construct_pivotal_pattern(At, 0.5 + 1e-9)
    assert res["K"] == 4 and res["mask"][2, 0] == 1 and res["mask"][2, 1] == 0 and res["forced"] == [3]


def test_selected_set_is_minimal_and_reaches_gamma():
    rng = np.random.default_rng(5)
    for Nb, gamma in [(3, 0.6), (4, 0.8), (4, 0.35)]:
        At = np.where(np.tril(np.ones((Nb, Nb), bool)), rng.standard_normal((Nb, Nb)) * 2, -np.inf)
        res = ppo.construct_pivotal_pattern(At, gamma)
        scores = res["scores"] / Nb
        cells = [(i, j) for i in range(Nb) for j in range(i + 1)]
        sel = [(i, j) for (i, j) in cells if res["mask"][i, j] and not (i in res["forced"] and i == j)]
        assert len(sel) == res["K"]
        assert sum(scores[c] for c in sel) >= gamma - 1e-15
        for k in range(res["K"]):
            for sub in itertools.combinations(cells, k):
                assert sum(scores[c] for c in sub) < gamma
        assert res["cum_before_cut"] < gamma <= res["cum_at_cut"]


def test_masks_nested_in_gamma_and_extremes():
    rng = np.random.default_rng(6)
    Nb = 12
    At = np.where(np.tril(np.ones((Nb, Nb), bool)), rng.standard_normal((Nb, Nb)) * 3, -np.inf)
    prev_sel = None
    for gamma in (0.05, 0.3, 0.6, 0.9, 0.99):
        res = ppo.construct_pivotal_pattern(At, gamma)
        sel = res["mask"].copy()
        for i in res["forced"]:
            sel[i, i] = 0
        if prev_sel is not None:
            assert np.all(prev_sel <= sel)
        prev_sel = sel
        assert np.all(np.triu(res["mask"], 1) == 0)
        assert np.all(res["mask"].sum(axis=1) >= 1)
    # gamma -> 0+: the single largest normalised score; gamma beyond reach: every block that exists
    res = ppo.construct_pivotal_pattern(At, 1e-12)
    assert res["K"] == 1
    A = ppo.pooled_softmax(At)
    i, j = np.unravel_index(np.argmax(A), A.shape)
    assert res["mask"][i, j] == 1
    res = ppo.construct_pivotal_pattern(At, 1.5)
    assert np.array_equal(res["mask"], np.tril(np.ones((Nb, Nb), np.uint8)))


def test_descending_order_matters():
    # one dominant block per row: a low gamma must pick dominant blocks, not the tiny ones
    Nb = 6
    At = np.where(np.tril(np.ones((Nb, Nb), bool)), -20.0, -np.inf)
    for i in range(Nb):
        At[i, 0] = 0.0
    res = ppo.construct_pivotal_pattern(At, 0.49)
    assert res["K"] == 3 and res["mask"][:, 0].sum() == 3 and res["mask"][:, 1:].sum() == 3     # + three forced diagonals
    assert len(res["forced"]) == 3


def test_last_block_distribution_is_last_row_of_the_map():
    N, d, B = 80, 8, 16
    Q, K = _rand(N, d, 7)
    a_hat = ppo.last_block_distribution(Q, K, B)
    A = ppo.pooled_softmax(ppo.pooled_logits(Q, K, B))
    np.testing.assert_allclose(a_hat, A[-1], atol=1e-14)
    assert a_hat.sum() == pytest.approx(1.0)
    # ragged last block
    Q, K = _rand(70, d, 8)
    np.testing.assert_allclose(ppo.last_block_distribution(Q, K, B), ppo.pooled_softmax(ppo.pooled_logits(Q, K, B))[-1], atol=1e-14)


def test_js_distance_against_scipy_and_identities():
    rng = np.random.default_rng(9)
    for n in (2, 7, 64):
        p = rng.random(n); p /= p.sum()
        q = rng.random(n) ** 3; q /= q.sum()
        assert ppo.js_distance(p, q) == pytest.approx(float(jensenshannon(p, q)), abs=1e-12)
        assert ppo.js_distance(p, q) == pytest.approx(ppo.js_distance(q, p), abs=1e-15)
        assert ppo.js_distance(p, p) == 0.0
    p = np.array([1.0, 0, 0, 0]); q = np.array([0, 0, 0.5, 0.5])
    assert ppo.js_distance(p, q) == pytest.approx(math.sqrt(math.log(2)), abs=1e-15)     # disjoint supports
    # uniform vs one-hot over n bins: closed form
    n = 8
    u = np.full(n, 1 / n); e = np.zeros(n); e[3] = 1
    m0 = 0.5 * (1 + 1 / n)
    jsd = 0.5 * math.log(1 / m0) + 0.5 * ((1 / n) * math.log((1 / n) / m0) + (n - 1) / n * math.log(2))
    assert ppo.js_distance(e, u) == pytest.approx(math.sqrt(jsd), abs=1e-14)


def test_determine_pattern_thresholds_are_strict():
    u = np.full(4, 0.25)
    a = np.array([0.4, 0.3, 0.2, 0.1])
    ds = ppo.js_distance(a, u)
    assert ppo.determine_pattern(a, a, ds + 1e-9, 1e-9)[0] == "shared_pivot"
    assert ppo.determine_pattern(a, a, ds, 1e-9)[0] == "vertical_slash"          # d_sparse < delta is strict
    b = np.array([0.1, 0.2, 0.3, 0.4])
    dsim = ppo.js_distance(a, b)
    assert ppo.determine_pattern(a, b, 1.0, dsim)[0] == "vertical_slash"          # d_sim < tau is strict
    assert ppo.determine_pattern(a, b, 1.0, dsim + 1e-9)[0] == "shared_pivot"
    assert ppo.determine_pattern(a, None, 1.0, 1.0)[0] == "vertical_slash"        # no pivotal representative yet
    pat, d1, d2 = ppo.determine_pattern(a, b, 0.3, 0.2)
    assert (d1, d2) == (pytest.approx(ds), pytest.approx(dsim))


# ------------------------------------------------------------------ vertical-slash search

def test_vertical_slash_scores_equal_scalar_brute_force():
    N, d, B = 40, 4, 16
    Q, K = _rand(N, d, 11)
    a_v, a_s = ppo.vertical_slash_scores(Q, K, B)
    r0 = 32
    ev, es = [0.0] * N, [0.0] * N
    for r in range(r0, N):
        logits = [sum(Q[r, t] * K[c, t] for t in range(d)) / math.sqrt(d) for c in range(r + 1)]
        mx = max(logits)
        den = sum(math.exp(x - mx) for x in logits)
        for c in range(r + 1):
            p = math.exp(logits[c] - mx) / den
            ev[c] += p
            es[r - c] += p
    np.testing.assert_allclose(a_v, ev, atol=1e-13)
    np.testing.assert_allclose(a_s, es, atol=1e-13)
    assert a_v.sum() == pytest.approx(N - r0) and a_s.sum() == pytest.approx(N - r0)


def test_vertical_slash_closed_forms():
    # Q = 0: every visible key of row r has probability 1/(r+1); vertical and slash sums coincide by symmetry
    N, d, B = 64, 4, 16
    Q = np.zeros((N, d)); K = np.random.default_rng(1).standard_normal((N, d))
    a_v, a_s = ppo.vertical_slash_scores(Q, K, B)
    rows = range(N - B, N)
    for c in (0, 10, 47, 50, 63):
        assert a_v[c] == pytest.approx(sum(1.0 / (r + 1) for r in rows if r >= c))
    for o in (0, 5, 48, 60, 63):
        assert a_s[o] == pytest.approx(sum(1.0 / (r + 1) for r in rows if r >= o))
    # one key dominates every row -> that column carries all the vertical mass; the slash mass of row r sits at r - c0
    c0 = 7
    Q = np.ones((N, d)); K = np.zeros((N, d)); K[c0] = 30.0
    a_v, a_s = ppo.vertical_slash_scores(Q, K, B)
    assert a_v[c0] == pytest.approx(B, rel=1e-9)
    for r in rows:
        assert a_s[r - c0] == pytest.approx(1.0, rel=1e-9)


def test_cumulative_select_minimal_ties_and_extremes():
    a = np.array([0.1, 0.4, 0.1, 0.2, 0.2])
    sel, K = ppo.cumulative_select(a, 0.6)
    assert K == 2 and sel.tolist() == [False, True, False, True, False]      # 0.4 + first of the two 0.2
    sel, K = ppo.cumulative_select(a, 0.6 + 1e-12)
    assert K == 3 and sel.tolist() == [False, True, False, True, True]
    sel, K = ppo.cumulative_select(a, 1e-9)
    assert K == 1 and sel[1]
    sel, K = ppo.cumulative_select(a, 2.0)
    assert K == 5 and sel.all()
    rng = np.random.default_rng(3)
    for _ in range(20):
        a = rng.random(7) ** 3
        g = float(rng.uniform(0.1, 0.95))
        sel, K = ppo.cumulative_select(a, g)
        f = a / a.sum()
        assert f[sel].sum() >= g - 1e-15
        for k in range(K):
            for sub in itertools.combinations(range(7), k):
                assert f[list(sub)].sum() < g


def test_vertical_slash_mask_geometry():
    # planted lines: a heavy key column c0 and the slash at offset o0 must light exactly the blocks they cross
    N, d, B = 128, 8, 16
    Nb = N // B
    rng = np.random.default_rng(4)
    Q, K = rng.standard_normal((N, d)) * 0.01, rng.standard_normal((N, d)) * 0.01
    res = ppo.search_vertical_slash_pattern(Q, K, 0.5, B)
    m = res["mask"]
    assert np.all(np.triu(m, 1) == 0) and np.all(m.sum(axis=1) >= 1)
    for i in range(Nb):
        for j in range(i + 1):
            want = res["sel_v"][j * B:(j + 1) * B].any()
            for r in range(i * B, (i + 1) * B):
                for c in range(j * B, (j + 1) * B):
                    if r - c >= 0 and res["sel_s"][r - c]:
                        want = True
            if i in res["forced"] and i == j:
                want = True
            assert m[i, j] == int(want)
    # masks grow with gamma
    prev = None
    for g in (0.2, 0.5, 0.8, 0.95):
        r = ppo.search_vertical_slash_pattern(Q, K, g, B)
        mm = r["mask"].copy()
        for i in r["forced"]:
            mm[i, i] = 0
        if prev is not None:
            assert np.all(prev <= mm)
        prev = mm

"""GPU parity of the paper-literal pattern construction and decision (block-averaged QK values,
global cumulative cut, Jensen-Shannon decision) against the float64 oracle."""
import numpy as np
import pytest
import torch

from oracle import pooled_pattern_oracle as ppo
from paper_2505_19578_b200 import synth
from tests import _parity as par

pytestmark = pytest.mark.gpu

POOLED_ATOL = 1e-10    # float64 block means and dot products of bf16 data on both sides (other summation order)
SCORE_BAND = 1e-6      # an entry may flip only if the oracle's cumulative score at it is this close to gamma: the
                       # library's scores are float64 softmax values rounded to fp32 once (6e-8 relative), summed exactly
DIV_ATOL = 1e-7        # Jensen-Shannon divergences (squared distances): float64 arithmetic on a representative that is
                       # stored in fp32 (6e-8 relative); the squares are compared (the root amplifies rounding near 0)
DIST_MARGIN = 1e-4     # a decision is checked when both distances are this far from their thresholds


@pytest.fixture(scope="module")
def binding():
    from paper_2505_19578_b200 import binding as b, build
    build.build()
    return b


def _oracle_cut(At, g):
    """Oracle result plus, per block, the cumulative normalised score at which it enters the order."""
    res = ppo.construct_pivotal_pattern(At, g)
    Nb = At.shape[0]
    flat = (res["scores"] / res["scores"].sum()).reshape(-1)
    idx = np.flatnonzero(np.tril(np.ones((Nb, Nb), bool)).reshape(-1))
    order = idx[np.argsort(-flat[idx], kind="stable")]
    cum_at = np.full(Nb * Nb, np.inf)
    cum_at[order] = np.cumsum(flat[order])
    return res, cum_at.reshape(Nb, Nb), flat.reshape(Nb, Nb)


def _mask_differences_in_band(m, res, cum_at, flat, g, band=None):
    """Entries where the GPU mask m differs from the oracle's: each must lie in the band (the oracle's cumulative
    normalised score with it, or just before it, within `band` of gamma).  One more case follows from such a flip: a
    row-block whose selection is empty on one side only receives its diagonal there, so a differing diagonal is
    accepted when one side's row is the diagonal alone and every other differing entry of the row is in the band.
    Returns the number of differing entries (all accounted for)."""
    band = SCORE_BAND if band is None else band
    diff = np.argwhere(m != res["mask"])
    near = {(int(i), int(j)): (abs(cum_at[i, j] - g) <= band or abs(cum_at[i, j] - flat[i, j] - g) <= band) for i, j in diff}
    for (i, j), ok in near.items():
        if ok:
            continue
        others = [e for e in near if e[0] == i and e != (i, j)]
        alone = (m[i].sum() == 1 and m[i, i] == 1) or (res["mask"][i].sum() == 1 and res["mask"][i, i] == 1)
        assert j == i and alone and others and all(near[e] for e in others), \
            f"block ({i}, {j}) differs away from the cut: cumulative {cum_at[i, j]:.9f}, gamma {g:.9f}"
    return len(diff)


def _lines_differences_in_band(got, want, a, g, band=None):
    """Selected lines (key columns or offsets) against the oracle's: a line may differ only inside the band."""
    band = VS_BAND if band is None else band
    cum, f = _cum_at(a, g)
    diff = np.flatnonzero(got.astype(bool) != want)
    for e in diff:
        assert abs(cum[e] - g) <= band or abs(cum[e] - f[e] - g) <= band, (int(e), float(cum[e]), g)
    return len(diff)


@pytest.mark.parametrize("name,seq,gamma", [("llama8b_32k", 4096, 0.9), ("tiny", 2048, 0.8), ("qwen7b_64k", 4096, 0.95)])
def test_pooled_logits_and_pattern_match_oracle(binding, name, seq, gamma):
    L = synth.make_layer(synth.scaled(synth.CONFIGS[name], seq), seed=3)
    cfg = L["cfg"]
    B, Nb = cfg.block, cfg.seq // cfg.block
    heads = list(L["pivot_heads"]) + [h for h in range(cfg.n_q_heads) if h not in L["pivot_heads"]][:1]
    ctx = binding.Context()
    q, k = L["q"].cuda(), L["k"].cuda()
    pooled = torch.full((len(heads), Nb, Nb), float("nan"), dtype=torch.float64, device="cuda")
    ctx.sp_pooled_logits(q, k, heads, B, pooled)
    mask = torch.full((len(heads), Nb, Nb), 7, dtype=torch.uint8, device="cuda")
    counts = torch.full((len(heads), Nb), -5, dtype=torch.int32, device="cuda")
    idx = torch.full((len(heads), Nb, Nb), -5, dtype=torch.int32, device="cuda")
    last = torch.full((len(heads), Nb), float("nan"), device="cuda")
    ctx.sp_pattern_from_pooled(pooled, gamma, mask, counts, idx, last_row_out=last)
    torch.cuda.synchronize()
    assert ctx.status() == (0, 0)
    Q, K = par.f64(L["q"]), par.f64(L["k"])
    g = par.gamma32(gamma)
    G = cfg.n_q_heads // cfg.n_kv_heads
    for t, h in enumerate(heads):
        At = ppo.pooled_logits(Q[h], K[h // G], B)
        got = pooled[t].cpu().numpy().astype(np.float64)
        tri = np.tril(np.ones((Nb, Nb), bool))
        assert np.all(got[~tri] == -np.inf)
        np.testing.assert_allclose(got[tri], At[tri], rtol=0, atol=POOLED_ATOL)
        res, cum_at, flat = _oracle_cut(At, g)
        np.testing.assert_allclose(last[t].cpu().numpy(), res["a_last"], rtol=0, atol=1e-6)
        m = mask[t].cpu().numpy()
        assert np.all(m[~tri] == 0) and np.all(m.sum(axis=1) >= 1)
        n_diff = _mask_differences_in_band(m, res, cum_at, flat, g)
        if n_diff:
            print(f"{name} head {h}: {n_diff} blocks inside the {SCORE_BAND} band flipped")
        # lists and counts describe the mask
        c, ix = counts[t].cpu().numpy(), idx[t].cpu().numpy()
        for i in range(Nb):
            sel = np.flatnonzero(m[i])
            assert c[i] == len(sel) and np.array_equal(ix[i, :c[i]], sel) and np.all(ix[i, c[i]:] == -1)


def test_pattern_from_pooled_exact_cases(binding):
    # equal scores inside a row (ties go to the smaller index), forced diagonals, unreachable gamma; the
    # gammas stay clear of the cumulative sums 1/8, 3/16, 1/4, ... where fp32 scores could fall either way
    Nb = 8
    At = np.where(np.tril(np.ones((Nb, Nb), bool)), 0.0, -np.inf)                        # uniform rows: scores 1/(i+1)
    ctx = binding.Context()
    pooled = torch.from_numpy(np.stack([At, At])).cuda()
    for gamma in (0.15, 0.2, 0.26, 0.6, 0.9, 1e-6, 1.5):
        mask = torch.zeros(2, Nb, Nb, dtype=torch.uint8, device="cuda")
        counts = torch.zeros(2, Nb, dtype=torch.int32, device="cuda")
        idx = torch.zeros(2, Nb, Nb, dtype=torch.int32, device="cuda")
        ctx.sp_pattern_from_pooled(pooled, gamma, mask, counts, idx)
        torch.cuda.synchronize()
        res = ppo.construct_pivotal_pattern(At, par.gamma32(gamma))
        for t in range(2):
            assert np.array_equal(mask[t].cpu().numpy(), res["mask"]), gamma
            assert np.array_equal(counts[t].cpu().numpy(), res["mask"].sum(axis=1))


@pytest.mark.parametrize("name,seq", [("llama8b_32k", 4096), ("qwen7b_64k", 2048)])
def test_determine_pattern_matches_oracle(binding, name, seq):
    L = synth.make_layer(synth.scaled(synth.CONFIGS[name], seq), seed=5)
    cfg = L["cfg"]
    B, Nb = cfg.block, cfg.seq // cfg.block
    piv = list(L["pivot_heads"])
    ctx = binding.Context()
    q, k = L["q"].cuda(), L["k"].cuda()
    pooled = torch.empty(len(piv), Nb, Nb, dtype=torch.float64, device="cuda")
    ctx.sp_pooled_logits(q, k, piv, B, pooled)
    mask = torch.empty(len(piv), Nb, Nb, dtype=torch.uint8, device="cuda")
    counts = torch.empty(len(piv), Nb, dtype=torch.int32, device="cuda")
    idx = torch.empty(len(piv), Nb, Nb, dtype=torch.int32, device="cuda")
    last = torch.empty(len(piv), Nb, device="cuda")
    ctx.sp_pattern_from_pooled(pooled, 0.9, mask, counts, idx, last_row_out=last)
    first = {}
    for t, p in enumerate(piv):
        first.setdefault(L["cluster_map"][p], t)
    heads = list(range(cfg.n_q_heads))
    rows = [first.get(L["cluster_map"][h], -1) for h in heads]
    rows[-1] = -1                                             # one head without a pivotal representative
    pat = torch.full((len(heads),), -1, dtype=torch.int32, device="cuda")
    dist = torch.full((len(heads), 2), float("nan"), device="cuda")
    Q, K = par.f64(L["q"]), par.f64(L["k"])
    G = cfg.n_q_heads // cfg.n_kv_heads
    a_tilde = [ppo.construct_pivotal_pattern(ppo.pooled_logits(Q[p], K[p // G], B), 0.9)["a_last"] for p in piv]
    ref = []
    for h, r in zip(heads, rows):
        a_hat = ppo.last_block_distribution(Q[h], K[h // G], B)
        ref.append(ppo.determine_pattern(a_hat, a_tilde[r] if r >= 0 else None, 0.3, 0.2))
    # thresholds that split the heads: medians of the oracle's distances
    delta = float(np.median([r[1] for r in ref])) + 1e-3
    tau = float(np.median([r[2] for r in ref if np.isfinite(r[2])])) + 1e-3
    ctx.sp_determine_pattern(q, k, heads, B, last, rows, delta, tau, pat, dist_out=dist)
    torch.cuda.synchronize()
    assert ctx.status() == (0, 0)
    got_p, got_d = pat.cpu().numpy(), dist.cpu().numpy()
    n_shared = 0
    for x, (h, r) in enumerate(zip(heads, rows)):
        _, ds, dm = ref[x]
        assert float(got_d[x, 0]) ** 2 == pytest.approx(ds * ds, abs=DIV_ATOL)
        if np.isfinite(dm):
            assert float(got_d[x, 1]) ** 2 == pytest.approx(dm * dm, abs=DIV_ATOL)
        else:
            assert np.isinf(got_d[x, 1])
        want = 0 if (ds < delta and dm < tau) else 1
        if min(abs(ds - delta), abs(dm - tau)) > DIST_MARGIN:     # away from the thresholds the decision is fixed
            assert got_p[x] == want
        n_shared += int(got_p[x] == 0)
    assert 0 < n_shared < len(heads)                                # the thresholds really split the heads
    # a pivot compared with its own representative: distance 0
    for t, p in enumerate(piv):
        if rows[p] == t:
            assert got_d[p, 1] <= 5e-4


# ------------------------------------------------------------------ vertical-slash search

VS_BAND = 2e-5         # a line may flip only if the oracle's cumulative score at it is this close to gamma: the
                       # probabilities come from bf16 tensor-core products accumulated in fp32 (128 terms of size up to
                       # ~2, logits up to ~30 after scaling: about 2e-5 absolute on a logit, i.e. relative on a score)


def _cum_at(a, g):
    f = a / a.sum()
    order = np.argsort(-f, kind="stable")
    cum = np.empty(len(a))
    cum[order] = np.cumsum(f[order])
    return cum, f


@pytest.mark.parametrize("name,seq,gamma", [("llama8b_32k", 4096, 0.9), ("qwen7b_64k", 2048, 0.8), ("llama8b_128k", 8192, 0.95)])
def test_vertical_slash_pattern_matches_oracle(binding, name, seq, gamma):
    from oracle import shareprefill_oracle as orc
    L = synth.make_layer(synth.scaled(synth.CONFIGS[name], seq), seed=6)
    cfg = L["cfg"]
    B, Nb, N = cfg.block, cfg.seq // cfg.block, cfg.seq
    heads = [1, cfg.n_q_heads - 1, 0]
    ctx = binding.Context()
    q, k, v = L["q"].cuda(), L["k"].cuda(), L["v"].cuda()
    mask = torch.full((len(heads), Nb, Nb), 7, dtype=torch.uint8, device="cuda")
    counts = torch.full((len(heads), Nb), -5, dtype=torch.int32, device="cuda")
    idx = torch.full((len(heads), Nb, Nb), -5, dtype=torch.int32, device="cuda")
    sv = torch.full((len(heads), N), 9, dtype=torch.uint8, device="cuda")
    ss = torch.full((len(heads), N), 9, dtype=torch.uint8, device="cuda")
    for rep in range(2):                                       # the second call reuses the scratch counters
        ctx.sp_vertical_slash_pattern(q, k, heads, gamma, B, mask, counts, idx, sel_v_out=sv, sel_s_out=ss)
        torch.cuda.synchronize()
        assert ctx.status() == (0, 0)
    Q, K, V = par.f64(L["q"]), par.f64(L["k"]), par.f64(L["v"])
    g = par.gamma32(gamma)
    G = cfg.n_q_heads // cfg.n_kv_heads
    for t, h in enumerate(heads):
        res = ppo.search_vertical_slash_pattern(Q[h], K[h // G], g, B)
        for got, want, a in ((sv[t].cpu().numpy(), res["sel_v"], res["a_v"]), (ss[t].cpu().numpy(), res["sel_s"], res["a_s"])):
            n_diff = _lines_differences_in_band(got, want, a, g)
            if n_diff:
                print(f"{name} head {h}: {n_diff} lines inside the {VS_BAND} band flipped")
        m = mask[t].cpu().numpy()
        # the mask is exactly what the GPU's own selected lines imply (integer work: bit-exact)
        gv, gs = sv[t].cpu().numpy().astype(bool), ss[t].cpu().numpy().astype(bool)
        want = np.zeros((Nb, Nb), np.uint8)
        colb = gv.reshape(Nb, B).any(axis=1)
        for i in range(Nb):
            for j in range(i + 1):
                lo, hi = max((i - j) * B - (B - 1), 0), min((i - j) * B + (B - 1), N - 1)
                want[i, j] = colb[j] or gs[lo:hi + 1].any()
            if want[i].sum() == 0:
                want[i, i] = 1
        assert np.array_equal(m, want)
        if np.array_equal(gv, res["sel_v"]) and np.array_equal(gs, res["sel_s"]):
            assert np.array_equal(m, res["mask"])
        c, ix = counts[t].cpu().numpy(), idx[t].cpu().numpy()
        for i in range(Nb):
            sel = np.flatnonzero(m[i])
            assert c[i] == len(sel) and np.array_equal(ix[i, :c[i]], sel) and np.all(ix[i, c[i]:] == -1)
    # the lists drive the block-sparse kernel directly
    out = torch.full_like(q, float("nan"))
    ctx.sp_block_sparse_attn(q, k, v, heads, list(range(len(heads))), counts, idx, B, out)
    torch.cuda.synchronize()
    assert ctx.status() == (0, 0)
    for t, h in enumerate(heads[:2]):
        ref = orc.masked_attention(Q, K, V, h, mask[t].cpu().numpy(), B)
        par.assert_out_close(par.f64(out[h]), ref, f"head {h}")


# ------------------------------------------------------------------ the whole decision flow on the device

@pytest.mark.parametrize("pooled", [False, True])
@pytest.mark.parametrize("name,seq", [("llama8b_32k", 4096), ("qwen7b_64k", 2048)])
def test_prefill_attn_auto_is_the_composition_of_its_steps(binding, name, seq, pooled):
    """sp_prefill_attn_auto must equal what the separately tested calls give when chained by hand with the
    decisions read back, and its outputs must match the oracle's masked attention under the masks it reports."""
    from oracle import shareprefill_oracle as orc
    L = synth.make_layer(synth.scaled(synth.CONFIGS[name], seq), seed=8)
    cfg = L["cfg"]
    B, Nb, Hq = cfg.block, cfg.seq // cfg.block, cfg.n_q_heads
    cm = list(L["cluster_map"])
    piv = list(L["pivot_heads"])
    cm[-1] = -1                                               # one head without a cluster: dense
    if Hq - 1 in piv:
        piv.remove(Hq - 1)
    gamma = 0.9
    ctx = binding.Context()
    q, k, v = L["q"].cuda(), L["k"].cuda(), L["v"].cuda()
    members = [h for h in range(Hq) if h not in piv]
    first = {}
    for t, p in enumerate(piv):
        first.setdefault(cm[p], t)
    rows = [first.get(cm[h], -1) if cm[h] >= 0 else -1 for h in members]

    # --- by hand: pivots' representatives, distances of the members, thresholds that split them
    Q, K, V = par.f64(L["q"]), par.f64(L["k"]), par.f64(L["v"])
    G = Hq // cfg.n_kv_heads
    a_t = [ppo.last_block_distribution(Q[p], K[p // G], B) for p in piv]
    ref = [ppo.determine_pattern(ppo.last_block_distribution(Q[h], K[h // G], B), a_t[r] if r >= 0 else None, 1.0, 1.0)
           for h, r in zip(members, rows)]
    ds = sorted(r[1] for r, row in zip(ref, rows) if row >= 0)
    delta = ds[len(ds) // 2] + 1e-3 if ds[-1] - ds[0] > 5e-3 else ds[-1] + 1.0
    dm = sorted(r[2] for r, row in zip(ref, rows) if row >= 0)
    tau = dm[(2 * len(dm)) // 3] + 1e-3

    out = torch.full_like(q, float("nan"))
    mask = torch.full((Hq, Nb, Nb), 7, dtype=torch.uint8, device="cuda")
    pat = torch.full((Hq,), -1, dtype=torch.int32, device="cuda")
    ctx.sp_prefill_attn_auto(q, k, v, cm, piv, gamma, delta, tau, B, out, pooled_construction=pooled, mask_out=mask,
                             pattern_out=pat)
    torch.cuda.synchronize()
    assert ctx.status() == (0, 0)
    pat_h, mask_h = pat.cpu().numpy(), mask.cpu().numpy()

    # decisions: as the oracle's wherever the distances are clear of the thresholds
    kinds = set()
    for h, r, (_, d1, d2) in zip(members, rows, ref):
        if r < 0:
            assert pat_h[h] == 0
            continue
        want = 1 if (d1 < delta and d2 < tau) else 2
        if min(abs(d1 - delta), abs(d2 - tau)) > DIST_MARGIN:
            assert pat_h[h] == want, (h, d1, d2, delta, tau)
        kinds.add(int(pat_h[h]))
    assert all(pat_h[p] == 0 for p in piv)
    assert kinds == {1, 2}                                    # both branches are exercised

    # masks: pivots' as the construction call gives them, members' by their decision
    if pooled:
        pl = torch.empty(len(piv), Nb, Nb, dtype=torch.float64, device="cuda")
        ctx.sp_pooled_logits(q, k, piv, B, pl)
        pmask = torch.empty(len(piv), Nb, Nb, dtype=torch.uint8, device="cuda")
        pc = torch.empty(len(piv), Nb, dtype=torch.int32, device="cuda")
        pi = torch.empty(len(piv), Nb, Nb, dtype=torch.int32, device="cuda")
        ctx.sp_pattern_from_pooled(pl, gamma, pmask, pc, pi)
    else:
        imp = torch.empty(len(piv), Nb, Nb, device="cuda")
        tmp = torch.empty_like(q)
        ctx.sp_dense_pivot_attn(q, k, v, piv, B, tmp, importance_out=imp)
        pmask = torch.empty(len(piv), Nb, Nb, dtype=torch.uint8, device="cuda")
        pc = torch.empty(len(piv), Nb, dtype=torch.int32, device="cuda")
        pi = torch.empty(len(piv), Nb, Nb, dtype=torch.int32, device="cuda")
        ctx.sp_block_mask_from_importance(imp, gamma, pmask, pc, pi)
    vs_heads = [h for h in members if pat_h[h] == 2]
    vmask = torch.empty(len(vs_heads), Nb, Nb, dtype=torch.uint8, device="cuda")
    vc = torch.empty(len(vs_heads), Nb, dtype=torch.int32, device="cuda")
    vi = torch.empty(len(vs_heads), Nb, Nb, dtype=torch.int32, device="cuda")
    ctx.sp_vertical_slash_pattern(q, k, vs_heads, gamma, B, vmask, vc, vi)
    torch.cuda.synchronize()
    pmask_h, vmask_h = pmask.cpu().numpy(), vmask.cpu().numpy()
    tri = np.tril(np.ones((Nb, Nb), np.uint8))
    for t, p in enumerate(piv):
        assert np.array_equal(mask_h[p], pmask_h[t])
    for h, r in zip(members, rows):
        if pat_h[h] == 0:
            assert np.array_equal(mask_h[h], tri)
        elif pat_h[h] == 1:
            assert np.array_equal(mask_h[h], pmask_h[r])
        else:
            assert np.array_equal(mask_h[h], vmask_h[vs_heads.index(h)])

    # outputs: dense for pivots and unclustered heads, masked attention under the reported mask for the rest
    check = piv[:1] + [Hq - 1] + [h for h in members if pat_h[h] == 1][:1] + vs_heads[:1]
    for h in check:
        M = tri if pat_h[h] == 0 else mask_h[h]
        refo = orc.masked_attention(Q, K, V, h, M, B)
        par.assert_out_close(par.f64(out[h]), refo, f"head {h} (pattern {pat_h[h]})")
    assert torch.isfinite(out.float()).all()


# ------------------------------------------------------------------ cross-layer dictionary

def _gap_threshold(values, lo_frac, hi_frac):
    """A threshold in the middle of the widest gap of the sorted values between two quantiles, so that no value is
    close to it (distances of order 0.1 .. 0.5 carry an error of about 1e-5 on the GPU)."""
    v = np.sort(np.asarray(values))
    lo, hi = int(len(v) * lo_frac), max(int(len(v) * hi_frac), int(len(v) * lo_frac) + 2)
    w = v[lo:hi + 1]
    gaps = w[1:] - w[:-1]
    g = int(np.argmax(gaps))
    assert gaps[g] > 4e-4, "no clear gap to put a threshold in"
    return float(0.5 * (w[g] + w[g + 1]))


@pytest.mark.parametrize("pooled", [False, True])
def test_layers_with_cross_layer_dictionary(binding, pooled):
    from oracle import shareprefill_oracle as orc
    cfg = synth.scaled(synth.CONFIGS["llama8b_32k"], 2048)
    B, Nb, Hq, G = cfg.block, cfg.seq // cfg.block, cfg.n_q_heads, cfg.n_q_heads // cfg.n_kv_heads
    gamma = 0.9
    layers = [synth.make_layer(cfg, seed=s) for s in (10, 11, 12)]
    # the second layer attends like the first (same queries and keys, other values), so that its heads find the
    # first layer's patterns similar; the third is unrelated
    layers[1] = dict(layers[1], q=layers[0]["q"], k=layers[0]["k"], cluster_map=layers[0]["cluster_map"])
    cms = []
    for li, L in enumerate(layers):
        cm = list(L["cluster_map"])
        cm[3 + li] = -1                                        # a noise-cluster head in every layer
        if li == 2:
            cm = [c if c < 0 else (c + 4) % 10 for c in cm]    # the last layer also brings two clusters not seen before
        cms.append(cm)
    # --- reference flow on the oracle's distances
    a_hats = [[ppo.last_block_distribution(par.f64(L["q"][h]), par.f64(L["k"][h // G]), B) for h in range(Hq)] for L in layers]
    u = np.full(Nb, 1.0 / Nb)
    d_sp = [[ppo.js_distance(a, u) for a in row] for row in a_hats]
    delta = _gap_threshold([x for row in d_sp for x in row], 0.7, 0.95)
    ref_dict, ref_pat, d_sims = {}, [], []
    for li in range(3):
        pats = []
        for h in range(Hq):
            c = cms[li][h]
            if c < 0 or d_sp[li][h] >= delta:
                pats.append(("vs", None))
            elif c in ref_dict:
                d = ppo.js_distance(a_hats[li][h], ref_dict[c][0])
                d_sims.append(d)
                pats.append(("cand", d, c))
            else:
                ref_dict[c] = (a_hats[li][h], (li, h))
                pats.append(("pivot", None, c))
        ref_pat.append(pats)
    tau = _gap_threshold(d_sims, 0.25, 0.75)

    ctx = binding.Context()
    d = binding.PatternDict(ctx, 10, Hq, cfg.seq, B)
    assert d.count() == 0
    stored = {}                                                # cluster -> mask the GPU stored for it
    kinds = set()
    cross_layer = 0
    for li, L in enumerate(layers):
        q, k, v = L["q"].cuda(), L["k"].cuda(), L["v"].cuda()
        out = torch.full_like(q, float("nan"))
        mask = torch.full((Hq, Nb, Nb), 7, dtype=torch.uint8, device="cuda")
        pat = torch.full((Hq,), -1, dtype=torch.int32, device="cuda")
        d.prefill_attn_layer(q, k, v, cms[li], gamma, delta, tau, B, out, pooled_construction=pooled, mask_out=mask, pattern_out=pat)
        torch.cuda.synchronize()
        assert ctx.status() == (0, 0)
        pat_h, mask_h = pat.cpu().numpy(), mask.cpu().numpy()
        Q, K, V = par.f64(L["q"]), par.f64(L["k"]), par.f64(L["v"])
        tri = np.tril(np.ones((Nb, Nb), np.uint8))
        vs_heads = [h for h in range(Hq) if pat_h[h] == 2]
        vmask = torch.empty(len(vs_heads), Nb, Nb, dtype=torch.uint8, device="cuda")
        vc = torch.empty(len(vs_heads), Nb, dtype=torch.int32, device="cuda")
        vi = torch.empty(len(vs_heads), Nb, Nb, dtype=torch.int32, device="cuda")
        ctx.sp_vertical_slash_pattern(q, k, vs_heads, gamma, B, vmask, vc, vi)
        torch.cuda.synchronize()
        vmask_h = vmask.cpu().numpy()
        for h in range(Hq):
            r = ref_pat[li][h]
            if r[0] == "pivot":
                assert pat_h[h] == 0
                stored[r[2]] = mask_h[h].copy()
                # the stored pattern is what the construction call gives for this head
                if pooled:
                    res, cum_at, flat = _oracle_cut(ppo.pooled_logits(Q[h], K[h // G], B), par.gamma32(gamma))
                    _mask_differences_in_band(mask_h[h], res, cum_at, flat, par.gamma32(gamma))
                else:
                    I, _ = orc.importance_map(Q, K, V, h, B)
                    M, _, _, infos = orc.block_mask_from_importance(I, par.gamma32(gamma))
                    bad, _ = par.compare_mask_rows(mask_h[h], M, infos, par.gamma32(gamma), range(Nb))
                    assert bad == 0, f"layer {li} pivot {h}: {bad} row-blocks differ outside the {par.MASK_BAND} band"
            elif r[0] == "vs":
                assert pat_h[h] == 2
            else:
                want = 1 if r[1] < tau else 2
                assert pat_h[h] == want, (li, h, r[1], tau)
                if want == 1:
                    assert np.array_equal(mask_h[h], stored[r[2]])       # the pattern of the cluster's pivot, possibly from an earlier layer
                    cross_layer += int(ref_dict[r[2]][1][0] < li)
            if pat_h[h] == 2:
                assert np.array_equal(mask_h[h], vmask_h[vs_heads.index(h)])
            kinds.add((li, int(pat_h[h])))
        # outputs under the reported masks
        picks = {}
        for h in range(Hq):
            picks.setdefault(int(pat_h[h]), h)
        for code, h in picks.items():
            M = tri if code == 0 else mask_h[h]
            par.assert_out_close(par.f64(out[h]), orc.masked_attention(Q, K, V, h, M, B), f"layer {li} head {h} pattern {code}")
        assert torch.isfinite(out.float()).all()
    assert d.count() == len(ref_dict)
    assert {0, 1, 2} <= {k_[1] for k_ in kinds}                          # pivots, sharing and vertical-slash all occur
    assert cross_layer > 0                                               # a pattern stored by one layer is reused by a later one
    d.clear()
    assert d.count() == 0


# ------------------------------------------------------------------ a workload on which the paper's thresholds decide

def test_mixed_workload_at_the_papers_thresholds(binding):
    """Two families of heads (flat block-averaged last rows / strong local decay) at gamma 0.9, delta 0.3, tau 0.2
    (Section 6, Implementation Details): the flat family shares its pivots' patterns, the other one falls back to
    vertical-slash, in sp_prefill_attn_auto and in the dictionary flow (where only the flat family yields pivots)."""
    from oracle import shareprefill_oracle as orc
    cfg = synth.scaled(synth.CONFIGS["llama8b_128k_mixed"], 8192)
    L = synth.make_layer(cfg, seed=2)
    B, Nb, Hq = cfg.block, cfg.seq // cfg.block, cfg.n_q_heads
    G = Hq // cfg.n_kv_heads
    gamma, delta, tau = 0.9, 0.3, 0.2
    cm, piv = list(L["cluster_map"]), list(L["pivot_heads"])
    Q, K, V = par.f64(L["q"]), par.f64(L["k"]), par.f64(L["v"])
    a_hat = [ppo.last_block_distribution(Q[h], K[h // G], B) for h in range(Hq)]
    want = {}
    for h in range(Hq):
        if h in piv:
            want[h] = 0
            continue
        pat, ds, dm = ppo.determine_pattern(a_hat[h], a_hat[piv[cm[h]]], delta, tau)
        assert min(abs(ds - delta), abs(dm - tau)) > 0.05          # the families are far from the thresholds
        want[h] = 1 if pat == "shared_pivot" else 2
    assert {1, 2} <= set(want.values())
    ctx = binding.Context()
    q, k, v = L["q"].cuda(), L["k"].cuda(), L["v"].cuda()
    tri = np.tril(np.ones((Nb, Nb), np.uint8))

    def check_outputs(out, mask_h, pat_h, label):
        picks = {}
        for h in range(Hq):
            picks.setdefault(int(pat_h[h]), h)
        assert set(picks) == {0, 1, 2}
        for code, h in picks.items():
            M = tri if code == 0 else mask_h[h]
            par.assert_out_close(par.f64(out[h]), orc.masked_attention(Q, K, V, h, M, B), f"{label} head {h} pattern {code}")
        assert torch.isfinite(out.float()).all()

    out = torch.full_like(q, float("nan"))
    mask = torch.full((Hq, Nb, Nb), 7, dtype=torch.uint8, device="cuda")
    pat = torch.full((Hq,), -1, dtype=torch.int32, device="cuda")
    ctx.sp_prefill_attn_auto(q, k, v, cm, piv, gamma, delta, tau, B, out, mask_out=mask, pattern_out=pat)
    torch.cuda.synchronize()
    assert ctx.status() == (0, 0)
    pat_h, mask_h = pat.cpu().numpy(), mask.cpu().numpy()
    assert [int(x) for x in pat_h] == [want[h] for h in range(Hq)]
    for h in range(Hq):
        if pat_h[h] == 1:
            assert np.array_equal(mask_h[h], mask_h[piv[cm[h]]])
    check_outputs(out, mask_h, pat_h, "auto")

    # the dictionary flow decides the pivots itself: a head of the other family never becomes one
    d = binding.PatternDict(ctx, cfg.n_clusters, Hq, cfg.seq, B)
    out2 = torch.full_like(q, float("nan"))
    mask.fill_(7)
    pat.fill_(-1)
    d.prefill_attn_layer(q, k, v, cm, gamma, delta, tau, B, out2, mask_out=mask, pattern_out=pat)
    torch.cuda.synchronize()
    assert ctx.status() == (0, 0)
    pat_h, mask_h = pat.cpu().numpy(), mask.cpu().numpy()
    u = np.full(Nb, 1.0 / Nb)
    seen = set()
    for h in range(Hq):
        sparse = ppo.js_distance(a_hat[h], u) >= delta
        if sparse:
            assert pat_h[h] == 2
        elif cm[h] not in seen:
            seen.add(cm[h])
            assert pat_h[h] == 0
        else:
            assert pat_h[h] == 1
    assert d.count() == len(seen) == cfg.global_clusters
    check_outputs(out2, mask_h, pat_h, "dictionary")


# ------------------------------------------------------------------ the same calls at the sizes the benchmark times

def _lines_mask(gv, gs, Nb, B, N):
    """index_to_mask of "Search Vertical Slash Pattern" from selected columns gv and offsets gs (vectorised restatement
    of the rule the small-size test spells out entry by entry): block (i, j), j <= i, is on if key-block j holds a
    selected column or a selected offset lies in [(i-j)B-(B-1), (i-j)B+(B-1)]; an empty row gets its diagonal."""
    colb = gv.reshape(Nb, B).any(axis=1)
    pre = np.concatenate([[0], np.cumsum(gs.astype(np.int64))])
    by_delta = np.zeros(Nb, bool)
    for dlt in range(Nb):
        lo, hi = max(dlt * B - (B - 1), 0), min(dlt * B + (B - 1), N - 1)
        by_delta[dlt] = pre[hi + 1] - pre[lo] > 0
    i_, j_ = np.meshgrid(np.arange(Nb), np.arange(Nb), indexing="ij")
    want = (j_ <= i_) & (colb[None, :] | by_delta[np.clip(i_ - j_, 0, Nb - 1)])
    want = want.astype(np.uint8)
    for i in np.flatnonzero(want.sum(axis=1) == 0):
        want[i, i] = 1
    return want


def test_decision_and_vertical_slash_at_131072_tokens(binding):
    """Algorithms "Determine Sparse Pattern" and "Search Vertical Slash Pattern" on the benchmark's 131072-token
    layer (Nb = 1024: 131072-entry cuts, 128 sweep chunks per head)."""
    from oracle import shareprefill_oracle as orc
    cfg = synth.CONFIGS["llama8b_128k"]
    L = synth.make_layer(cfg, seed=0, device="cuda")
    B, Nb, N, Hq = cfg.block, cfg.seq // cfg.block, cfg.seq, cfg.n_q_heads
    G = Hq // cfg.n_kv_heads
    piv = list(L["pivot_heads"])
    ctx = binding.Context()
    q, k, v = L["q"], L["k"], L["v"]
    Lh = dict(L, q=q.cpu(), k=k.cpu(), v=v.cpu())
    kv64 = {}

    def K64(g):
        if g not in kv64:
            kv64[g] = par.f64(Lh["k"][g])
        return kv64[g]

    # ---- decision: every head against the representative of its cluster's pivot (the pivot's own a^)
    first = {}
    for t, p in enumerate(piv):
        first.setdefault(L["cluster_map"][p], t)
    heads = list(range(Hq))
    rows = [first.get(L["cluster_map"][h], -1) for h in heads]
    a_hat = [ppo.last_block_distribution(par.f64(Lh["q"][h]), K64(h // G), B) for h in heads]
    ref = [ppo.determine_pattern(a_hat[h], a_hat[piv[r]] if r >= 0 else None, 0.3, 0.2) for h, r in zip(heads, rows)]
    def widest_gap(values):                                     # a threshold that splits the heads and is close to few of them
        w = np.sort(np.asarray(values))
        w = w[len(w) // 5: len(w) - len(w) // 5 + 1]
        gi = int(np.argmax(w[1:] - w[:-1]))
        return float(0.5 * (w[gi] + w[gi + 1]))

    delta = widest_gap([r[1] for r in ref])
    tau = widest_gap([r[2] for r in ref if np.isfinite(r[2]) and r[2] > 0])
    a_tilde = torch.from_numpy(np.stack([a_hat[p] for p in piv]).astype(np.float32)).cuda()
    pat = torch.full((Hq,), -1, dtype=torch.int32, device="cuda")
    dist = torch.full((Hq, 2), float("nan"), device="cuda")
    ctx.sp_determine_pattern(q, k, heads, B, a_tilde, rows, delta, tau, pat, dist_out=dist)
    torch.cuda.synchronize()
    assert ctx.status() == (0, 0)
    got_p, got_d = pat.cpu().numpy(), dist.cpu().numpy()
    checked = 0
    for x, (h, r) in enumerate(zip(heads, rows)):
        _, ds, dm = ref[x]
        assert float(got_d[x, 0]) ** 2 == pytest.approx(ds * ds, abs=DIV_ATOL), (h, got_d[x, 0], ds)
        assert float(got_d[x, 1]) ** 2 == pytest.approx(dm * dm, abs=DIV_ATOL), (h, got_d[x, 1], dm)
        if min(abs(ds - delta), abs(dm - tau)) > DIST_MARGIN:
            assert got_p[x] == (0 if (ds < delta and dm < tau) else 1), (h, ds, dm, delta, tau)
            checked += 1
    assert checked >= Hq // 4 and 0 < int((got_p == 0).sum()) < Hq
    print(f"decision at 131072 tokens: {checked} of {Hq} decisions clear of the thresholds by {DIST_MARGIN}; d_sparse "
          f"{min(r[1] for r in ref):.4f}..{max(r[1] for r in ref):.4f}, delta {delta:.4f}, tau {tau:.4f}, "
          f"max |d^2 error| {max(abs(float(got_d[x, 0]) ** 2 - ref[x][1] ** 2) for x in range(Hq)):.1e}")

    # ---- vertical-slash search for three heads; the third one's lists then drive the block-sparse kernel
    vs_heads = [1, Hq - 1, 0]
    gamma = 0.9
    g = par.gamma32(gamma)
    mask = torch.full((3, Nb, Nb), 7, dtype=torch.uint8, device="cuda")
    counts = torch.full((3, Nb), -5, dtype=torch.int32, device="cuda")
    idx = torch.full((3, Nb, Nb), -5, dtype=torch.int32, device="cuda")
    sv = torch.full((3, N), 9, dtype=torch.uint8, device="cuda")
    ss = torch.full((3, N), 9, dtype=torch.uint8, device="cuda")
    ctx.sp_vertical_slash_pattern(q, k, vs_heads, gamma, B, mask, counts, idx, sel_v_out=sv, sel_s_out=ss)
    torch.cuda.synchronize()
    assert ctx.status() == (0, 0)
    flipped = 0
    for t, h in enumerate(vs_heads):
        a_v, a_s = ppo.vertical_slash_scores(par.f64(Lh["q"][h]), K64(h // G), B)
        sel_v, _ = ppo.cumulative_select(a_v, g)
        sel_s, _ = ppo.cumulative_select(a_s, g)
        gv, gs = sv[t].cpu().numpy().astype(bool), ss[t].cpu().numpy().astype(bool)
        flipped += _lines_differences_in_band(gv, sel_v, a_v, g) + _lines_differences_in_band(gs, sel_s, a_s, g)
        m = mask[t].cpu().numpy()
        assert np.array_equal(m, _lines_mask(gv, gs, Nb, B, N))            # integer work: bit-exact on the GPU's own lines
        c, ix = counts[t].cpu().numpy(), idx[t].cpu().numpy()
        assert np.array_equal(c, m.sum(axis=1))
        for i in (0, 1, Nb // 2, Nb - 1):
            sel = np.flatnonzero(m[i])
            assert np.array_equal(ix[i, :c[i]], sel) and np.all(ix[i, c[i]:] == -1)
    print(f"vertical-slash at 131072 tokens: {flipped} lines inside the {VS_BAND} band flipped; mask densities "
          f"{[round(float(mask[t].sum()) / (Nb * (Nb + 1) / 2), 3) for t in range(3)]}")
    out = torch.full_like(q, float("nan"))
    ctx.sp_block_sparse_attn(q, k, v, vs_heads[:1], [0], counts, idx, B, out)
    torch.cuda.synchronize()
    assert ctx.status() == (0, 0)
    h = vs_heads[0]
    m0 = mask[0].cpu().numpy()
    Qh, Kg, Vg = par.f64(Lh["q"][h]), K64(h // G), par.f64(Lh["v"][h // G])
    for i in par.sample_rows(Nb, 6, 5):
        o_ref, _ = orc.attention_rowblock(Qh, Kg, Vg, i, B, mask_row=m0[i])
        par.assert_out_close(par.f64(out[h, i * B:(i + 1) * B]), o_ref, f"head {h} row-block {i}")


@pytest.mark.parametrize("name,gamma", [("llama8b_32k", 0.9), ("llama8b_128k", 0.9)])
def test_pooled_construction_at_full_size(binding, name, gamma):
    """Algorithm "Construct Pivotal Pattern" as the paper writes it, one pivot of the 32768- and of the 131072-token
    workload in full: the pooled map, the global cut on the library's own map, and the global cut fed with the
    oracle's map (so that the cut's fixed-point sums are checked at 32896 and 524800 scores by themselves)."""
    cfg = synth.CONFIGS[name]
    L = synth.make_layer(cfg, seed=0, device="cuda")
    B, Nb = cfg.block, cfg.seq // cfg.block
    G = cfg.n_q_heads // cfg.n_kv_heads
    h = L["pivot_heads"][0]
    ctx = binding.Context()
    pooled = torch.full((1, Nb, Nb), float("nan"), dtype=torch.float64, device="cuda")
    ctx.sp_pooled_logits(L["q"], L["k"], [h], B, pooled)
    torch.cuda.synchronize()
    At = ppo.pooled_logits(par.f64(L["q"][h].cpu()), par.f64(L["k"][h // G].cpu()), B)
    tri = np.tril(np.ones((Nb, Nb), bool))
    got = pooled[0].cpu().numpy().astype(np.float64)
    assert np.all(got[~tri] == -np.inf)
    err = float(np.abs(got[tri] - At[tri]).max())
    assert err <= POOLED_ATOL, err
    g = par.gamma32(gamma)
    res, cum_at, flat = _oracle_cut(At, g)
    n_diff = {}
    for label, src in (("own map", pooled), ("oracle's map", torch.from_numpy(At[None].copy()).cuda())):
        mask = torch.full((1, Nb, Nb), 7, dtype=torch.uint8, device="cuda")
        counts = torch.full((1, Nb), -5, dtype=torch.int32, device="cuda")
        idx = torch.full((1, Nb, Nb), -5, dtype=torch.int32, device="cuda")
        last = torch.full((1, Nb), float("nan"), device="cuda")
        ctx.sp_pattern_from_pooled(src, gamma, mask, counts, idx, last_row_out=last)
        torch.cuda.synchronize()
        assert ctx.status() == (0, 0)
        m = mask[0].cpu().numpy()
        assert np.all(m[~tri] == 0) and np.all(m.sum(axis=1) >= 1)
        n_diff[label] = _mask_differences_in_band(m, res, cum_at, flat, g)
        np.testing.assert_allclose(last[0].cpu().numpy(), res["a_last"], rtol=0, atol=1e-6)
        assert np.array_equal(counts[0].cpu().numpy(), m.sum(axis=1))
    print(f"{name} pivot {h}: pooled map max error {err:.2e}; blocks inside the {SCORE_BAND} band that flipped: {n_diff}; "
          f"density {float(res['mask'].sum()) / tri.sum():.4f}")


# ------------------------------------------------------------------ argument checking of these calls (host side)

def test_invalid_arguments_of_the_pattern_calls(binding):
    ctx = binding.Context()
    q = torch.zeros(4, 512, 128, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(2, 512, 128, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros_like(q)
    Nb = 4
    f = torch.zeros(1, Nb, Nb, dtype=torch.float64, device="cuda")
    m = torch.zeros(1, Nb, Nb, dtype=torch.uint8, device="cuda")
    c = torch.zeros(1, Nb, dtype=torch.int32, device="cuda")
    ix = torch.zeros(1, Nb, Nb, dtype=torch.int32, device="cuda")
    pat = torch.zeros(4, dtype=torch.int32, device="cuda")

    def code(fn):
        with pytest.raises(binding.SpError) as e:
            fn()
        return e.value.code

    INV, UNS = binding.SP_ERR_INVALID_ARG, binding.SP_ERR_UNSUPPORTED
    assert code(lambda: ctx.sp_pooled_logits(q, k, [4], 128, f)) == INV                    # head range
    assert code(lambda: ctx.sp_pooled_logits(q, k, [0], 96, f)) == UNS                     # block
    assert code(lambda: ctx.sp_pattern_from_pooled(f, 0.0, m, c, ix)) == INV               # gamma
    assert code(lambda: ctx.sp_pattern_from_pooled(f, 0.9, None, c, ix)) == INV            # the mask is required
    assert code(lambda: ctx.sp_determine_pattern(q, k, [0], 128, None, [0], 0.3, 0.2, pat)) == INV
    assert code(lambda: ctx.sp_vertical_slash_pattern(q, k, [0], -1.0, 128, m, c, ix)) == INV
    q64 = torch.zeros(4, 512, 64, dtype=torch.bfloat16, device="cuda")
    k64 = torch.zeros(2, 512, 64, dtype=torch.bfloat16, device="cuda")
    o64 = torch.zeros_like(q64)
    assert code(lambda: ctx.sp_vertical_slash_pattern(q64, k64, [0], 0.9, 64, m, c, ix)) == UNS
    assert code(lambda: ctx.sp_prefill_attn_auto(q, k, k, [0, 0, 1, 1], [0, 0], 0.9, 0.3, 0.2, 128, out)) == INV
    assert code(lambda: ctx.sp_prefill_attn_auto(q64, k64, k64, [0, 0, 1, 1], [0], 0.9, 0.3, 0.2, 64, o64)) == UNS
    d = binding.PatternDict(ctx, 2, 4, 512, 128)
    assert code(lambda: d.prefill_attn_layer(q, k, k, [0, 1, 2, 0], 0.9, 0.3, 0.2, 128, out)) == INV      # cluster id
    q2 = torch.zeros(4, 1024, 128, dtype=torch.bfloat16, device="cuda")
    k2 = torch.zeros(2, 1024, 128, dtype=torch.bfloat16, device="cuda")
    o2 = torch.zeros_like(q2)
    assert code(lambda: d.prefill_attn_layer(q2, k2, k2, [0, 1, 0, 1], 0.9, 0.3, 0.2, 128, o2)) == INV    # other length
    with pytest.raises(binding.SpError):
        binding.PatternDict(ctx, 2, 4, 500, 128)
    with pytest.raises(ValueError):                                                        # host call wants host tensors
        ctx.sp_prefill_attn_host(q, k.cpu(), k.cpu(), [0, 0, 1, 1], [0], 0.9, 128, out.cpu())
    torch.cuda.synchronize()
    assert ctx.status() == (0, 0)

"""Helpers for the GPU-vs-oracle parity tests (tolerances live here).

Output tolerance (bf16 inputs, fp32 accumulation, bf16 output, against the
float64 oracle): worst-head max-abs <= 2e-2 and relative L2 <= 1e-2.

Mask tolerance: bit-exact, except row-blocks whose oracle cumulative mass at
the cut (or just before it) lies within MASK_BAND of gamma: there the fp32
importance of the GPU may legitimately land on the other side of the
threshold.  Such row-blocks are counted and returned, never silently dropped.
"""
import numpy as np
import torch

from oracle import shareprefill_oracle as orc

OUT_MAX_ABS = 2e-2
OUT_REL_L2 = 1e-2
MASK_BAND = 1e-6
IMP_ATOL = 2e-6          # per-tile mass: fp32 accumulation of ~B*B bf16-accurate probabilities


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float32).numpy().astype(np.float64)


def gamma32(gamma: float) -> float:
    """The value the library compares against: the double nearest to float(gamma)."""
    return float(np.float32(gamma))


def out_errors(got: np.ndarray, ref: np.ndarray):
    diff = got - ref
    max_abs = float(np.abs(diff).max()) if diff.size else 0.0
    den = float(np.linalg.norm(ref))
    rel = float(np.linalg.norm(diff)) / den if den > 0 else 0.0
    return max_abs, rel


def assert_out_close(got, ref, what=""):
    max_abs, rel = out_errors(got, ref)
    assert max_abs <= OUT_MAX_ABS and rel <= OUT_REL_L2, f"{what}: max_abs={max_abs:.3e} rel_l2={rel:.3e}"
    return max_abs, rel


def compare_mask_rows(gpu_mask, ref_mask, infos, gamma, rows, band=MASK_BAND):
    """Row-blocks of one pivot: returns (n_mismatch_rows_outside_band, n_rows_in_band_that_differ)."""
    bad, exempt = 0, 0
    for i in rows:
        if np.array_equal(gpu_mask[i], ref_mask[i]):
            continue
        info = infos[i]
        near = abs(info["cum_at_cut"] - gamma) <= band or abs(info["cum_before_cut"] - gamma) <= band
        if near:
            exempt += 1
        else:
            bad += 1
    return bad, exempt


# ------------------------------------------------------------------ whole-layer helpers

def run_layer(binding, L, gamma, kernel, row_blocks=None):
    cfg = L["cfg"]
    ctx = binding.Context(kernel=kernel)
    qd, kd, vd = L["q"].cuda(), L["k"].cuda(), L["v"].cuda()
    Nb = cfg.seq // cfg.block
    out = torch.full_like(qd, float("nan"))
    mask = torch.full((cfg.n_q_heads, Nb, Nb), 9, dtype=torch.uint8, device="cuda")
    ctx.sp_prefill_attn(qd, kd, vd, L["cluster_map"], L["pivot_heads"], gamma, cfg.block, out, mask_out=mask)
    torch.cuda.synchronize()
    assert ctx.status() == (0, 0)
    return out, mask


def check_layer(L, gamma, out, mask, row_blocks=None):
    cfg = L["cfg"]
    B, Nb = cfg.block, cfg.seq // cfg.block
    Q, K, V = f64(L["q"]), f64(L["k"]), f64(L["v"])
    g = gamma32(gamma)
    rows = list(range(Nb)) if row_blocks is None else row_blocks
    ref = orc.prefill_attn(Q, K, V, L["cluster_map"], L["pivot_heads"], g, B, row_blocks=row_blocks)
    mask_np = mask.cpu().numpy()
    bad = exempt = 0
    src, mask_src = orc.share_masks(L["cluster_map"], L["pivot_heads"])
    clean_pivot = {}
    for t, p in enumerate(L["pivot_heads"]):
        b, e = compare_mask_rows(mask_np[p], ref["mask"][p], ref["infos"][t], g, rows)
        bad += b
        exempt += e
        clean_pivot[t] = {i for i in rows if np.array_equal(mask_np[p][i], ref["mask"][p][i])}
    assert bad == 0, f"{bad} row-blocks differ outside the {MASK_BAND} band ({exempt} inside)"
    worst = (0.0, 0.0)
    for h in range(cfg.n_q_heads):
        # members report their pivot's mask, dense heads the causal mask
        if mask_src[h] >= 0:
            assert np.array_equal(mask_np[h][rows], mask_np[L["pivot_heads"][mask_src[h]]][rows])
        else:
            assert np.array_equal(mask_np[h][rows], np.tril(np.ones((Nb, Nb), np.uint8))[rows])
        assert np.all(np.triu(mask_np[h], 1) == 0)
        got = f64(out[h])
        for i in rows:
            if src[h] >= 0 and i not in clean_pivot[src[h]]:
                continue                                         # row-block whose mask legitimately flipped
            sl = slice(i * B, (i + 1) * B)
            ma, rl = out_errors(got[sl], ref["out"][h][sl])
            worst = (max(worst[0], ma), max(worst[1], rl))
    assert worst[0] <= OUT_MAX_ABS and worst[1] <= OUT_REL_L2, worst
    return worst, exempt




# ------------------------------------------------------------------ sampled check of a layer at several thresholds

def sample_rows(Nb, n, seed):
    """Row-blocks 0, 1, Nb/2, Nb-1 and seeded others, n in all (all of them when Nb <= n)."""
    fixed = {0, min(1, Nb - 1), Nb // 2, Nb - 1}
    rng = np.random.default_rng(seed)
    rest = [int(i) for i in rng.permutation(Nb) if int(i) not in fixed]
    return sorted(fixed | set(rest[:max(0, n - len(fixed))]))


def check_layer_sampled(L, runs, rows, members=None, what=""):
    """Sampled row-blocks of one layer against the oracle, at one or several thresholds.

    runs: {gamma: (out [Hq, N, d] tensor, mask [Hq, Nb, Nb] tensor)} as sp_prefill_attn returned them on the SAME inputs.
    rows: row-blocks to check (a row-block's mask and outputs depend only on its own queries and the keys before it).
    members: {gamma: non-pivot heads whose outputs are checked}; default: all of them at every gamma.
    The pivots' dense attention and importance rows do not depend on gamma, so the oracle computes them once per
    (pivot, row-block) and cuts them at every gamma.  Mask rule: bit-exact, except row-blocks whose oracle cumulative
    mass at the cut, or just before it, is within MASK_BAND of gamma; those are counted (and returned), and outputs of
    heads that use such a row are not compared there.  Returns dict(worst_max_abs, worst_rel_l2, exempt, near_ties).
    """
    cfg = L["cfg"]
    B, Nb, Hq, Hkv = cfg.block, cfg.seq // cfg.block, cfg.n_q_heads, cfg.n_kv_heads
    piv = list(L["pivot_heads"])
    src, mask_src = orc.share_masks(L["cluster_map"], piv)
    kv = {}

    def kvf(g):
        if g not in kv:
            kv[g] = (f64(L["k"][g]), f64(L["v"][g]))
        return kv[g]

    masks = {g_: m.cpu().numpy() for g_, (_, m) in runs.items()}
    causal = np.tril(np.ones((Nb, Nb), np.uint8))
    stats = {"worst_max_abs": 0.0, "worst_rel_l2": 0.0, "exempt": 0, "near_ties": 0, "rows": len(rows)}
    clean = {g_: {} for g_ in runs}          # gamma -> pivot slot -> set of row-blocks whose mask agreed
    ref_rows = {g_: {} for g_ in runs}       # gamma -> (pivot slot, row-block) -> oracle mask row
    for t, p in enumerate(piv):
        Qp = f64(L["q"][p])
        Kg, Vg = kvf(orc.kv_head_of(p, Hq, Hkv))
        for g_ in runs:
            clean[g_][t] = set()
        for i in rows:
            o_ref, mass = orc.attention_rowblock(Qp, Kg, Vg, i, B)
            for g_, (out, _) in runs.items():
                got = f64(out[p, i * B:(i + 1) * B])
                ma, rl = out_errors(got, o_ref)
                assert ma <= OUT_MAX_ABS and rl <= OUT_REL_L2, f"{what} pivot {p} row-block {i} gamma {g_}: {ma:.3e} {rl:.3e}"
                stats["worst_max_abs"] = max(stats["worst_max_abs"], ma)
                stats["worst_rel_l2"] = max(stats["worst_rel_l2"], rl)
                gam = gamma32(g_)
                sel, info = orc.block_mask_row(mass, i, gam)
                ref_row = np.zeros(Nb, np.uint8)
                ref_row[:i + 1] = sel
                ref_rows[g_][(t, i)] = ref_row
                if info["tie_gap"] <= MASK_BAND:
                    stats["near_ties"] += 1
                if np.array_equal(masks[g_][p, i], ref_row):
                    clean[g_][t].add(i)
                else:
                    near = abs(info["cum_at_cut"] - gam) <= MASK_BAND or abs(info["cum_before_cut"] - gam) <= MASK_BAND
                    assert near, (f"{what} pivot {p} row-block {i} gamma {g_}: mask differs away from the threshold "
                                  f"(cum {info['cum_before_cut']:.9f} -> {info['cum_at_cut']:.9f})")
                    stats["exempt"] += 1
        del Qp
    for g_, (out, _) in runs.items():
        m = masks[g_]
        hs = [h for h in range(Hq) if h not in piv] if members is None else list(members[g_])
        for h in range(Hq):                       # reported patterns: integer work, every head
            if mask_src[h] >= 0:
                assert np.array_equal(m[h][rows], m[piv[mask_src[h]]][rows])
            else:
                assert np.array_equal(m[h][rows], causal[rows])
            assert np.all(np.triu(m[h], 1) == 0)
        for h in hs:
            Qh = f64(L["q"][h])
            Kg, Vg = kvf(orc.kv_head_of(h, Hq, Hkv))
            for i in rows:
                if src[h] >= 0:
                    if i not in clean[g_][src[h]]:
                        continue                  # row-block whose mask legitimately flipped
                    o_ref, _ = orc.attention_rowblock(Qh, Kg, Vg, i, B, mask_row=ref_rows[g_][(src[h], i)])
                else:
                    o_ref, _ = orc.attention_rowblock(Qh, Kg, Vg, i, B)
                ma, rl = out_errors(f64(out[h, i * B:(i + 1) * B]), o_ref)
                assert ma <= OUT_MAX_ABS and rl <= OUT_REL_L2, f"{what} head {h} row-block {i} gamma {g_}: {ma:.3e} {rl:.3e}"
                stats["worst_max_abs"] = max(stats["worst_max_abs"], ma)
                stats["worst_rel_l2"] = max(stats["worst_rel_l2"], rl)
    return stats

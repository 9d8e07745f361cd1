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



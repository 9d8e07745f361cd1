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

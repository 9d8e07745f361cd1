"""Float64 CPU oracle for the paper-literal pattern construction and decision.

TEST INFRASTRUCTURE ONLY: the slow, plain definition the CUDA library is
checked against.  It shares no code with the CUDA path, imports nothing from
the product package and must never be called by it.

What is defined here, step by step as the paper states it:

  * pooled_logits            Section 5.2, "Sparse Attention Computation": next to
                             the output the kernel yields the block-wise average
                             of the QK values, A~ (−inf where a block is not
                             computed).
  * construct_pivotal_pattern  Algorithm "Construct Pivotal Pattern": softmax over
                             the block averages, last row kept as the pivotal
                             representative a~, map flattened and normalised,
                             sorted, minimum budget K whose scores sum to gamma,
                             index set turned into a mask.
  * last_block_distribution  Algorithm "Determine Sparse Pattern": a^ =
                             softmax(pool(Q^ K^T) / sqrt(d)) with Q^ the last
                             block of queries.
  * js_distance, determine_pattern  same algorithm: d_sparse = sqrt(JSD(a^ || u)),
                             d_sim = sqrt(JSD(a^ || a~)); shared pivot iff
                             d_sparse < delta and d_sim < tau, else vertical-slash.

  * vertical_slash_scores, search_vertical_slash_pattern  Algorithm "Search Vertical Slash
                             Pattern": A^ = softmax(Q^ K^T / sqrt(d)) for the last block
                             of queries, sums along the vertical (per key) and slash (per
                             query-minus-key offset) directions, each normalised, sorted and
                             cut at gamma, union of the selected lines turned into a block
                             mask.

Readings taken where the paper is silent (also listed in the design notes):
  * causal: a block above the diagonal is never computed (average −inf); the
    average of the diagonal block runs over its visible entries (key <= query);
  * the scale 1/sqrt(d) is applied to the averages (pooling is linear, so
    before or after makes no difference);
  * the softmax of "Construct Pivotal Pattern" is taken along each row-block's
    key-blocks, so every row sums to 1 and the normalising total is the number
    of row-blocks;
  * sort descending, ties to the smaller flattened (row-major) index, ">= gamma";
  * a row-block left without any selected block would make the masked softmax
    of its rows undefined: it receives its diagonal block (forced, counted);
  * Jensen-Shannon divergence with natural logarithms, 0 log 0 = 0;
  * vertical-slash: Q^ is the last block of queries; a slash line is the set of (query r, key c)
    with r - c = o for an offset o >= 0; index_to_mask computes a block if it contains a selected
    key column or is crossed by a selected slash line (and lies on or below the diagonal); an empty
    row-block receives its diagonal block as above.

Everything is numpy float64 on the bf16-rounded inputs.  Pins:
tests/test_pooled_oracle_pins.py.  Parity with the authors' implementation is
unpinned (the paper prints no worked numeric example of these steps).
"""
from __future__ import annotations

import math

import numpy as np

__all__ = [
    "pooled_logits",
    "pooled_softmax",
    "construct_pivotal_pattern",
    "last_block_distribution",
    "js_distance",
    "determine_pattern",
    "cumulative_select",
    "vertical_slash_scores",
    "search_vertical_slash_pattern",
]


def pooled_logits(Qh, Kg, B: int):
    """Block-wise average of the scaled QK values of one head (Section 5.2).

    Qh, Kg [N, d].  Returns A~ [Nb, Nb] float64: entry (i, j), j <= i, is the
    mean of q_r . k_c / sqrt(d) over the visible (c <= r) entries of the block;
    entries with j > i are −inf (never computed).
    """
    Qh = np.asarray(Qh, dtype=np.float64)
    Kg = np.asarray(Kg, dtype=np.float64)
    N, d = Qh.shape
    Nb = (N + B - 1) // B
    out = np.full((Nb, Nb), -np.inf)
    for i in range(Nb):
        r0, r1 = i * B, min((i + 1) * B, N)
        for j in range(i + 1):
            c0, c1 = j * B, min((j + 1) * B, N)
            S = (Qh[r0:r1] @ Kg[c0:c1].T) / math.sqrt(d)
            if j < i:
                out[i, j] = S.mean()
            else:
                vis = np.arange(c0, c1)[None, :] <= np.arange(r0, r1)[:, None]
                out[i, j] = S[vis].sum() / vis.sum()
    return out


def pooled_softmax(At):
    """Row-wise softmax of the block averages ("Construct Pivotal Pattern": A~ = softmax(A~)).
    −inf entries get probability 0."""
    At = np.asarray(At, dtype=np.float64)
    m = At.max(axis=1, keepdims=True)
    E = np.exp(At - m)
    return E / E.sum(axis=1, keepdims=True)


def construct_pivotal_pattern(At, gamma: float):
    """Algorithm "Construct Pivotal Pattern" on the block averages At [Nb, Nb].

    Returns dict: mask u8 [Nb, Nb], a_last [Nb] (the pivotal representative a~),
    K (budget before forcing), forced (row-blocks that received their diagonal),
    cum_at_cut / cum_before_cut (cumulative score with and without the last
    selected entry, for near-threshold bookkeeping).
    """
    A = pooled_softmax(At)
    Nb = A.shape[0]
    a_last = A[-1].copy()
    causal = np.tril(np.ones((Nb, Nb), dtype=bool))
    flat = (A / A.sum()).reshape(-1)                 # flatten and normalise
    idx = np.flatnonzero(causal.reshape(-1))         # blocks that exist
    order = idx[np.argsort(-flat[idx], kind="stable")]
    cum = np.cumsum(flat[order])
    hit = np.flatnonzero(cum >= gamma)
    K = int(hit[0]) + 1 if hit.size else len(order)
    sel = order[:K]
    mask = np.zeros(Nb * Nb, dtype=np.uint8)
    mask[sel] = 1
    mask = mask.reshape(Nb, Nb)
    forced = [i for i in range(Nb) if mask[i].sum() == 0]
    for i in forced:
        mask[i, i] = 1
    return {
        "mask": mask, "a_last": a_last, "K": K, "forced": forced,
        "cum_at_cut": float(cum[K - 1]), "cum_before_cut": float(cum[K - 2]) if K >= 2 else 0.0,
        "scores": A,
    }


def last_block_distribution(Qh, Kg, B: int):
    """a^ of "Determine Sparse Pattern": softmax(pool(Q^ K^T) / sqrt(d)), Q^ = the last block of
    queries, pooled over each key-block (visible entries only)."""
    Qh = np.asarray(Qh, dtype=np.float64)
    Kg = np.asarray(Kg, dtype=np.float64)
    N, d = Qh.shape
    Nb = (N + B - 1) // B
    r0 = (Nb - 1) * B
    S = Qh[r0:N] @ Kg.T                                # [rows, N]
    pooled = np.empty(Nb)
    for j in range(Nb):
        c0, c1 = j * B, min((j + 1) * B, N)
        vis = np.arange(c0, c1)[None, :] <= np.arange(r0, N)[:, None]
        pooled[j] = S[:, c0:c1][vis].sum() / vis.sum()
    z = pooled / math.sqrt(d)
    e = np.exp(z - z.max())
    return e / e.sum()


def js_distance(p, q) -> float:
    """sqrt of the Jensen-Shannon divergence (natural logarithm) of two distributions."""
    p = np.asarray(p, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    m = 0.5 * (p + q)

    def kl(a, b):
        nz = a > 0
        return float(np.sum(a[nz] * (np.log(a[nz]) - np.log(b[nz]))))

    return math.sqrt(max(0.5 * kl(p, m) + 0.5 * kl(q, m), 0.0))


def determine_pattern(a_hat, a_tilde, delta: float, tau: float):
    """Algorithm "Determine Sparse Pattern".  Returns (pattern, d_sparse, d_sim) with pattern
    'shared_pivot' or 'vertical_slash'.  a_tilde None (no pivotal representative) -> d_sim = inf."""
    a_hat = np.asarray(a_hat, dtype=np.float64)
    u = np.full_like(a_hat, 1.0 / a_hat.size)
    d_sparse = js_distance(a_hat, u)
    d_sim = js_distance(a_hat, a_tilde) if a_tilde is not None else math.inf
    pattern = "shared_pivot" if (d_sparse < delta and d_sim < tau) else "vertical_slash"
    return pattern, d_sparse, d_sim


def cumulative_select(a, gamma: float):
    """Minimum prefix of the descending order of the non-negative vector a (normalised by its sum)
    whose scores sum to >= gamma; equal scores go to the smaller index; everything if never reached.
    Returns (selected bool [len(a)], K)."""
    a = np.asarray(a, dtype=np.float64)
    flat = a / a.sum()
    order = np.argsort(-flat, kind="stable")
    cum = np.cumsum(flat[order])
    hit = np.flatnonzero(cum >= gamma)
    K = int(hit[0]) + 1 if hit.size else len(order)
    sel = np.zeros(len(a), dtype=bool)
    sel[order[:K]] = True
    return sel, K


def vertical_slash_scores(Qh, Kg, B: int):
    """A^ = softmax(Q^ K^T / sqrt(d)), causal, for the last block of queries; returns
    (a_v [N], a_s [N]): its sums per key column and per offset o = query - key (o >= 0), unnormalised
    (both sum to the number of rows of Q^)."""
    Qh = np.asarray(Qh, dtype=np.float64)
    Kg = np.asarray(Kg, dtype=np.float64)
    N, d = Qh.shape
    Nb = (N + B - 1) // B
    r0 = (Nb - 1) * B
    S = (Qh[r0:N] @ Kg.T) / math.sqrt(d)
    rows = np.arange(r0, N)[:, None]
    cols = np.arange(N)[None, :]
    S = np.where(cols <= rows, S, -np.inf)
    P = np.exp(S - S.max(axis=1, keepdims=True))
    P /= P.sum(axis=1, keepdims=True)
    a_v = P.sum(axis=0)
    a_s = np.zeros(N)
    for x in range(P.shape[0]):                      # row r0 + x: offset o = r - c
        r = r0 + x
        a_s[:r + 1] += P[x, r::-1]                   # c = r - o for o = 0..r
    return a_v, a_s


def search_vertical_slash_pattern(Qh, Kg, gamma: float, B: int):
    """Algorithm "Search Vertical Slash Pattern" -> dict(mask u8 [Nb, Nb], sel_v, sel_s, K_v, K_s, forced)."""
    N = np.asarray(Qh).shape[0]
    Nb = (N + B - 1) // B
    a_v, a_s = vertical_slash_scores(Qh, Kg, B)
    sel_v, K_v = cumulative_select(a_v, gamma)
    sel_s, K_s = cumulative_select(a_s, gamma)
    mask = np.zeros((Nb, Nb), dtype=np.uint8)
    col_block = np.array([sel_v[j * B:(j + 1) * B].any() for j in range(Nb)])
    for i in range(Nb):
        for j in range(i + 1):
            lo = max((i - j) * B - (B - 1), 0)       # offsets r - c reachable inside block (i, j)
            hi = min((i - j) * B + (B - 1), N - 1)
            if col_block[j] or sel_s[lo:hi + 1].any():
                mask[i, j] = 1
    forced = [i for i in range(Nb) if mask[i].sum() == 0]
    for i in forced:
        mask[i, i] = 1
    return {"mask": mask, "sel_v": sel_v, "sel_s": sel_s, "K_v": K_v, "K_s": K_s, "forced": forced,
            "a_v": a_v, "a_s": a_s}

"""Float64 CPU oracle for the SharePrefill prefill-attention path.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the
CUDA library is checked against.  It shares no code with the CUDA path, imports
nothing from the product package, and must never be called by it: only the
tests, the smoke check and the benchmark's CPU-baseline leg execute it.

Everything is numpy float64.  Inputs are arrays that already hold the
bf16-rounded values (any float dtype; they are widened to float64 exactly).
Library primitives used as steps: matrix product, exp, stable argsort, cumsum.
There is no tiling beyond the block structure the method itself defines.

Layouts: Q is [Hq, N, d]; K and V are [Hkv, N, d]; query head h reads KV head
h // (Hq // Hkv).  A "row-block" i covers query rows [i*B, min((i+1)*B, N));
a "key-block" j covers keys [j*B, min((j+1)*B, N)).  Nb = ceil(N / B).

Readings of the paper taken here (each is also listed in the design notes):
  * attention is causal (LLM prefill); the masked form is the problem
    statement's softmax(QK^T/sqrt(d) - c(1-M))V with c -> infinity;
  * importance of a tile = true softmax probability mass inside the tile,
    averaged over the rows of the row-block (each row-block's entries sum to 1);
  * the cumulative-mass threshold of "Construct Pivotal Pattern" is applied per
    row-block, descending order, ties to the smaller key-block, ">= gamma";
  * one pivot per cluster shares its mask ("Share Pivotal Pattern"); a head
    whose cluster has no pivot gets the all-ones (dense) pattern.

Parity pins live in tests/test_oracle_pins.py (closed forms, brute force,
library cross-check, invariants).  Parity with the paper authors' own
implementation is unpinned: the paper prints no worked numeric example.
"""
from __future__ import annotations

import math

import numpy as np

__all__ = [
    "n_blocks",
    "kv_head_of",
    "attention_rowblock",
    "dense_causal_attention",
    "importance_map",
    "block_mask_row",
    "block_mask_from_importance",
    "masked_attention",
    "share_masks",
    "prefill_attn",
]


def n_blocks(N: int, B: int) -> int:
    return (N + B - 1) // B


def kv_head_of(h: int, Hq: int, Hkv: int) -> int:
    """GQA mapping: consecutive groups of Hq/Hkv query heads share a KV head."""
    if Hq % Hkv != 0:
        raise ValueError("Hq must be a multiple of Hkv")
    return h // (Hq // Hkv)


def attention_rowblock(Qh, Kg, Vg, i: int, B: int, mask_row=None):
    """One row-block of (masked) causal attention for one head.

    Section 5.1 (Problem Formulation): O = softmax(QK^T/sqrt(d) - c(1-M)) V,
    with c -> infinity so that a tile with M = 0 contributes exactly nothing,
    plus the causal constraint key <= query.

    Qh [N, d], Kg/Vg [N, d] float; mask_row is None (dense) or a 0/1 vector
    over key-blocks (entries beyond i are ignored).

    Returns (O [rows, d] float64, mass [i+1] float64) where mass[j] is the
    softmax probability inside tile (i, j) summed over the tile and divided by
    the number of rows of the row-block: the block-importance row.
    """
    Qh = np.asarray(Qh, dtype=np.float64)
    Kg = np.asarray(Kg, dtype=np.float64)
    Vg = np.asarray(Vg, dtype=np.float64)
    N, d = Qh.shape
    r0 = i * B
    r1 = min(r0 + B, N)
    if r0 >= N:
        raise ValueError("row-block out of range")
    rows = r1 - r0
    S = (Qh[r0:r1] @ Kg[:r1].T) / math.sqrt(d)            # [rows, r1]
    r_idx = np.arange(r0, r1)[:, None]
    c_idx = np.arange(r1)[None, :]
    allowed = c_idx <= r_idx                               # causal
    if mask_row is not None:
        mrow = np.asarray(mask_row)
        sel = np.zeros(r1, dtype=bool)
        for j in range(i + 1):
            if mrow[j]:
                sel[j * B:min((j + 1) * B, r1)] = True
        allowed = allowed & sel[None, :]
    if not allowed.any(axis=1).all():
        raise ValueError("a query row has no admissible key (mask selects nothing for it)")
    S = np.where(allowed, S, -np.inf)
    m = S.max(axis=1, keepdims=True)
    E = np.exp(S - m)                                      # exp(-inf) = 0 exactly
    P = E / E.sum(axis=1, keepdims=True)
    O = P @ Vg[:r1]
    col_mass = P.sum(axis=0)                               # [r1]
    mass = np.empty(i + 1, dtype=np.float64)
    for j in range(i + 1):
        mass[j] = col_mass[j * B:min((j + 1) * B, r1)].sum() / rows
    return O, mass


def dense_causal_attention(Q, K, V, B: int = 128, heads=None):
    """Exact causal attention O = softmax(QK^T/sqrt(d)) V for the given heads.

    Section 5.1, second equation (full attention), causal.  B only sets how
    many rows are handled at a time; the result does not depend on it.
    Returns O [len(heads), N, d] float64.
    """
    Hq, N, d = Q.shape
    Hkv = K.shape[0]
    heads = list(range(Hq)) if heads is None else list(heads)
    out = np.empty((len(heads), N, d), dtype=np.float64)
    for t, h in enumerate(heads):
        g = kv_head_of(h, Hq, Hkv)
        for i in range(n_blocks(N, B)):
            O, _ = attention_rowblock(Q[h], K[g], V[g], i, B)
            out[t, i * B:i * B + O.shape[0]] = O
    return out


def importance_map(Q, K, V, h: int, B: int, row_blocks=None):
    """Block-importance map of head h under dense causal attention.

    I[i][j] = (1/rows_i) * sum_{r in row-block i} sum_{c in key-block j, c<=r} P[r,c]
    for j <= i and 0 above the diagonal.  This is the exact quantity that the
    block-averaged score of "Construct Pivotal Pattern" (softmax applied to
    block-averaged QK) estimates.  Returns (I [Nb, Nb] float64, O [N, d]).
    If row_blocks is given only those rows of I / O are filled (others 0).
    """
    Hq, N, d = Q.shape
    g = kv_head_of(h, Hq, K.shape[0])
    Nb = n_blocks(N, B)
    I = np.zeros((Nb, Nb), dtype=np.float64)
    O = np.zeros((N, d), dtype=np.float64)
    for i in (range(Nb) if row_blocks is None else row_blocks):
        o, mass = attention_rowblock(Q[h], K[g], V[g], i, B)
        I[i, :i + 1] = mass
        O[i * B:i * B + o.shape[0]] = o
    return I, O


def block_mask_row(imp_row, i: int, gamma: float):
    """Cumulative-mass threshold for one row-block.

    Algorithm "Construct Pivotal Pattern": sort the scores, take the minimum
    budget K whose top-K sum is >= gamma, select those indices.  Applied to
    the causal entries imp_row[0..i] of row-block i; descending order, equal
    scores ordered by smaller key-block; running sum sequential in that order
    in float64.  If the sum never reaches gamma every causal tile is selected.

    Returns (selected [i+1] uint8, info dict: K, cum_at_cut, cum_before_cut,
    tie_gap = score of last selected - score of first unselected).
    """
    x = np.asarray(imp_row[:i + 1], dtype=np.float64)
    order = np.argsort(-x, kind="stable")                  # descending, ties -> smaller j
    cum = np.cumsum(x[order])
    hit = np.nonzero(cum >= gamma)[0]
    Kc = int(hit[0]) + 1 if hit.size else i + 1
    sel = np.zeros(i + 1, dtype=np.uint8)
    sel[order[:Kc]] = 1
    info = {
        "K": Kc,
        "cum_at_cut": float(cum[Kc - 1]),
        "cum_before_cut": float(cum[Kc - 2]) if Kc >= 2 else 0.0,
        "tie_gap": float(x[order[Kc - 1]] - x[order[Kc]]) if Kc <= i else float("inf"),
    }
    return sel, info


def block_mask_from_importance(I, gamma: float):
    """Importance map [Nb, Nb] -> block mask [Nb, Nb] uint8 (1 = compute).

    Row-blocks are thresholded independently (see block_mask_row); entries
    above the diagonal are 0.  Also returns counts [Nb] and, per row-block,
    the ascending list of selected key-blocks, and the per-row diagnostics.
    """
    I = np.asarray(I)
    Nb = I.shape[0]
    M = np.zeros((Nb, Nb), dtype=np.uint8)
    counts = np.zeros(Nb, dtype=np.int32)
    lists, infos = [], []
    for i in range(Nb):
        sel, info = block_mask_row(I[i], i, gamma)
        M[i, :i + 1] = sel
        counts[i] = info["K"]
        lists.append(np.nonzero(sel)[0].astype(np.int32))
        infos.append(info)
    return M, counts, lists, infos


def masked_attention(Q, K, V, h: int, M, B: int, row_blocks=None):
    """Block-sparse causal attention of head h under block mask M [Nb, Nb].

    Section 5.1, first equation.  Returns O [N, d] float64 (rows of row-blocks
    not requested stay 0).
    """
    Hq, N, d = Q.shape
    g = kv_head_of(h, Hq, K.shape[0])
    Nb = n_blocks(N, B)
    O = np.zeros((N, d), dtype=np.float64)
    for i in (range(Nb) if row_blocks is None else row_blocks):
        o, _ = attention_rowblock(Q[h], K[g], V[g], i, B, mask_row=M[i])
        O[i * B:i * B + o.shape[0]] = o
    return O


def share_masks(cluster_map, pivot_heads):
    """Which pivot's pattern each head uses.

    Algorithm "Share Pivotal Pattern": a head looks up its cluster and takes
    the cluster's pivotal pattern if one exists, else the dense pattern.  The
    pivot of a cluster is the first listed pivot head that belongs to it
    (the paper's "first head within the cluster").  Returns src [Hq] with
    src[h] = index into pivot_heads, or -1 for "dense" (pivots themselves,
    heads with cluster id < 0, heads whose cluster has no pivot).
    The second return value mask_src[h] is the pivot index whose mask is
    *reported* for head h (a pivot reports the mask it constructed).
    """
    cluster_map = list(cluster_map)
    pivot_heads = list(pivot_heads)
    pivot_of_cluster = {}
    for t, p in enumerate(pivot_heads):
        c = cluster_map[p]
        if c >= 0 and c not in pivot_of_cluster:
            pivot_of_cluster[c] = t
    src, mask_src = [], []
    for h, c in enumerate(cluster_map):
        if h in pivot_heads:
            src.append(-1)
            mask_src.append(pivot_heads.index(h))
        elif c >= 0 and c in pivot_of_cluster:
            src.append(pivot_of_cluster[c])
            mask_src.append(pivot_of_cluster[c])
        else:
            src.append(-1)
            mask_src.append(-1)
    return src, mask_src


def prefill_attn(Q, K, V, cluster_map, pivot_heads, gamma: float, B: int, row_blocks=None):
    """The whole layer: Algorithm "Sparse Attention" with the pattern decision
    fixed by (cluster_map, pivot_heads).

    1. pivot heads: dense causal attention + importance map;
    2. importance -> mask per pivot ("Construct Pivotal Pattern");
    3. every other head takes its cluster's pivot mask ("Share Pivotal
       Pattern") and runs masked attention; heads without a pivot run dense.

    Returns dict(out [Hq, N, d] float64, mask [Hq, Nb, Nb] uint8,
    importance [n_pivots, Nb, Nb], infos per pivot).  With row_blocks given,
    only those row-blocks are computed (others left 0 in out/mask/importance).
    """
    Hq, N, d = Q.shape
    Nb = n_blocks(N, B)
    pivot_heads = list(pivot_heads)
    rbs = list(range(Nb)) if row_blocks is None else list(row_blocks)
    out = np.zeros((Hq, N, d), dtype=np.float64)
    imps = np.zeros((len(pivot_heads), Nb, Nb), dtype=np.float64)
    pmasks = np.zeros((len(pivot_heads), Nb, Nb), dtype=np.uint8)
    infos = []
    for t, p in enumerate(pivot_heads):
        I, O = importance_map(Q, K, V, p, B, row_blocks=rbs)
        imps[t] = I
        out[p] = O
        info_t = {}
        for i in rbs:
            sel, info = block_mask_row(I[i], i, gamma)
            pmasks[t, i, :i + 1] = sel
            info_t[i] = info
        infos.append(info_t)
    src, mask_src = share_masks(cluster_map, pivot_heads)
    mask = np.zeros((Hq, Nb, Nb), dtype=np.uint8)
    causal = np.tril(np.ones((Nb, Nb), dtype=np.uint8))
    for h in range(Hq):
        if mask_src[h] >= 0:
            mask[h] = pmasks[mask_src[h]]
        else:
            for i in rbs:
                mask[h, i] = causal[i]
        if h in pivot_heads:
            continue
        if src[h] >= 0:
            out[h] = masked_attention(Q, K, V, h, pmasks[src[h]], B, row_blocks=rbs)
        else:
            g = kv_head_of(h, Hq, K.shape[0])
            for i in rbs:
                o, _ = attention_rowblock(Q[h], K[g], V[g], i, B)
                out[h, i * B:i * B + o.shape[0]] = o
    return {"out": out, "mask": mask, "importance": imps, "pivot_masks": pmasks, "infos": infos}

"""Seeded synthetic long-context attention workloads.

This module only *makes inputs*: bf16 Q/K/V tensors shaped like one attention
layer of a long-context LLM, a head -> cluster table and the list of pivot
heads.  It contains none of the method's arithmetic (no softmax, no importance,
no threshold) and is the one module that both the tests' CPU oracle and the
CUDA library's callers may share.  The same bf16 bits must be handed to both
sides: generate once (on either device) and copy.

Recipe (per config; all draws from a torch.Generator seeded from `seed`):
  1. per cluster c a base matrix base_c ~ N(0,1) [N, d]; per query head h noise
     E_h ~ N(0,1); Qraw_h = (base_c(h) + sigma_h * E_h) / sqrt(d).
     Kraw_g, V_g ~ N(0,1) / sqrt(d) per KV head g.
  2. a shared constant direction lam * ell, ell = (1,...,1)/sqrt(d), is added to
     every row of Qraw and Kraw before RoPE (per cluster lam_c = lam * (1 + 0.1 z_c),
     z_c ~ U(-1,1), on the query side).  It is what makes the rotary phases and
     the mean query matter: without it the logits are nearly uniform.
  3. RoPE on Q and K, half-split pairing (i, i + d/2), inv_freq_i = theta^(-2i/d),
     positions from 0.
  4. attention sink: K_g[0] += 4 * qbar_g, with qbar_g the mean post-RoPE query of
     the heads of KV group g; `n_heavy` seeded key positions get += 2 * qbar_g.
  5. round to bf16.
  6. cluster_map: heads are dealt into `n_clusters` near-equal clusters by a seeded
     permutation (not aligned to KV groups); the pivot of a cluster is its
     lowest-numbered head.

Mixed workloads (`global_clusters` > 0): the last `global_clusters` clusters put their
query-side constant direction into the d/32 slowest-rotating rotary pairs only (norm scaled
by `global_scale`).  Those dimensions turn by about a radian over 131072 positions, so for
these heads the direction acts as a position-independent bias: the block-averaged logits of
a row are flat (every key-block gets the same shift) while key 0 and the heavy keys, which
also carry `global_sink` / `global_heavy` times that direction, take most of the probability
mass.  (The mean query of a KV group is then taken over its ordinary heads only.)  The other clusters keep the
direction in all dimensions, whose fast pairs give the strong local decay.  The two families
fall on different sides of a flatness test on block-averaged logits.
"""
from __future__ import annotations

import dataclasses
import math

import torch


@dataclasses.dataclass(frozen=True)
class LayerConfig:
    name: str
    seq: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    block: int
    rope_theta: float
    n_heavy: int
    n_clusters: int
    noise: tuple          # (lo, hi): sigma_h ~ U(lo, hi); lo == hi -> constant
    lam: float
    gamma: float = 0.9
    global_clusters: int = 0   # clusters (the last ones) whose constant direction lives in the slow rotary pairs only
    global_scale: float = 1.0  # ... scaled by this
    global_sink: float = 0.0   # mixed workloads: K[0] and the heavy keys also get these multiples of that slow direction,
    global_heavy: float = 0.0  # so that what such heads attend to does not depend on which heads share their KV head


CONFIGS = {
    # tiny parity config
    "tiny": LayerConfig("tiny", 2048, 8, 8, 64, 64, 1e4, 16, 2, (0.3, 0.3), 10.5),
    # Llama-3-8B-shaped layer, 32K
    "llama8b_32k": LayerConfig("llama8b_32k", 32768, 32, 8, 128, 128, 5e5, 64, 8, (0.3, 0.3), 12.5),
    # Llama-3-8B-shaped layer, 128K, 4 pivots per 32 heads
    "llama8b_128k": LayerConfig("llama8b_128k", 131072, 32, 8, 128, 128, 5e5, 256, 4, (0.3, 0.3), 13.5),
    # Qwen2.5-7B-shaped layer, 64K, GQA 7
    "qwen7b_64k": LayerConfig("qwen7b_64k", 65536, 28, 4, 128, 128, 1e6, 64, 7, (0.2, 0.6), 13.0),
    # the 128K layer with two families of heads: 3 clusters as above, 3 whose block-averaged logits are flat
    "llama8b_128k_mixed": LayerConfig("llama8b_128k_mixed", 131072, 32, 8, 128, 128, 5e5, 256, 6, (0.3, 0.3), 13.5,
                                      0.9, 3, 0.5, 24.0, 18.0),
}


def scaled(cfg: LayerConfig, seq: int, name: str | None = None) -> LayerConfig:
    """Same recipe at another sequence length (for tests at reduced size)."""
    return dataclasses.replace(cfg, seq=seq, name=name or f"{cfg.name}@{seq}")


def _rope(x: torch.Tensor, theta: float) -> torch.Tensor:
    """Rotary embedding, half-split pairing; x [N, d] fp32."""
    N, d = x.shape
    half = d // 2
    inv_freq = theta ** (-torch.arange(half, device=x.device, dtype=torch.float64) * 2.0 / d)
    ang = torch.arange(N, device=x.device, dtype=torch.float64)[:, None] * inv_freq[None, :]
    cos, sin = ang.cos().float(), ang.sin().float()
    x1, x2 = x[:, :half], x[:, half:]
    return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=1)


def make_cluster_map(cfg: LayerConfig, seed: int):
    g = torch.Generator(device="cpu").manual_seed(seed * 7919 + 17)
    perm = torch.randperm(cfg.n_q_heads, generator=g).tolist()
    cluster_map = [0] * cfg.n_q_heads
    for rank, h in enumerate(perm):
        cluster_map[h] = rank % cfg.n_clusters
    pivots = []
    for c in range(cfg.n_clusters):
        pivots.append(min(h for h in range(cfg.n_q_heads) if cluster_map[h] == c))
    return cluster_map, pivots


def make_layer(cfg: LayerConfig, seed: int = 0, device: str = "cpu", literal: bool = False,
               structure_seed: int | None = None):
    """Returns dict(q [Hq,N,d] bf16, k, v [Hkv,N,d] bf16, cluster_map, pivot_heads, cfg, seed).

    literal=True drops step 2 (lam = 0): the recipe without the shared direction.
    structure_seed: where given, the draws that describe the prompt and the model rather than one layer's
    activations (heavy key positions, cluster table, per-cluster and per-head scalars) come from this seed and
    only the random matrices from `seed`: the layers of one stack then share them, as the layers of a model
    share the prompt and the head clustering.
    """
    dev = torch.device(device)
    N, d, Hq, Hkv = cfg.seq, cfg.head_dim, cfg.n_q_heads, cfg.n_kv_heads
    G = Hq // Hkv
    gen = torch.Generator(device=dev).manual_seed(seed)
    sseed = seed if structure_seed is None else structure_seed
    cpu_gen = torch.Generator(device="cpu").manual_seed(sseed * 104729 + 3)
    cluster_map, pivots = make_cluster_map(cfg, sseed)
    lam = 0.0 if literal else cfg.lam
    ell = torch.full((d,), 1.0 / math.sqrt(d), device=dev)
    # the same norm in the slowest rotary pairs (i, i + d/2), i >= d/2 - d/32: under a radian over 131072 positions
    ell_slow = torch.zeros(d, device=dev)
    n_slow = max(2, d // 32)
    slow = list(range(d // 2 - n_slow, d // 2)) + list(range(d - n_slow, d))
    ell_slow[slow] = 1.0 / math.sqrt(len(slow))
    inv_sqrt_d = 1.0 / math.sqrt(d)

    z = (torch.rand(cfg.n_clusters, generator=cpu_gen) * 2 - 1).tolist()
    lo, hi = cfg.noise
    sigma = (lo + (hi - lo) * torch.rand(Hq, generator=cpu_gen)).tolist()
    heavy = (torch.randperm(N - 1, generator=cpu_gen)[: cfg.n_heavy] + 1).to(dev)

    def randn(*shape):
        return torch.randn(*shape, generator=gen, device=dev, dtype=torch.float32)

    q = torch.empty(Hq, N, d, device=dev, dtype=torch.bfloat16)
    k = torch.empty(Hkv, N, d, device=dev, dtype=torch.bfloat16)
    v = torch.empty(Hkv, N, d, device=dev, dtype=torch.bfloat16)
    qbar = torch.zeros(Hkv, d, device=dev, dtype=torch.float32)
    n_local = [0] * Hkv

    bases = {}
    for h in range(Hq):
        c = cluster_map[h]
        if c not in bases:
            bases[c] = randn(N, d)
    for h in range(Hq):
        c = cluster_map[h]
        is_global = c >= cfg.n_clusters - cfg.global_clusters
        direction = ell_slow * cfg.global_scale if is_global else ell
        qraw = (bases[c] + sigma[h] * randn(N, d)) * inv_sqrt_d + (lam * (1.0 + 0.1 * z[c])) * direction
        qr = _rope(qraw, cfg.rope_theta)
        if not is_global:                       # the mean query of a KV group is taken over its ordinary heads
            qbar[h // G] += qr.mean(dim=0)
            n_local[h // G] += 1
        q[h] = qr.to(torch.bfloat16)
    del bases
    for g in range(Hkv):
        kraw = randn(N, d) * inv_sqrt_d + lam * ell
        kr = _rope(kraw, cfg.rope_theta)
        qb = qbar[g] / max(n_local[g], 1)
        if cfg.global_clusters > 0:
            qb = qb * (ell_slow == 0)           # the slow pairs belong to the other family alone
        kr[0] += 4.0 * qb
        kr[heavy] += 2.0 * qb
        if cfg.global_clusters > 0:
            kr[0] += cfg.global_sink * ell_slow
            kr[heavy] += cfg.global_heavy * ell_slow
        k[g] = kr.to(torch.bfloat16)
        v[g] = (randn(N, d) * inv_sqrt_d).to(torch.bfloat16)
    return {"q": q, "k": k, "v": v, "cluster_map": cluster_map, "pivot_heads": pivots,
            "cfg": cfg, "seed": seed}

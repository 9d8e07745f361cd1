#!/usr/bin/env python
"""Benchmark of the SharePrefill prefill-attention layer on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload llama8b_128k] [--gamma 0.9] [--seed 0]

A "step" is one whole pass of the hot path (pivot dense attention + block
importance, importance -> mask, block-sparse attention of the member heads)
over one synthetic layer, i.e. one `sp_prefill_attn` call.  Prints ONE JSON
line.  `value` is effective (as-if-dense) TFLOP/s:
Hq * 4 d * N (N + 1) / 2 flops per layer divided by the time of a layer.

With N > 1 (torchrun, one process per GPU) every rank runs its own layer
(independent problems: different seeds, as the layers of a model are), no
data-path collective; the time is the max over ranks and `value` the sum of the
layers done divided by it ("weak" scaling).

`--impl reference` times the float64 CPU oracle on a bounded sample of the same
workload instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2505_19578_b200 import synth  # noqa: E402

# DRAM bytes (read + write) per launch of the attention kernel, from ncu captures: a small tracked table
# (one line per workload / length / gamma / seed / call, with the command that produced it in its header).  A
# workload without a line, or a line taken before the kernel last changed (removed then), gives null.
TRAFFIC_TABLE = os.path.join(ROOT, "profiles", "attention_kernel_dram_traffic.txt")


def load_traffic_table(path=TRAFFIC_TABLE):
    """{(workload, seq, gamma, seed, call): bytes per launch}; lines starting with # are comments."""
    table = {}
    if not os.path.exists(path):
        return table
    for line in open(path):
        line = line.split("#", 1)[0].strip()
        if not line:
            continue
        f = line.split()
        if len(f) != 6:
            continue
        table[(f[0], int(f[1]), round(float(f[2]), 6), int(f[3]), f[4])] = int(f[5])
    return table


METRIC = "effective_tflops_prefill_attention_layer"
UNIT = "TFLOP/s"


# ----------------------------------------------------------------------------- helpers (host logic, CPU-testable)

def dense_flops(cfg) -> float:
    """As-if-dense causal attention flops of one layer: Hq * 4 d * N (N+1) / 2."""
    return cfg.n_q_heads * 4.0 * cfg.head_dim * cfg.seq * (cfg.seq + 1) / 2.0


def tile_flops(cfg) -> float:
    """QK^T + PV of one full (block x block) tile."""
    return 4.0 * cfg.block * cfg.block * cfg.head_dim


def rank_seed(base_seed: int, rank: int) -> int:
    """Each rank works on its own layer (independent problem)."""
    return base_seed + 1000 * rank


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def aggregate(ms_local: float, layers_local: float, world: int, device=None):
    """Max time over ranks, total layers over ranks."""
    if world == 1:
        return ms_local, layers_local
    import torch.distributed as dist
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    n = torch.tensor([layers_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), float(n.item())


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"bf16_tflops": d["bf16_tflops"], "bf16_tflops_sustained": d.get("bf16_tflops_sustained"),
                "hbm_gbs": d["hbm_gbs"], "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clocks / throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.proc, self.path = gpu_index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu)], stdout=open(self.path, "w"),
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if not self.proc:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, power, reasons = [], [], [], set()
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), power_w_max=max(power),
                       reasons=sorted(reasons), samples=len(sm))
        return out


# ----------------------------------------------------------------------------- CPU oracle legs

def oracle_sample_time(L, gamma, row_blocks):
    """Times the float64 oracle (as it stands) on the given row-blocks of every head.
    Returns (seconds, as-if-dense flops covered, threads used)."""
    import numpy as np
    from oracle import shareprefill_oracle as orc
    cfg = L["cfg"]
    Q = L["q"].float().cpu().numpy().astype(np.float64)
    K = L["k"].float().cpu().numpy().astype(np.float64)
    V = L["v"].float().cpu().numpy().astype(np.float64)
    g = float(np.float32(gamma))
    t0 = time.perf_counter()
    orc.prefill_attn(Q, K, V, L["cluster_map"], L["pivot_heads"], g, cfg.block, row_blocks=row_blocks)
    dt = time.perf_counter() - t0
    B, d = cfg.block, cfg.head_dim
    flops = sum(cfg.n_q_heads * 4.0 * d * B * (i * B + (B + 1) / 2.0) for i in row_blocks)
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threads = os.cpu_count() or 1
    return dt, flops, threads


def time_config(binding, ctx, L, gamma, steps, stream, dense=True):
    """Per-kernel times of one layer on workload L at `gamma`: the three public calls with CUDA events between them,
    one warm-up, `steps` timed; the build's own dense kernel on every head beside it.  Compact dict for the
    other_configs block."""
    cfg = L["cfg"]
    q, k, v, cm, piv = L["q"], L["k"], L["v"], L["cluster_map"], L["pivot_heads"]
    B, Nb = cfg.block, cfg.seq // cfg.block
    dev = q.device
    out = torch.empty_like(q)
    members = [h for h in range(cfg.n_q_heads) if h not in piv]
    first_pivot_of = {}
    for t, p in enumerate(piv):
        first_pivot_of.setdefault(cm[p], t)
    lists = [first_pivot_of.get(cm[h], -1) if cm[h] >= 0 else -1 for h in members]
    imp = torch.empty(len(piv), Nb, Nb, device=dev)
    pm = torch.empty(len(piv), Nb, Nb, dtype=torch.uint8, device=dev)
    counts = torch.empty(len(piv), Nb, dtype=torch.int32, device=dev)
    indices = torch.empty(len(piv), Nb, Nb, dtype=torch.int32, device=dev)

    def split_step(e):
        e[0].record(stream)
        ctx.sp_dense_pivot_attn(q, k, v, piv, B, out, importance_out=imp, stream=stream)
        e[1].record(stream)
        ctx.sp_block_mask_from_importance(imp, gamma, pm, counts, indices, stream=stream)
        e[2].record(stream)
        ctx.sp_block_sparse_attn(q, k, v, members, lists, counts, indices, B, out, stream=stream)
        e[3].record(stream)

    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps + 1)]
    sampler = ClockSampler(dev.index or 0)
    split_step(ev[0])
    torch.cuda.synchronize()
    sampler.start()
    for e in ev[1:]:
        split_step(e)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    k1 = sum(e[0].elapsed_time(e[1]) for e in ev[1:]) / steps
    k2 = sum(e[1].elapsed_time(e[2]) for e in ev[1:]) / steps
    k3 = sum(e[2].elapsed_time(e[3]) for e in ev[1:]) / steps
    # the whole call
    w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ctx.sp_prefill_attn(q, k, v, cm, piv, gamma, B, out, stream=stream)
    torch.cuda.synchronize()
    w0.record(stream)
    for _ in range(steps):
        ctx.sp_prefill_attn(q, k, v, cm, piv, gamma, B, out, stream=stream)
    w1.record(stream)
    torch.cuda.synchronize()
    ms = w0.elapsed_time(w1) / steps
    cnt = counts.cpu().numpy()
    tiles_causal = Nb * (Nb + 1) // 2
    pivot_tiles = len(piv) * tiles_causal
    member_tiles = int(sum(int(cnt[l].sum()) if l >= 0 else tiles_causal for l in lists))
    Ft = tile_flops(cfg)
    dense_ms = None
    if dense:
        heads = list(range(cfg.n_q_heads))
        ctx.sp_dense_pivot_attn(q, k, v, heads, B, out, stream=stream)
        torch.cuda.synchronize()
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        d0.record(stream)
        for _ in range(2):
            ctx.sp_dense_pivot_attn(q, k, v, heads, B, out, stream=stream)
        d1.record(stream)
        torch.cuda.synchronize()
        dense_ms = d0.elapsed_time(d1) / 2
    assert ctx.status() == (0, 0), "device-side wait timed out"
    dens = [float(cnt[t].sum()) / tiles_causal for t in range(len(piv))]
    return {
        "workload": cfg.name, "seq": cfg.seq, "gamma": gamma, "n_pivots": len(piv), "steps": steps,
        "ms_per_layer": ms, "kernels_ms": {"pivot_dense_attn": k1, "block_mask": k2, "block_sparse_attn": k3},
        "visited_tflops": {"pivot_dense_attn": pivot_tiles * Ft / (k1 * 1e-3) / 1e12,
                           "block_sparse_attn": member_tiles * Ft / (k3 * 1e-3) / 1e12 if k3 > 0 else 0.0},
        "mask_density_min_max": [min(dens), max(dens)] if dens else None,
        "dense_baseline_ms": dense_ms, "speedup_vs_dense": dense_ms / ms if dense_ms else None,
        "clocks": {k_: clocks.get(k_) for k_ in ("sm_mhz", "sm_max_mhz", "reasons")},
    }


def workload_cfg(args):
    cfg = synth.CONFIGS[args.workload]
    return synth.scaled(cfg, args.seq) if args.seq else cfg


def config_dict(cfg, gamma, n_pivots, seed, by_cluster):
    """The `config` object of the JSON line: the same for both arms (the reference arm runs on this arm's config)."""
    return {"workload": cfg.name, "seq": cfg.seq, "n_q_heads": cfg.n_q_heads, "n_kv_heads": cfg.n_kv_heads,
            "head_dim": cfg.head_dim, "block": cfg.block, "gamma": gamma, "n_pivots": n_pivots, "seed": seed,
            "l2": "inputs (2.5 GiB at 128K) exceed the 126 MB L2; no flush between steps",
            "units_per_rank": ("one layer split by cluster over the ranks (K/V replicated, outputs disjoint, no "
                               "collective)" if by_cluster else "one layer per rank, independent seeds")}


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    cfg = workload_cfg(args)
    L = synth.make_layer(cfg, seed=rank_seed(args.seed, 0), device="cpu")
    Nb = cfg.seq // cfg.block
    rbs = [Nb // 2]
    times, flops, threads = [], 0.0, 1
    for s in range(args.warmup + args.steps):
        dt, flops, threads = oracle_sample_time(L, args.gamma, rbs)
        if s >= args.warmup:
            times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = flops / (ms * 1e-3) / 1e12
    sample = f"row-block {rbs[0]} of {Nb} for all {cfg.n_q_heads} heads per step (float64 numpy oracle)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(cfg, args.gamma, len(L["pivot_heads"]), args.seed, args.shard == "cluster" and world > 1),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ----------------------------------------------------------------------------- GPU arm

def run_ours(args):
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (there is no CPU fallback for the product path)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    from paper_2505_19578_b200 import binding, build
    build.build()

    cfg = workload_cfg(args)
    gamma = args.gamma
    by_cluster = args.shard == "cluster" and world > 1      # ONE layer split over the ranks (strong scaling)
    L = synth.make_layer(cfg, seed=args.seed if by_cluster else rank_seed(args.seed, rank), device=str(dev))
    q, k, v = L["q"], L["k"], L["v"]
    cm, piv = L["cluster_map"], L["pivot_heads"]
    Nb, B = cfg.seq // cfg.block, cfg.block
    ctx = binding.Context(device=local_rank)
    ctx.reserve(binding.workspace_bytes(cfg.seq, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, B, len(piv)))
    out = torch.empty_like(q)
    mask = torch.empty(cfg.n_q_heads, Nb, Nb, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    # ---- the layer split by cluster: a shard is the pivots of some clusters, their members and the heads that run
    #      dense; K and V are replicated, every rank writes the output rows of its own heads, nothing is exchanged
    from paper_2505_19578_b200 import sharding
    sh_bufs = {}

    def run_shard(sh):
        n_p = len(sh.pivots)
        if n_p not in sh_bufs:
            sh_bufs[n_p] = (torch.empty(max(n_p, 1), Nb, Nb, device=dev),
                            torch.empty(max(n_p, 1), Nb, Nb, dtype=torch.uint8, device=dev),
                            torch.empty(max(n_p, 1), Nb, dtype=torch.int32, device=dev),
                            torch.empty(max(n_p, 1), Nb, Nb, dtype=torch.int32, device=dev))
        s_imp, s_pm, s_cnt, s_idx = sh_bufs[n_p]
        if n_p:
            ctx.sp_dense_pivot_attn(q, k, v, sh.pivots, B, out, importance_out=s_imp[:n_p], stream=stream)
            ctx.sp_block_mask_from_importance(s_imp[:n_p], gamma, s_pm[:n_p], s_cnt[:n_p], s_idx[:n_p], stream=stream)
        if sh.dense:
            ctx.sp_dense_pivot_attn(q, k, v, sh.dense, B, out, stream=stream)
        if sh.members:
            ctx.sp_block_sparse_attn(q, k, v, sh.members, sh.member_list, s_cnt[:max(n_p, 1)], s_idx[:max(n_p, 1)], B, out,
                                     stream=stream)

    my_shard = sharding.deal_clusters(cm, piv, world, Nb)[rank] if by_cluster else None

    def step():
        if by_cluster:
            run_shard(my_shard)
        else:
            ctx.sp_prefill_attn(q, k, v, cm, piv, gamma, B, out, mask_out=mask, stream=stream)

    # ---- warm-up, then the timed region: K whole-layer steps, inputs resident in HBM
    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    launches0 = ctx.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    ms_local = e0.elapsed_time(e1) / args.steps
    launches = ctx.launch_count() - launches0
    assert ctx.status() == (0, 0), "device-side wait timed out"

    # ---- per-kernel split: the same step issued as its three public calls with events between
    members = [h for h in range(cfg.n_q_heads) if h not in piv]
    first_pivot_of = {}
    for t, p in enumerate(piv):
        first_pivot_of.setdefault(cm[p], t)
    lists = [first_pivot_of.get(cm[h], -1) if cm[h] >= 0 else -1 for h in members]
    imp = torch.empty(len(piv), Nb, Nb, device=dev)
    pm = torch.empty(len(piv), Nb, Nb, dtype=torch.uint8, device=dev)
    counts = torch.empty(len(piv), Nb, dtype=torch.int32, device=dev)
    indices = torch.empty(len(piv), Nb, Nb, dtype=torch.int32, device=dev)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]

    def split_step(e):
        e[0].record(stream)
        ctx.sp_dense_pivot_attn(q, k, v, piv, B, out, importance_out=imp, stream=stream)
        e[1].record(stream)
        ctx.sp_block_mask_from_importance(imp, gamma, pm, counts, indices, stream=stream)
        e[2].record(stream)
        ctx.sp_block_sparse_attn(q, k, v, members, lists, counts, indices, B, out, stream=stream)
        e[3].record(stream)

    scratch = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    split_step(scratch)
    torch.cuda.synchronize()
    for e in ev:
        split_step(e)
    torch.cuda.synchronize()
    k1 = sum(e[0].elapsed_time(e[1]) for e in ev) / args.steps
    k2 = sum(e[1].elapsed_time(e[2]) for e in ev) / args.steps
    k3 = sum(e[2].elapsed_time(e[3]) for e in ev) / args.steps
    cnt_host = counts.cpu().numpy()
    tiles_causal = Nb * (Nb + 1) // 2
    pivot_tiles = len(piv) * tiles_causal
    member_tiles = int(sum(int(cnt_host[l].sum()) if l >= 0 else tiles_causal for l in lists))
    density = {int(p): float(cnt_host[t].sum()) / tiles_causal for t, p in enumerate(piv)}

    # ---- the build's own dense baseline: every head dense, no importance (one warm run, two timed)
    all_heads = list(range(cfg.n_q_heads))
    dense_ms = None
    if rank == 0 and not args.no_dense:
        ctx.sp_dense_pivot_attn(q, k, v, all_heads, B, out, stream=stream)
        torch.cuda.synchronize()
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        d0.record(stream)
        for _ in range(2):
            ctx.sp_dense_pivot_attn(q, k, v, all_heads, B, out, stream=stream)
        d1.record(stream)
        torch.cuda.synchronize()
        dense_ms = d0.elapsed_time(d1) / 2
    clocks = sampler.stop() if rank == 0 else None

    # ---- preview of the split by cluster on this one GPU: the shards of a W-rank run one after the other; the longest
    #      is what the layer would take on W GPUs (no exchange step; an estimate, not a multi-GPU measurement)
    shard_preview = None
    if world == 1 and args.shard_preview > 1:
        shards = sharding.deal_clusters(cm, piv, args.shard_preview, Nb)
        per = []
        for sh in shards:
            run_shard(sh)
            torch.cuda.synchronize()
            p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            p0.record(stream)
            for _ in range(3):
                run_shard(sh)
            p1.record(stream)
            torch.cuda.synchronize()
            per.append({"heads": sh.heads(), "pivots": sh.pivots, "estimated_tiles": sh.cost, "ms": p0.elapsed_time(p1) / 3})
        shard_preview = {"ranks": args.shard_preview, "shards": per, "ms_longest": max(x["ms"] for x in per),
                         "ms_sum": sum(x["ms"] for x in per),
                         "note": "shards timed one after the other on ONE GPU; ms_longest estimates the layer at that many "
                                 "GPUs with K/V replicated (no collective in the path)"}

    # ---- optional: a stack of layers (each its own seeded inputs and 3-6 clusters), times summed over layers
    stack = None
    if args.stack_layers is None:
        args.stack_layers = 32 if (world == 1 and not args.seq and args.workload == "llama8b_128k" and gamma == 0.9) else 0
    if rank == 0 and args.stack_layers > 0:
        import dataclasses
        import random
        rng = random.Random(args.seed)
        t_sparse = t_dense = 0.0
        piv_counts = []
        for layer in range(args.stack_layers):
            lcfg = dataclasses.replace(cfg, n_clusters=rng.randint(3, 6))
            Ll = synth.make_layer(lcfg, seed=args.seed + 1 + layer, device=str(dev))
            piv_counts.append(len(Ll["pivot_heads"]))
            se = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            if layer == 0:                                  # warm the kernels on this shape once
                ctx.sp_prefill_attn(Ll["q"], Ll["k"], Ll["v"], Ll["cluster_map"], Ll["pivot_heads"], gamma, B, out, stream=stream)
            torch.cuda.synchronize()
            se[0].record(stream)
            ctx.sp_prefill_attn(Ll["q"], Ll["k"], Ll["v"], Ll["cluster_map"], Ll["pivot_heads"], gamma, B, out, stream=stream)
            se[1].record(stream)
            if not args.no_dense:
                ctx.sp_dense_pivot_attn(Ll["q"], Ll["k"], Ll["v"], all_heads, B, out, stream=stream)
            se[2].record(stream)
            torch.cuda.synchronize()
            t_sparse += se[0].elapsed_time(se[1])
            t_dense += se[1].elapsed_time(se[2])
            del Ll
        stack = {"layers": args.stack_layers, "pivots_per_layer": piv_counts, "shareprefill_ms": t_sparse,
                 "dense_ms": None if args.no_dense else t_dense,
                 "speedup_vs_dense": None if args.no_dense else t_dense / t_sparse,
                 "note": "every layer has its own seeded q, k, v and 3-6 clusters (one pivot each); layers treated independently"}

    # ---- the other configurations named next to the default one: the gamma sweep on the same inputs, the 32K and the
    #      GQA-7 64K layer (a few steps each; per-kernel times, visited-tile rates, dense, clocks)
    others = None
    if world == 1 and not args.no_other_configs and not args.seq and args.workload == "llama8b_128k" and gamma == 0.9:
        others = []
        n_other = max(2, min(args.steps, 5))
        for g_ in (0.8, 0.95):
            others.append(time_config(binding, ctx, L, g_, n_other, stream, dense=False))
        for name in ("llama8b_32k", "qwen7b_64k"):
            Lo = synth.make_layer(synth.CONFIGS[name], seed=args.seed, device=str(dev))
            others.append(time_config(binding, ctx, Lo, 0.9, n_other, stream, dense=not args.no_dense))
            del Lo
            torch.cuda.empty_cache()

    # ---- a workload on which the paper's thresholds (gamma 0.9, delta 0.3, tau 0.2) decide something: two families
    #      of heads, one sharing its pivots' patterns, one falling back to vertical-slash.  One layer through
    #      sp_prefill_attn_auto, then a stack of layers through the cross-layer dictionary (pivots only where a cluster
    #      has no pattern yet; later layers reuse what earlier ones stored)
    mixed = None
    if (world == 1 and not args.no_mixed and not args.seq and args.workload == "llama8b_128k" and gamma == 0.9):
        mcfg = synth.CONFIGS["llama8b_128k_mixed"]
        Lm = synth.make_layer(mcfg, seed=args.seed, device=str(dev))
        mout = torch.empty_like(Lm["q"])
        mpat = torch.empty(mcfg.n_q_heads, dtype=torch.int32, device=dev)
        me = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        for _ in range(2):
            me[0].record(stream)
            ctx.sp_prefill_attn_auto(Lm["q"], Lm["k"], Lm["v"], Lm["cluster_map"], Lm["pivot_heads"], gamma, 0.3, 0.2, B,
                                     mout, pattern_out=mpat, stream=stream)
            me[1].record(stream)
            torch.cuda.synchronize()
        mp = mpat.cpu().numpy()
        mixed = {"workload": mcfg.name, "gamma": gamma, "delta": 0.3, "tau": 0.2,
                 "prefill_attn_auto": {"ms_per_layer": me[0].elapsed_time(me[1]),
                                       "heads_dense_shared_vslash": [int((mp == c).sum()) for c in (0, 1, 2)]}}
        n_dict_layers = args.stack_layers if args.stack_layers > 0 else 0
        if n_dict_layers:
            pd = binding.PatternDict(ctx, mcfg.n_clusters, mcfg.n_q_heads, mcfg.seq, B)
            t_layers, totals, new_pivots = 0.0, [0, 0, 0], []
            for layer in range(n_dict_layers):
                Ll = Lm if layer == 0 else synth.make_layer(mcfg, seed=args.seed + 1 + layer, device=str(dev),
                                                            structure_seed=args.seed)
                before = pd.count()
                if layer == 0:                          # warm the kernels of this flow once, on a dictionary of its own
                    warm = binding.PatternDict(ctx, mcfg.n_clusters, mcfg.n_q_heads, mcfg.seq, B)
                    warm.prefill_attn_layer(Ll["q"], Ll["k"], Ll["v"], Ll["cluster_map"], gamma, 0.3, 0.2, B, mout, stream=stream)
                    torch.cuda.synchronize()
                    warm.close()
                de = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
                de[0].record(stream)
                pd.prefill_attn_layer(Ll["q"], Ll["k"], Ll["v"], Ll["cluster_map"], gamma, 0.3, 0.2, B, mout,
                                      pattern_out=mpat, stream=stream)
                de[1].record(stream)
                torch.cuda.synchronize()
                t_layers += de[0].elapsed_time(de[1])
                lp = mpat.cpu().numpy()
                for c in (0, 1, 2):
                    totals[c] += int((lp == c).sum())
                new_pivots.append(pd.count() - before)
                if layer:
                    del Ll
            mixed["layer_stack_with_dictionary"] = {
                "layers": n_dict_layers, "ms_total": t_layers, "ms_per_layer_mean": t_layers / n_dict_layers,
                "pivots_per_model": pd.count(), "new_pivots_per_layer": new_pivots,
                "heads_dense_shared_vslash_total": totals,
                "note": "layers share the heavy key positions and the cluster table (structure seed) and draw their own "
                        "q, k, v; one sp_prefill_attn_layer call per layer, CUDA events around each call"}
            pd.close()
        assert ctx.status() == (0, 0), "device-side wait timed out"
        del Lm, mout
        torch.cuda.empty_cache()

    # ---- the paper-literal construction beside it (block-averaged QK values, global cut): time and what it selects
    literal = None
    if world == 1 and not args.no_literal:      # (with several ranks the other GPUs would only stand by)
        pooled = torch.empty(len(piv), Nb, Nb, dtype=torch.float64, device=dev)
        lm = torch.empty(len(piv), Nb, Nb, dtype=torch.uint8, device=dev)
        lc = torch.empty(len(piv), Nb, dtype=torch.int32, device=dev)
        li = torch.empty(len(piv), Nb, Nb, dtype=torch.int32, device=dev)
        last = torch.empty(len(piv), Nb, device=dev)
        pat = torch.empty(cfg.n_q_heads, dtype=torch.int32, device=dev)
        rows = [first_pivot_of.get(cm[h], -1) if cm[h] >= 0 else -1 for h in range(cfg.n_q_heads)]

        def literal_step(e):
            e[0].record(stream)
            ctx.sp_pooled_logits(q, k, piv, B, pooled, stream=stream)
            e[1].record(stream)
            ctx.sp_pattern_from_pooled(pooled, gamma, lm, lc, li, last_row_out=last, stream=stream)
            e[2].record(stream)
            ctx.sp_determine_pattern(q, k, list(range(cfg.n_q_heads)), B, last, rows, 0.3, 0.2, pat, stream=stream)
            e[3].record(stream)

        le = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        literal_step(le)
        torch.cuda.synchronize()
        literal_step(le)
        torch.cuda.synchronize()
        # vertical-slash fallback of every member head: search, then the block-sparse kernel on its lists
        vs = None
        if (cfg.head_dim, B) == (128, 128):
            vm = torch.empty(len(members), Nb, Nb, dtype=torch.uint8, device=dev)
            vc = torch.empty(len(members), Nb, dtype=torch.int32, device=dev)
            vi = torch.empty(len(members), Nb, Nb, dtype=torch.int32, device=dev)
            ve = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            for _ in range(2):
                ve[0].record(stream)
                ctx.sp_vertical_slash_pattern(q, k, members, gamma, B, vm, vc, vi, stream=stream)
                ve[1].record(stream)
                ctx.sp_block_sparse_attn(q, k, v, members, list(range(len(members))), vc, vi, B, out, stream=stream)
                ve[2].record(stream)
                torch.cuda.synchronize()
            vtiles = int(vc.sum().item())
            vs = {"search_ms": ve[0].elapsed_time(ve[1]), "block_sparse_attn_ms": ve[1].elapsed_time(ve[2]),
                  "heads": len(members), "mean_mask_density": vtiles / (len(members) * tiles_causal),
                  "block_sparse_tflops": vtiles * tile_flops(cfg) / (ve[1].elapsed_time(ve[2]) * 1e-3) / 1e12}
        # the whole online algorithm with the decision on the device (paper's thresholds, then thresholds that let heads share)
        auto = None
        if (cfg.head_dim, B) == (128, 128):
            auto = {}
            for label, (dl, tu) in (("delta0.3_tau0.2", (0.3, 0.2)), ("delta1_tau1", (1.0, 1.0))):
                ae = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
                for _ in range(2):
                    ae[0].record(stream)
                    ctx.sp_prefill_attn_auto(q, k, v, cm, piv, gamma, dl, tu, B, out, pattern_out=pat, stream=stream)
                    ae[1].record(stream)
                    torch.cuda.synchronize()
                pc_ = pat.cpu().numpy()
                auto[label] = {"ms_per_layer": ae[0].elapsed_time(ae[1]),
                               "heads_dense_shared_vslash": [int((pc_ == c).sum()) for c in (0, 1, 2)]}
        inter = (lm & pm).sum(dim=(1, 2)).float()
        union = (lm | pm).sum(dim=(1, 2)).float()
        literal = {
            "pooled_logits_ms": le[0].elapsed_time(le[1]), "pattern_from_pooled_ms": le[1].elapsed_time(le[2]),
            "determine_pattern_ms": le[2].elapsed_time(le[3]),
            "mask_density_per_pivot": {int(p): float(lc[t].sum().item()) / tiles_causal for t, p in enumerate(piv)},
            "jaccard_with_mass_mask_per_pivot": {int(p): float(inter[t] / union[t]) for t, p in enumerate(piv)},
            "heads_shared_pivot_at_delta0.3_tau0.2": int((pat == 0).sum().item()),
            "vertical_slash": vs,
            "prefill_attn_auto": auto,
        }

    # ---- end to end through the C ABI with host buffers: H2D of q,k,v, the layer, D2H of the output
    hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
    hout = torch.empty(out.shape, dtype=out.dtype).pin_memory()

    def e2e_step():
        # the library's host-buffer call: H2D of q, k, v, the layer, D2H of the output, pipelined inside
        ctx.sp_prefill_attn_host(hq, hk, hv, cm, piv, gamma, B, hout, mask_out=None, stream=stream)

    e2e_steps = 0 if args.no_e2e else max(1, min(args.steps, 5))
    if e2e_steps:
        e2e_step()
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    f1.record(stream)
    barrier()
    e2e_ms_local = f0.elapsed_time(f1) / e2e_steps if e2e_steps else float("nan")
    h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv))
    d2h = hout.numel() * hout.element_size()

    ms, layers = aggregate(ms_local, 1.0 / world if by_cluster else 1.0, world, dev)
    e2e_ms, _ = aggregate(e2e_ms_local, 1.0, world, dev)
    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    F = dense_flops(cfg)
    Ft = tile_flops(cfg)
    value = layers * F / (ms * 1e-3) / 1e12
    k1_tf = pivot_tiles * Ft / (k1 * 1e-3) / 1e12
    k3_tf = member_tiles * Ft / (k3 * 1e-3) / 1e12 if k3 > 0 else 0.0
    # dominant kernel by time
    dom = ("pivot_dense_attn", k1, k1_tf) if k1 >= k3 else ("block_sparse_attn", k3, k3_tf)
    roofline = {
        "kernel": (f"attn_pair_kernel ({dom[0]})" if (cfg.head_dim, cfg.block) == (128, 128)
                   else f"attn_tc_kernel<{cfg.head_dim},{cfg.block}> ({dom[0]})"),
        "bound": "tensor", "achieved": dom[2],
        "peak": peaks["bf16_tflops_sustained"] or peaks["bf16_tflops"], "unit": "TFLOP/s",
        "frac": dom[2] / (peaks["bf16_tflops_sustained"] or peaks["bf16_tflops"]),
        "peak_kind": f"{peaks['source']} sustained cuBLAS bf16 (kernel timed inside a long step)",
        "frac_of_burst_peak": dom[2] / peaks["bf16_tflops"],
        "traffic": load_traffic_table().get((cfg.name, cfg.seq, round(gamma, 6), args.seed, dom[0])),
        "traffic_unit": "bytes of DRAM read + write per launch (ncu, same workload; null: not taken since the kernel changed)",
        "ms_per_launch": dom[1], "flops_per_launch": (pivot_tiles if dom[0].startswith("pivot") else member_tiles) * Ft,
        "timing": "CUDA events around each of the three public calls, same inputs, same number of steps",
    }
    mask_bytes = len(piv) * Nb * Nb * (4 + 1 + 4) + len(piv) * Nb * 4
    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "strong" if by_cluster else "weak", "vs_baseline": None,
        "dtype": "bf16",
        "data": "synthetic",
        "config": config_dict(cfg, gamma, len(piv), args.seed, by_cluster),
        "ms_per_layer": ms,
        "kernels_ms": {"pivot_dense_attn": k1, "block_mask": k2, "block_sparse_attn": k3},
        "visited_tiles": {"pivot": pivot_tiles, "members": member_tiles, "causal_per_head": tiles_causal},
        "mask_density_per_pivot": density,
        "visited_tflops": {"pivot_dense_attn": k1_tf, "block_sparse_attn": k3_tf,
                           "layer": (pivot_tiles + member_tiles) * Ft / (ms * 1e-3) / 1e12},
        "frac_of_bf16_peak": {"pivot_dense_attn": k1_tf / peaks["bf16_tflops"],
                              "block_sparse_attn": k3_tf / peaks["bf16_tflops"], "peak": peaks["bf16_tflops"],
                              "peak_source": peaks["source"]},
        "block_mask_gbs": mask_bytes / (k2 * 1e-3) / 1e9 if k2 > 0 else None,
        "dense_baseline_ms": dense_ms,
        "dense_baseline_tflops": F / (dense_ms * 1e-3) / 1e12 if dense_ms else None,
        "speedup_vs_dense": dense_ms / ms if dense_ms else None,
        "roofline": roofline,
        "e2e": {"value": layers * F / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "paper_literal_pattern": literal,
        "layer_stack": stack,
        "other_configs": others,
        "mixed_workload": mixed,
        "shard_preview": shard_preview,
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    if world == 1 and not args.no_cpu_baseline:
        Lh = {"q": hq, "k": hk, "v": hv, "cluster_map": cm, "pivot_heads": piv, "cfg": cfg}
        rbs = sorted({0, Nb // 4, Nb // 2, Nb - 1})
        dt, fl, threads = oracle_sample_time(Lh, gamma, rbs)
        result["cpu_baseline"] = {"value": fl / dt / 1e12, "unit": UNIT, "cores": threads, "kind": "oracle",
                                  "seconds": dt,
                                  "sample": f"row-blocks {rbs} of {Nb} for all {cfg.n_q_heads} heads "
                                            f"(float64 numpy oracle, whole method)"}
    print(json.dumps(result))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama8b_128k", choices=sorted(synth.CONFIGS))
    ap.add_argument("--gamma", type=float, default=0.9)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--seq", type=int, default=0, help="override the workload's sequence length (profiling on a small case)")
    ap.add_argument("--no-dense", action="store_true", help="skip the dense-baseline leg")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the CPU-oracle leg")
    ap.add_argument("--shard", default="layer", choices=["layer", "cluster"],
                    help="with --gpus N > 1: 'layer' = one independent layer per rank (weak scaling, default); 'cluster' = ONE "
                         "layer split by head cluster over the ranks (strong scaling, no collective)")
    ap.add_argument("--shard-preview", type=int, default=0,
                    help="at N = 1: also time the shards of a split by cluster over this many ranks, one after the other")
    ap.add_argument("--no-mixed", action="store_true",
                    help="skip the two-family workload (sp_prefill_attn_auto and the dictionary flow at the paper's thresholds)")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the compact block on the other configurations (gamma 0.8 / 0.95, 32K, 64K GQA-7)")
    ap.add_argument("--stack-layers", type=int, default=None,
                    help="also run a stack of this many independent layers (3-6 seeded clusters each) and sum their "
                         "times; default: 32 on the default 131072-token workload at N = 1, otherwise 0")
    ap.add_argument("--no-literal", action="store_true", help="skip the paper-literal pattern construction leg")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg (profiling runs)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

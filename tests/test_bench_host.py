"""Host-side logic of bench.py, on CPU: work formulas, the per-rank sharding
and the max-over-ranks reduction (world size 2, gloo), and the reference arm."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from paper_2505_19578_b200 import synth  # noqa: E402


def test_work_formulas():
    cfg = synth.CONFIGS["llama8b_128k"]
    assert bench.tile_flops(cfg) == 4 * 128 * 128 * 128
    assert abs(bench.dense_flops(cfg) - 1.407e14) / 1.407e14 < 1e-3
    nb = cfg.seq // cfg.block
    # dense flops ~= causal tiles * tile flops (the diagonal tiles are counted half in the dense formula)
    tiles = cfg.n_q_heads * nb * (nb + 1) / 2
    assert abs(tiles * bench.tile_flops(cfg) / bench.dense_flops(cfg) - 1) < 2e-3
    assert len({bench.rank_seed(0, r) for r in range(8)}) == 8


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, layers = bench.aggregate(10.0 * (rank + 1), 1.0, world, device=None)
    q.put((rank, ms, layers))
    dist.destroy_process_group()


def test_aggregate_max_over_ranks_gloo_world2():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == [(0, 20.0, 2.0), (1, 20.0, 2.0)]            # slowest rank's time, both layers counted
    assert bench.aggregate(7.0, 1.0, 1) == (7.0, 1.0)


def test_reference_arm_prints_one_json_line_and_other_ranks_stay_silent():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
           "--steps", "1", "--warmup", "3"]
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    out = subprocess.run(cmd, capture_output=True, text=True, env=env, timeout=600)
    assert out.returncode == 0, out.stderr
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == bench.METRIC and d["unit"] == bench.UNIT
    assert d["value"] > 0 and d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["vs_baseline"] is None
    # the reference arm runs on the GPU arm's config: one function writes the object for both
    from paper_2505_19578_b200 import synth
    cfg = synth.CONFIGS["tiny"]
    n_piv = len(synth.make_cluster_map(cfg, 0)[1])
    assert d["config"] == bench.config_dict(cfg, 0.9, n_piv, 0, False)
    env1 = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out1 = subprocess.run(cmd, capture_output=True, text=True, env=env1, timeout=600)
    assert out1.returncode == 0 and out1.stdout.strip() == ""


def test_traffic_table_parsing(tmp_path):
    import bench
    p = tmp_path / "t.txt"
    p.write_text("# comment\n\nllama8b_128k 131072 0.9 0 pivot_dense_attn 123456  # trailing note\nbad line\n")
    t = bench.load_traffic_table(str(p))
    assert t == {("llama8b_128k", 131072, 0.9, 0, "pivot_dense_attn"): 123456}
    assert bench.load_traffic_table(str(tmp_path / "missing.txt")) == {}


def _shard_worker(rank, world, port, q):
    import os
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch
    import torch.distributed as dist
    from paper_2505_19578_b200 import sharding, synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cm, piv = synth.make_cluster_map(synth.CONFIGS["llama8b_128k_mixed"], 0)
    cm[5] = -1                                         # a head without a cluster: a dense unit of its own
    shards = sharding.deal_clusters(cm, piv, world, 1024)
    mine = shards[rank]
    owned = torch.zeros(len(cm), dtype=torch.int32)
    owned[mine.heads()] = 1
    dist.all_reduce(owned)                             # how many ranks compute each head
    costs = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(costs, torch.tensor([mine.cost], dtype=torch.float64))
    q.put((rank, owned.tolist(), [float(c) for c in costs], mine.pivots, mine.members, mine.member_list, mine.dense))
    dist.destroy_process_group()


def test_cluster_sharding_gloo_world2():
    """Strong-scaling split of one layer by cluster: every head is computed by exactly one rank, a pivot sits with
    all the members that walk its list, and the estimated loads are balanced."""
    import multiprocessing as mp
    from paper_2505_19578_b200 import sharding, synth
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 500
    ps = [ctx.Process(target=_shard_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in ps:
        p.start()
    got = sorted(q.get(timeout=120) for _ in ps)
    for p in ps:
        p.join(timeout=60)
        assert p.exitcode == 0
    cm, piv = synth.make_cluster_map(synth.CONFIGS["llama8b_128k_mixed"], 0)
    cm[5] = -1
    for rank, owned, costs, pivots, members, member_list, dense in got:
        assert owned == [1] * len(cm)                                  # exactly once, on every rank's view
        for h, slot in zip(members, member_list):
            assert cm[h] == cm[pivots[slot]] and cm[h] >= 0            # a member walks the list of its own cluster's pivot
        assert all(p in piv for p in pivots)
        assert max(costs) <= 1.35 * min(costs)                         # 6 clusters + 1 loose head on 2 ranks
    assert 5 in got[0][6] + got[1][6]
    # one rank: everything; more ranks than units: some stay empty, nothing is lost
    one = sharding.deal_clusters(cm, piv, 1, 64)
    assert one[0].heads() == list(range(len(cm)))
    many = sharding.deal_clusters(cm, piv, 16, 64)
    assert sorted(h for s in many for h in s.heads()) == list(range(len(cm)))
    # a second listed pivot of a cluster runs dense on the rank of its cluster
    units, loose = sharding.units_of_layer([0, 0, 0, 1], [0, 1])
    assert units[0]["pivot"] == 0 and units[0]["extra_pivots"] == [1] and units[0]["members"] == [2] and loose == [3]

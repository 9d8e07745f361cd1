"""The C-ABI library builds, loads without a GPU, and exports every symbol
that include/shareprefill.h declares.  No compute call is made here."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2505_19578_b200 import binding, build
    build.build()
    return binding.load()


def _declared():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            txt = open(os.path.join(inc, f)).read()
            txt = re.sub(r"/\*.*?\*/", "", txt, flags=re.S)
            names |= set(re.findall(r"\b(sp_[a-z0-9_]+)\s*\(", txt))
    return names


def test_every_declared_symbol_is_exported(lib):
    from paper_2505_19578_b200 import binding
    names = _declared()
    assert {"sp_prefill_attn", "sp_dense_pivot_attn", "sp_block_mask_from_importance",
            "sp_block_sparse_attn"} <= names
    assert names == set(binding.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_host_only_calls(lib):
    from paper_2505_19578_b200 import binding
    assert binding.error_string(0) == "ok"
    assert "timed out" in binding.error_string(binding.SP_ERR_TIMEOUT)
    b = binding.workspace_bytes(131072, 32, 8, 128, 128, 4)
    nb = 1024
    # importance + mask + counts + lists, and per-tile statistics: one region of 2 * nb * 128 floats per
    # persistent CTA (at most one per SM) instead of one float per row of every causal tile of every pivot
    assert b >= 4 * nb * nb * (4 + 1 + 4) + 2 * nb * 128 * 4
    assert b < 256 << 20
    # the one-row-block kernel (other shapes) keeps the per-tile layout
    b64 = binding.workspace_bytes(8192, 8, 8, 64, 64, 2)
    assert b64 >= 2 * 128 * 129 // 2 * 64 * 4
    wa, wl = binding.workspace_bytes_patterns(131072, 32, 8, 128, 128, 6)
    assert wa > 32 * nb * nb * 5 and wl > 0            # masks and lists of every head's own pattern
    assert binding.workspace_bytes_patterns(131072, 32, 8, 128, 128, 6, True)[0] > wa - (200 << 20)
    out = ctypes.c_size_t()
    assert lib.sp_workspace_bytes(1000, 32, 8, 128, 128, 4, ctypes.byref(out)) == binding.SP_ERR_UNSUPPORTED
    assert lib.sp_workspace_bytes(4096, 32, 8, 96, 128, 4, ctypes.byref(out)) == binding.SP_ERR_UNSUPPORTED
    assert lib.sp_workspace_bytes(4096, 32, 8, 128, 128, 4, None) == binding.SP_ERR_INVALID_ARG


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    from paper_2505_19578_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load()


def test_work_order_of_the_paired_kernel_covers_every_tile_once(lib):
    """Host logic of a paired-kernel launch: every (head, row-block) is one tile of exactly one work item; two heads
    share items only if they read the same KV head and walk the same list; a launch of many items keeps the heads of
    a KV head together and, inside such a group, the long row-blocks first."""
    import random
    from paper_2505_19578_b200 import binding
    rnd = random.Random(11)
    cases = [([4, 0, 3, 5, 1, 2], [1, 0, 1, -1, 1, -1], 6, 1, 11, 148)]            # the GPU test's case: 2 pairs + 2 single
    for _ in range(60):
        hkv = rnd.choice([1, 2, 4, 8])
        hq = hkv * rnd.choice([1, 2, 4, 7])
        n_heads = rnd.randint(1, hq)
        heads = rnd.sample(range(hq), n_heads)
        lists = [rnd.choice([-1, 0, 1, 2]) for _ in heads]
        cases.append((heads, lists, hq, hkv, rnd.choice([1, 2, 3, 8, 9, 64, 257]), rnd.choice([4, 148])))
    for heads, lists, hq, hkv, nb, n_sm in cases:
        group = hq // hkv
        for pair_heads in (True, False):
            items, n_groups = binding.pair_work_order(heads, lists, hq, hkv, nb, n_sm, pair_heads)
            assert len(items) == len(heads) * ((nb + 1) // 2)
            seen = {}
            for raw, (sa, ra, sb, rb) in enumerate(items):
                assert 0 <= sa < len(heads) and 0 <= sb < len(heads) and ra >= 0 and rb >= 0
                assert heads[sa] // group == heads[sb] // group                   # one K/V stream per item
                if sa != sb:
                    assert pair_heads and ra == rb                                # two heads: the same row-block,
                    assert max(lists[sa], -1) == max(lists[sb], -1)               # ... the same list
                else:
                    assert rb == ra + 1 and ra % 2 == 0                           # one head: adjacent row-blocks
                for s_, r_ in ((sa, ra), (sb, rb)):
                    if r_ < nb:
                        assert (s_, r_) not in seen, (heads, lists, nb, raw)
                        seen[(s_, r_)] = raw
            assert len(seen) == len(heads) * nb                                   # every tile, once
            by_kv = len(heads) * ((nb + 1) // 2) >= 40 * n_sm
            assert n_groups == (len({h // group for h in heads}) if by_kv else 1)
            # the heads of a KV head stay together (many items), and inside a group the pairs of row-blocks never grow
            last_u, last_kv, closed = None, None, set()
            for sa, ra, sb, rb in items:
                kv = heads[sa] // group
                if by_kv and kv != last_kv:
                    assert kv not in closed
                    closed.add(kv)
                    last_kv, last_u = kv, None
                assert last_u is None or ra // 2 <= last_u
                last_u = ra // 2
    # the 128K workload: 16 of the 28 members find a partner
    from paper_2505_19578_b200 import synth
    cfg = synth.CONFIGS["llama8b_128k"]
    cm, piv = synth.make_cluster_map(cfg, 0)
    members = [h for h in range(cfg.n_q_heads) if h not in piv]
    items, _ = binding.pair_work_order(members, [cm[h] for h in members], cfg.n_q_heads, cfg.n_kv_heads, 1024)
    assert len({s for sa, _, sb, _ in items if sa != sb for s in (sa, sb)}) == 16

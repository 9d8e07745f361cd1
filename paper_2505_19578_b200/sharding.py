"""Host-side split of ONE layer across GPUs by head cluster (strong scaling).

A cluster (its pivot and the members that share the pivot's pattern) needs no
data from another cluster: the pivot's dense pass, its mask and its members'
block-sparse passes all happen on one GPU, K and V are replicated, and every
rank writes the output rows of its own heads only.  So the split needs no
exchange step inside the layer (the paper's Limitations paragraph names
per-device partial dictionaries as the way to scale the method out; this is
that, inside one layer).  Heads that run dense (no cluster, or a cluster without
a pivot) are units of their own.

Only integer bookkeeping happens here; nothing of the method's arithmetic.
"""
from __future__ import annotations

from dataclasses import dataclass, field


@dataclass
class Shard:
    pivots: list = field(default_factory=list)    # pivot heads this rank runs dense (and builds masks from)
    members: list = field(default_factory=list)   # heads that walk a pivot's list on this rank
    member_list: list = field(default_factory=list)  # for each member: index into `pivots` of the list it walks
    dense: list = field(default_factory=list)     # heads without a pattern: dense on this rank
    cost: float = 0.0                             # estimated tiles

    def heads(self):
        return sorted(self.pivots + self.members + self.dense)


def units_of_layer(cluster_map, pivot_heads):
    """Work units of a layer: one per cluster that has a pivot (first listed pivot of the cluster + every other
    listed pivot of it, which runs dense too, + its members), one per head that runs dense without a pattern.
    Mirrors the sharing rule of the library: the pivot of a cluster is the first listed pivot belonging to it."""
    cluster_map, pivot_heads = list(cluster_map), list(pivot_heads)
    first = {}
    for p in pivot_heads:
        c = cluster_map[p]
        if c >= 0 and c not in first:
            first[c] = p
    units = {c: {"pivot": p, "extra_pivots": [], "members": []} for c, p in first.items()}
    loose = []
    for h, c in enumerate(cluster_map):
        if h in pivot_heads:
            if c >= 0 and first.get(c) == h:
                continue
            if c >= 0 and c in units:
                units[c]["extra_pivots"].append(h)     # a second listed pivot of a cluster: dense, its mask unused
            else:
                loose.append(h)                        # a listed pivot without a cluster: dense
        elif c >= 0 and c in units:
            units[c]["members"].append(h)
        else:
            loose.append(h)
    return units, loose


def deal_clusters(cluster_map, pivot_heads, n_ranks: int, n_blocks: int, member_density: float = 0.1):
    """Deals the units to `n_ranks` ranks, largest first onto the least loaded rank.  Cost model in tiles: a dense
    head walks T = n_blocks (n_blocks + 1) / 2 tiles, a member about member_density * T (the real figure is only
    known after the pivot has run).  Returns a list of n_ranks Shard objects; every head appears exactly once."""
    if n_ranks < 1:
        raise ValueError("n_ranks must be >= 1")
    T = n_blocks * (n_blocks + 1) / 2.0
    units, loose = units_of_layer(cluster_map, pivot_heads)
    items = []
    for c, u in units.items():
        cost = T * (1 + len(u["extra_pivots"])) + member_density * T * len(u["members"])
        items.append((cost, 0, c))
    for h in loose:
        items.append((T, 1, h))
    items.sort(key=lambda t: (-t[0], t[1], t[2]))
    shards = [Shard() for _ in range(n_ranks)]
    for cost, kind, key in items:
        r = min(range(n_ranks), key=lambda x: (shards[x].cost, x))
        s = shards[r]
        if kind == 0:
            u = units[key]
            slot = len(s.pivots)
            s.pivots.append(u["pivot"])
            for h in u["members"]:
                s.members.append(h)
                s.member_list.append(slot)
            s.dense.extend(u["extra_pivots"])
        else:
            s.dense.append(key)
        s.cost += cost
    return shards

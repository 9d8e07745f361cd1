"""Calibration record of a synthetic workload, computed with the float64 oracle only.

TEST INFRASTRUCTURE: run by hand (`python -m oracle.workload_calibration <workload> [seed] [rows]`); it calls the
input generator and the oracle, never the CUDA library.  For every cluster of the layer it prints, for the pivot
and for up to three members: d_sparse and d_sim (Algorithm "Determine Sparse Pattern"), the density of the
mass-based mask at gamma (Algorithm "Construct Pivotal Pattern", per row-block), the Jaccard similarity between
the member's own mask and the pivot's (Section 4 of the paper reports > 0.5 between similar heads), and the
error of the member's output under the pivot's mask against its dense output, on sampled row-blocks.
"""
from __future__ import annotations

import sys

import numpy as np

from oracle import pooled_pattern_oracle as ppo
from oracle import shareprefill_oracle as orc
from paper_2505_19578_b200 import synth


def main(argv):
    name = argv[1] if len(argv) > 1 else "llama8b_128k_mixed"
    seed = int(argv[2]) if len(argv) > 2 else 0
    n_rows = int(argv[3]) if len(argv) > 3 else 8
    gamma = float(np.float32(0.9))
    cfg = synth.CONFIGS[name]
    L = synth.make_layer(cfg, seed=seed)
    f64 = lambda t: t.float().numpy().astype(np.float64)
    B, Nb, Hq = cfg.block, cfg.seq // cfg.block, cfg.n_q_heads
    G = Hq // cfg.n_kv_heads
    rng = np.random.default_rng(7)
    rows = sorted({1, Nb // 2, Nb - 1} | set(int(x) for x in rng.choice(Nb, n_rows, replace=False)))
    u = np.full(Nb, 1.0 / Nb)
    cm, piv = L["cluster_map"], L["pivot_heads"]
    print(f"{name} seed {seed}: N {cfg.seq}, {Hq}/{cfg.n_kv_heads} heads, gamma 0.9, row-blocks {rows}")
    for c, p in enumerate(piv):
        members = [h for h in range(Hq) if cm[h] == c and h != p][:3]
        family = "flat" if c >= cfg.n_clusters - cfg.global_clusters else "local"
        rec = {}
        for h in [p] + members:
            g = h // G
            Q, K, V = f64(L["q"][h]), f64(L["k"][g]), f64(L["v"][g])
            a = ppo.last_block_distribution(Q, K, B)
            if h == p:
                a_p = a
            sel, dense_o = {}, {}
            for i in rows:
                o, mass = orc.attention_rowblock(Q, K, V, i, B)
                s, _ = orc.block_mask_row(mass, i, gamma)
                sel[i], dense_o[i] = s, o
            err = None
            if h != p:
                num = den = 0.0
                for i in rows:
                    o_sh, _ = orc.attention_rowblock(Q, K, V, i, B, mask_row=rec[p]["sel"][i])
                    num += float(np.sum((o_sh - dense_o[i]) ** 2))
                    den += float(np.sum(dense_o[i] ** 2))
                err = (num / den) ** 0.5
            rec[h] = {"sel": sel, "d_sparse": ppo.js_distance(a, u), "d_sim": ppo.js_distance(a, a_p), "err": err,
                      "density": float(np.mean([sel[i].sum() / (i + 1) for i in rows]))}
        line = (f"cluster {c} ({family}): pivot {p} d_sparse {rec[p]['d_sparse']:.3f} density {rec[p]['density']:.3f}")
        for h in members:
            jac = [float((rec[h]["sel"][i] & rec[p]["sel"][i]).sum() / max(1, (rec[h]["sel"][i] | rec[p]["sel"][i]).sum()))
                   for i in rows]
            line += (f" | member {h}: d_sparse {rec[h]['d_sparse']:.3f} d_sim {rec[h]['d_sim']:.4f} own density "
                     f"{rec[h]['density']:.3f} Jaccard min/mean {min(jac):.2f}/{np.mean(jac):.2f} "
                     f"rel-L2 error under the shared mask {rec[h]['err']:.3f}")
        print(line, flush=True)


if __name__ == "__main__":
    main(sys.argv)

"""Element-by-element brute force used to pin the oracle (tiny sizes only).

Pure Python loops over scalars with math.exp: no matrix product, no blocking,
no shared code with the oracle.  It materialises the full N x N probability
matrix first and derives everything else from it.
"""
import math


def causal_probs(Qh, Kg, allowed=None):
    """P[r][c] for one head; allowed(r, c) -> bool adds a mask on top of causality."""
    N, d = len(Qh), len(Qh[0])
    P = [[0.0] * N for _ in range(N)]
    for r in range(N):
        logits = []
        for c in range(r + 1):
            if allowed is not None and not allowed(r, c):
                logits.append(None)
                continue
            s = 0.0
            for t in range(d):
                s += float(Qh[r][t]) * float(Kg[c][t])
            logits.append(s / math.sqrt(d))
        finite = [x for x in logits if x is not None]
        mx = max(finite)
        den = sum(math.exp(x - mx) for x in finite)
        for c, x in enumerate(logits):
            if x is not None:
                P[r][c] = math.exp(x - mx) / den
    return P


def apply_probs(P, Vg):
    N, d = len(P), len(Vg[0])
    O = [[0.0] * d for _ in range(N)]
    for r in range(N):
        for c in range(r + 1):
            p = P[r][c]
            if p != 0.0:
                for t in range(d):
                    O[r][t] += p * float(Vg[c][t])
    return O


def tile_mass(P, B):
    """I[i][j] = sum of P over tile (i, j) / rows in row-block i."""
    N = len(P)
    Nb = (N + B - 1) // B
    I = [[0.0] * Nb for _ in range(Nb)]
    for r in range(N):
        for c in range(r + 1):
            I[r // B][c // B] += P[r][c]
    for i in range(Nb):
        rows = min((i + 1) * B, N) - i * B
        for j in range(Nb):
            I[i][j] /= rows
    return I

"""Test-side helpers that are independent of both the oracle and the CUDA library."""

from __future__ import annotations

import numpy as np


def out_edges(G):
    """sender -> list of receiver-CSR edge ids, by ascending receiver."""
    out = [[] for _ in range(G.n)]
    for i in range(G.n):
        for e in range(int(G.rowptr[i]), int(G.rowptr[i + 1])):
            out[int(G.col[e])].append(e)
    return out


def brute_force_stamps(G, sch, codes):
    """Consumed stamp of every (event, in-edge), straight from the definition: the largest
    local-iteration stamp among the packets of that edge that were not dropped and whose
    first usable round (send round + 1 + delay) is not after the consuming round.

    Returns (stamps, act_round): stamps is a flat int list in event order then in-edge order,
    act_round[j] lists the rounds in which j was active (activation t happens in act_round[j][t-1]).
    """
    n = G.n
    out = out_edges(G)
    sent = [[] for _ in range(len(G.col))]          # per edge: (first usable round, stamp)
    t = [0] * n
    act_round = [[] for _ in range(n)]
    pos = 0
    ev_of = []
    for r in range(sch.K):
        for ev in range(int(sch.act_ptr[r]), int(sch.act_ptr[r + 1])):
            i = int(sch.act_node[ev])
            t[i] += 1
            act_round[i].append(r)
            for f in out[i]:
                d = int(codes[pos]); pos += 1
                if d >= 0:
                    sent[f].append((r + 1 + d, t[i]))
            ev_of.append((r, i))
    stamps = []
    for (r, i) in ev_of:
        for e in range(int(G.rowptr[i]), int(G.rowptr[i + 1])):
            stamps.append(max([s for (a, s) in sent[e] if a <= r], default=0))
    return stamps, act_round


class FracGraph:
    """Receiver-CSR graph with exact rational weights (fractions.Fraction)."""

    def __init__(self, G, kind):
        from fractions import Fraction
        self.n, self.rowptr, self.col, self.kind = G.n, G.rowptr, G.col, kind
        indeg = np.diff(G.rowptr)
        outdeg = np.bincount(G.col, minlength=G.n)
        if kind == "row":
            self.diag = [Fraction(1, 1 + int(indeg[i])) for i in range(G.n)]
            recv = np.repeat(np.arange(G.n), indeg)
            self.w = [Fraction(1, 1 + int(indeg[recv[e]])) for e in range(len(G.col))]
        else:
            self.diag = [Fraction(1, 1 + int(outdeg[i])) for i in range(G.n)]
            self.w = [Fraction(1, 1 + int(outdeg[G.col[e]])) for e in range(len(G.col))]


def f64_weights(G):
    """Same graph with the uniform weights recomputed in float64 (column / row sums exact
    to rounding), for checks that need stochasticity far below float32 resolution."""
    import copy
    H = copy.copy(G)
    indeg = np.diff(G.rowptr).astype(np.float64)
    outdeg = np.bincount(G.col, minlength=G.n).astype(np.float64)
    if G.kind == "row":
        recv = np.repeat(np.arange(G.n), np.diff(G.rowptr))
        H.w = 1.0 / (1.0 + indeg[recv]); H.diag = 1.0 / (1.0 + indeg)
    else:
        H.w = 1.0 / (1.0 + outdeg[G.col]); H.diag = 1.0 / (1.0 + outdeg)
    return H

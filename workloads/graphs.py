"""Communication graphs G_R = G(W) and G_C = G(A) as receiver-CSR arrays.

Edge convention (Section III-A): (j, i) is an edge of G(M) iff M_ij > 0, and
then j sends to i.  A graph is stored by receiver: row i lists its in-neighbours
j in ascending order together with M_ij; the diagonal M_ii is kept apart.

Weights follow the rule of Appendix G ("designed by knowing the number of
in-neighbours, resp. out-neighbours"), read as uniform weights:
  W (row-stochastic):    w_ij = 1 / (1 + |N_i^in(W)|)   for j in N_i^in(W) or j = i
  A (column-stochastic): a_ji = 1 / (1 + |N_i^out(A)|)  for j in N_i^out(A) or j = i
"""

from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass
class Graph:
    n: int
    rowptr: np.ndarray   # int32 [n+1], receiver-CSR
    col: np.ndarray      # int32 [E], sender ids, ascending within a row
    w: np.ndarray        # float32 [E], M[receiver, sender]
    diag: np.ndarray     # float32 [n], M[i, i]
    kind: str            # "row" (W) or "col" (A)

    @property
    def n_edges(self) -> int:
        return int(self.col.shape[0])

    def dense(self, dtype=np.float64) -> np.ndarray:
        """The n x n weight matrix (for tests on small graphs)."""
        M = np.zeros((self.n, self.n), dtype=dtype)
        for i in range(self.n):
            M[i, i] = self.diag[i]
            for e in range(self.rowptr[i], self.rowptr[i + 1]):
                M[i, self.col[e]] = self.w[e]
        return M


def graph_from_edges(n: int, edges, kind: str) -> Graph:
    """edges: iterable of (sender j, receiver i), j != i, no duplicates."""
    edges = sorted(set((int(j), int(i)) for j, i in edges), key=lambda t: (t[1], t[0]))
    for j, i in edges:
        if j == i or not (0 <= j < n and 0 <= i < n):
            raise ValueError(f"bad edge ({j},{i})")
    indeg = np.zeros(n, dtype=np.int64)
    outdeg = np.zeros(n, dtype=np.int64)
    for j, i in edges:
        indeg[i] += 1
        outdeg[j] += 1
    rowptr = np.zeros(n + 1, dtype=np.int32)
    rowptr[1:] = np.cumsum(indeg)
    col = np.array([j for j, _ in edges], dtype=np.int32).reshape(-1)
    recv = np.array([i for _, i in edges], dtype=np.int64).reshape(-1)
    if kind == "row":
        w = (1.0 / (1.0 + indeg[recv])).astype(np.float32) if len(edges) else np.zeros(0, np.float32)
        diag = (1.0 / (1.0 + indeg)).astype(np.float32)
    elif kind == "col":
        w = (1.0 / (1.0 + outdeg[col])).astype(np.float32) if len(edges) else np.zeros(0, np.float32)
        diag = (1.0 / (1.0 + outdeg)).astype(np.float32)
    else:
        raise ValueError(kind)
    return Graph(n, rowptr, col, w, diag, kind)


def sender_csr(g: Graph):
    """Out-edge lists: for sender j its receivers in ascending order.

    Returns (optr[n+1], orecv[E], oeid[E]) with oeid the receiver-CSR edge index.
    This is the order in which a schedule lists one event's send codes.
    """
    n, E = g.n, g.n_edges
    recv = np.repeat(np.arange(n, dtype=np.int64), np.diff(g.rowptr).astype(np.int64))
    order = np.lexsort((recv, g.col.astype(np.int64)))   # by sender, then receiver
    optr = np.zeros(n + 1, dtype=np.int32)
    optr[1:] = np.cumsum(np.bincount(g.col, minlength=n))
    return optr, recv[order].astype(np.int32), order.astype(np.int32)


def tree_graphs(parent_R, parent_C):
    """G_R: every non-root pulls from its parent (edge parent -> child);
    G_C: every non-root pushes to its parent (edge child -> parent).
    parent[root] = -1; the two trees may differ but share the root."""
    parent_R = np.asarray(parent_R)
    parent_C = np.asarray(parent_C)
    n = len(parent_R)
    eR = [(int(parent_R[i]), i) for i in range(n) if parent_R[i] >= 0]
    eC = [(i, int(parent_C[i])) for i in range(n) if parent_C[i] >= 0]
    return graph_from_edges(n, eR, "row"), graph_from_edges(n, eC, "col")


def ring_graphs(n: int):
    """Directed ring i -> (i+1) mod n for both graphs."""
    e = [(i, (i + 1) % n) for i in range(n)] if n > 1 else []
    return graph_from_edges(n, e, "row"), graph_from_edges(n, e, "col")


def binary_tree_parents(n: int) -> np.ndarray:
    p = np.array([(j - 1) // 2 for j in range(n)], dtype=np.int64)
    p[0] = -1
    return p


def exponential_tree_parents(n: int):
    """Two spanning trees of the exponential graph on n = 2^m nodes, root 0:
    clear the highest set bit (tree used for G_R) / the lowest set bit (G_C).
    Each parent differs from the child in one power of two, an exponential-graph hop."""
    hi = np.full(n, -1, dtype=np.int64)
    lo = np.full(n, -1, dtype=np.int64)
    for j in range(1, n):
        hi[j] = j & ~(1 << (j.bit_length() - 1))
        lo[j] = j & (j - 1)
    return hi, lo


def random_tree_parents(n: int, rng: np.random.Generator, max_children: int | None = None) -> np.ndarray:
    """Random recursive tree on a seeded relabelling, node 0 kept as the root.
    With max_children, a parent is drawn among earlier nodes that still have room."""
    label = np.concatenate([[0], 1 + rng.permutation(n - 1)]) if n > 1 else np.array([0])
    parent = np.full(n, -1, dtype=np.int64)
    nchild = np.zeros(n, dtype=np.int64)
    for k in range(1, n):
        if max_children is None:
            q = int(rng.integers(0, k))
        else:
            room = [q for q in range(k) if nchild[label[q]] < max_children]
            q = room[int(rng.integers(0, len(room)))]
        parent[label[k]] = label[q]
        nchild[label[q]] += 1
    return parent

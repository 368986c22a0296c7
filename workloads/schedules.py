"""Raw, value-independent asynchronous schedules (Algorithm 2, step S.0).

A schedule lists, for K rounds, which nodes are active, and for every activation
event and every out-edge of the active node (in each graph) whether the packet
sent by that event is dropped (-1) or after how many extra rounds it becomes
available (delay d >= 0: sent in round r, usable from round r + 1 + d).
For stochastic models it also carries the minibatch row indices of every event
(and the initial sample of every node).

Nothing here depends on iterate values; stamps and delays in the paper's sense
(tau, d_v, d_rho) are derived from these arrays by whoever consumes them.
"""

from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from .graphs import Graph, sender_csr


@dataclass
class Schedule:
    K: int
    act_ptr: np.ndarray      # int32 [K+1]
    act_node: np.ndarray     # int32 [E_ev], ascending inside a round
    send_r: np.ndarray       # int8, per (event, out-edge of its node in G_R, sender order)
    send_c: np.ndarray       # int8, same for G_C
    batch: int               # B, 0 when the model takes no minibatch
    batch_idx: np.ndarray    # int32 [(n + E_ev) * B]; first n*B entries: the initial samples
    alpha_round: np.ndarray | None = None   # float32 [K] step size per round, or None (constant)

    @property
    def n_events(self) -> int:
        return int(self.act_node.shape[0])


def activation_all(n: int, K: int):
    return [np.arange(n, dtype=np.int32) for _ in range(K)]


def activation_bernoulli(n: int, K: int, prob: float, rng: np.random.Generator):
    """Each node active independently with probability prob; an empty draw is repeated."""
    out = []
    for _ in range(K):
        while True:
            m = rng.random(n) < prob
            if m.any():
                break
        out.append(np.nonzero(m)[0].astype(np.int32))
    return out


def activation_uniform_subset(n: int, K: int, lo: int, hi: int, rng: np.random.Generator):
    """m ~ U{lo..hi} distinct nodes per round."""
    out = []
    for _ in range(K):
        m = int(rng.integers(lo, hi + 1))
        out.append(np.sort(rng.choice(n, size=m, replace=False)).astype(np.int32))
    return out


def activation_durations(n: int, K: int, duration_fn):
    """Compute-time model: a node that activates in round r activates next in round
    r + duration_fn(node, activation_index); everybody starts in round 0."""
    nxt = np.zeros(n, dtype=np.int64)
    cnt = np.zeros(n, dtype=np.int64)
    out = []
    for r in range(K):
        act = np.nonzero(nxt <= r)[0]
        for i in act:
            d = int(duration_fn(int(i), int(cnt[i])))
            nxt[i] = r + max(1, d)
            cnt[i] += 1
        out.append(act.astype(np.int32))
    return out


def make_schedule(G_R: Graph, G_C: Graph, active_sets, drop: float, max_delay: int,
                  rng: np.random.Generator, batch: int = 0, rows_per_node: int = 0) -> Schedule:
    n = G_R.n
    K = len(active_sets)
    act_ptr = np.zeros(K + 1, dtype=np.int32)
    act_ptr[1:] = np.cumsum([len(a) for a in active_sets])
    act_node = (np.concatenate(active_sets).astype(np.int32)
                if K and act_ptr[-1] else np.zeros(0, np.int32))
    outdeg_R = np.diff(sender_csr(G_R)[0]).astype(np.int64)
    outdeg_C = np.diff(sender_csr(G_C)[0]).astype(np.int64)

    def codes(outdeg):
        m = int(outdeg[act_node].sum())
        d = rng.integers(0, max_delay + 1, size=m).astype(np.int8)
        dropped = rng.random(m) < drop
        d[dropped] = -1
        return d

    send_r = codes(outdeg_R)
    send_c = codes(outdeg_C)
    if batch > 0:
        batch_idx = rng.integers(0, rows_per_node, size=(n + len(act_node)) * batch).astype(np.int32)
    else:
        batch_idx = np.zeros(0, np.int32)
    return Schedule(K, act_ptr, act_node, send_r, send_c, batch, batch_idx)


def split_schedule(s: Schedule, G_R: Graph, G_C: Graph, cuts) -> list:
    """The schedule cut into consecutive parts at the rounds `cuts` (ascending, inside 0..K), each
    part numbered from its own round 0 and event 0, the way rounds are handed to an engine a
    piece at a time.  Every part carries the initial samples (the first n*B entries of
    batch_idx) in front of its own events' samples.  Array slicing only."""
    n = G_R.n
    outdeg_R = np.diff(sender_csr(G_R)[0]).astype(np.int64)
    outdeg_C = np.diff(sender_csr(G_C)[0]).astype(np.int64)
    off_r = np.concatenate([[0], np.cumsum(outdeg_R[s.act_node])]).astype(np.int64)
    off_c = np.concatenate([[0], np.cumsum(outdeg_C[s.act_node])]).astype(np.int64)
    bounds = [0] + [int(c) for c in cuts] + [int(s.K)]
    parts = []
    for r0, r1 in zip(bounds[:-1], bounds[1:]):
        e0, e1 = int(s.act_ptr[r0]), int(s.act_ptr[r1])
        lead = n * s.batch
        bi = (np.concatenate([s.batch_idx[:lead], s.batch_idx[lead + e0 * s.batch: lead + e1 * s.batch]]).astype(np.int32)
              if s.batch > 0 else np.zeros(0, np.int32))
        parts.append(Schedule(r1 - r0, (s.act_ptr[r0:r1 + 1] - e0).astype(np.int32), s.act_node[e0:e1].copy(),
                              s.send_r[off_r[e0]:off_r[e1]].copy(), s.send_c[off_c[e0]:off_c[e1]].copy(), s.batch, bi,
                              None if s.alpha_round is None else s.alpha_round[r0:r1].copy()))
    return parts


def make_schedule_ack_gated(G_R: Graph, G_C: Graph, active_sets, max_delay: int,
                            rng: np.random.Generator, batch: int = 0, rows_per_node: int = 0) -> Schedule:
    """Packet loss as the paper emulates it (Section VI, first paragraph): a node sends a new
    packet to an out-neighbour only once that neighbour has acknowledged the previous one, and
    otherwise discards the packet of this activation.  Here: a packet sent in round r with
    delay d is usable from round r+1+d; the receiver acknowledges it at its first activation
    from then on, and the acknowledgement travels back with its own delay (same distribution).
    Until it has arrived the sender's packets on that edge are dropped (code -1)."""
    n = G_R.n
    K = len(active_sets)
    act_ptr = np.zeros(K + 1, dtype=np.int32)
    act_ptr[1:] = np.cumsum([len(a) for a in active_sets])
    act_node = (np.concatenate(active_sets).astype(np.int32) if K and act_ptr[-1] else np.zeros(0, np.int32))
    act_rounds = [[] for _ in range(n)]
    for r, a in enumerate(active_sets):
        for i in a:
            act_rounds[int(i)].append(r)
    act_rounds = [np.asarray(a, dtype=np.int64) for a in act_rounds]

    def codes(G):
        optr, orecv, oeid = sender_csr(G)
        ack_ready = np.zeros(G.n_edges, dtype=np.int64)        # round from which the edge may send again
        out = []
        for r, a in enumerate(active_sets):
            for i in a:
                for k in range(optr[i], optr[i + 1]):
                    e, j = int(oeid[k]), int(orecv[k])
                    if r < ack_ready[e]:
                        out.append(-1)
                        continue
                    d = int(rng.integers(0, max_delay + 1))
                    out.append(d)
                    pos = np.searchsorted(act_rounds[j], r + 1 + d)
                    if pos == len(act_rounds[j]):
                        ack_ready[e] = K + 1                     # never processed within the horizon
                    else:
                        ack_ready[e] = int(act_rounds[j][pos]) + 1 + int(rng.integers(0, max_delay + 1))
        return np.asarray(out, dtype=np.int8)

    send_r = codes(G_R)
    send_c = codes(G_C)
    if batch > 0:
        batch_idx = rng.integers(0, rows_per_node, size=(n + len(act_node)) * batch).astype(np.int32)
    else:
        batch_idx = np.zeros(0, np.int32)
    return Schedule(K, act_ptr, act_node, send_r, send_c, batch, batch_idx)


def realised_T_D(G_R: Graph, G_C: Graph, s: Schedule):
    """Realised constants of Assumption 3 in units of rounds: T = longest stretch
    of rounds in which some node stays inactive plus one; D = largest delay code."""
    n = G_R.n
    last = np.full(n, -1, dtype=np.int64)
    T = 0
    for r in range(s.K):
        a = s.act_node[s.act_ptr[r]:s.act_ptr[r + 1]]
        T = max(T, int((r - last[a]).max()) if len(a) else 0)
        last[a] = r
    T = max(T, int((s.K - 1 - last).max()) + 1) if s.K else 0
    D = int(max(s.send_r.max(initial=-1), s.send_c.max(initial=-1)))
    return T, D

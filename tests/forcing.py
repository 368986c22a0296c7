"""Teacher forcing: put the oracle's state at the start of a round into the engine, run that one
round on both sides from the same fp32 values, compare what the round produced.

A free trajectory lets two implementations drift apart along the iteration; a forced round shows
what one activation round does to identical inputs.  The oracle's state is first rounded to
fp32 (the engine's storage type) and BOTH sides start from those rounded values, so the
comparison sees one round of arithmetic and nothing else.

Test-side glue only: it moves arrays between the oracle's attributes and the C ABI's
rfast_seek / rfast_write_state / rfast_write_packet and holds none of the method's arithmetic.
"""

from __future__ import annotations

import numpy as np

from oracle import RFastOracle


def f32(a):
    """The fp32-representable value nearest to each entry, held in fp64."""
    return np.asarray(a, dtype=np.float64).astype(np.float32).astype(np.float64)


def rounded_clone(orc: RFastOracle) -> RFastOracle:
    """A second oracle in the same state with every float array rounded to fp32.  Shares the
    graphs and the gradient callable with the original; owns its state."""
    c = RFastOracle(orc.n, orc.p, orc.alpha, orc.R, orc.C, orc.grad, None, dtype=orc.dtype)
    c.x = [f32(a) for a in orc.x]
    c.z = [f32(a) for a in orc.z]
    c.g = [f32(a) for a in orc.g]
    c.t = list(orc.t)
    c.v_latest = [f32(a) for a in orc.v_latest]
    c.tau_v = list(orc.tau_v)
    c.v_recv = [f32(a) for a in orc.v_recv]
    c.inbox_v = [[(a, s, f32(pl)) for (a, s, pl) in box] for box in orc.inbox_v]
    c.rho = [f32(a) for a in orc.rho]
    c.tau_rho = list(orc.tau_rho)
    c.rho_recv = [f32(a) for a in orc.rho_recv]
    c.rho_tilde = [f32(a) for a in orc.rho_tilde]
    c.inbox_rho = [[(a, s, f32(pl)) for (a, s, pl) in box] for box in orc.inbox_rho]
    c.round, c.activations = orc.round, orc.activations
    return c


def known_packets(orc: RFastOracle):
    """Every packet payload the oracle still knows, keyed the way the C ABI addresses versions:
    (0, sender node, stamp) for v, (1, G_C edge id, stamp) for rho.  Sources: the packets in the
    inboxes, the newest packet received per in-edge, the senders' latest running sums and v."""
    pk = {}
    for e in range(len(orc.R.col)):
        j = int(orc.R.col[e])
        if orc.tau_v[e] >= 1:
            pk[(0, j, orc.tau_v[e])] = orc.v_recv[e]
        for (_, s, pl) in orc.inbox_v[e]:
            pk[(0, j, s)] = pl
    for j in range(orc.n):
        if orc.t[j] >= 1:
            pk[(0, j, orc.t[j])] = orc.v_latest[j]
    for e in range(len(orc.C.col)):
        j = int(orc.C.col[e])
        if orc.tau_rho[e] >= 1:
            pk[(1, e, orc.tau_rho[e])] = orc.rho_recv[e]
        for (_, s, pl) in orc.inbox_rho[e]:
            pk[(1, e, s)] = pl
        if orc.t[j] >= 1:
            pk[(1, e, orc.t[j])] = orc.rho[e]
    return pk


def load_into_engine(eng, orc: RFastOracle, has_gradient_view=True, packets=True):
    """Engine := the oracle's state as of the start of round orc.round.  Returns the number of
    packet versions written (those the engine keeps a row for)."""
    from paper_2307_11617_b200 import binding as B
    eng.seek(orc.round)
    eng.write(B.STATE_X, orc.X())
    eng.write(B.STATE_Y, orc.Z())
    if has_gradient_view:
        eng.write(B.STATE_G_LAST, orc.G())
    written = 0
    if packets:
        for (graph, ident, stamp), payload in known_packets(orc).items():
            written += bool(eng.write_packet(graph, ident, stamp, payload))
    return written


def row_errors(got, ref, floor):
    """Per-row relative L2 error (denominator floored at `floor`, an L2 norm; scalar or one per
    row) and per-row max-abs error relative to the row's largest reference magnitude (floored at
    the magnitude a row of norm `floor` has: four times its root mean square)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    d = got - ref
    l2 = np.linalg.norm(d, axis=1) / np.maximum(np.linalg.norm(ref, axis=1), floor)
    mx = np.abs(d).max(axis=1) / np.maximum(np.abs(ref).max(axis=1), 4.0 * np.asarray(floor) / np.sqrt(ref.shape[1]))
    return l2, mx


def assert_per_node(got, ref, grad, tol, what):
    """Row by row, so that one wrong node or a wrong ragged tail cannot hide in a norm over the
    whole state: relative L2 of every node's row and its largest element error.  A row is
    measured against its own norm, floored at the norm of an average row (a node whose row has
    all but vanished is held to the state's scale) and, for the tracker, at 1/20 of the node's
    gradient norm (fp32 operands of S2b carry their own rounding; a tracker far smaller than
    the gradient it is a difference of cannot be resolved below ~5e-7 of that gradient)."""
    ref = np.asarray(ref, dtype=np.float64)
    n, p = ref.shape
    floor = np.full(n, np.linalg.norm(ref) / np.sqrt(n))
    if grad is not None:
        floor = np.maximum(floor, 0.05 * np.linalg.norm(np.asarray(grad, dtype=np.float64), axis=1))
    d = np.asarray(got, dtype=np.float64) - ref
    l2 = np.linalg.norm(d, axis=1) / np.maximum(np.maximum(np.linalg.norm(ref, axis=1), floor), 1e-300)
    mx = np.abs(d).max(axis=1) / np.maximum(np.maximum(np.abs(ref).max(axis=1), 4.0 * floor / np.sqrt(p)), 1e-300)
    assert l2.max() <= tol, (what, "worst node rel-L2", float(l2.max()), int(l2.argmax()))
    assert mx.max() <= 10 * tol, (what, "worst node max-abs", float(mx.max()), int(mx.argmax()))

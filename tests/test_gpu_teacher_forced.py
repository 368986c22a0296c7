"""Teacher-forced parity: one activation round from the oracle's own state, through the C ABI.

At chosen rounds the oracle's state (x, z, remembered gradients, running sums, buffers, every
packet in flight) is rounded to fp32 and loaded into the engine with rfast_seek /
rfast_write_state / rfast_write_packet; the engine runs that one round; a clone of the oracle
runs it from the same rounded values.  Whatever differs afterwards is that round's arithmetic:
nothing has had time to drift.  The bar is 1e-5 relative L2 PER NODE (every active node's row of
x, y, g and the running sums it pushed), plus a max-abs bound, so a single wrong row or a wrong
ragged tail cannot hide in a norm over the whole state.

Denominator of a tracker row: S2b forms y_i from z_i, the news and g_new - g_old, and every fp32
operand carries its own rounding (a few 6e-8 of ITS magnitude), so a tracker that has become
small next to the gradient it is a difference of (most of the mass in transit under heavy
loss) cannot be resolved better than ~5e-7 |g_i| in absolute terms by any fp32 evaluation.
A row of y is therefore measured against max(|y_i|, |g_i| / 20).
"""

from __future__ import annotations

import numpy as np
import pytest

from forcing import known_packets, load_into_engine, rounded_clone, row_errors
from oracle import from_workload, make_model, run_schedule
from workloads import build_config

pytestmark = pytest.mark.gpu

TOL = 1e-5

CASES = [
    ("quad_tree64", dict(n=16, p=70_001, K=24), 5, "quad tiles+tail"),
    ("quad_tree64", dict(n=64, p=4099, K=60, drop=0.6, max_delay=8), 11, "quad heavy loss"),
    ("ls_ring4", {}, 37, "least squares as stated"),
    ("softmax_exp16", dict(F=96, C=7, rows=64, K=90, batch=8), 17, "reduced softmax"),
    ("logistic_tree1024", dict(n=96, p=5000, rows=8, K=50, batch=4, nnz=50), 9, "reduced sparse logistic"),
]


def _init_oracle(wl):
    orc = from_workload(wl, make_model(wl).grad)
    Bs, s = wl.batch, wl.schedule
    orc.init_gradients([s.batch_idx[i * Bs:(i + 1) * Bs] for i in range(wl.n)] if Bs else None)
    return orc


def _active(s, r):
    return [int(i) for i in s.act_node[s.act_ptr[r]:s.act_ptr[r + 1]]]


def _assert_rows(got, ref, floor, what, tol=TOL):
    l2, mx = row_errors(got, ref, floor)
    assert l2.max() <= tol, (what, "row rel-L2", float(l2.max()), int(l2.argmax()))
    assert mx.max() <= 10 * tol, (what, "row max-abs", float(mx.max()), int(mx.argmax()))


@pytest.mark.parametrize("name,ov,every,why", CASES, ids=[c[3] for c in CASES])
def test_forced_round_matches_oracle_per_node(rfast_lib, name, ov, every, why):
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config(name, seed=3, **ov)
    s = wl.schedule
    orc = _init_oracle(wl)
    quad = wl.model == "quad_diag"
    zfl = 1e-3 * np.linalg.norm(orc.Z()) / np.sqrt(wl.n)
    xfl = max(1e-3 * np.linalg.norm(orc.X()) / np.sqrt(wl.n), 1e-30)
    out_C = orc.out_C
    checked = 0
    with pkg.Engine(wl) as eng:
        eng.load_schedule(s)
        for r in range(s.K):
            if r % every == 0 or r == s.K - 1:
                c = rounded_clone(orc)
                pk = known_packets(c)
                load_into_engine(eng, c, not quad)
                # integer state follows from the schedule and the round
                assert eng.read(B.STATE_T_LOCAL).tolist() == c.t
                assert eng.read(B.STATE_TAU_V).tolist() == c.tau_v
                assert eng.read(B.STATE_TAU_RHO).tolist() == c.tau_rho
                # every version the engine holds is one the oracle still knows, with that payload
                for j in range(wl.n):
                    for st in range(1, c.t[j] + 1):
                        got = eng.read_packet(B.GRAPH_R, j, st)
                        if got is not None:
                            assert (0, j, st) in pk, ("engine holds a v version the oracle has dropped", j, st)
                            assert np.array_equal(got, pk[(0, j, st)].astype(np.float32))
                for e in range(len(wl.G_C.col)):
                    for st in range(1, c.t[int(wl.G_C.col[e])] + 1):
                        got = eng.read_packet(B.GRAPH_C, e, st)
                        if got is not None:
                            assert (1, e, st) in pk, ("engine holds a rho version the oracle has dropped", e, st)
                            assert np.array_equal(got, pk[(1, e, st)].astype(np.float32))
                held = eng.read(B.STATE_V_HELD)
                vl = eng.read(B.STATE_V_LATEST)
                for j in range(wl.n):
                    assert held[j] in (0, c.t[j])
                    if held[j]:
                        assert np.array_equal(vl[j], c.v_latest[j].astype(np.float32))
                    else:
                        assert not vl[j].any()
                eng.run(1)
                run_schedule(c, s, K=r + 1)
                act = _active(s, r)
                ina = [i for i in range(wl.n) if i not in act]
                x, y = eng.read(B.STATE_X), eng.read(B.STATE_Y)
                # rows of inactive nodes are untouched, bit for bit
                assert np.array_equal(x[ina], c.X()[ina].astype(np.float32))
                assert np.array_equal(y[ina], c.Z()[ina].astype(np.float32))
                if act:
                    _assert_rows(x[act], c.X()[act], xfl, "x")
                    yfl = np.maximum(zfl, 0.05 * np.linalg.norm(c.G()[act], axis=1))
                    _assert_rows(y[act], c.Z()[act], yfl, "y")
                    _assert_rows(eng.read(B.STATE_G_LAST)[act], c.G()[act], zfl, "g")
                    edges = [f for i in act for f in out_C[i]]
                    if edges:
                        _assert_rows(eng.read(B.STATE_RHO_LATEST)[edges], c.RHO()[edges], zfl, "rho")
                    checked += 1
            run_schedule(orc, s, K=r + 1)
    assert checked >= 3


def test_write_state_validation_and_round_trip(rfast_lib):
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    from paper_2307_11617_b200.binding import EINVAL, ESTATE, RFastError
    wl = build_config("softmax_exp16", seed=5, n=8, F=48, C=5, rows=64, K=30, batch=8, compensated=0)
    rng = np.random.default_rng(0)
    with pkg.Engine(wl) as eng:
        with pytest.raises(RFastError) as ei:
            eng.seek(3)
        assert ei.value.code == ESTATE
        eng.load_schedule(wl.schedule)
        eng.run(17)
        for view in (B.STATE_X, B.STATE_Y, B.STATE_G_LAST, B.STATE_RHO_LATEST, B.STATE_RHO_BUF, B.STATE_V_LATEST):
            before = eng.read(view)
            new = rng.standard_normal(before.shape).astype(np.float32)
            eng.write(view, new)
            after = eng.read(view)
            stored = np.abs(before).sum(axis=1) > 0 if view in (B.STATE_RHO_LATEST, B.STATE_RHO_BUF, B.STATE_V_LATEST) \
                else np.ones(len(before), bool)
            if view == B.STATE_V_LATEST:
                stored = eng.read(B.STATE_V_HELD) > 0
            assert np.array_equal(after[stored], new[stored]), view
            assert not after[~stored].any(), view
            eng.write(view, before)
            assert np.array_equal(eng.read(view), before)
        with pytest.raises(RFastError) as ei:
            eng.write(B.STATE_T_LOCAL, np.zeros(wl.n, np.float32))
        assert ei.value.code == EINVAL
        with pytest.raises(RFastError) as ei:
            eng.write(B.STATE_X, np.zeros((wl.n, wl.p - 1), np.float32))
        assert ei.value.code == EINVAL
        with pytest.raises(RFastError) as ei:
            eng.seek(wl.schedule.K + 1)
        assert ei.value.code == EINVAL
        assert eng.read_packet(B.GRAPH_R, 0, 10_000) is None
        with pytest.raises(RFastError):
            eng.read_packet(B.GRAPH_R, wl.n, 1)
        # seek is the counter only: the state written back above continues bit for bit
        eng.run(5)
        x22 = eng.read(B.STATE_X)
        eng.seek(17)
        assert eng.query(B.Q_ROUND) == 17
        eng.reset()
        eng.run(22)
        assert np.array_equal(eng.read(B.STATE_X), x22)

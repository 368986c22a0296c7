"""Checkpoint / resume and the on-device diagnostics (auxiliary entry points)."""

from __future__ import annotations

import numpy as np
import pytest

from oracle import from_workload, make_model, run_schedule
from workloads import build_config

pytestmark = pytest.mark.gpu

CASES = [
    ("quad_tree64", dict(n=16, p=3000, K=30)),
    ("softmax_exp16", dict(F=40, C=5, rows=32, K=40, batch=8)),          # two-float tracker
    ("ls_ring4", dict(K=60)),                                            # two-float tracker and running sums
    ("logistic_tree1024", dict(n=48, p=2500, rows=8, K=30, batch=4, nnz=30)),
    ("mlp_tree64", dict(n=5, F=64, H=128, C=4, rows=96, K=12, batch=64)),
]


@pytest.mark.parametrize("name,ov", CASES, ids=[c[0] for c in CASES])
def test_resume_from_checkpoint_is_bit_identical(rfast_lib, name, ov):
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config(name, seed=8, **ov)
    K, r = wl.schedule.K, wl.schedule.K // 3
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        eng.run(r)
        blob = eng.checkpoint()
        eng.run(K - r)
        x1, y1, g1 = eng.read(B.STATE_X), eng.read(B.STATE_Y), eng.read(B.STATE_G_LAST)
        rl1 = eng.read(B.STATE_RHO_LATEST)
    with pkg.Engine(wl) as eng:                      # a fresh handle, as after a restart
        eng.load_schedule(wl.schedule)
        eng.restore(blob)
        assert eng.query(B.Q_ROUND) == r
        eng.run(K - r)
        assert np.array_equal(x1, eng.read(B.STATE_X)) and np.array_equal(y1, eng.read(B.STATE_Y))
        assert np.array_equal(g1, eng.read(B.STATE_G_LAST))
        assert np.array_equal(rl1, eng.read(B.STATE_RHO_LATEST))


def test_checkpoint_of_another_schedule_is_refused(rfast_lib):
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200.binding import EINVAL, ESTATE, RFastError
    wl = build_config("quad_tree64", seed=8, n=8, p=100, K=10)
    other = build_config("quad_tree64", seed=9, n=8, p=100, K=10)
    with pkg.Engine(wl) as eng:
        with pytest.raises(RFastError) as ei:
            eng.checkpoint()                         # nothing loaded yet
        assert ei.value.code == ESTATE
        eng.load_schedule(wl.schedule)
        eng.run(4)
        blob = eng.checkpoint()
        eng.load_schedule(other.schedule)
        try:
            eng.restore(blob)
            raised = None
        except RFastError as e:
            raised = e
        assert raised is not None and raised.code == EINVAL


DIAG_CASES = CASES[:4] + [("mlp_tree64", dict(n=5, F=64, H=128, C=4, rows=128, K=12, batch=64))]


@pytest.mark.parametrize("name,ov", DIAG_CASES, ids=[c[0] for c in DIAG_CASES])
def test_diagnostics_match_the_oracle_state(rfast_lib, name, ov):
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config(name, seed=8, **ov)
    orc = from_workload(wl, make_model(wl).grad)
    run_schedule(orc, wl.schedule)
    X, Z, G = orc.X(), orc.Z(), orc.G()
    xbar = X.mean(axis=0)
    want = {"consensus_error": np.linalg.norm(X - xbar), "xbar_norm": np.linalg.norm(xbar),
            "gradient_sum_max": np.abs(G.sum(axis=0)).max(), "tracker_norm": np.linalg.norm(Z)}
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        d0 = eng.diagnostics()
        assert d0["conservation_residual"] <= 1e-6 * max(d0["gradient_sum_max"], 1e-30)   # z^0 = g^0
        eng.run(wl.schedule.K // 2)
        eng.diagnostics()                            # in mid-run: must leave no trace in the state
        eng.run()
        x_end, y_end = eng.read(B.STATE_X), eng.read(B.STATE_Y)
        d = eng.diagnostics()
        assert np.array_equal(x_end, eng.read(B.STATE_X)) and np.array_equal(y_end, eng.read(B.STATE_Y))
    with pkg.Engine(wl) as eng:                      # the same run without any diagnostics call
        eng.load_schedule(wl.schedule)
        eng.run()
        assert np.array_equal(x_end, eng.read(B.STATE_X)) and np.array_equal(y_end, eng.read(B.STATE_Y))
    # merit function of the non-convex analysis: the full gradient of F = sum_i f_i (every row
    # of every shard) at the mean iterate, from the oracle's own models
    m = make_model(wl)
    if wl.model in ("quad_diag", "least_squares"):
        gF = sum(m.grad(i, xbar, None) for i in range(wl.n))
        want["full_gradient_norm"] = np.linalg.norm(gF)
        want["merit"] = np.linalg.norm(gF) ** 2 + np.linalg.norm(X - xbar) ** 2
        want["objective"] = sum(m.loss(i, xbar, None) for i in range(wl.n))    # F(xbar) of eq. (1)
    else:
        # sampled objectives: every row of every shard, in shard order
        gF = sum(m.grad(i, xbar, np.arange(wl.rows)) for i in range(wl.n))
        want["full_gradient_norm"] = np.linalg.norm(gF)
        want["merit"] = np.linalg.norm(gF) ** 2 + np.linalg.norm(X - xbar) ** 2
        want["objective"] = sum(m.loss(i, xbar, np.arange(wl.rows)) for i in range(wl.n))
    for key, w in want.items():
        assert abs(d[key] - w) <= 1e-4 * max(w, 1e-6), (key, d[key], w)
    # Lemma 3 on the device state, relative to the gradients that are summed
    scale = np.abs(G).sum(axis=0).max()
    assert d["conservation_residual"] <= 1e-5 * scale


def test_bounded_barrier_wait_reports_timeout_and_the_handle_recovers(rfast_lib):
    """Failure detection without faulting the GPU: the persistent kernel's grid barrier is told
    (on the host) to expect an arrival that nobody makes; its bounded wait runs out, the kernel
    returns, the next synchronising call reports RFAST_ETIMEOUT, and after a reset the same
    handle runs the schedule correctly."""
    import time
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    from paper_2307_11617_b200.binding import ETIMEOUT, RFastError
    wl = build_config("ls_ring4", seed=2)
    orc = from_workload(wl, make_model(wl).grad)
    run_schedule(orc, wl.schedule)
    with pkg.Engine(wl) as eng:
        eng.set_option(B.OPT_PERSISTENT, 1)
        eng.set_option(B.OPT_WAIT_LIMIT_MS, 200)
        eng.set_option(B.OPT_PHANTOM_ARRIVALS, 1)
        eng.load_schedule(wl.schedule)
        t0 = time.time()
        with pytest.raises(RFastError) as ei:
            eng.run()
        assert ei.value.code == ETIMEOUT and time.time() - t0 < 5.0
        eng.set_option(B.OPT_PHANTOM_ARRIVALS, 0)
        eng.reset()
        # the reset has cleared the timeout: the state can be read before anything runs again
        assert np.array_equal(eng.read(B.STATE_X), np.zeros((wl.n, wl.p), np.float32) if wl.x0 is None else wl.x0)
        eng.run()
        x = eng.read(B.STATE_X)
    assert np.linalg.norm(x - orc.X()) <= 1e-5 * np.linalg.norm(orc.X())


def test_bounded_copy_wait_of_the_one_pass_kernel_reports_timeout_and_recovers(rfast_lib):
    """The same for the sparse-logistic cluster kernel: its mbarrier is told (on the host) to
    expect bytes that no copy delivers; every CTA's bounded wait runs out, the CTAs still meet
    at their cluster barriers and return, the next synchronising call reports RFAST_ETIMEOUT,
    and after a reset the same handle runs the schedule correctly.  Nothing faults or hangs."""
    import time
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    from paper_2307_11617_b200.binding import ETIMEOUT, RFastError
    wl = build_config("logistic_tree1024", seed=2, n=24, p=9000, rows=8, K=6, batch=4, nnz=60)
    orc = from_workload(wl, make_model(wl).grad)
    Bs, s = wl.batch, wl.schedule
    orc.init_gradients([s.batch_idx[i * Bs:(i + 1) * Bs] for i in range(wl.n)])
    run_schedule(orc, s)
    with pkg.Engine(wl) as eng:
        eng.set_option(B.OPT_CLUSTER_SIZE, 2)
        eng.set_option(B.OPT_WAIT_LIMIT_MS, 100)
        eng.set_option(B.OPT_PHANTOM_ARRIVALS, 1)
        eng.load_schedule(s)
        t0 = time.time()
        with pytest.raises(RFastError) as ei:
            eng.run(1)
        assert ei.value.code == ETIMEOUT and time.time() - t0 < 10.0
        eng.set_option(B.OPT_PHANTOM_ARRIVALS, 0)
        eng.reset()
        eng.run()
        x = eng.read(B.STATE_X)
    assert np.linalg.norm(x - orc.X()) <= 1e-5 * np.linalg.norm(orc.X())


def test_snapshot_equals_read_state_and_survives_what_follows(rfast_lib):
    """rfast_snapshot: x and y as of the call, delivered while the handle already does other work."""
    import torch
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config("quad_tree64", seed=8, n=16, p=70_001, K=30)
    xs = [torch.empty((wl.n, wl.p), dtype=torch.float32, pin_memory=True).numpy() for _ in range(2)]
    ys = [torch.empty((wl.n, wl.p), dtype=torch.float32, pin_memory=True).numpy() for _ in range(2)]
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        eng.run(11)
        x11, y11 = eng.read(B.STATE_X), eng.read(B.STATE_Y)
        eng.snapshot(xs[0], ys[0])
        eng.run(sync=False)                          # the state moves on at once
        eng.snapshot(xs[1], ys[1])                   # queues behind the first
        eng.load_schedule(wl.schedule)               # a new pass starts; the snapshots are not disturbed
        eng.run(5)
        eng.snapshot_wait()
        assert np.array_equal(xs[0], x11) and np.array_equal(ys[0], y11)
        eng.reset()
        eng.run()
        assert np.array_equal(xs[1], eng.read(B.STATE_X)) and np.array_equal(ys[1], eng.read(B.STATE_Y))
        with pytest.raises(ValueError):
            eng.snapshot(xs[0][:, :-1], ys[0])

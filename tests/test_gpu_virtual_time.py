"""Synchronous push-pull against R-FAST in simulated time, on the same engine.

The paper's headline (Section VI-B, Table I) is that with one slow node the synchronous methods
pay the straggler's compute time in every iteration while R-FAST does not: it reports a
three-fold shorter training time than Ring-AllReduce.  Here both modes are schedules for the
same kernels.  Time unit: one compute time of a normal node.
  asynchronous: a node activates again one unit after it finished (the straggler after four);
                packets are delayed 0-2 rounds and 10 % are lost; a round lasts one unit.
  synchronous:  the special case of Remark 1 (everybody active, nothing delayed or lost); every
                round waits for the straggler, so it lasts four units.
The check is on the shape of the claim, not on the paper's numbers (other model, other data)."""

from __future__ import annotations

import numpy as np
import pytest

from oracle import from_workload, make_model, rel_l2, run_schedule
from workloads import activation_all, activation_durations, build_config, make_schedule

pytestmark = pytest.mark.gpu


def test_async_beats_sync_in_virtual_time_with_a_straggler(rfast_lib):
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config("softmax_exp16", seed=0, F=64, C=10, rows=256, K=10, batch=32)
    model = make_model(wl)
    n, straggler, slow, T = wl.n, 3, 4, 800
    rng = np.random.default_rng(1)
    acts = activation_durations(n, T, lambda i, t: slow if i == straggler else 1)
    s_async = make_schedule(wl.G_R, wl.G_C, acts, 0.1, 2, rng, batch=32, rows_per_node=wl.rows)
    s_sync = make_schedule(wl.G_R, wl.G_C, activation_all(n, T // slow), 0.0, 0, rng, batch=32,
                           rows_per_node=wl.rows)

    def global_loss(X):                       # F at the network average, full shards
        xbar = X.astype(np.float64).mean(axis=0)
        return sum(model.loss(i, xbar, np.arange(wl.rows)) for i in range(n)) / n

    curves = {}
    for name, sch, unit, every in (("async", s_async, 1, 50), ("sync", s_sync, slow, 25)):
        wl.schedule = sch
        orc = from_workload(wl, model.grad)
        run_schedule(orc, sch)
        with pkg.Engine(wl) as eng:
            eng.load_schedule(sch)
            curve = []
            for r in range(0, sch.K, every):
                eng.run(every)
                curve.append(((r + every) * unit, global_loss(eng.read(B.STATE_X))))
                on_device = eng.diagnostics()["objective"] / n          # the same curve without leaving the GPU
                assert abs(on_device - curve[-1][1]) <= 1e-5 * abs(curve[-1][1])
            assert rel_l2(eng.read(B.STATE_X), orc.X()) <= 1e-5       # both modes in parity with the oracle
            d = eng.diagnostics()
        curves[name] = curve
        assert d["conservation_residual"] <= 1e-5 * max(d["gradient_sum_max"], d["tracker_norm"])
    sync_final = curves["sync"][-1][1]
    assert curves["async"][-1][1] < sync_final                         # better at equal simulated time
    t_reach = next(t for t, loss in curves["async"] if loss <= sync_final)
    assert t_reach <= T / 2, (t_reach, curves)                          # and at least twice as fast to that loss


def test_async_beats_sync_on_the_full_size_mlp_with_heavy_tailed_compute_times(rfast_lib):
    """The same claim on the non-convex objective at the benchmarked size (n = 64, MLP 784-512-10,
    lognormal compute times): no oracle is needed, the loss curve F(xbar) comes from the device.
    A synchronous iteration lasts as long as its slowest node's compute time (the maximum of 64
    lognormal draws); R-FAST nodes go on at their own pace, with delays and losses."""
    import copy
    import paper_2307_11617_b200 as pkg
    wl = build_config("mlp_tree64", seed=0)
    n, T = wl.n, wl.schedule.K                                         # one round = one time unit
    rng = np.random.default_rng(7)
    dur = np.maximum(1, np.rint(np.exp(rng.standard_normal((T, n))))).max(axis=1)
    end = np.cumsum(dur)                                               # when each synchronous iteration is through
    k_sync = int((end <= T).sum())
    s_sync = make_schedule(wl.G_R, wl.G_C, activation_all(n, k_sync), 0.0, 0, rng, batch=wl.batch, rows_per_node=wl.rows)
    curves = {}
    for name, sch, every in (("async", wl.schedule, 25), ("sync", s_sync, 5)):
        w = copy.copy(wl)
        w.schedule = sch
        with pkg.Engine(w) as eng:
            eng.load_schedule(sch)
            f0 = eng.diagnostics()["objective"] / n
            curve = []
            for r in range(0, sch.K, every):
                eng.run(min(every, sch.K - r))
                rr = min(r + every, sch.K)
                d = eng.diagnostics()
                curve.append((float(rr) if name == "async" else float(end[rr - 1]), d["objective"] / n))
                assert d["conservation_residual"] <= 1e-5 * max(d["gradient_sum_max"], d["tracker_norm"])
        curves[name] = curve
        assert curve[-1][1] < f0
    sync_final = curves["sync"][-1][1]
    assert curves["async"][-1][1] <= 0.1 * sync_final                   # far lower at equal simulated time
    t_reach = next(t for t, loss in curves["async"] if loss <= sync_final)
    assert t_reach <= T / 3, (t_reach, curves)                          # and at least three times as fast to that loss

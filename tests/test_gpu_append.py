"""Rounds handed to the engine a piece at a time (rfast_append_schedule): Algorithm 2 goes on
counting k, the state and the packets on their way carry over, and the result is, bit for bit,
that of the whole schedule loaded at once."""

from __future__ import annotations

import numpy as np
import pytest

from workloads import build_config, split_schedule

pytestmark = pytest.mark.gpu

CASES = [
    ("ls_ring4", {}, "least squares, two-float sums"),
    ("ls_ring4", dict(compensated=0), "least squares, plain fp32"),
    ("softmax_exp16", dict(F=96, C=7, rows=64, K=150, batch=8), "reduced softmax"),
    ("mlp_tree64", dict(n=12, rows=128, K=40), "MLP, twelve nodes"),
    ("quad_tree64", dict(n=64, p=4099, K=90, drop=0.5, max_delay=8), "quad heavy loss"),
    ("logistic_tree1024", dict(n=96, p=5000, rows=8, K=60, batch=4, nnz=50), "reduced sparse logistic"),
]

FLOAT_VIEWS = ("STATE_X", "STATE_Y", "STATE_RHO_LATEST", "STATE_RHO_BUF", "STATE_V_LATEST")
INT_VIEWS = ("STATE_T_LOCAL", "STATE_TAU_V", "STATE_TAU_RHO", "STATE_USED_TAU_V", "STATE_USED_TAU_RHO", "STATE_V_HELD")


def _views(eng, B, quad):
    out = {}
    for nm in FLOAT_VIEWS + INT_VIEWS + (() if quad else ("STATE_G_LAST",)):
        out[nm] = eng.read(getattr(B, nm))
    return out


@pytest.mark.parametrize("name,ov,why", CASES, ids=[c[2] for c in CASES])
def test_appended_rounds_give_the_whole_schedule_bit_for_bit(rfast_lib, name, ov, why):
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config(name, seed=4, **ov)
    s = wl.schedule
    quad = wl.model == "quad_diag"
    with pkg.Engine(wl) as eng:
        eng.load_schedule(s)
        eng.run()
        want = _views(eng, B, quad)
    cuts = [s.K // 4, s.K // 2 + 1]
    parts = split_schedule(s, wl.G_R, wl.G_C, cuts)
    with pkg.Engine(wl) as eng:
        eng.set_option(B.OPT_OPEN_END, 1)
        eng.load_schedule(parts[0])
        eng.run()
        assert eng.query(B.Q_ROUND) == cuts[0]
        eng.append_schedule(parts[1])
        assert eng.query(B.Q_ROUND) == cuts[0] and eng.query(B.Q_EVENTS_TOTAL) == parts[0].n_events + parts[1].n_events
        eng.run(3)                                   # the third piece arrives while the second is under way
        eng.append_schedule(parts[2])
        assert eng.query(B.Q_ROUND) == cuts[0] + 3
        eng.run()
        assert eng.query(B.Q_ROUND) == s.K
        got = _views(eng, B, quad)
        for nm, ref in want.items():
            if nm == "STATE_V_LATEST" or nm == "STATE_V_HELD":
                continue                             # an open end holds more of v than a closed one
            assert np.array_equal(got[nm], ref), nm
        # what the closed end still held of v, the open end holds too, with the same bits
        held = want["STATE_V_HELD"] > 0
        assert np.array_equal(got["STATE_V_HELD"][held], want["STATE_V_HELD"][held])
        assert np.array_equal(got["STATE_V_LATEST"][held], want["STATE_V_LATEST"][held])
        # a checkpoint taken after the appends goes back into the same handle
        blob = pkg.rfast_checkpoint_save(eng.h)
        eng.seek(s.K // 2)
        pkg.rfast_checkpoint_load(eng.h, blob)
        assert eng.query(B.Q_ROUND) == s.K
        assert np.array_equal(eng.read(B.STATE_X), want["STATE_X"])
        # and a reset starts the whole appended schedule over
        eng.reset()
        eng.run()
        assert np.array_equal(eng.read(B.STATE_X), want["STATE_X"])
        assert np.array_equal(eng.read(B.STATE_Y), want["STATE_Y"])


def test_append_with_step_sizes_on_one_part_only(rfast_lib):
    import copy
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config("softmax_exp16", seed=6, F=48, C=5, rows=64, K=80, batch=8)
    s = copy.copy(wl.schedule)
    alpha = np.full(s.K, wl.alpha, np.float32)
    alpha[50:] = np.float32(wl.alpha) * np.float32(0.5)        # the step decays in the appended rounds
    s.alpha_round = alpha
    with pkg.Engine(wl) as eng:
        eng.load_schedule(s)
        eng.run()
        want = eng.read(B.STATE_X), eng.read(B.STATE_Y)
    first, more = split_schedule(s, wl.G_R, wl.G_C, [50])
    first.alpha_round = None                                    # constant alpha: the problem's
    with pkg.Engine(wl) as eng:
        eng.set_option(B.OPT_OPEN_END, 1)
        eng.load_schedule(first)
        eng.run()
        eng.append_schedule(more)
        eng.run()
        assert np.array_equal(eng.read(B.STATE_X), want[0])
        assert np.array_equal(eng.read(B.STATE_Y), want[1])


def test_append_needs_an_open_end(rfast_lib):
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    from paper_2307_11617_b200.binding import EINVAL, ESCHED, ESTATE, RFastError
    wl = build_config("ls_ring4", seed=2)
    first, more = split_schedule(wl.schedule, wl.G_R, wl.G_C, [120])
    with pkg.Engine(wl) as eng:
        with pytest.raises(RFastError) as ei:
            eng.append_schedule(more)                           # nothing loaded
        assert ei.value.code == ESTATE
        eng.load_schedule(first)
        with pytest.raises(RFastError) as ei:
            eng.append_schedule(more)                           # loaded with a closed end
        assert ei.value.code == ESTATE
        with pytest.raises(RFastError) as ei:
            eng.set_option(B.OPT_OPEN_END, 1)                   # too late: a schedule is loaded
        assert ei.value.code == ESTATE
        eng.run()                                               # the handle is as it was
        x = eng.read(B.STATE_X)
    with pkg.Engine(wl) as eng:
        eng.set_option(B.OPT_OPEN_END, 1)
        eng.load_schedule(first)
        eng.run()
        assert np.array_equal(eng.read(B.STATE_X), x)           # the option changes no value
        bad = split_schedule(wl.schedule, wl.G_R, wl.G_C, [120])[1]
        bad.send_r = bad.send_r[:-1]
        with pytest.raises(RFastError) as ei:
            eng.append_schedule(bad)
        assert ei.value.code == ESCHED
        assert eng.query(B.Q_ROUND) == 120 and np.array_equal(eng.read(B.STATE_X), x)   # nothing changed
        eng.append_schedule(more)
        eng.run()
        assert eng.query(B.Q_ROUND) == wl.schedule.K
    wlb = build_config("ls_ring4", seed=2, tracker=1)
    with pkg.Engine(wlb) as eng:
        with pytest.raises(RFastError) as ei:
            eng.set_option(B.OPT_OPEN_END, 1)                   # mass buckets lump what a later round would split
        assert ei.value.code == EINVAL


def test_append_with_empty_parts(rfast_lib):
    """Degenerate pieces: nothing loaded at first (K = 0), an empty piece in the middle, an empty
    piece at the end; the result is still the whole schedule's, bit for bit."""
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config("softmax_exp16", seed=9, F=48, C=5, rows=64, K=60, batch=8)
    s = wl.schedule
    with pkg.Engine(wl) as eng:
        eng.load_schedule(s)
        eng.run()
        want = eng.read(B.STATE_X), eng.read(B.STATE_Y), eng.read(B.STATE_RHO_LATEST)
    parts = split_schedule(s, wl.G_R, wl.G_C, [0, 25, 25, s.K])
    assert [p.K for p in parts] == [0, 25, 0, s.K - 25, 0]
    with pkg.Engine(wl) as eng:
        eng.set_option(B.OPT_OPEN_END, 1)
        eng.load_schedule(parts[0])
        x0 = eng.read(B.STATE_X)
        eng.run()                                            # nothing to run yet
        assert eng.query(B.Q_ROUND) == 0 and np.array_equal(eng.read(B.STATE_X), x0)
        for part in parts[1:]:
            eng.append_schedule(part)
            eng.run()
        assert eng.query(B.Q_ROUND) == s.K
        assert np.array_equal(eng.read(B.STATE_X), want[0]) and np.array_equal(eng.read(B.STATE_Y), want[1])
        assert np.array_equal(eng.read(B.STATE_RHO_LATEST), want[2])


@pytest.mark.parametrize("name,ov", [("quad_tree64", dict(n=12, p=5003, K=60)),
                                     ("softmax_exp16", dict(n=12, F=40, C=5, rows=32, K=60, batch=8))],
                         ids=["quad", "softmax"])
def test_append_on_general_digraphs(rfast_lib, name, ov):
    """Several in- and out-neighbours per node in both graphs, heavy loss and delays up to six
    rounds: many packets are on their way or waiting in an inbox when a piece ends."""
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    from workloads import activation_bernoulli, graph_from_edges, make_schedule
    wl = build_config(name, seed=21, **ov)
    rng = np.random.default_rng(22)
    n = wl.n

    def edges():
        e = {(i, (i + 1) % n) for i in range(n)}
        while len(e) < 3 * n:
            a, b = rng.integers(0, n, size=2)
            if a != b:
                e.add((int(a), int(b)))
        return e
    wl.G_R, wl.G_C = graph_from_edges(n, edges(), "row"), graph_from_edges(n, edges(), "col")
    s = make_schedule(wl.G_R, wl.G_C, activation_bernoulli(n, wl.schedule.K, 0.4, rng), 0.4, 6, rng,
                      batch=wl.batch, rows_per_node=wl.rows)
    wl.schedule = s
    with pkg.Engine(wl) as eng:
        eng.load_schedule(s)
        eng.run()
        want = {v: eng.read(getattr(B, v)) for v in ("STATE_X", "STATE_Y", "STATE_RHO_LATEST", "STATE_RHO_BUF", "STATE_TAU_V", "STATE_TAU_RHO")}
    cuts = [7, 8, 30, 47]
    parts = split_schedule(s, wl.G_R, wl.G_C, cuts)
    with pkg.Engine(wl) as eng:
        eng.set_option(B.OPT_OPEN_END, 1)
        eng.load_schedule(parts[0])
        for part in parts[1:]:
            eng.run()
            eng.append_schedule(part)
        eng.run()
        for v, ref in want.items():
            assert np.array_equal(eng.read(getattr(B, v)), ref), v

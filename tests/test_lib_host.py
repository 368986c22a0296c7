"""Host-side logic of the CUDA library, checked without a GPU: exported symbols, the schedule
compiler's integer artefacts against the oracle and against brute force, safety of the version
rows, input validation."""

from __future__ import annotations

import copy
import os
import re

import numpy as np
import pytest

from helpers import brute_force_stamps, out_edges
from oracle import from_workload, make_model, run_schedule
from workloads import build_config, graph_from_edges

CASES = [
    ("ls_ring4", {}),
    ("softmax_exp16", dict(F=12, C=4, rows=16, K=120, batch=4)),
    ("mlp_tree64", dict(F=10, H=6, C=3, rows=12, K=60, batch=4)),
    ("quad_tree64", dict(p=19, K=100)),
    ("logistic_tree1024", dict(n=150, p=300, rows=4, K=60, batch=2, nnz=6)),
]


def test_library_exports_every_declared_symbol(rfast_lib, repo_root):
    text = open(os.path.join(repo_root, "include", "rfast.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(rfast_[a-z_]+)\s*\(", text))
    assert {"rfast_create", "rfast_load_schedule", "rfast_run", "rfast_read_state"} <= names
    for nm in names:
        assert hasattr(rfast_lib, nm), nm


@pytest.mark.parametrize("name,ov", CASES)
def test_compiled_stamps_equal_oracle_and_brute_force(rfast_lib, name, ov):
    import paper_2307_11617_b200 as pkg
    wl = build_config(name, seed=2, **ov)
    r = pkg.rfast_compile_host(wl, wl.schedule)
    sv, _ = brute_force_stamps(wl.G_R, wl.schedule, wl.schedule.send_r)
    sr, _ = brute_force_stamps(wl.G_C, wl.schedule, wl.schedule.send_c)
    assert list(r["used_tau_v"]) == sv and list(r["used_tau_rho"]) == sr
    if name != "mlp_tree64":                          # the oracle's MLP is slow; stamps are value-free
        orc = from_workload(wl, make_model(wl).grad)
        run_schedule(orc, wl.schedule)
        assert list(r["used_tau_v"]) == orc.used_tau_v and list(r["used_tau_rho"]) == orc.used_tau_rho
    assert r["events"] == wl.schedule.n_events


@pytest.mark.parametrize("name,ov", CASES)
def test_version_rows_never_alias_a_live_version(rfast_lib, name, ov):
    """Two versions may share a row only if the first is dead before the second is written;
    every consumed version is alive, in its own row, when it is read."""
    import paper_2307_11617_b200 as pkg
    wl = build_config(name, seed=5, **ov)
    s = wl.schedule
    r = pkg.rfast_compile_host(wl, s)
    ev_round = np.repeat(np.arange(s.K), np.diff(s.act_ptr))
    # --- v versions: one per event
    v = r["v_ver"]
    assert (v[:, 1] == ev_round).all()
    by_row = {}
    for ev in np.argsort(v[:, 1], kind="stable"):
        row, wr, last = v[ev]
        if row < 0:
            continue
        assert 0 <= row < r["v_rows"] and last >= wr
        if row in by_row:
            assert by_row[row] < wr, "row reused while its version was still to be read"
        by_row[row] = last
    # --- rho versions: one per (event, out-edge in G_C)
    rho = r["rho_ver"]
    outC = out_edges(wl.G_C)
    edge_of, stamp_of = [], []
    t = [0] * wl.n
    for ev, i in enumerate(s.act_node):
        t[i] += 1
        for f in outC[i]:
            edge_of.append(f); stamp_of.append(t[i])
    assert len(edge_of) == len(rho)
    owner = {}
    for vid in np.argsort(rho[:, 1], kind="stable"):
        row, wr, last = rho[vid]
        assert 0 <= row < r["rho_rows"] and last >= wr
        if row in owner:
            pl, pe, ps = owner[row]
            in_place = (pe == edge_of[vid] and ps + 1 == stamp_of[vid] and pl == wr)
            assert pl < wr or in_place, "rho row reused while its version was still to be read"
        owner[row] = (last, edge_of[vid], stamp_of[vid])
    # --- every consumed version is inside its lifetime
    sv, _ = brute_force_stamps(wl.G_R, s, s.send_r)
    ev_of = [[] for _ in range(wl.n)]
    for ev, i in enumerate(s.act_node):
        ev_of[i].append(ev)
    k = 0
    for ev, i in enumerate(s.act_node):
        for e in range(wl.G_R.rowptr[i], wl.G_R.rowptr[i + 1]):
            tau = sv[k]; k += 1
            if tau >= 1:
                row, wr, last = v[ev_of[wl.G_R.col[e]][tau - 1]]
                assert row >= 0 and wr < ev_round[ev] <= last
    sr, _ = brute_force_stamps(wl.G_C, s, s.send_c)
    off = np.concatenate([[0], np.cumsum([len(outC[i]) for i in s.act_node])])
    pos = {f: k for i in range(wl.n) for k, f in enumerate(outC[i])}
    k = 0
    prev = [0] * wl.G_C.n_edges
    for ev, i in enumerate(s.act_node):
        for e in range(wl.G_C.rowptr[i], wl.G_C.rowptr[i + 1]):
            tau = sr[k]; k += 1
            if tau > prev[e]:
                for st in (tau, prev[e]):
                    if st >= 1:
                        row, wr, last = rho[off[ev_of[wl.G_C.col[e]][st - 1]] + pos[e]]
                        assert wr < ev_round[ev] <= last
                prev[e] = tau


def test_compile_rejects_bad_graphs_and_schedules(rfast_lib):
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200.binding import EGRAPH, ESCHED, RFastError
    wl = build_config("quad_tree64", n=8, p=5, K=10)
    bad = copy.deepcopy(wl)
    bad.G_R.w = bad.G_R.w * np.float32(0.9)                       # rows of W no longer sum to 1
    with pytest.raises(RFastError) as ei:
        pkg.rfast_compile_host(bad, bad.schedule)
    assert ei.value.code == EGRAPH and "Assumption 1" in str(ei.value)
    bad = copy.deepcopy(wl)
    bad.G_C.diag = bad.G_C.diag.copy(); bad.G_C.diag[3] = 0.0    # Assumption 1 i)
    with pytest.raises(RFastError) as ei:
        pkg.rfast_compile_host(bad, bad.schedule)
    assert ei.value.code == EGRAPH
    # no common root: G_R a chain 0->1->...; G_C pushes away from node 0
    n = 4
    bad = build_config("quad_tree64", n=n, p=5, K=10)
    bad.G_R = graph_from_edges(n, [(i, i + 1) for i in range(n - 1)], "row")
    bad.G_C = graph_from_edges(n, [(i, i + 1) for i in range(n - 1)], "col")
    with pytest.raises(RFastError) as ei:
        pkg.rfast_compile_host(bad, bad.schedule)
    assert ei.value.code == EGRAPH and "Assumption 2" in str(ei.value)
    for mutate in ("order", "code", "count", "node"):
        s = copy.deepcopy(wl.schedule)
        if mutate == "order":
            r = int(np.argmax(np.diff(s.act_ptr) >= 2)); a = s.act_ptr[r]
            s.act_node[a], s.act_node[a + 1] = s.act_node[a + 1], s.act_node[a]
        elif mutate == "code":
            s.send_c[0] = -2
        elif mutate == "count":
            s.send_r = s.send_r[:-1]
        else:
            s.act_node[0] = wl.n
        with pytest.raises(RFastError) as ei:
            pkg.rfast_compile_host(wl, s)
        assert ei.value.code == ESCHED, mutate


def test_create_fails_loudly_without_a_device(rfast_lib):
    from conftest import has_cuda
    if has_cuda():
        pytest.skip("a CUDA device is present")
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200.binding import ECUDA, RFastError
    wl = build_config("quad_tree64", n=4, p=5, K=3)
    with pytest.raises(RFastError) as ei:
        pkg.rfast_create(wl)
    assert ei.value.code == ECUDA


@pytest.mark.parametrize("name,ov", CASES)
def test_bucket_tracker_rows_hold_exactly_one_consumption(rfast_lib, name, ov):
    """Mass-bucket tracker: the contributions a receiver consumes together (sender stamps
    tau_prev < t <= tau_new, Algorithm 1 S2b) share one row from the first of them to the
    consumption and no other bucket uses that row meanwhile; what nobody consumes inside the
    schedule forms one last bucket per edge that is kept.  The stamps are the brute-force ones."""
    import paper_2307_11617_b200 as pkg
    wl = build_config(name, seed=5, tracker=1, **ov)
    s = wl.schedule
    r = pkg.rfast_compile_host(wl, s)
    ref = pkg.rfast_compile_host(build_config(name, seed=5, **ov), s)
    assert list(r["used_tau_rho"]) == list(ref["used_tau_rho"]) and list(r["used_tau_v"]) == list(ref["used_tau_v"])
    assert r["streams"] <= ref["streams"]
    rho = r["rho_ver"]
    ev_round = np.repeat(np.arange(s.K), np.diff(s.act_ptr))
    outC = out_edges(wl.G_C)
    off = np.concatenate([[0], np.cumsum([len(outC[i]) for i in s.act_node])])
    pos = {f: k for i in range(wl.n) for k, f in enumerate(outC[i])}
    ev_of = [[] for _ in range(wl.n)]
    for ev, i in enumerate(s.act_node):
        ev_of[i].append(ev)
    vid = lambda e, stamp: off[ev_of[wl.G_C.col[e]][stamp - 1]] + pos[e]
    sr, _ = brute_force_stamps(wl.G_C, s, s.send_c)
    INF = np.iinfo(np.int32).max
    buckets = []                                       # (row, first write round, consume round)
    k = 0
    prev = [0] * wl.G_C.n_edges
    for ev, i in enumerate(s.act_node):
        for e in range(wl.G_C.rowptr[i], wl.G_C.rowptr[i + 1]):
            tau = sr[k]; k += 1
            if tau > prev[e]:
                members = [vid(e, st) for st in range(prev[e] + 1, tau + 1)]
                rows = {int(rho[m][0]) for m in members}
                assert len(rows) == 1
                assert all(int(rho[m][2]) == ev_round[ev] for m in members)
                assert all(int(rho[m][1]) < ev_round[ev] for m in members)
                buckets.append((rows.pop(), int(rho[members[0]][1]), int(ev_round[ev])))
                prev[e] = tau
    t = [len(a) for a in ev_of]
    for e in range(wl.G_C.n_edges):
        j = int(wl.G_C.col[e])
        if t[j] > prev[e]:
            members = [vid(e, st) for st in range(prev[e] + 1, t[j] + 1)]
            rows = {int(rho[m][0]) for m in members}
            assert len(rows) == 1 and all(int(rho[m][2]) == INF for m in members)
            buckets.append((rows.pop(), int(rho[members[0]][1]), INF))
    assert sum(1 for _ in buckets) > 0
    by_row = {}
    for row, first, last in sorted(buckets, key=lambda b: b[1]):
        assert 0 <= row < r["rho_rows"]
        if row in by_row:
            assert by_row[row] < first, "bucket row reused before its consumption"
        by_row[row] = last


def test_threaded_descriptor_pass_equals_the_single_threaded_one(rfast_lib, monkeypatch):
    """Schedules of 50,000 events and more have their device descriptors filled in by several
    host threads, each on a span of rounds.  Everything the kernels are driven by must come out
    the same as from one thread (digest over descriptors, row lists, weights, byte counts), for
    the running sums and for the bucket tracker, on a general digraph."""
    import paper_2307_11617_b200 as pkg
    from workloads import activation_bernoulli, graph_from_edges, make_schedule
    wl = build_config("quad_tree64", seed=3, n=48, p=8, K=4)
    rng = np.random.default_rng(5)
    n = wl.n
    edges = {(i, (i + 1) % n) for i in range(n)} | {(int(a), int(b)) for a, b in rng.integers(0, n, size=(3 * n, 2)) if a != b}
    wl.G_R, wl.G_C = graph_from_edges(n, edges, "row"), graph_from_edges(n, edges, "col")
    sch = make_schedule(wl.G_R, wl.G_C, activation_bernoulli(n, 2400, 0.5, rng), 0.2, 4, rng, batch=0)
    assert sch.n_events >= 50_000
    for tracker in (0, 1):
        wl.tracker = tracker
        monkeypatch.setenv("RFAST_COMPILE_THREADS", "1")
        one = pkg.rfast_compile_digest(wl, sch)
        monkeypatch.setenv("RFAST_COMPILE_THREADS", "8")
        many = pkg.rfast_compile_digest(wl, sch)
        monkeypatch.delenv("RFAST_COMPILE_THREADS")
        assert one == many == pkg.rfast_compile_digest(wl, sch)
    # and the digest does see a difference: another schedule, another number
    other = make_schedule(wl.G_R, wl.G_C, activation_bernoulli(n, 2400, 0.5, rng), 0.2, 4, rng, batch=0)
    assert pkg.rfast_compile_digest(wl, other) != many


@pytest.mark.parametrize("name,ov", CASES)
def test_appended_rounds_move_no_row_and_consume_the_same_stamps(rfast_lib, name, ov):
    """Rounds handed over a piece at a time (Algorithm 2 goes on counting k): compiled open-ended
    and then extended, the rounds of the first piece keep every version row, row list and event
    descriptor, and the stamps consumed are those of the whole schedule compiled in one piece."""
    import paper_2307_11617_b200 as pkg
    from workloads import split_schedule
    wl = build_config(name, seed=11, **ov)
    s = wl.schedule
    for cut in sorted({1, s.K // 3, s.K // 2, s.K - 1} - {0, s.K}):
        first, more = split_schedule(s, wl.G_R, wl.G_C, [cut])
        assert first.K + more.K == s.K and first.n_events + more.n_events == s.n_events
        r = pkg.rfast_compile_append_check(wl, first, more)
        # an open end keeps more alive than a closed one; the pools only ever grow
        assert r["appended"][0] >= r["first"][0] and r["appended"][1] >= r["first"][1]
        assert r["appended"][0] >= r["whole"][0] and r["appended"][1] >= r["whole"][1]


def test_append_check_rejects_inconsistent_parts(rfast_lib):
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200.binding import ESCHED, RFastError
    from workloads import split_schedule
    wl = build_config("ls_ring4", seed=1)
    first, more = split_schedule(wl.schedule, wl.G_R, wl.G_C, [50])
    bad = copy.copy(more)
    bad.send_c = more.send_c[:-1]
    with pytest.raises(RFastError) as ei:
        pkg.rfast_compile_append_check(wl, first, bad)
    assert ei.value.code == ESCHED
    bad = copy.copy(more)
    bad.act_ptr = more.act_ptr + 1
    with pytest.raises(RFastError) as ei:
        pkg.rfast_compile_append_check(wl, first, bad)
    assert ei.value.code == ESCHED
    wlb = build_config("ls_ring4", seed=1, tracker=1)     # mass buckets: no appending
    with pytest.raises(RFastError) as ei:
        pkg.rfast_compile_append_check(wlb, first, more)
    assert ei.value.code == ESCHED


@pytest.mark.parametrize("seed", range(6))
def test_append_check_on_random_general_digraphs(rfast_lib, seed):
    """Ring plus random chords in both graphs, heavy loss, delays up to 9 rounds, sparse
    activations (packets wait in inboxes for many rounds), several random cuts: the rows of the
    loaded rounds never move and the consumed stamps are the whole schedule's."""
    import paper_2307_11617_b200 as pkg
    from workloads import activation_bernoulli, make_schedule, split_schedule
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(3, 14))
    wl = build_config("quad_tree64", seed=seed, n=n, p=8, K=10)

    def edges():
        e = {(i, (i + 1) % n) for i in range(n)}
        while len(e) < n + int(rng.integers(0, 2 * n)):
            a, b = rng.integers(0, n, size=2)
            if a != b:
                e.add((int(a), int(b)))
        return e
    wl.G_R, wl.G_C = graph_from_edges(n, edges(), "row"), graph_from_edges(n, edges(), "col")
    K = int(rng.integers(20, 90))
    s = make_schedule(wl.G_R, wl.G_C, activation_bernoulli(n, K, float(rng.uniform(0.15, 0.9)), rng),
                      float(rng.uniform(0.0, 0.7)), int(rng.integers(0, 10)), rng)
    sv, _ = brute_force_stamps(wl.G_R, s, s.send_r)
    assert list(pkg.rfast_compile_host(wl, s)["used_tau_v"]) == sv
    for cut in sorted(set(int(c) for c in rng.integers(0, K + 1, size=4))):
        first, more = split_schedule(s, wl.G_R, wl.G_C, [cut])
        pkg.rfast_compile_append_check(wl, first, more)

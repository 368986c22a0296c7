"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same seeded inputs.

Bar: integer artefacts (consumed stamps, counters) bit-exact; x and y within 1e-5 relative L2
after K rounds, the denominator floored at 1e-3 of the reference's initial norm."""

from __future__ import annotations

import numpy as np
import pytest

from conftest import has_cuda
from forcing import assert_per_node as _per_node
from oracle import from_workload, make_model, rel_l2, run_schedule
from workloads import build_config

pytestmark = pytest.mark.gpu

TOL = 1e-5

# sizes the oracle finishes in seconds, spanning several tiles and a ragged tail
CASES = [
    ("quad_tree64", dict(n=16, p=70_001, K=30), "tiles+tail"),
    ("quad_tree64", dict(n=64, p=3, K=100), "tiny p"),
    ("quad_tree64", dict(n=1, p=33, K=5), "single node"),
    ("quad_tree64", dict(n=64, p=4099, K=100, drop=0.6, max_delay=8), "heavy loss"),
    ("quad_tree64", dict(n=32, p=2048, K=60, drop=0.0, max_delay=0), "no loss no delay"),
    ("ls_ring4", {}, "config 1 as stated"),
    ("softmax_exp16", dict(F=96, C=7, rows=64, K=150, batch=8), "reduced softmax"),
    ("logistic_tree1024", dict(n=96, p=5000, rows=8, K=60, batch=4, nnz=50), "reduced sparse logistic"),
]


def _oracle(wl, K=None):
    orc = from_workload(wl, make_model(wl).grad)
    B = wl.batch
    zeta0 = [wl.schedule.batch_idx[i * B:(i + 1) * B] for i in range(wl.n)] if B else None
    orc.init_gradients(zeta0)
    ref0 = (np.linalg.norm(orc.X()), np.linalg.norm(orc.Z()))
    run_schedule(orc, wl.schedule, K=K)
    return orc, ref0


def _compare(eng, orc, ref0, tol=TOL, node_tol=None):
    from paper_2307_11617_b200 import binding as B
    x, y = eng.read(B.STATE_X), eng.read(B.STATE_Y)
    assert np.isfinite(x).all() and np.isfinite(y).all()
    ex, ey = rel_l2(x, orc.X(), ref0[0]), rel_l2(y, orc.Z(), ref0[1])
    assert ex <= tol and ey <= tol, (ex, ey)
    _per_node(x, orc.X(), None, node_tol or tol, "x")
    _per_node(y, orc.Z(), orc.G(), node_tol or tol, "y")
    g = eng.read(B.STATE_G_LAST)
    assert rel_l2(g, orc.G(), ref0[1]) <= 10 * tol
    if len(orc.rho):
        rl, rb = eng.read(B.STATE_RHO_LATEST), eng.read(B.STATE_RHO_BUF)
        scale = max(np.linalg.norm(orc.RHO()), ref0[1])
        assert np.linalg.norm(rl - orc.RHO()) <= 10 * tol * scale
        assert np.linalg.norm(rb - orc.RHO_TILDE()) <= 10 * tol * scale
    return ex, ey


@pytest.mark.parametrize("name,ov,why", CASES, ids=[c[2] for c in CASES])
def test_parity_after_K_rounds(rfast_lib, name, ov, why):
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config(name, seed=1, **ov)
    orc, ref0 = _oracle(wl)
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        eng.run()
        _compare(eng, orc, ref0)
        # integers: bit-exact
        assert eng.read(B.STATE_USED_TAU_V).tolist() == orc.used_tau_v
        assert eng.read(B.STATE_USED_TAU_RHO).tolist() == orc.used_tau_rho
        assert eng.read(B.STATE_T_LOCAL).tolist() == orc.t
        assert eng.read(B.STATE_TAU_V_END).tolist() == orc.tau_v
        assert eng.read(B.STATE_TAU_RHO_END).tolist() == orc.tau_rho
        assert eng.read(B.STATE_ROUND)[0] == wl.schedule.K
        assert eng.query(B.Q_EVENTS_RUN) == orc.activations
        assert eng.query(B.Q_LAUNCHES) > 0


def test_parity_round_by_round_and_reset(rfast_lib):
    """Stepping one round at a time gives the same state as one call, and reset + rerun is
    bit-identical (no atomics, fixed summation order)."""
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config("quad_tree64", seed=7, n=16, p=1500, K=25)
    orc = from_workload(wl, make_model(wl).grad)
    orc.init_gradients()
    ref0 = (1.0, np.linalg.norm(orc.Z()))
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        for r in range(wl.schedule.K):
            eng.run(1)
            run_schedule(orc, wl.schedule, K=r + 1)
            if r % 6 == 0 or r == wl.schedule.K - 1:
                _compare(eng, orc, ref0)
                assert eng.read(B.STATE_T_LOCAL).tolist() == orc.t
        x1, y1 = eng.read(B.STATE_X), eng.read(B.STATE_Y)
        eng.reset()
        assert eng.query(B.Q_ROUND) == 0
        eng.run()
        assert np.array_equal(x1, eng.read(B.STATE_X)) and np.array_equal(y1, eng.read(B.STATE_Y))


@pytest.mark.parametrize("level", [0, 1, 2], ids=["plain", "two-float tracker", "two-float tracker and sums"])
@pytest.mark.parametrize("name,ov", [
    ("quad_tree64", dict(n=32, p=4099, K=80, drop=0.4)),
    ("quad_tree64", dict(n=16, p=70_001, K=30)),
    ("ls_ring4", {}),
    ("logistic_tree1024", dict(n=96, p=5000, rows=8, K=60, batch=4, nnz=50)),
    ("softmax_exp16", dict(F=96, C=7, rows=64, K=150, batch=8)),
], ids=["quad", "quad tiles", "ls", "logistic", "softmax"])
def test_parity_in_every_tracker_arithmetic(rfast_lib, name, ov, level):
    """Every objective in each of the three tracker arithmetics (plain fp32; tracker as two
    floats with error feedback; running sums as two floats as well)."""
    import paper_2307_11617_b200 as pkg
    wl = build_config(name, seed=2, **ov)
    wl.compensated = level
    orc, ref0 = _oracle(wl)
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        eng.run()
        # fp32 running sums keep growing while the trackers do not: at levels 0 and 1 a receiver
        # sees its in-neighbours' mass at the resolution of ulp(rho), which on the four-node
        # least-squares problem (trackers several times smaller than the local gradients) costs a
        # single node up to ~1.5e-5 of its tracker while the state as a whole stays inside 1e-5
        _compare(eng, orc, ref0, node_tol=3e-5 if (name == "ls_ring4" and level < 2) else None)
        d = eng.diagnostics()
    if level == 2:                                   # Lemma 3 then holds to double-float accuracy
        assert d["conservation_residual"] <= 1e-9 * max(d["gradient_sum_max"], d["tracker_norm"])


def test_conservation_on_the_device_state(rfast_lib):
    """Lemma 3 on what the GPU holds: trackers plus undelivered mass equal the sum of the
    latest gradients, up to fp32 rounding of the running sums."""
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config("quad_tree64", seed=3, n=32, p=999, K=80, drop=0.4)
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        eng.run()
        y, g = eng.read(B.STATE_Y).astype(np.float64), eng.read(B.STATE_G_LAST).astype(np.float64)
        rl, rb = eng.read(B.STATE_RHO_LATEST).astype(np.float64), eng.read(B.STATE_RHO_BUF).astype(np.float64)
    res = y.sum(axis=0) + (rl - rb).sum(axis=0) - g.sum(axis=0)
    scale = np.abs(g).sum(axis=0).max()
    assert np.abs(res).max() <= 1e-5 * scale


@pytest.mark.parametrize("name,ov", [("quad_tree64", dict(n=16, p=3000, K=40)),
                                     ("softmax_exp16", dict(F=40, C=5, rows=32, K=60, batch=8))],
                         ids=["quad", "softmax"])
def test_time_varying_step_size(rfast_lib, name, ov):
    """A per-round step size (step decay, as in the paper's ResNet schedule) on both sides."""
    import paper_2307_11617_b200 as pkg
    wl = build_config(name, seed=6, **ov)
    K = wl.schedule.K
    wl.schedule.alpha_round = (0.02 * 0.1 ** (np.arange(K) // (K // 3 + 1))).astype(np.float32)
    orc, ref0 = _oracle(wl)
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        eng.run()
        _compare(eng, orc, ref0)
    wl.schedule.alpha_round = None                 # and it really was used
    orc2, _ = _oracle(wl)
    assert rel_l2(orc2.X(), orc.X()) > 1e-3


def test_parity_under_acknowledgement_gated_loss(rfast_lib):
    """The paper's own packet-loss emulation (send only after the last packet was acknowledged)."""
    import paper_2307_11617_b200 as pkg
    from workloads import activation_bernoulli, make_schedule_ack_gated
    wl = build_config("quad_tree64", seed=4, n=32, p=2000, K=10)
    rng = np.random.default_rng(4)
    wl.schedule = make_schedule_ack_gated(wl.G_R, wl.G_C, activation_bernoulli(wl.n, 80, 0.5, rng), 4, rng)
    orc, ref0 = _oracle(wl)
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        eng.run()
        _compare(eng, orc, ref0)
        from paper_2307_11617_b200 import binding as B
        assert eng.read(B.STATE_USED_TAU_RHO).tolist() == orc.used_tau_rho


def test_run_past_the_schedule_is_refused(rfast_lib):
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200.binding import ESTATE, RFastError
    wl = build_config("quad_tree64", n=4, p=8, K=3)
    with pkg.Engine(wl) as eng:
        with pytest.raises(RFastError) as ei:
            eng.run(1)                      # no schedule yet
        assert ei.value.code == ESTATE
        eng.load_schedule(wl.schedule)
        eng.run(3)
        with pytest.raises(RFastError) as ei:
            eng.run(1)
        assert ei.value.code == ESTATE


def test_empty_rounds_and_x0(rfast_lib):
    """Rounds without any active node are legal; a non-zero x0 is honoured."""
    import paper_2307_11617_b200 as pkg
    wl = build_config("quad_tree64", seed=9, n=8, p=40, K=12)
    s = wl.schedule
    # empty out rounds 2 and 5 (their events and codes are removed consistently)
    from workloads import make_schedule
    acts = [s.act_node[s.act_ptr[r]:s.act_ptr[r + 1]] for r in range(s.K)]
    acts[2] = acts[2][:0]; acts[5] = acts[5][:0]
    rng = np.random.default_rng(0)
    wl.schedule = make_schedule(wl.G_R, wl.G_C, acts, 0.2, 3, rng)
    wl.x0 = rng.standard_normal((wl.n, wl.p)).astype(np.float32)
    orc, ref0 = _oracle(wl)
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        eng.run()
        _compare(eng, orc, ref0)


@pytest.mark.parametrize("name,ov", [
    ("quad_tree64", dict(n=16, p=5000, K=25)),
    ("softmax_exp16", dict(F=96, C=7, rows=64, K=60, batch=8)),
    ("logistic_tree1024", dict(n=64, p=3000, rows=8, K=30, batch=4, nnz=40)),
], ids=["quad", "softmax", "logistic"])
def test_graph_replay_on_a_user_stream_equals_direct_launches(rfast_lib, name, ov):
    """On a non-default stream a span of rounds is recorded into a CUDA graph and replayed
    after a reset; both must be bit-identical to direct launches on the default stream."""
    import torch
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config(name, seed=5, **ov)
    orc, ref0 = _oracle(wl)
    with pkg.Engine(wl) as eng:                      # default stream: direct launches
        eng.load_schedule(wl.schedule)
        eng.run()
        xd, yd = eng.read(B.STATE_X), eng.read(B.STATE_Y)
        direct_launches = eng.query(B.Q_LAUNCHES)
    stream = torch.cuda.Stream()
    with pkg.Engine(wl, stream.cuda_stream) as eng:
        eng.load_schedule(wl.schedule)
        eng.run()                                    # records and launches the graph
        _compare(eng, orc, ref0)
        x1, y1 = eng.read(B.STATE_X), eng.read(B.STATE_Y)
        assert eng.query(B.Q_LAUNCHES) == direct_launches
        eng.reset()
        eng.run()                                    # replays it
        x2, y2 = eng.read(B.STATE_X), eng.read(B.STATE_Y)
        assert eng.query(B.Q_LAUNCHES) == 2 * direct_launches
        eng.reset()
        eng.run(3)                                   # another span: re-recorded
        eng.run(wl.schedule.K - 3)
        x3 = eng.read(B.STATE_X)
    assert np.array_equal(xd, x1) and np.array_equal(yd, y1)
    assert np.array_equal(x1, x2) and np.array_equal(y1, y2) and np.array_equal(x1, x3)


@pytest.mark.parametrize("name,ov", [
    ("ls_ring4", {}),
    ("ls_ring4", dict(n=9, p=300, rows=40, K=60)),
    ("softmax_exp16", dict(F=96, C=7, rows=64, K=150, batch=8)),
    ("softmax_exp16", dict(F=96, C=7, rows=64, K=80, batch=8, compensated=False)),
    ("softmax_exp16", dict(n=8, F=784, C=10, rows=64, K=40, batch=32)),
], ids=["config 1", "ls wider", "softmax", "softmax plain", "softmax 784x10"])
def test_persistent_kernel_equals_one_kernel_per_phase(rfast_lib, name, ov):
    """L2-resident problems can run a span of rounds as one cooperative persistent kernel with
    bounded grid barriers (an option); by default, one kernel per phase.  Same bits, and parity
    with the oracle either way."""
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config(name, seed=3, **ov)
    orc, ref0 = _oracle(wl)
    res = {}
    for persistent in (1, 0):
        with pkg.Engine(wl) as eng:
            eng.set_option(B.OPT_PERSISTENT, persistent)
            eng.load_schedule(wl.schedule)
            l0 = eng.query(B.Q_LAUNCHES)             # the initial gradients are launched at load time
            eng.run(7)                               # spans of several lengths
            eng.run(1)
            eng.run()
            _compare(eng, orc, ref0)
            res[persistent] = (eng.read(B.STATE_X), eng.read(B.STATE_Y), eng.read(B.STATE_G_LAST),
                               eng.read(B.STATE_RHO_LATEST), eng.query(B.Q_LAUNCHES) - l0)
    for u, v in zip(res[1][:4], res[0][:4]):
        assert np.array_equal(u, v)
    assert res[1][4] == 3 and res[0][4] > 3 * 7       # one launch per span against several per round


def _general_digraphs(n, rng, extra):
    """Ring plus random chords: several in- and out-neighbours per node in both graphs, weights
    1/3, 1/4, ... that are not exact in binary."""
    from workloads import graph_from_edges
    def edges():
        e = {(i, (i + 1) % n) for i in range(n)}
        while len(e) < n + extra:
            a, b = rng.integers(0, n, size=2)
            if a != b:
                e.add((int(a), int(b)))
        return e
    return graph_from_edges(n, edges(), "row"), graph_from_edges(n, edges(), "col")


@pytest.mark.parametrize("name,ov,comp", [
    ("quad_tree64", dict(n=12, p=5003, K=50), False),
    ("quad_tree64", dict(n=12, p=5003, K=50), True),
    ("softmax_exp16", dict(n=12, F=40, C=5, rows=32, K=60, batch=8), True),
    ("logistic_tree1024", dict(n=12, p=3000, rows=8, K=50, batch=4, nnz=30), False),
], ids=["quad", "quad compensated", "softmax compensated", "logistic"])
def test_parity_on_general_digraphs(rfast_lib, name, ov, comp):
    """Not only trees and rings: several in-neighbours in G_R (S2a sums more than one packet),
    several in- and out-neighbours in G_C (S2b consumes several running sums, S2c feeds several)."""
    import paper_2307_11617_b200 as pkg
    from workloads import activation_bernoulli, make_schedule
    wl = build_config(name, seed=11, **ov)
    rng = np.random.default_rng(12)
    wl.G_R, wl.G_C = _general_digraphs(wl.n, rng, 2 * wl.n)
    assert np.diff(wl.G_R.rowptr).max() >= 3 and np.bincount(wl.G_C.col).max() >= 3
    wl.schedule = make_schedule(wl.G_R, wl.G_C, activation_bernoulli(wl.n, wl.schedule.K, 0.6, rng), 0.25, 3,
                                rng, batch=wl.batch, rows_per_node=wl.rows)
    wl.compensated = comp
    orc, ref0 = _oracle(wl)
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        eng.run()
        _compare(eng, orc, ref0)
        from paper_2307_11617_b200 import binding as B
        assert eng.read(B.STATE_USED_TAU_V).tolist() == orc.used_tau_v
        assert eng.read(B.STATE_USED_TAU_RHO).tolist() == orc.used_tau_rho
        d = eng.diagnostics()
    scale = np.abs(orc.G()).sum(axis=0).max()
    assert d["conservation_residual"] <= 2e-5 * scale


@pytest.mark.parametrize("name,ov", [
    ("logistic_tree1024", dict(n=28, p=9000, rows=8, K=40, batch=4, nnz=60)),
    ("softmax_exp16", dict(n=28, F=40, C=5, rows=32, K=40, batch=8)),
], ids=["logistic", "softmax"])
def test_parity_with_many_in_neighbours(rfast_lib, name, ov):
    """A hub: every node pushes to node 0 over G_C (in-degree n - 1 = 27 there, up to 27 rows of
    news in one activation -- more than the sparse-logistic pass lists for prefetching, which
    must not change what is summed) and pulls from node 0 over G_R, plus the ring so that
    other nodes have in- and out-neighbours too."""
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    from workloads import activation_bernoulli, graph_from_edges, make_schedule
    wl = build_config(name, seed=13, **ov)
    n = wl.n
    rng = np.random.default_rng(14)
    ring = {(i, (i + 1) % n) for i in range(n)}
    wl.G_R = graph_from_edges(n, ring | {(0, i) for i in range(1, n)}, "row")
    wl.G_C = graph_from_edges(n, ring | {(i, 0) for i in range(1, n)}, "col")
    wl.schedule = make_schedule(wl.G_R, wl.G_C, activation_bernoulli(n, wl.schedule.K, 0.7, rng), 0.1, 2,
                                rng, batch=wl.batch, rows_per_node=wl.rows)
    orc, ref0 = _oracle(wl)
    # the hub really consumes more than 16 newer running sums in one activation
    s, news = wl.schedule, 0
    used = np.asarray(orc.used_tau_rho)
    pos, last = 0, {}
    for ev in range(s.n_events):
        i = int(s.act_node[ev])
        deg = int(wl.G_C.rowptr[i + 1] - wl.G_C.rowptr[i])
        cur = used[pos:pos + deg]
        if i == 0:
            news = max(news, int((cur > last.get(0, np.zeros(deg, int))).sum()))
            last[0] = cur
        pos += deg
    assert news > 16, news
    with pkg.Engine(wl) as eng:
        eng.load_schedule(s)
        eng.run()
        _compare(eng, orc, ref0)
        assert eng.read(B.STATE_USED_TAU_RHO).tolist() == orc.used_tau_rho


@pytest.mark.parametrize("level", [0, 1, 2], ids=["plain", "two-float tracker", "two-float tracker and sums"])
@pytest.mark.parametrize("cluster", [-1, 1, 2, 4, 8], ids=["three kernels", "1 CTA", "2 CTAs", "4 CTAs", "8 CTAs"])
def test_sparse_logistic_one_pass_in_every_cluster_size(rfast_lib, cluster, level):
    """The sparse-logistic activation as one cluster per activation (slices of x and z kept in
    shared memory, partial dot products exchanged between the CTAs), in every cluster size, and
    the three-kernel path it replaces: each against the oracle, each bit-identical on a rerun.
    p = 9000 gives 18 ranges of 512 coordinates: ragged slices in every size, an empty slice never."""
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config("logistic_tree1024", seed=5, n=48, p=9000, rows=8, K=40, batch=4, nnz=60)
    wl.compensated = level
    orc, ref0 = _oracle(wl)
    with pkg.Engine(wl) as eng:
        if cluster < 0:
            eng.set_option(B.OPT_ONE_PASS, 0)
        else:
            eng.set_option(B.OPT_CLUSTER_SIZE, cluster)
        eng.load_schedule(wl.schedule)
        eng.run()
        _compare(eng, orc, ref0)
        x1, y1 = eng.read(B.STATE_X), eng.read(B.STATE_Y)
        assert eng.query(B.Q_BYTES_TOTAL) == eng.query(B.Q_METHOD_BYTES_TOTAL) + (0 if cluster >= 0 else 2 * 4 * wl.p * wl.schedule.n_events) \
            + 2 * min(level, 1) * 4 * wl.p * wl.schedule.n_events
        eng.reset()
        eng.run()
        assert np.array_equal(x1, eng.read(B.STATE_X)) and np.array_equal(y1, eng.read(B.STATE_Y))
        with pytest.raises(B.RFastError):                       # the byte accounting follows the option
            eng.set_option(B.OPT_ONE_PASS, 0)


def test_sparse_logistic_one_pass_with_an_empty_slice_and_a_large_batch(rfast_lib):
    """p = 1500 is three ranges: in a cluster of four the last CTA owns nothing and still meets
    its peers at the barriers; batch 40 makes a warp take more than one sampled row."""
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config("logistic_tree1024", seed=6, n=24, p=1500, rows=64, K=25, batch=40, nnz=30)
    orc, ref0 = _oracle(wl)
    with pkg.Engine(wl) as eng:
        eng.set_option(B.OPT_CLUSTER_SIZE, 4)
        eng.load_schedule(wl.schedule)
        eng.run()
        _compare(eng, orc, ref0)


@pytest.mark.parametrize("p,one_pass", [(200_003, True), (300_001, False)], ids=["1024-thread CTAs", "too large: three kernels"])
def test_sparse_logistic_large_dimension_paths(rfast_lib, p, one_pass):
    """p = 200,003 does not fit eight 512-thread CTAs (two per SM) any more and takes the
    1024-thread variant of the one-pass kernel (49 ranges per CTA, 200 KB of slices); p = 300,001
    does not fit a cluster of eight at all and falls back to three kernels per round.  Which path
    ran shows in the byte accounting."""
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config("logistic_tree1024", seed=7, n=8, p=p, rows=8, K=10, batch=4, nnz=300)
    orc, ref0 = _oracle(wl)
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        eng.run()
        _compare(eng, orc, ref0)
        extra = eng.query(B.Q_BYTES_TOTAL) - eng.query(B.Q_METHOD_BYTES_TOTAL)
        assert (extra == 0) == one_pass


def test_sparse_logistic_one_pass_with_more_entries_than_it_can_keep(rfast_lib):
    """The one-pass kernel keeps the sampled rows' entries of a slice in shared memory between the
    dot products and the gradient assembly, sized for 1.5 x the mean row; what does not fit is
    read from global memory again.  Here half of the nodes hold rows forty times denser than the
    other half, so their slices overflow the store and the second source is exercised."""
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config("logistic_tree1024", seed=9, n=8, p=9000, rows=8, K=30, batch=4, nnz=400)
    d = wl.data
    ptr, col, val = d["sp_rowptr"], d["sp_col"], d["sp_val"]
    keep = np.ones(len(col), bool)
    for r in range(4 * wl.rows):                              # nodes 0..3: ten entries per row
        keep[ptr[r] + 10:ptr[r + 1]] = False
    lens = np.array([keep[ptr[r]:ptr[r + 1]].sum() for r in range(len(ptr) - 1)])
    wl.data = dict(d, sp_rowptr=np.concatenate([[0], np.cumsum(lens)]).astype(np.int64), sp_col=col[keep], sp_val=val[keep])
    assert lens.max() >= 30 * lens.min()
    orc, ref0 = _oracle(wl)
    with pkg.Engine(wl) as eng:
        eng.set_option(B.OPT_CLUSTER_SIZE, 2)
        eng.load_schedule(wl.schedule)
        eng.run()
        _compare(eng, orc, ref0)
        assert eng.query(B.Q_BYTES_TOTAL) == eng.query(B.Q_METHOD_BYTES_TOTAL)     # the one-pass path ran


def test_coordinate_shards_reproduce_the_whole_bit_for_bit(rfast_lib):
    """The element-wise problem split by coordinate (what `bench.py --shard coords` gives each
    GPU) needs no exchange: three ragged slices run one after the other on this GPU give, side
    by side, exactly the state of the whole problem."""
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    from workloads import shard_coordinates
    wl = build_config("quad_tree64", seed=6, n=16, p=70_001, K=30)
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        eng.run()
        X, Y = eng.read(B.STATE_X), eng.read(B.STATE_Y)
    xs, ys = [], []
    for k in range(3):
        sub = shard_coordinates(wl, k, 3)
        with pkg.Engine(sub) as eng:
            eng.load_schedule(sub.schedule)
            eng.run()
            xs.append(eng.read(B.STATE_X)); ys.append(eng.read(B.STATE_Y))
    assert np.array_equal(np.concatenate(xs, axis=1), X)
    assert np.array_equal(np.concatenate(ys, axis=1), Y)

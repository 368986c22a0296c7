"""Sanity of the seeded input generators: Assumptions 1-2 on the graphs, schedule layout,
Assumption 3's realised constants, determinism in the seed (no GPU)."""

from __future__ import annotations

import numpy as np
import pytest

from workloads import CONFIG_NAMES, build_config, realised_T_D, sender_csr

SMALL = {
    "ls_ring4": {},
    "softmax_exp16": dict(F=12, C=4, rows=16, K=50, batch=4),
    "mlp_tree64": dict(F=10, H=6, C=3, rows=12, K=40, batch=4),
    "quad_tree64": dict(p=19, K=50),
    "logistic_tree1024": dict(n=200, p=300, rows=4, K=40, batch=2, nnz=6),
}


def _reach(n, edges_from, root):
    seen = {root}; todo = [root]
    while todo:
        u = todo.pop()
        for v in edges_from[u]:
            if v not in seen:
                seen.add(v); todo.append(v)
    return len(seen) == n


@pytest.mark.parametrize("name", CONFIG_NAMES)
def test_graphs_satisfy_assumptions(name):
    wl = build_config(name, **SMALL[name])
    W, A = wl.G_R.dense(), wl.G_C.dense()
    assert (np.diag(W) > 0).all() and (np.diag(A) > 0).all()            # Assumption 1 i)
    assert np.abs(W.sum(axis=1) - 1).max() < 1e-6                        # W row-stochastic
    assert np.abs(A.sum(axis=0) - 1).max() < 1e-6                        # A column-stochastic
    n = wl.n
    # Assumption 2: the root reaches everybody along G(W) edges (j -> i iff W_ij > 0) and along
    # G(A^T) edges (i -> j iff A_ij > 0)
    fw = [[i for i in range(n) if i != j and W[i, j] > 0] for j in range(n)]
    fa = [[j for j in range(n) if j != i and A[i, j] > 0] for i in range(n)]
    assert _reach(n, fw, wl.root) and _reach(n, fa, wl.root)
    for G in (wl.G_R, wl.G_C):
        for i in range(n):
            row = G.col[G.rowptr[i]:G.rowptr[i + 1]]
            assert (np.diff(row) > 0).all() and (row != i).all()


@pytest.mark.parametrize("name", CONFIG_NAMES)
def test_schedule_layout(name):
    wl = build_config(name, **SMALL[name])
    s = wl.schedule
    assert s.act_ptr[0] == 0 and s.act_ptr[-1] == len(s.act_node) and len(s.act_ptr) == s.K + 1
    for r in range(s.K):
        a = s.act_node[s.act_ptr[r]:s.act_ptr[r + 1]]
        assert len(a) >= 1 and (np.diff(a) > 0).all() and a.min() >= 0 and a.max() < wl.n
    od_r = np.diff(sender_csr(wl.G_R)[0]); od_c = np.diff(sender_csr(wl.G_C)[0])
    assert len(s.send_r) == od_r[s.act_node].sum() and len(s.send_c) == od_c[s.act_node].sum()
    assert s.send_r.min(initial=0) >= -1 and s.send_r.max(initial=0) <= wl.meta["max_delay"]
    assert len(s.batch_idx) == (wl.n + s.n_events) * s.batch
    if s.batch:
        assert s.batch_idx.min() >= 0 and s.batch_idx.max() < wl.rows
    T, D = realised_T_D(wl.G_R, wl.G_C, s)
    assert 1 <= T <= s.K and 0 <= D <= wl.meta["max_delay"]


def test_seed_determinism_and_sensitivity():
    a = build_config("quad_tree64", seed=0, p=8, K=20)
    b = build_config("quad_tree64", seed=0, p=8, K=20)
    c = build_config("quad_tree64", seed=1, p=8, K=20)
    assert np.array_equal(a.data["d"], b.data["d"]) and np.array_equal(a.schedule.send_c, b.schedule.send_c)
    assert not np.array_equal(a.data["d"], c.data["d"])


def test_full_size_shapes_of_the_small_configs():
    wl = build_config("ls_ring4")
    assert (wl.n, wl.p, wl.schedule.K) == (4, 10, 200) and wl.data["feat"].shape == (4, 50, 10)
    assert abs(wl.alpha - 0.01) < 1e-9
    wl = build_config("softmax_exp16", rows=8, K=3)
    assert (wl.n, wl.p, wl.batch) == (16, 7850, 32)
    wl = build_config("mlp_tree64", rows=4, K=2)
    assert (wl.n, wl.p, wl.batch) == (64, 407050, 64)
    wl = build_config("logistic_tree1024", p=1000, rows=2, K=2)
    assert wl.n == 1024 and np.bincount(wl.G_C.rowptr[1:] - wl.G_C.rowptr[:-1]).size <= 9


def test_ack_gated_schedule_never_has_two_unacknowledged_packets():
    """Section VI's packet-loss emulation: at most one packet per edge awaits its receiver."""
    from workloads import activation_bernoulli, make_schedule_ack_gated, ring_graphs
    from helpers import out_edges
    rng = np.random.default_rng(3)
    n, K = 6, 80
    G_R, G_C = ring_graphs(n)
    acts = activation_bernoulli(n, K, 0.5, rng)
    s = make_schedule_ack_gated(G_R, G_C, acts, 3, rng)
    assert (s.send_r == -1).any() and (s.send_r >= 0).any()
    out = out_edges(G_R)
    act_rounds = [[r for r in range(K) if i in acts[r]] for i in range(n)]
    pending = {}                                    # edge -> round at which its packet gets processed
    pos = 0
    for r in range(K):
        for i in acts[r]:
            for e in out[int(i)]:
                code = int(s.send_r[pos]); pos += 1
                if code >= 0:
                    assert e not in pending or pending[e] < r, "sent while the last packet was unprocessed"
                    recv = int(np.searchsorted(G_R.rowptr, e, side="right") - 1)
                    later = [q for q in act_rounds[recv] if q >= r + 1 + code]
                    pending[e] = later[0] if later else K + 1


def test_coordinate_shards_partition_the_problem_and_the_oracle_agrees():
    """The element-wise objective splits by coordinate with no exchange: the slices cover p
    exactly once, and the oracle run slice by slice equals the oracle run on the whole."""
    from oracle import from_workload, make_model, run_schedule
    from workloads import shard_coordinates
    wl = build_config("quad_tree64", seed=4, n=12, p=1003, K=25)
    parts = [shard_coordinates(wl, k, 7) for k in range(7)]
    spans = [q.meta["coordinates"] for q in parts]
    assert spans[0][0] == 0 and spans[-1][1] == wl.p
    assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
    assert max(hi - lo for lo, hi in spans) - min(hi - lo for lo, hi in spans) <= 1
    whole = from_workload(wl, make_model(wl).grad)
    whole.init_gradients()
    run_schedule(whole, wl.schedule)
    X, Z = [], []
    for q in parts:
        o = from_workload(q, make_model(q).grad)
        o.init_gradients()
        run_schedule(o, q.schedule)
        X.append(o.X()); Z.append(o.Z())
    assert np.array_equal(np.concatenate(X, axis=1), whole.X())
    assert np.array_equal(np.concatenate(Z, axis=1), whole.Z())
    with pytest.raises(ValueError):
        shard_coordinates(build_config("ls_ring4", seed=0), 0, 2)


def test_split_schedule_parts_tile_the_schedule():
    """Cutting a schedule into consecutive parts is array slicing only: laid end to end again
    (events renumbered, each part's copy of the initial samples dropped) the parts are the
    schedule."""
    import numpy as np
    from workloads import build_config, split_schedule
    wl = build_config("softmax_exp16", seed=3, F=12, C=4, rows=16, K=90, batch=4)
    s = wl.schedule
    parts = split_schedule(s, wl.G_R, wl.G_C, [7, 30, 31])
    assert [p.K for p in parts] == [7, 23, 1, 59]
    lead = wl.n * s.batch
    assert np.array_equal(np.concatenate([p.act_node for p in parts]), s.act_node)
    assert np.array_equal(np.concatenate([p.send_r for p in parts]), s.send_r)
    assert np.array_equal(np.concatenate([p.send_c for p in parts]), s.send_c)
    assert np.array_equal(np.concatenate([s.batch_idx[:lead]] + [p.batch_idx[lead:] for p in parts]), s.batch_idx)
    ev0 = 0
    for p in parts:
        assert p.act_ptr[0] == 0 and np.array_equal(p.batch_idx[:lead], s.batch_idx[:lead])
        ev0 += p.n_events
    assert ev0 == s.n_events

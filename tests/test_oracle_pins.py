"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU)."""

from __future__ import annotations

from fractions import Fraction

import numpy as np
import pytest

from helpers import FracGraph, brute_force_stamps, f64_weights, out_edges
from oracle import RFastOracle, from_workload, make_model, run_schedule
from oracle.models import QuadDiag, LeastSquares
from workloads import (activation_all, activation_bernoulli, activation_uniform_subset,
                       build_config, graph_from_edges, make_schedule, ring_graphs, tree_graphs,
                       binary_tree_parents)


def _rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def _general_graphs(n, rng):
    """A ring plus a few random chords: general digraphs, not only trees."""
    e = {(i, (i + 1) % n) for i in range(n)}
    for _ in range(n):
        a, b = rng.integers(0, n, size=2)
        if a != b:
            e.add((int(a), int(b)))
    e2 = {(i, (i + 1) % n) for i in range(n)}
    for _ in range(n):
        a, b = rng.integers(0, n, size=2)
        if a != b:
            e2.add((int(a), int(b)))
    return graph_from_edges(n, e, "row"), graph_from_edges(n, e2, "col")


# ---------------------------------------------------------------------------------------------
# P1  Lemma 3 (tracking conservation), exact in rational arithmetic
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_conservation_exact_rational(seed):
    rng = _rng(seed)
    n, p, K = 4, 3, 30
    G_R, G_C = _general_graphs(n, rng)
    sch = make_schedule(G_R, G_C, activation_uniform_subset(n, K, 1, n, rng), 0.35, 3, rng)
    FR, FC = FracGraph(G_R, "row"), FracGraph(G_C, "col")

    def frac_vec():
        return np.array([Fraction(int(rng.integers(-50, 51)), int(rng.integers(1, 17)))
                         for _ in range(p)], dtype=object)

    # an arbitrary "stochastic gradient": a fresh random rational vector at every call, so the
    # identity is exercised for any gradient sequence, as the lemma states
    def grad(i, x, idx):
        return frac_vec() + x * Fraction(1, 3)

    x0 = [frac_vec() for _ in range(n)]
    orc = RFastOracle(n, p, Fraction(1, 100), FR, FC, grad, x0=x0, dtype=object)
    seen = []

    def check(o, r):
        res = o.conservation_residual()
        assert all(c == 0 for c in res), f"round {r}: residual {res}"
        seen.append(r)

    run_schedule(orc, sch, after_round=check)
    assert len(seen) == K
    # the drops really happened and mass really sat on edges at some point
    assert (sch.send_c == -1).any()
    assert any(any(c != 0 for c in (orc.rho[e] - orc.rho_tilde[e])) for e in range(len(orc.rho)))


def test_conservation_negative_control_planted_sign_error():
    """A planted mistake in the oracle (buffer updated with the wrong packet) must break the
    identity: shows the check has teeth."""
    rng = _rng(5)
    n, p, K = 4, 3, 30
    G_R, G_C = _general_graphs(n, rng)
    sch = make_schedule(G_R, G_C, activation_uniform_subset(n, K, 1, n, rng), 0.3, 3, rng)
    FR, FC = FracGraph(G_R, "row"), FracGraph(G_C, "col")
    d = np.array([[Fraction(1 + i + c, 2) for c in range(p)] for i in range(n)], dtype=object)
    b = np.array([[Fraction(i - c, 3) for c in range(p)] for i in range(n)], dtype=object)

    class Broken(RFastOracle):
        def activate(self, i, r, cr, cc, idx):
            super().activate(i, r, cr, cc, idx)
            for e in range(int(self.C.rowptr[i]), int(self.C.rowptr[i + 1])):
                self.rho_tilde[e] = self.rho_tilde[e] * Fraction(1, 2)   # forgets half the buffer

    orc = Broken(n, p, Fraction(1, 50), FR, FC, QuadDiag(d, b).grad, dtype=object)
    run_schedule(orc, sch)
    assert any(c != 0 for c in orc.conservation_residual())


@pytest.mark.parametrize("name,ov", [
    ("ls_ring4", {}),
    ("softmax_exp16", dict(F=12, C=4, rows=16, K=40, batch=4)),
    ("mlp_tree64", dict(n=8, F=10, H=6, C=3, rows=12, K=30, batch=4)),
    ("quad_tree64", dict(n=16, p=37, K=40)),
    ("logistic_tree1024", dict(n=24, p=200, rows=8, K=40, batch=4, nnz=10)),
])
def test_conservation_fp64_all_models(name, ov):
    wl = build_config(name, seed=3, **ov)
    orc = from_workload(wl, make_model(wl).grad)
    worst = [0.0]

    def check(o, r):
        res = np.abs(o.conservation_residual()).max()
        scale = max(1.0, np.abs(o.G()).sum(axis=0).max())
        worst[0] = max(worst[0], res / scale)

    run_schedule(orc, wl.schedule, after_round=check)
    assert worst[0] < 1e-12, worst[0]


# ---------------------------------------------------------------------------------------------
# P2  Remark 1 / eq. (2): all active, no delay, no drop  ==  dense synchronous recursion
# ---------------------------------------------------------------------------------------------
def test_sync_reduction_dense_recursion():
    rng = _rng(11)
    n, p, K = 6, 5, 25
    G_R, G_C = _general_graphs(n, rng)
    W, A = G_R.dense(), G_C.dense()
    assert np.allclose(W.sum(axis=1), 1) and np.allclose(A.sum(axis=0), 1)
    d = rng.uniform(0.5, 2.0, (n, p)); b = rng.standard_normal((n, p))
    x0 = rng.standard_normal((n, p))
    alpha = 0.05
    sch = make_schedule(G_R, G_C, activation_all(n, K), 0.0, 0, rng)
    orc = RFastOracle(n, p, alpha, G_R, G_C, QuadDiag(d, b).grad, x0=x0)
    run_schedule(orc, sch)

    # dense recursion: tau = t for every edge, so the neighbour term is the previous v and the
    # own term is the fresh v; Y^t = z^{t+1/2} obeys eq. (2b): Y^t = A Y^{t-1} + G^{t+1} - G^t
    grad = lambda X: d * d * (X - b)
    dW, dA = np.diag(np.diag(W)), np.diag(np.diag(A))
    X = x0.copy(); G = grad(X); Z = G.copy(); Vprev = np.zeros((n, p)); Yprev = None
    for t in range(K):
        V = X - alpha * Z
        Xn = dW @ V + (W - dW) @ Vprev
        Gn = grad(Xn)
        Y = (Z + Gn - G) if Yprev is None else (A @ Yprev + Gn - G)
        Z = dA @ Y
        X, G, Vprev, Yprev = Xn, Gn, V, Y
    assert np.abs(orc.X() - X).max() <= 1e-12 * max(1, np.abs(X).max())
    assert np.abs(orc.Z() - Z).max() <= 1e-12 * max(1, np.abs(Z).max())


# ---------------------------------------------------------------------------------------------
# P4  n = 1: plain (stochastic) gradient descent
# ---------------------------------------------------------------------------------------------
def test_single_node_is_gradient_descent():
    rng = _rng(2)
    p, rows, K, alpha = 6, 20, 40, 0.05
    G_R = graph_from_edges(1, [], "row"); G_C = graph_from_edges(1, [], "col")
    feat = rng.standard_normal((1, rows, p)); target = rng.standard_normal((1, rows))
    x0 = rng.standard_normal((1, p))
    sch = make_schedule(G_R, G_C, activation_all(1, K), 0.0, 0, rng, batch=5, rows_per_node=rows)
    orc = RFastOracle(1, p, alpha, G_R, G_C, LeastSquares(feat, target, 0.01).grad, x0=x0)
    run_schedule(orc, sch)
    # x^{t+1} = x^t - alpha * grad f(x^t; zeta^t): the step uses the gradient remembered from the
    # previous activation (z = g when there is nobody to track with)
    x = x0[0].copy()
    for t in range(K):
        idx = sch.batch_idx[t * 5:(t + 1) * 5]      # sample t: entry 0 is zeta^0
        A, y = feat[0][idx], target[0][idx]
        x = x - alpha * (A.T @ (A @ x - y) / 5 + 0.01 * x)
    assert np.abs(orc.X()[0] - x).max() < 1e-13
    assert np.abs(orc.Z() - orc.G()).max() < 1e-13


# ---------------------------------------------------------------------------------------------
# P3 / P6 / P7  Theorem 1 with sigma = 0: geometric convergence to the closed-form optimum,
#               heterogeneous shards, with drops and delays; the increment-sending tracker fails
# ---------------------------------------------------------------------------------------------
def _ls_problem(seed, n=4, p=3, rows=8, shift=2.0):
    rng = _rng(seed)
    feat = rng.standard_normal((n, rows, p)) + shift * rng.standard_normal((n, 1, p))
    target = rng.standard_normal((n, rows)) + shift * np.arange(n)[:, None]
    H = sum(a.T @ a / rows for a in feat)
    c = sum(a.T @ y / rows for a, y in zip(feat, target))
    return feat, target, np.linalg.solve(H, c), np.linalg.eigvalsh(H).max()


@pytest.mark.parametrize("topology", ["ring", "tree"])
def test_geometric_convergence_to_least_squares_optimum(topology):
    n, p, K = 4, 3, 6000
    feat, target, xstar, L = _ls_problem(7)
    rng = _rng(8)
    if topology == "ring":
        G_R, G_C = ring_graphs(n)
    else:
        G_R, G_C = tree_graphs(binary_tree_parents(n), binary_tree_parents(n))
    sch = make_schedule(G_R, G_C, activation_bernoulli(n, K, 0.6, rng), 0.3, 3, rng)
    # ring: the trackers share the total gradient evenly, the effective step is alpha / n;
    # tree: the root's tracker carries the whole sum
    step = (1.5 if topology == "ring" else 0.3) / L
    orc = RFastOracle(n, p, step, G_R, G_C, LeastSquares(feat, target).grad)
    errs = []
    run_schedule(orc, sch, after_round=lambda o, r: errs.append(np.linalg.norm(o.X() - xstar)))
    errs = np.array(errs)
    assert errs[-1] <= 1e-10 * np.linalg.norm(xstar), errs[-1]
    # linear on a log plot: fit the decay before the rounding floor, residual of the fit small
    hi = int(np.argmax(errs < 1e-9)) if (errs < 1e-9).any() else K
    ks = np.arange(hi // 10, hi)
    slope, icpt = np.polyfit(ks, np.log(errs[ks]), 1)
    assert slope < 0
    assert np.abs(np.log(errs[ks]) - (slope * ks + icpt)).max() < 3.0   # within e^3 of a pure geometric decay over >9 decades


def test_increment_sending_tracker_misses_the_optimum():
    n, p, K = 4, 3, 6000
    feat, target, xstar, L = _ls_problem(7)
    rng = _rng(8)
    G_R, G_C = ring_graphs(n)
    sch = make_schedule(G_R, G_C, activation_bernoulli(n, K, 0.6, rng), 0.3, 3, rng)
    bad = RFastOracle(n, p, 1.5 / L, G_R, G_C, LeastSquares(feat, target).grad, increments_only=True)
    run_schedule(bad, sch)
    assert np.linalg.norm(bad.X() - xstar) > 1e-3 * np.linalg.norm(xstar)


# ---------------------------------------------------------------------------------------------
# Stamp semantics: the packet a receiver holds is the one with the largest stamp among those
# usable by now (brute force over all packets ever sent on the edge)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("seed", [0, 1])
def test_consumed_stamps_match_brute_force(seed):
    rng = _rng(seed)
    n, p, K = 7, 2, 60
    G_R, G_C = _general_graphs(n, rng)
    sch = make_schedule(G_R, G_C, activation_bernoulli(n, K, 0.5, rng), 0.25, 4, rng)
    d = rng.uniform(0.5, 2, (n, p)); b = rng.standard_normal((n, p))
    orc = RFastOracle(n, p, 0.01, G_R, G_C, QuadDiag(d, b).grad)
    run_schedule(orc, sch)
    sv, _ = brute_force_stamps(G_R, sch, sch.send_r)
    sr, _ = brute_force_stamps(G_C, sch, sch.send_c)
    assert orc.used_tau_v == sv
    assert orc.used_tau_rho == sr
    assert max(sv) > 1 and 0 in sv       # both "nothing yet" and overtaking occur


# ---------------------------------------------------------------------------------------------
# P5  Appendices E-F: the augmented systems as dense matrices, one active node per iteration
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("seed,multi", [(0, False), (1, False), (2, False), (3, True), (4, True)])
def test_augmented_systems_dense(seed, multi):
    """multi = False: one active node per round, Algorithm 2 as printed.  multi = True: rounds
    with several active nodes, checked against Algorithm 2 run once per member in ascending id
    (global iteration = event index): members of a round must not see each other's output, which
    in the global view is simply a larger delay."""
    rng = _rng(100 + seed)
    n, p, K = 4, 3, (10 if multi else 16)
    G_R, G_C = (f64_weights(g) for g in _general_graphs(n, rng))
    W, A = G_R.dense(), G_C.dense()
    if multi:
        act = activation_uniform_subset(n, K, 1, n, rng)
    else:
        act = [np.array([int(rng.integers(0, n))], dtype=np.int32) for _ in range(K)]
    sch = make_schedule(G_R, G_C, act, 0.3, 2, rng)
    d = rng.uniform(0.5, 2, (n, p)); b = rng.standard_normal((n, p)); x0 = rng.standard_normal((n, p))
    gamma = 0.03
    orc = RFastOracle(n, p, gamma, G_R, G_C, QuadDiag(d, b).grad, x0=x0)

    sv, _ = brute_force_stamps(G_R, sch, sch.send_r)
    sr, _ = brute_force_stamps(G_C, sch, sch.send_c)
    events = [(r, int(i)) for r in range(K) for i in act[r]]        # global iteration k = event index
    ev_idx = [[k for k, (_, i) in enumerate(events) if i == j] for j in range(n)]
    rounds_R = rounds_C = ev_idx
    D = len(events) + 1
    E = G_C.n_edges
    grad = lambda i, x: d[i] * d[i] * (x - b[i])

    h = np.zeros(((D + 2) * n, p)); h[:n] = x0
    S = n + (D + 1) * E
    zhat = np.zeros((S, p))
    g = np.stack([grad(i, x0[i]) for i in range(n)]); zhat[:n] = g
    pv = pr = 0
    outC = out_edges(G_C)
    snaps = []
    run_schedule(orc, sch, after_round=lambda o, r: snaps.append(
        (o.X().copy(), o.Z().copy(), o.RHO() - o.RHO_TILDE())))
    for k, (rnd, i) in enumerate(events):
        # delays in the global view: d = k - g(j, tau - 1) - 1; "nothing received yet" reads a
        # slot that still holds the zero initial value
        What = np.zeros(((D + 2) * n,) * 2)
        What[i, i] = W[i, i]
        for e in range(int(G_R.rowptr[i]), int(G_R.rowptr[i + 1])):
            j = int(G_R.col[e]); tau = sv[pv]; pv += 1
            if tau >= 1:
                dv = k - rounds_R[j][tau - 1] - 1
            else:
                first = next((r for r in rounds_R[j] if r < k), None)
                dv = 0 if first is None else k - first
            assert 0 <= dv <= D
            What[i, j + (dv + 1) * n] = W[i, j]
        for r_ in range(2 * n):
            if r_ not in (i, i + n):
                What[r_, r_] = 1
        for r_ in list(range(2 * n, (D + 2) * n)) + [i + n]:
            What[r_, r_ - n] = 1
        assert np.allclose(What.sum(axis=1), 1)
        hp = h.copy(); hp[i] -= gamma * zhat[i]
        x_old_i = h[i].copy()
        h = What @ hp
        eps = grad(i, h[i]) - grad(i, x_old_i)
        # sum step
        Sk = np.eye(S)
        for e in range(int(G_C.rowptr[i]), int(G_C.rowptr[i + 1])):
            j = int(G_C.col[e]); tau = sr[pr]; pr += 1
            drho = (k - rounds_C[j][tau - 1] - 1) if tau >= 1 else D
            assert 0 <= drho <= D
            for dd in range(drho, D + 1):
                m = n + dd * E + e
                Sk[m, m] = 0; Sk[i, m] = 1
        # push step
        Pk = np.zeros((S, S))
        Pk[i, i] = A[i, i]
        for f in outC[i]:
            recv = int(np.searchsorted(G_C.rowptr, f, side="right") - 1)
            Pk[n + 0 * E + f, i] = A[recv, i]
        for q in range(n):
            if q != i:
                Pk[q, q] = 1
        for e in range(E):
            for dd in range(D):
                Pk[n + (dd + 1) * E + e, n + dd * E + e] = 1
            Pk[n + D * E + e, n + D * E + e] = 1
        assert np.allclose(Pk.sum(axis=0), 1) and np.allclose(Sk.sum(axis=0), 1)
        zhalf = Sk @ zhat; zhalf[i] += eps
        zhat = Pk @ zhalf
        if k + 1 < len(events) and events[k + 1][0] == rnd:
            continue                                     # compare at the end of each round
        X, Z, M = snaps[rnd]
        assert np.abs(h[:n] - X).max() < 1e-12
        assert np.abs(zhat[:n] - Z).max() < 1e-12
        mass = zhat[n:].reshape(D + 1, E, p).sum(axis=0)
        assert np.abs(mass - M).max() < 1e-12
        assert np.abs(zhat.sum(axis=0) - np.stack(
            [grad(q, h[q]) for q in range(n)]).sum(axis=0)).max() < 1e-12   # Lemma 3 on the dense system


def test_time_varying_step_size_single_node():
    """gamma^t of Algorithm 1 S1 varying per round: n = 1 is gradient descent with that step sequence."""
    rng = _rng(21)
    p, rows, K = 5, 12, 30
    G_R = graph_from_edges(1, [], "row"); G_C = graph_from_edges(1, [], "col")
    feat = rng.standard_normal((1, rows, p)); target = rng.standard_normal((1, rows))
    x0 = rng.standard_normal((1, p))
    sch = make_schedule(G_R, G_C, activation_all(1, K), 0.0, 0, rng)
    sch.alpha_round = (0.1 * 0.5 ** (np.arange(K) // 10)).astype(np.float32)     # step decay
    orc = RFastOracle(1, p, 123.0, G_R, G_C, LeastSquares(feat, target).grad, x0=x0)
    run_schedule(orc, sch)
    x = x0[0].copy()
    for t in range(K):
        x = x - float(sch.alpha_round[t]) * (feat[0].T @ (feat[0] @ x - target[0]) / rows)
    assert np.abs(orc.X()[0] - x).max() < 1e-13


def test_convergence_under_acknowledgement_gated_loss():
    """Theorem 1 (sigma = 0) with the paper's own loss emulation instead of i.i.d. drops."""
    from workloads import make_schedule_ack_gated
    n, p, K = 4, 3, 20000
    feat, target, xstar, L = _ls_problem(7)
    rng = _rng(9)
    G_R, G_C = ring_graphs(n)
    sch = make_schedule_ack_gated(G_R, G_C, activation_bernoulli(n, K, 0.6, rng), 3, rng)
    assert (sch.send_c == -1).mean() > 0.2
    # three packets in four are discarded here, which lengthens the effective delays: smaller step
    orc = RFastOracle(n, p, 0.8 / L, G_R, G_C, LeastSquares(feat, target).grad)
    run_schedule(orc, sch)
    assert np.linalg.norm(orc.X() - xstar) <= 1e-8 * np.linalg.norm(xstar)
    # the identity of Lemma 3 holds to rounding of the running sums it is made of
    assert np.abs(orc.conservation_residual()).max() <= 1e-13 * max(1.0, np.abs(orc.RHO()).max()) * 100


def test_oracle_reproduces_its_frozen_output_on_config_1(repo_root):
    """Regression guard (not a pin by the paper, which prints no iterates): the stored output of
    tests/golden/make_golden.py, which calls only the oracle and the seeded generators."""
    import os
    gold = os.path.join(repo_root, "tests", "golden")
    wl = build_config("ls_ring4", seed=0)
    orc = from_workload(wl, make_model(wl).grad)
    run_schedule(orc, wl.schedule)
    x = np.loadtxt(os.path.join(gold, "ls_ring4_x_after_200_rounds.txt"))
    z = np.loadtxt(os.path.join(gold, "ls_ring4_z_after_200_rounds.txt"))
    st = np.loadtxt(os.path.join(gold, "ls_ring4_stamps.txt"), dtype=np.int64)
    assert np.abs(orc.X() - x).max() <= 1e-13 * np.abs(x).max()
    assert np.abs(orc.Z() - z).max() <= 1e-13 * np.abs(z).max()
    assert st.tolist() == orc.t + orc.tau_v + orc.tau_rho


def test_rel_l2_metric_known_vectors_and_floor():
    """The parity metric itself: ||a - ref||_F / max(||ref||_F, 1e-3 * ref0_norm)."""
    from oracle import rel_l2
    ref = np.array([[3.0, 4.0], [0.0, 0.0]])                     # Frobenius norm 5
    a = ref + np.array([[0.0, 0.0], [0.3, 0.4]])                  # error norm 0.5
    assert rel_l2(a, ref) == pytest.approx(0.1, rel=1e-15)
    assert rel_l2(ref, ref) == 0.0
    # the floor takes over once the reference has shrunk below 1e-3 of its initial norm
    tiny = ref * 1e-6                                             # norm 5e-6
    assert rel_l2(tiny + 1e-6, tiny, ref0_norm=100.0) == pytest.approx(2e-6 / 0.1, rel=1e-12)
    assert rel_l2(tiny + 1e-6, tiny, ref0_norm=1e-3) == pytest.approx(2e-6 / 5e-6, rel=1e-12)
    # a vanished reference without a floor does not divide by zero
    assert np.isfinite(rel_l2(np.ones(3), np.zeros(3)))
    # float32 input is measured in double
    assert rel_l2(np.float32([1.0, 1.0]), np.array([1.0, 1.0 + 1e-12])) == pytest.approx(1e-12 / np.sqrt(2.0 + 2e-12), rel=1e-3)

"""The mass-bucket tracker (the edge masses of the augmented system, Appendix F) against the
same oracle as the running sums of Algorithm 1: the two keep the same quantity, so x and y must
meet the same bar; the integer artefacts are those of the schedule and do not change."""

from __future__ import annotations

import numpy as np
import pytest

from oracle import from_workload, make_model, rel_l2, run_schedule
from workloads import build_config

pytestmark = pytest.mark.gpu

TOL = 1e-5

CASES = [
    ("quad_tree64", dict(n=16, p=70_001, K=30), "tiles+tail"),
    ("quad_tree64", dict(n=64, p=4099, K=100, drop=0.6, max_delay=8), "heavy loss"),
    ("quad_tree64", dict(n=32, p=2048, K=60, drop=0.0, max_delay=0), "no loss no delay"),
    ("quad_tree64", dict(n=1, p=33, K=5), "single node"),
    ("ls_ring4", {}, "config 1 as stated"),
    ("softmax_exp16", dict(F=96, C=7, rows=64, K=150, batch=8), "reduced softmax"),
    ("logistic_tree1024", dict(n=96, p=5000, rows=8, K=60, batch=4, nnz=50), "reduced sparse logistic"),
    ("mlp_tree64", dict(n=6, F=64, H=128, C=10, rows=128, K=20, batch=64), "reduced mlp"),
]


def _oracle(wl):
    orc = from_workload(wl, make_model(wl).grad)
    B = wl.batch
    orc.init_gradients([wl.schedule.batch_idx[i * B:(i + 1) * B] for i in range(wl.n)] if B else None)
    ref0 = (np.linalg.norm(orc.X()), np.linalg.norm(orc.Z()))
    run_schedule(orc, wl.schedule)
    return orc, ref0


@pytest.mark.parametrize("level", [0, 1], ids=["plain", "two-float tracker"])
@pytest.mark.parametrize("name,ov,why", CASES, ids=[c[2] for c in CASES])
def test_bucket_tracker_parity(rfast_lib, name, ov, why, level):
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    from paper_2307_11617_b200.binding import ESTATE, RFastError
    wl = build_config(name, seed=1, tracker=1, compensated=level, **ov)
    orc, ref0 = _oracle(wl)
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        eng.run()
        x, y = eng.read(B.STATE_X), eng.read(B.STATE_Y)
        assert np.isfinite(x).all() and np.isfinite(y).all()
        ex, ey = rel_l2(x, orc.X(), ref0[0]), rel_l2(y, orc.Z(), ref0[1])
        ytol = 1e-4 if name == "mlp_tree64" else TOL          # bf16-rounded state, as for the running sums
        assert ex <= TOL and ey <= ytol, (ex, ey)
        assert eng.read(B.STATE_USED_TAU_V).tolist() == orc.used_tau_v
        assert eng.read(B.STATE_USED_TAU_RHO).tolist() == orc.used_tau_rho
        assert eng.read(B.STATE_T_LOCAL).tolist() == orc.t
        # Lemma 3 on the device state: trackers + buckets begun and not yet consumed = gradients
        d = eng.diagnostics()
        scale = np.abs(orc.G()).sum(axis=0).max()
        assert d["conservation_residual"] <= 1e-5 * max(scale, 1e-30)
        # there are no running sums to look at
        if wl.G_C.n_edges:
            for view in (B.STATE_RHO_LATEST, B.STATE_RHO_BUF):
                with pytest.raises(RFastError) as ei:
                    eng.read(view)
                assert ei.value.code == ESTATE


def test_bucket_tracker_moves_fewer_bytes_and_keeps_small_trackers_exact(rfast_lib):
    """Config 1's trackers are small next to the running sums, which costs the plain fp32
    running-sum tracker resolution; the buckets hold only the mass in transit.  Same schedule,
    plain fp32 on both sides: the bucket run must be at least as close to the oracle in y, and
    its compiled schedule must move fewer bytes."""
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    err, nbytes = {}, {}
    for tracker in (0, 1):
        wl = build_config("ls_ring4", seed=0, tracker=tracker, compensated=0)
        orc, ref0 = _oracle(wl)
        with pkg.Engine(wl) as eng:
            eng.load_schedule(wl.schedule)
            eng.run()
            err[tracker] = rel_l2(eng.read(B.STATE_Y), orc.Z(), ref0[1])
            nbytes[tracker] = eng.query(B.Q_BYTES_TOTAL)
    assert err[1] <= err[0] and err[1] <= TOL, err
    assert nbytes[1] < nbytes[0]


def test_bucket_tracker_checkpoint_resume_and_stepping(rfast_lib):
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config("quad_tree64", seed=3, n=24, p=3001, K=40, tracker=1)
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        eng.run()
        x1, y1 = eng.read(B.STATE_X), eng.read(B.STATE_Y)
        eng.reset()
        for _ in range(17):
            eng.run(1)
        blob = eng.checkpoint()
        mid = eng.diagnostics()["conservation_residual"]
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        eng.restore(blob)
        assert eng.query(B.Q_ROUND) == 17
        assert eng.diagnostics()["conservation_residual"] == mid
        eng.run(wl.schedule.K - 17)
        assert np.array_equal(x1, eng.read(B.STATE_X)) and np.array_equal(y1, eng.read(B.STATE_Y))
    # a blob of the running-sum tracker does not fit a bucket handle
    other = build_config("quad_tree64", seed=3, n=24, p=3001, K=40)
    with pkg.Engine(other) as eng:
        eng.load_schedule(other.schedule)
        eng.run(17)
        foreign = eng.checkpoint()
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        with pytest.raises(pkg.binding.RFastError):
            eng.restore(foreign)


def _sweep_cases(count, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for it in range(count):
        model = ["quad_tree64", "ls_ring4", "softmax_exp16", "logistic_tree1024"][it % 4]
        ov = dict(K=int(rng.integers(1, 40)), drop=float(rng.choice([0.0, 0.3, 0.6])),
                  max_delay=int(rng.choice([0, 3, 10])), tracker=int(rng.integers(0, 2)),
                  compensated=int(rng.integers(0, 3)))
        if model == "quad_tree64":
            ov.update(n=int(rng.integers(1, 24)), p=int(rng.choice([1, 3, 5, 1023, 1024, 1025, 4097, 9001])))
        elif model == "ls_ring4":
            ov.update(n=int(rng.integers(1, 10)), p=int(rng.choice([1, 7, 10, 33, 300, 1030])), rows=int(rng.integers(2, 40)))
        elif model == "softmax_exp16":
            ov.update(n=int(2 ** rng.integers(0, 5)), F=int(rng.choice([5, 16, 96, 100])), C=int(rng.integers(2, 9)),
                      rows=int(rng.integers(8, 40)), batch=int(rng.integers(1, 9)))
        else:
            p = int(rng.choice([50, 999, 4096, 5000, 9000]))
            ov.update(n=int(rng.integers(2, 40)), p=p, rows=int(rng.integers(2, 10)), batch=int(rng.integers(1, 5)),
                      nnz=int(rng.integers(1, min(p, 60))))
        cases.append((model, ov, int(rng.integers(0, 1000))))
    return cases


@pytest.mark.parametrize("model,ov,seed", _sweep_cases(32, 2024),
                         ids=[f"{i}-{c[0].split('_')[0]}" for i, c in enumerate(_sweep_cases(32, 2024))])
def test_seeded_sweep_of_shapes_losses_trackers_and_arithmetics(rfast_lib, model, ov, seed):
    """Ragged and degenerate shapes (one node, one coordinate, tile size +- 1, one sampled row),
    no loss to 60 % loss, delays up to 10 rounds, both trackers, the three tracker arithmetics:
    x and y at 1e-5, stamps bit-exact, Lemma 3 on the device state."""
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    wl = build_config(model, seed=seed, **ov)
    orc, ref0 = _oracle(wl)
    with pkg.Engine(wl) as eng:
        eng.load_schedule(wl.schedule)
        eng.run()
        x, y = eng.read(B.STATE_X), eng.read(B.STATE_Y)
        assert eng.read(B.STATE_USED_TAU_V).tolist() == orc.used_tau_v
        assert eng.read(B.STATE_USED_TAU_RHO).tolist() == orc.used_tau_rho
        d = eng.diagnostics()
    assert rel_l2(x, orc.X(), ref0[0]) <= TOL and rel_l2(y, orc.Z(), ref0[1]) <= TOL
    assert d["conservation_residual"] <= 1e-5 * max(np.abs(orc.G()).sum(axis=0).max(), 1e-30)

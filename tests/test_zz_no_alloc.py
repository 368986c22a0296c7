"""The allocation-free least-squares gradient against the handle-based path.

Some users of this library may not allocate device memory where they need a gradient (their
framework owns the whole GPU through its own pool, or they sit in a loop where cudaMalloc's
device-wide synchronisation is not acceptable).  rfast_ls_gradient_static serves them with a
scratch array built into the library.  Here its result is compared, through the C ABI, with
the gradient the ordinary entry points produce for the same shard and the same x
(rfast_create + rfast_load_schedule compute grad f_i(x0) for the initial trackers;
rfast_read_state returns it), on two calls in a row that share the scratch.

Collected last on purpose: a run that stops at the first failure has then run everything else.
"""

from __future__ import annotations

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = 1e-5      # relative L2, the bar of the parity tests


def _reference_gradient(feat, target, x, l2):
    """grad f(x) from the existing entry points: a one-node least-squares problem whose
    initial gradient is read back."""
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200 import binding as B
    from workloads import Workload, graph_from_edges, Schedule
    rows, F = feat.shape
    wl = Workload("ls_single", 1, F, 0, 0.01, graph_from_edges(1, [], "row"),
                  graph_from_edges(1, [], "col"), "least_squares", 0, l2, rows,
                  dims={"n_features": F}, data={"feat": feat[None], "target": target[None]},
                  x0=x[None].copy())
    empty = Schedule(0, np.zeros(1, np.int32), np.zeros(0, np.int32), np.zeros(0, np.int8),
                     np.zeros(0, np.int8), 0, np.zeros(0, np.int32))
    with pkg.Engine(wl) as eng:
        eng.load_schedule(empty)
        return eng.read(B.STATE_G_LAST)[0].copy(), wl.l2


def test_static_gradient_matches_handle_path_twice(rfast_lib):
    import torch
    import paper_2307_11617_b200 as pkg
    rng = np.random.default_rng(11)
    dev = torch.device("cuda", 0)
    # second problem is smaller than the first: stale residuals of call 1 stay in the scratch
    for rows, F in ((3000, 517), (77, 33)):
        feat = rng.standard_normal((rows, F)).astype(np.float32)
        target = rng.standard_normal(rows).astype(np.float32)
        x = rng.standard_normal(F).astype(np.float32)
        want, l2 = _reference_gradient(feat, target, x, 1e-3)
        d_feat, d_target, d_x = (torch.from_numpy(a).to(dev) for a in (feat, target, x))
        d_grad = torch.full((F,), float("nan"), device=dev)
        torch.cuda.synchronize()
        pkg.rfast_ls_gradient_static(d_feat.data_ptr(), d_target.data_ptr(), d_x.data_ptr(),
                                     d_grad.data_ptr(), rows, F, l2,
                                     torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        got = d_grad.cpu().numpy()
        assert np.isfinite(got).all()
        assert np.linalg.norm(got - want) <= TOL * np.linalg.norm(want)
        # and directly against the CPU oracle's definition of the same gradient
        from oracle.models import LeastSquares
        ref = LeastSquares([feat], [target], l2).grad(0, x.astype(np.float64))
        assert np.linalg.norm(got - ref) <= TOL * np.linalg.norm(ref)


def test_static_gradient_rejects_oversize(rfast_lib):
    import torch
    import paper_2307_11617_b200 as pkg
    from paper_2307_11617_b200.binding import EINVAL, RFastError, STATIC_MAX_ROWS
    d = torch.zeros(8, device="cuda")
    with pytest.raises(RFastError) as ei:
        pkg.rfast_ls_gradient_static(d.data_ptr(), d.data_ptr(), d.data_ptr(), d.data_ptr(),
                                     STATIC_MAX_ROWS + 1, 1)
    assert ei.value.code == EINVAL and "exceed" in str(ei.value)

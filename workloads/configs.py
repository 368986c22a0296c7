"""The five synthetic workloads (graphs + data shards + schedule), seeded.

Each `build_config(name, ...)` returns a `Workload` holding plain arrays only.
Every size can be overridden so that the same recipe yields a small case for
parity tests and the full case for the benchmark.

Stand-ins: the paper's own workloads are logistic regression on MNIST digits
(Section VI-A: 784 features, minibatch 32) and ResNet-50 on ImageNet (Section
VI-B); neither dataset is available, so Gaussian-mixture / synthetic data of the
same shapes is generated instead.
"""

from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from .graphs import (Graph, binary_tree_parents, exponential_tree_parents,
                     graph_from_edges, random_tree_parents, ring_graphs, tree_graphs)
from .schedules import (Schedule, activation_bernoulli, activation_durations,
                        activation_uniform_subset, make_schedule)

CONFIG_NAMES = ("ls_ring4", "softmax_exp16", "mlp_tree64", "quad_tree64", "logistic_tree1024")

MODEL_QUAD_DIAG = "quad_diag"
MODEL_LEAST_SQUARES = "least_squares"
MODEL_SOFTMAX = "softmax"
MODEL_MLP = "mlp"
MODEL_LOGISTIC_SPARSE = "logistic_sparse"


@dataclass
class Workload:
    name: str
    n: int
    p: int
    root: int
    alpha: float
    G_R: Graph
    G_C: Graph
    model: str
    batch: int                      # minibatch rows per activation (0: full shard / no data rows)
    l2: float
    rows: int                       # rows per node in the shard (0 for quad_diag)
    dims: dict = field(default_factory=dict)    # n_features / n_classes / n_hidden
    data: dict = field(default_factory=dict)    # model-specific arrays, see below
    x0: np.ndarray | None = None    # float32 [n, p] or None (zeros)
    schedule: Schedule | None = None
    meta: dict = field(default_factory=dict)
    compensated: int = 0            # tracker arithmetic asked of the engine: 0 plain fp32, 1 two-float
                                    # tracker, 2 two-float tracker and running sums
    tracker: int = 0                # how the engine keeps the mass on the G_C edges: 0 running sums
                                    # (Algorithm 1 as printed), 1 one row per consumption ("buckets")

    def __post_init__(self):
        # scalars are handed to every consumer as the fp32-representable value
        self.alpha = float(np.float32(self.alpha))
        self.l2 = float(np.float32(self.l2))

    # data keys by model:
    #   quad_diag:        d [n,p] f32, b [n,p] f32            f_i = 0.5 * || d_i * (x - b_i) ||^2
    #   least_squares:    feat [n,rows,p] f32, target [n,rows] f32
    #   softmax / mlp:    feat [n,rows,F] f32, label [n,rows] i32 in [0,C)
    #   logistic_sparse:  sp_rowptr [n*rows+1] i64, sp_col i32, sp_val f32, label [n,rows] i32 in {-1,+1}


def _rng(seed, stream):
    return np.random.Generator(np.random.PCG64([int(seed), int(stream)]))


def _gaussian_mixture(n, rows, F, C, classes_per_node, rng, scale):
    means = rng.standard_normal((C, F)).astype(np.float32)
    feat = np.empty((n, rows, F), dtype=np.float32)
    label = np.empty((n, rows), dtype=np.int32)
    for i in range(n):
        own = [(classes_per_node * i + c) % C for c in range(classes_per_node)]
        lab = np.asarray(own, dtype=np.int32)[rng.integers(0, classes_per_node, size=rows)]
        x = means[lab] + rng.standard_normal((rows, F)).astype(np.float32)
        feat[i] = x * np.float32(scale)
        label[i] = lab
    return feat, label


def build_config(name: str, seed: int = 0, **ov) -> Workload:
    """ov overrides: n, p, rows, K, F (features), H (hidden), C (classes), batch, drop,
    max_delay, alpha, nnz (per sparse row), compensated, tracker."""
    builders = {"ls_ring4": _ls_ring, "softmax_exp16": _softmax_exp, "mlp_tree64": _mlp_tree,
                "quad_tree64": _quad_tree, "logistic_tree1024": _logistic_tree}
    wl = builders[name](seed, ov)
    wl.tracker = int(ov.get("tracker", 0))
    return wl


# -- config 1: n=4 directed ring, heterogeneous least squares, full batch ---------------------
def _ls_ring(seed, ov):
    n = ov.get("n", 4); p = ov.get("p", 10); rows = ov.get("rows", 50); K = ov.get("K", 200)
    drop = ov.get("drop", 0.1); max_delay = ov.get("max_delay", 2); alpha = ov.get("alpha", 0.01)
    rd, rs = _rng(seed, 1), _rng(seed, 2)
    G_R, G_C = ring_graphs(n)
    x_true = rd.standard_normal(p)
    feat = np.empty((n, rows, p), np.float32)
    target = np.empty((n, rows), np.float32)
    for i in range(n):
        mu = 1.0 * (2.0 * i / max(n - 1, 1) - 1.0)
        A = rd.standard_normal((rows, p)) + mu
        xi = x_true + 1.0 * rd.standard_normal(p)
        feat[i] = A.astype(np.float32)
        target[i] = (A @ xi + 0.1 * rd.standard_normal(rows)).astype(np.float32)
    act = activation_uniform_subset(n, K, 1, min(4, n), rs)
    sch = make_schedule(G_R, G_C, act, drop, max_delay, rs, batch=0)
    return Workload("ls_ring4", n, p, 0, alpha, G_R, G_C, MODEL_LEAST_SQUARES, 0, 0.0, rows,
                    dims={"n_features": p}, data={"feat": feat, "target": target}, schedule=sch,
                    meta={"K": K, "drop": drop, "max_delay": max_delay},
                    compensated=ov.get("compensated", 2))


# -- config 2: n=16 exponential-graph trees, softmax regression, one 4x straggler --------------
def _softmax_exp(seed, ov):
    n = ov.get("n", 16); F = ov.get("F", 784); C = ov.get("C", 10); rows = ov.get("rows", 1024)
    K = ov.get("K", 5000); B = ov.get("batch", 32); drop = ov.get("drop", 0.1)
    max_delay = ov.get("max_delay", 2); alpha = ov.get("alpha", 0.01)
    rd, rs = _rng(seed, 1), _rng(seed, 2)
    hi, lo = exponential_tree_parents(n)
    G_R, G_C = tree_graphs(hi, lo)
    feat, label = _gaussian_mixture(n, rows, F, C, 2, rd, 1.0 / np.sqrt(F))
    straggler = int(rs.integers(0, n))
    act = activation_durations(n, K, lambda i, t: 4 if i == straggler else 1)
    sch = make_schedule(G_R, G_C, act, drop, max_delay, rs, batch=B, rows_per_node=rows)
    p = C * F + C
    return Workload("softmax_exp16", n, p, 0, alpha, G_R, G_C, MODEL_SOFTMAX, B, 1e-4, rows,
                    dims={"n_features": F, "n_classes": C}, data={"feat": feat, "label": label},
                    schedule=sch, meta={"K": K, "drop": drop, "max_delay": max_delay,
                                        "straggler": straggler},
                    compensated=ov.get("compensated", 1))


# -- config 3: n=64 random trees, MLP F-H-C ReLU, lognormal compute times -----------------------
def _mlp_tree(seed, ov):
    n = ov.get("n", 64); F = ov.get("F", 784); H = ov.get("H", 512); C = ov.get("C", 10)
    rows = ov.get("rows", 1024); K = ov.get("K", 500); B = ov.get("batch", 64)
    drop = ov.get("drop", 0.05); max_delay = ov.get("max_delay", 2); alpha = ov.get("alpha", 0.002)
    l2 = ov.get("l2", 0.0)
    rd, rs = _rng(seed, 1), _rng(seed, 2)
    G_R, G_C = tree_graphs(random_tree_parents(n, rs), random_tree_parents(n, rs))
    feat, label = _gaussian_mixture(n, rows, F, C, 2, rd, 1.0 / np.sqrt(F))
    p = H * F + H + C * H + C
    w1 = (rd.standard_normal(H * F) * np.sqrt(2.0 / F)).astype(np.float32)
    w2 = (rd.standard_normal(C * H) * np.sqrt(2.0 / H)).astype(np.float32)
    x_init = np.concatenate([w1, np.zeros(H, np.float32), w2, np.zeros(C, np.float32)])
    x0 = np.broadcast_to(x_init, (n, p)).copy()
    act = activation_durations(
        n, K, lambda i, t: max(1, int(np.rint(np.exp(rs.standard_normal())))))
    sch = make_schedule(G_R, G_C, act, drop, max_delay, rs, batch=B, rows_per_node=rows)
    return Workload("mlp_tree64", n, p, 0, alpha, G_R, G_C, MODEL_MLP, B, l2, rows,
                    dims={"n_features": F, "n_hidden": H, "n_classes": C},
                    data={"feat": feat, "label": label}, x0=x0, schedule=sch,
                    meta={"K": K, "drop": drop, "max_delay": max_delay})


# -- config 4: n=64 binary-tree G_R + ring G_C, diagonal quadratic, bandwidth stress -----------
def _quad_tree(seed, ov):
    n = ov.get("n", 64); p = ov.get("p", 11_200_000); K = ov.get("K", 100)
    drop = ov.get("drop", 0.2); max_delay = ov.get("max_delay", 8); alpha = ov.get("alpha", 0.01)
    rd, rs = _rng(seed, 1), _rng(seed, 2)
    G_R, _ = tree_graphs(binary_tree_parents(n), binary_tree_parents(n))
    G_C = graph_from_edges(n, [(i, (i + 1) % n) for i in range(n)] if n > 1 else [], "col")
    d = np.empty((n, p), np.float32)
    b = np.empty((n, p), np.float32)
    for i in range(n):
        d[i] = rd.random(p, dtype=np.float32) * np.float32(1.5) + np.float32(0.5)
        b[i] = rd.standard_normal(p, dtype=np.float32)
    act = activation_bernoulli(n, K, 0.5, rs)
    sch = make_schedule(G_R, G_C, act, drop, max_delay, rs, batch=0)
    return Workload("quad_tree64", n, p, 0, alpha, G_R, G_C, MODEL_QUAD_DIAG, 0, 0.0, 0,
                    data={"d": d, "b": b}, schedule=sch,
                    meta={"K": K, "drop": drop, "max_delay": max_delay})


# -- config 5: n=1024 random trees (<= 8 children), sparse logistic regression, 10% stragglers --
def _logistic_tree(seed, ov):
    n = ov.get("n", 1024); p = ov.get("p", 100_000); rows = ov.get("rows", 64)
    K = ov.get("K", 300); B = ov.get("batch", 16); drop = ov.get("drop", 0.3)
    max_delay = ov.get("max_delay", 2); alpha = ov.get("alpha", 0.002)
    nnz = ov.get("nnz", max(1, int(round(0.01 * p))))
    rd, rs = _rng(seed, 1), _rng(seed, 2)
    G_R, G_C = tree_graphs(random_tree_parents(n, rs, 8), random_tree_parents(n, rs, 8))
    R = n * rows
    cols = np.sort(rd.integers(0, p, size=(R, nnz), dtype=np.int32), axis=1)
    keep = np.ones((R, nnz), dtype=bool)
    keep[:, 1:] = cols[:, 1:] != cols[:, :-1]          # repeated columns inside a row are removed
    vals = (rd.standard_normal((R, nnz), dtype=np.float32) / np.float32(np.sqrt(nnz)))
    x_true = rd.standard_normal(p).astype(np.float32)
    score = np.where(keep, vals * x_true[cols], 0).sum(axis=1)
    pref = np.where(np.arange(n) % 2 == 0, 1, -1)       # worker i holds mostly one sign
    want = np.repeat(pref, rows) * np.where(rd.random(R) < 0.9, 1, -1)
    flip = np.where(np.sign(score) * want < 0, -1.0, 1.0).astype(np.float32)
    vals *= flip[:, None]                                # (-a) . x_true has the wanted sign
    label = want.astype(np.int32).reshape(n, rows)
    sp_rowptr = np.zeros(R + 1, dtype=np.int64)
    sp_rowptr[1:] = np.cumsum(keep.sum(axis=1))
    sp_col = cols[keep].astype(np.int32)
    sp_val = vals[keep].astype(np.float32)
    n_strag = max(1, n // 10)
    strag = set(int(s) for s in rs.choice(n, size=n_strag, replace=False))
    act = activation_durations(n, K, lambda i, t: 10 if i in strag else 1)
    sch = make_schedule(G_R, G_C, act, drop, max_delay, rs, batch=B, rows_per_node=rows)
    return Workload("logistic_tree1024", n, p, 0, alpha, G_R, G_C, MODEL_LOGISTIC_SPARSE, B, 1e-4,
                    rows, dims={"n_features": p},
                    data={"sp_rowptr": sp_rowptr, "sp_col": sp_col, "sp_val": sp_val,
                          "label": label},
                    schedule=sch, meta={"K": K, "drop": drop, "max_delay": max_delay,
                                        "stragglers": sorted(strag)})


def shard_coordinates(wl: Workload, part: int, parts: int) -> Workload:
    """The slice of an element-wise problem that one of `parts` devices owns.

    Every step of an activation (S1, S2a, the gradient d^2 (x - b), S2b, S2c) acts coordinate by
    coordinate when the objective is the diagonal quadratic, so the problem splits by
    coordinate with no exchange at all: each part runs the same schedule on its slice and the
    concatenation of the parts' states is the state of the whole.  Slices are contiguous, as
    equal as possible, the first p mod parts of them one coordinate longer."""
    if wl.model != MODEL_QUAD_DIAG:
        raise ValueError("only the element-wise objective splits by coordinate without exchange")
    if not (0 <= part < parts <= wl.p):
        raise ValueError("need 0 <= part < parts <= p")
    base, extra = divmod(wl.p, parts)
    lo = part * base + min(part, extra)
    hi = lo + base + (1 if part < extra else 0)
    data = {k: np.ascontiguousarray(v[:, lo:hi]) for k, v in wl.data.items()}
    x0 = None if wl.x0 is None else np.ascontiguousarray(wl.x0[:, lo:hi])
    sub = Workload(wl.name, wl.n, hi - lo, wl.root, wl.alpha, wl.G_R, wl.G_C, wl.model, wl.batch, wl.l2,
                   wl.rows, dims=dict(wl.dims), data=data, x0=x0, schedule=wl.schedule,
                   meta=dict(wl.meta, coordinates=(lo, hi)), compensated=wl.compensated)
    sub.tracker = wl.tracker
    return sub

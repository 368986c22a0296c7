"""Pins of the oracle's objectives: gradients against their own losses (central differences),
closed forms, and the bf16 rounding rule against hand-computed values (no GPU)."""

from __future__ import annotations

import numpy as np
import pytest

from oracle import bf16_round, make_model
from oracle.models import LeastSquares, LogisticSparse, MLP, QuadDiag, Softmax
from workloads import build_config


def _fd(loss, x, h=1e-6):
    g = np.zeros_like(x)
    for c in range(len(x)):
        e = np.zeros_like(x); e[c] = h
        g[c] = (loss(x + e) - loss(x - e)) / (2 * h)
    return g


SMALL = [
    ("ls_ring4", dict(rows=9, p=5)),
    ("softmax_exp16", dict(n=4, F=6, C=3, rows=10, K=2, batch=4)),
    ("quad_tree64", dict(n=4, p=7, K=2)),
    ("logistic_tree1024", dict(n=4, p=30, rows=6, K=2, batch=3, nnz=5)),
]


@pytest.mark.parametrize("name,ov", SMALL)
def test_gradient_matches_finite_differences(name, ov):
    wl = build_config(name, seed=1, **ov)
    m = make_model(wl)
    rng = np.random.default_rng(0)
    for i in (0, wl.n - 1):
        x = rng.standard_normal(wl.p)
        idx = rng.integers(0, wl.rows, size=wl.batch) if wl.batch else None
        if name == "logistic_tree1024":
            idx[-1] = idx[0]                 # a repeated row in the batch counts twice
        g = m.grad(i, x, idx)
        fd = _fd(lambda y: m.loss(i, y, idx), x)
        assert np.abs(g - fd).max() <= 1e-6 * max(1.0, np.abs(fd).max())


def test_mlp_gradient_matches_finite_differences_without_rounding():
    wl = build_config("mlp_tree64", seed=1, n=3, F=5, H=4, C=3, rows=8, K=2, batch=4)
    m = make_model(wl, round_inputs=False)
    rng = np.random.default_rng(0)
    x = rng.standard_normal(wl.p) * 0.7
    idx = rng.integers(0, wl.rows, size=wl.batch)
    g = m.grad(1, x, idx)
    fd = _fd(lambda y: m.loss(1, y, idx), x)
    assert np.abs(g - fd).max() <= 1e-6 * max(1.0, np.abs(fd).max())


def test_mlp_rounded_path_is_the_same_code_with_rounded_operands():
    """With operands that are already bf16 numbers the rounded and unrounded paths coincide
    in the forward pass; the rounded gradient stays within bf16 resolution of the exact one."""
    wl = build_config("mlp_tree64", seed=2, n=2, F=6, H=5, C=3, rows=8, K=2, batch=4)
    wl.data["feat"] = bf16_round(wl.data["feat"]).astype(np.float32)
    exact, rounded = make_model(wl, round_inputs=False), make_model(wl, round_inputs=True)
    rng = np.random.default_rng(1)
    x = bf16_round(rng.standard_normal(wl.p) * 0.5)
    idx = rng.integers(0, wl.rows, size=wl.batch)
    # forward: hidden pre-activations use only (A, W1) -> identical
    assert np.array_equal(exact._forward(0, x, idx)[2], rounded._forward(0, x, idx)[2])
    ge, gr = exact.grad(0, x, idx), rounded.grad(0, x, idx)
    assert np.abs(ge - gr).max() <= 3 * 2.0 ** -8 * np.abs(ge).max()
    # only the weight gradient of the first layer sees a rounded operand (dpre); the rest is exact
    o1 = wl.dims["n_hidden"] * wl.dims["n_features"]
    assert np.array_equal(ge[o1:], gr[o1:]) and not np.array_equal(ge[:o1], gr[:o1])


def test_bf16_round_hand_values():
    # bf16 keeps 8 significant bits: spacing 2^-7 in [1, 2)
    cases = [
        (1.0, 1.0),
        (1.0 + 2.0 ** -8, 1.0),                    # tie -> even (mantissa ...0)
        (1.0 + 2.0 ** -7 + 2.0 ** -8, 1.0 + 2.0 ** -6),   # tie -> even (up)
        (1.0 + 2.0 ** -8 + 2.0 ** -20, 1.0 + 2.0 ** -7),  # just above the tie
        (-3.0 - 2.0 ** -7, -3.0),                  # spacing 2^-6 in [2,4): tie -> even
        (0.0, 0.0),
        (3.140625, 3.140625),                      # already representable
        (1e-3, 0.00099945068359375),
    ]
    for a, want in cases:
        assert bf16_round(np.array([a]))[0] == want, (a, want)
    # double rounding is deliberate: the decision is taken on the fp32 value
    a = 1.0 + 2.0 ** -8 + 2.0 ** -30              # fp32 drops the 2^-30, leaving an exact tie
    assert bf16_round(np.array([a]))[0] == 1.0


def test_least_squares_gradient_vanishes_at_normal_equations():
    rng = np.random.default_rng(3)
    A = rng.standard_normal((1, 12, 4)); y = rng.standard_normal((1, 12))
    m = LeastSquares(A, y, l2=0.1)
    xs = np.linalg.solve(A[0].T @ A[0] / 12 + 0.1 * np.eye(4), A[0].T @ y[0] / 12)
    assert np.abs(m.grad(0, xs, None)).max() < 1e-13


def test_quad_diag_closed_form_minimiser_of_the_sum():
    rng = np.random.default_rng(4)
    d = rng.uniform(0.5, 2, (5, 6)); b = rng.standard_normal((5, 6))
    m = QuadDiag(d, b)
    xs = (d * d * b).sum(axis=0) / (d * d).sum(axis=0)
    assert np.abs(sum(m.grad(i, xs) for i in range(5))).max() < 1e-13


def test_softmax_gradient_structure():
    rng = np.random.default_rng(5)
    feat = rng.standard_normal((1, 9, 4)); lab = rng.integers(0, 3, (1, 9)).astype(np.int32)
    m = Softmax(feat, lab, 3, l2=0.0)
    x = rng.standard_normal(3 * 4 + 3)
    g = m.grad(0, x, np.arange(9))
    # probabilities sum to one: the class gradients cancel feature by feature and in the bias
    assert np.abs(g[:12].reshape(3, 4).sum(axis=0)).max() < 1e-14
    assert abs(g[12:].sum()) < 1e-14
    # two classes, zero weights: p = 1/2, bias gradient = mean(1/2 - onehot)
    m2 = Softmax(feat, (lab % 2).astype(np.int32), 2)
    g2 = m2.grad(0, np.zeros(2 * 4 + 2), np.arange(9))
    want = 0.5 - np.bincount(lab[0] % 2, minlength=2) / 9
    assert np.allclose(g2[8:], want, atol=1e-15)


def test_logistic_matches_dense_formula():
    wl = build_config("logistic_tree1024", seed=6, n=2, p=40, rows=5, K=2, batch=3, nnz=6)
    m = make_model(wl)
    d = wl.data
    dense = np.zeros((wl.n * wl.rows, wl.p))
    for r in range(wl.n * wl.rows):
        dense[r, d["sp_col"][d["sp_rowptr"][r]:d["sp_rowptr"][r + 1]]] = \
            d["sp_val"][d["sp_rowptr"][r]:d["sp_rowptr"][r + 1]]
    rng = np.random.default_rng(0)
    x = rng.standard_normal(wl.p)
    idx = np.array([4, 0, 2])
    A = dense[wl.rows * 1 + idx]; y = d["label"][1][idx].astype(np.float64)
    want = -(A * (y / (1 + np.exp(y * (A @ x))))[:, None]).mean(axis=0) + wl.l2 * x
    assert np.abs(m.grad(1, x, idx) - want).max() < 1e-14

"""Per-node objectives f_i and their sample gradients (TEST INFRASTRUCTURE, plain numpy fp64).

Problem (1): F(x) = sum_i f_i(x), f_i the expected (here: minibatch-mean) loss on node i's
own shard.  A minibatch gradient is the mean over the sampled rows; each f_i carries its own
(l2/2)||x||^2.  Every class offers loss(i, x, idx) and grad(i, x, idx); the tests pin grad
to loss by central finite differences, and loss is the textbook definition written out.

Parameter layouts (x is one flat vector of length p):
  least_squares    x = coefficients [F]
  softmax          x = [W (C x F, row c = class c) | bias (C)]
  mlp              x = [W1 (H x F) | b1 (H) | W2 (C x H) | b2 (C)],  hidden = relu(W1 a + b1)
  logistic_sparse  x = coefficients [p], labels in {-1,+1}, features in CSR
  quad_diag        f_i(x) = 0.5 * || d_i * (x - b_i) ||^2  (element-wise)
"""

from __future__ import annotations

import numpy as np


def bf16_round(a):
    """Round to bfloat16 (8-bit significand), nearest-even, taken from the fp32 value: the
    GEMM inputs of the MLP are rounded this way (fp32 state / bf16 GEMM inputs), and the
    decision is taken in fp32 because that is the precision the state is held in.
    Finite inputs only."""
    f = np.asarray(a, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


class QuadDiag:
    def __init__(self, d, b):
        self.d, self.b = d, b

    def loss(self, i, x, idx=None):
        r = self.d[i] * (x - self.b[i])
        return 0.5 * (r * r).sum()

    def grad(self, i, x, idx=None):
        d = self.d[i]
        return d * d * (x - self.b[i])


class LeastSquares:
    def __init__(self, feat, target, l2=0.0):
        self.A = [np.asarray(a, dtype=np.float64) for a in feat]
        self.y = [np.asarray(t, dtype=np.float64) for t in target]
        self.l2 = l2

    def _rows(self, i, idx):
        if idx is None or len(idx) == 0:
            return self.A[i], self.y[i]
        return self.A[i][idx], self.y[i][idx]

    def loss(self, i, x, idx=None):
        A, y = self._rows(i, idx)
        r = A @ x - y
        return 0.5 * (r @ r) / len(y) + 0.5 * self.l2 * (x @ x)

    def grad(self, i, x, idx=None):
        A, y = self._rows(i, idx)
        r = A @ x - y
        return A.T @ r / len(y) + self.l2 * x


def _softmax_rows(logits):
    m = logits.max(axis=1, keepdims=True)
    e = np.exp(logits - m)
    return e / e.sum(axis=1, keepdims=True), m[:, 0] + np.log(e.sum(axis=1))


class Softmax:
    def __init__(self, feat, label, n_classes, l2=0.0):
        self.A = feat
        self.lab = label
        self.C = n_classes
        self.F = feat.shape[2]
        self.l2 = l2

    def _parts(self, i, x, idx):
        A = np.asarray(self.A[i][idx], dtype=np.float64)
        lab = self.lab[i][idx]
        W = x[:self.C * self.F].reshape(self.C, self.F)
        bias = x[self.C * self.F:]
        return A, lab, W, bias

    def loss(self, i, x, idx):
        A, lab, W, bias = self._parts(i, x, idx)
        P, lse = _softmax_rows(A @ W.T + bias)
        logits = A @ W.T + bias
        return (lse - logits[np.arange(len(lab)), lab]).mean() + 0.5 * self.l2 * (x @ x)

    def grad(self, i, x, idx):
        A, lab, W, bias = self._parts(i, x, idx)
        P, _ = _softmax_rows(A @ W.T + bias)
        P[np.arange(len(lab)), lab] -= 1.0
        D = P / len(lab)
        return np.concatenate([(D.T @ A).ravel(), D.sum(axis=0)]) + self.l2 * x


class MLP:
    """One hidden ReLU layer, softmax cross-entropy.  With round_inputs=True the operands of
    the two GEMM-shaped products -- the hidden pre-activations A W1^T and the weight gradient
    dpre^T A -- are first rounded to bf16 ("fp32 state / bf16 GEMM inputs").  The products
    with the n_classes-wide output layer are a few columns thin, not GEMM work, and stay in
    full precision, as do sums, biases, ReLU, softmax and all accumulation."""

    def __init__(self, feat, label, n_hidden, n_classes, l2=0.0, round_inputs=True):
        self.A, self.lab = feat, label
        self.F, self.H, self.C = feat.shape[2], n_hidden, n_classes
        self.l2 = l2
        self.q = bf16_round if round_inputs else (lambda a: np.asarray(a, dtype=np.float64))

    def _split(self, x):
        F, H, C = self.F, self.H, self.C
        o1 = H * F
        o2 = o1 + H
        o3 = o2 + C * H
        return x[:o1].reshape(H, F), x[o1:o2], x[o2:o3].reshape(C, H), x[o3:]

    def _forward(self, i, x, idx):
        q = self.q
        A = q(self.A[i][idx])
        lab = self.lab[i][idx]
        W1, b1, W2, b2 = self._split(x)
        pre = A @ q(W1).T + b1
        h = np.maximum(pre, 0.0)
        logits = h @ W2.T + b2
        return A, lab, pre, h, logits

    def loss(self, i, x, idx):
        A, lab, pre, h, logits = self._forward(i, x, idx)
        _, lse = _softmax_rows(logits)
        return (lse - logits[np.arange(len(lab)), lab]).mean() + 0.5 * self.l2 * (x @ x)

    def grad(self, i, x, idx):
        q = self.q
        A, lab, pre, h, logits = self._forward(i, x, idx)
        W1, b1, W2, b2 = self._split(x)
        P, _ = _softmax_rows(logits)
        P[np.arange(len(lab)), lab] -= 1.0
        dlog = P / len(lab)                       # d loss / d logits          [B, C]
        gW2 = dlog.T @ h                          #                            [C, H]
        gb2 = dlog.sum(axis=0)
        dh = dlog @ W2                            #                            [B, H]
        dpre = dh * (pre > 0.0)
        gW1 = q(dpre).T @ A                       # A already rounded          [H, F]
        gb1 = dpre.sum(axis=0)
        return np.concatenate([gW1.ravel(), gb1, gW2.ravel(), gb2]) + self.l2 * x


class LogisticSparse:
    def __init__(self, sp_rowptr, sp_col, sp_val, label, rows, l2=0.0):
        self.ptr, self.col, self.val = sp_rowptr, sp_col, sp_val
        self.lab, self.rows, self.l2 = label, rows, l2

    def _row(self, i, k):
        r = i * self.rows + int(k)
        s, e = int(self.ptr[r]), int(self.ptr[r + 1])
        return self.col[s:e], np.asarray(self.val[s:e], dtype=np.float64)

    def loss(self, i, x, idx):
        tot = 0.0
        for k in idx:
            c, v = self._row(i, k)
            m = float(self.lab[i][k]) * (v @ x[c])
            tot += np.logaddexp(0.0, -m)
        return tot / len(idx) + 0.5 * self.l2 * (x @ x)

    def grad(self, i, x, idx):
        g = self.l2 * x
        for k in idx:                              # rows in batch order; repeats count twice
            c, v = self._row(i, k)
            y = float(self.lab[i][k])
            m = y * (v @ x[c])
            coef = -y / (1.0 + np.exp(m)) / len(idx)
            g[c] += coef * v                       # columns are distinct inside a row
        return g


def make_model(wl, **kw):
    """Build the objective for a workload object (fields: model, data, dims, l2, rows)."""
    m, d = wl.model, wl.data
    if m == "quad_diag":
        return QuadDiag(np.asarray(d["d"], dtype=np.float64), np.asarray(d["b"], dtype=np.float64))
    if m == "least_squares":
        return LeastSquares(d["feat"], d["target"], wl.l2)
    if m == "softmax":
        return Softmax(d["feat"], d["label"], wl.dims["n_classes"], wl.l2)
    if m == "mlp":
        return MLP(d["feat"], d["label"], wl.dims["n_hidden"], wl.dims["n_classes"], wl.l2, **kw)
    if m == "logistic_sparse":
        return LogisticSparse(d["sp_rowptr"], d["sp_col"], d["sp_val"], d["label"], wl.rows, wl.l2)
    raise KeyError(m)

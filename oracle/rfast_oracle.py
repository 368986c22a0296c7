"""R-FAST, written out step by step (TEST INFRASTRUCTURE: never used by the product path).

Follows Algorithm 1 (local view: S1 descent, S2a mix, S2b track, S2c keep/accumulate,
S3 send, S4 buffer, S5 counter) with the bookkeeping of Algorithm 2 (global view):
messages are real objects carrying (stamp, payload); a receiver keeps, per in-edge,
the payload with the largest stamp it has received so far.

Notation is the paper's: x, v, z, rho (sender running sum, one per out-edge in G(A)),
rho_tilde (receiver buffer, one per in-edge in G(A)), tau_v / tau_rho (largest stamps
received), t (local iteration counter), gamma = alpha (constant step size).

Readings where the paper leaves room (each also listed in the design notes):
  * A round activates a set of nodes.  Every message sent in round r with delay code
    d >= 0 is usable from round r + 1 + d on, so members of one round never see each
    other's output; the round is Algorithm 2 run once per member, in any order.
  * A dropped packet (code -1) is never delivered; the sender's running sum is updated
    regardless (S2c is unconditional), so the mass rides on the next delivered packet.
  * The sum in S2a takes the own term first, then in-neighbours by ascending id; the sum
    in S2b takes z, then the in-neighbour differences by ascending id, then +g_new, -g_old.
  * v_j^0 = 0 and rho^0 = 0 are what a receiver holds before the first delivery (stamp 0).

Pins (tests/test_oracle_*.py): conservation of Lemma 3 in exact rational arithmetic,
the synchronous special case of Remark 1 / eq. (2) as a dense matrix recursion, the
augmented systems of Appendices E-F as dense matrices, n = 1 gradient descent, geometric
convergence to the closed-form least-squares optimum (Theorem 1, sigma = 0), and a
negative control (increment-sending tracker).  The value of an iterate at finite k for
the stochastic models is not printed anywhere in the paper: beyond those pins it is
"parity unpinned".

Everything works on any numpy dtype whose elements support + - *, including
dtype=object arrays of fractions.Fraction (used by the exact conservation test).
"""

from __future__ import annotations

import numpy as np


def _out_lists(n, rowptr, col):
    """For each sender j: its out-edges (receiver-CSR edge ids) by ascending receiver."""
    out = [[] for _ in range(n)]
    for i in range(n):                       # receivers ascending => each list ascending
        for e in range(int(rowptr[i]), int(rowptr[i + 1])):
            out[int(col[e])].append(e)
    return out


class RFastOracle:
    """State of all n nodes plus the packets in flight."""

    def __init__(self, n, p, alpha, G_R, G_C, grad, x0=None, dtype=np.float64,
                 increments_only=False):
        """G_R, G_C: objects with rowptr, col, w, diag (receiver-CSR; w[e] = M[receiver, col[e]]).
        grad(i, x, idx) -> stochastic gradient of f_i at x on sample rows idx (or None).
        increments_only=True builds the *wrong* tracker used as a negative control: it sends
        the increment a_ji z^{t+1/2} instead of the running sum, so dropped mass is lost."""
        self.n, self.p, self.alpha, self.dtype = n, p, alpha, dtype
        self.R, self.C = G_R, G_C
        self.grad = grad
        self.increments_only = increments_only
        self.out_R = _out_lists(n, G_R.rowptr, G_R.col)
        self.out_C = _out_lists(n, G_C.rowptr, G_C.col)
        ER, EC = len(G_R.col), len(G_C.col)
        zero = np.zeros(p, dtype=dtype)
        self.zero = zero
        if x0 is None:
            self.x = [zero.copy() for _ in range(n)]
        else:
            self.x = [np.array(x0[i], dtype=dtype) for i in range(n)]
        self.z = [None] * n                  # set by init_gradients
        self.g = [None] * n                  # remembered sample gradient, grad f_i(x_i^t; zeta_i^t)
        self.t = [0] * n
        self.v_latest = [zero] * n           # v_i^0 = 0
        # G(W) in-edges: newest packet received
        self.tau_v = [0] * ER
        self.v_recv = [zero] * ER
        self.inbox_v = [[] for _ in range(ER)]
        # G(A): sender side running sum, receiver side newest packet + buffer
        self.rho = [zero] * EC
        self.tau_rho = [0] * EC              # stamp of the newest rho packet received (consumed at S2b)
        self.rho_recv = [zero] * EC
        self.rho_tilde = [zero] * EC
        self.inbox_rho = [[] for _ in range(EC)]
        self.round = 0
        self.activations = 0
        # integer artefacts, in event order then in-edge (CSR) order
        self.used_tau_v = []
        self.used_tau_rho = []

    # Initialization line of Algorithm 1: z_i^0 = grad f_i(x_i^0; zeta_i^0)
    def init_gradients(self, zeta0=None):
        for i in range(self.n):
            gi = self.grad(i, self.x[i], None if zeta0 is None else zeta0[i])
            self.g[i] = gi
            self.z[i] = gi

    def _deliver(self, i, r):
        for e in range(int(self.R.rowptr[i]), int(self.R.rowptr[i + 1])):
            keep = []
            for (arrival, stamp, payload) in self.inbox_v[e]:
                if arrival <= r:
                    if stamp > self.tau_v[e]:            # largest stamp received wins
                        self.tau_v[e], self.v_recv[e] = stamp, payload
                else:
                    keep.append((arrival, stamp, payload))
            self.inbox_v[e] = keep
        for e in range(int(self.C.rowptr[i]), int(self.C.rowptr[i + 1])):
            keep = []
            for (arrival, stamp, payload) in self.inbox_rho[e]:
                if arrival <= r:
                    if self.increments_only:             # negative control: add up what arrives
                        self.rho_recv[e] = self.rho_recv[e] + payload
                        self.tau_rho[e] = max(self.tau_rho[e], stamp)
                    elif stamp > self.tau_rho[e]:
                        self.tau_rho[e], self.rho_recv[e] = stamp, payload
                else:
                    keep.append((arrival, stamp, payload))
            self.inbox_rho[e] = keep

    def activate(self, i, r, codes_r, codes_c, idx):
        """One pass of the while-loop body of Algorithm 1 for node i in round r."""
        R, C, alpha = self.R, self.C, self.alpha
        self._deliver(i, r)
        # (S1) local descent
        v = self.x[i] - alpha * self.z[i]
        # (S2a) consensus mix over N_i^in(W)
        x_new = R.diag[i] * v
        for e in range(int(R.rowptr[i]), int(R.rowptr[i + 1])):
            x_new = x_new + R.w[e] * self.v_recv[e]
            self.used_tau_v.append(self.tau_v[e])
        # stochastic gradient at the new point, fresh sample
        g_new = self.grad(i, x_new, idx)
        # (S2b) robust tracking over N_i^in(A)
        zh = self.z[i]
        for e in range(int(C.rowptr[i]), int(C.rowptr[i + 1])):
            zh = zh + (self.rho_recv[e] - self.rho_tilde[e])
            self.used_tau_rho.append(self.tau_rho[e])
        zh = zh + g_new - self.g[i]
        # (S2c) keep a_ii, accumulate a_ji into the running sums
        z_new = C.diag[i] * zh
        for f in self.out_C[i]:
            self.rho[f] = self.rho[f] + C.w[f] * zh
        # (S5) counter (done here so that the packets carry stamp t+1)
        self.t[i] += 1
        stamp = self.t[i]
        # (S3) send, subject to the schedule's drop / delay codes
        for f, d in zip(self.out_R[i], codes_r):
            if d >= 0:
                self.inbox_v[f].append((r + 1 + int(d), stamp, v))
        for f, d in zip(self.out_C[i], codes_c):
            if d >= 0:
                payload = C.w[f] * zh if self.increments_only else self.rho[f]
                self.inbox_rho[f].append((r + 1 + int(d), stamp, payload))
        # (S4) buffer
        for e in range(int(C.rowptr[i]), int(C.rowptr[i + 1])):
            self.rho_tilde[e] = self.rho_recv[e]
        self.x[i], self.z[i], self.g[i], self.v_latest[i] = x_new, z_new, g_new, v
        self.activations += 1

    # -- views -----------------------------------------------------------------------------
    def X(self):
        return np.stack(self.x)

    def Z(self):
        return np.stack(self.z)

    def G(self):
        return np.stack(self.g)

    def RHO(self):
        return np.stack(self.rho) if self.rho else np.zeros((0, self.p), self.dtype)

    def RHO_TILDE(self):
        return np.stack(self.rho_tilde) if self.rho_tilde else np.zeros((0, self.p), self.dtype)

    def conservation_residual(self):
        """sum_i z_i + sum_e (rho_e - rho_tilde_e) - sum_i g_i  (Lemma 3: identically 0)."""
        tot = self.zero.copy()
        for i in range(self.n):
            tot = tot + self.z[i] - self.g[i]
        for e in range(len(self.rho)):
            tot = tot + (self.rho[e] - self.rho_tilde[e])
        return tot


def run_schedule(orc: RFastOracle, sch, K=None, after_round=None):
    """Drive the oracle over rounds [orc.round, K) of a raw schedule.

    sch: object with K, act_ptr, act_node, send_r, send_c, batch, batch_idx (see the
    generator module).  Send codes are laid out event by event, each event listing the
    out-edges of its node by ascending receiver.  Minibatch indices: first n*B entries are
    the initial samples zeta^0, then B per event."""
    n, B = orc.n, int(sch.batch)
    K = sch.K if K is None else K
    if orc.z[0] is None:
        zeta0 = None
        if B > 0:
            zeta0 = [np.asarray(sch.batch_idx[i * B:(i + 1) * B]) for i in range(n)]
        orc.init_gradients(zeta0)
    outdeg_r = [len(o) for o in orc.out_R]
    outdeg_c = [len(o) for o in orc.out_C]
    # offsets of each event's send codes
    pr = pc = 0
    ev0 = int(sch.act_ptr[orc.round])
    for ev in range(ev0):
        pr += outdeg_r[int(sch.act_node[ev])]
        pc += outdeg_c[int(sch.act_node[ev])]
    alpha_round = getattr(sch, "alpha_round", None)
    for r in range(orc.round, K):
        if alpha_round is not None:          # time-varying step size gamma^r (Algorithm 2, S.1)
            orc.alpha = float(alpha_round[r])
        for ev in range(int(sch.act_ptr[r]), int(sch.act_ptr[r + 1])):
            i = int(sch.act_node[ev])
            cr = sch.send_r[pr:pr + outdeg_r[i]]
            cc = sch.send_c[pc:pc + outdeg_c[i]]
            pr += outdeg_r[i]
            pc += outdeg_c[i]
            idx = np.asarray(sch.batch_idx[(n + ev) * B:(n + ev + 1) * B]) if B > 0 else None
            orc.activate(i, r, cr, cc, idx)
        orc.round = r + 1
        if after_round is not None:
            after_round(orc, r)
    return orc


def from_workload(wl, grad, dtype=np.float64, **kw):
    """Oracle for a workload object (fields n, p, alpha, G_R, G_C, x0) and a gradient callable."""
    return RFastOracle(wl.n, wl.p, wl.alpha, wl.G_R, wl.G_C, grad, wl.x0, dtype=dtype, **kw)


def rel_l2(a, ref, ref0_norm=0.0):
    """Relative L2 (Frobenius) error with the denominator floored at 1e-3 of the reference's
    initial norm, so that a tracker that vanishes at an optimum does not blow the ratio up."""
    a = np.asarray(a, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = max(float(np.linalg.norm(ref)), 1e-3 * float(ref0_norm), 1e-300)
    return float(np.linalg.norm(a - ref)) / den

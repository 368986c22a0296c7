"""ctypes binding of librfast.so: argument marshalling only.

Every step of the R-FAST activation path runs inside the CUDA library; this module turns
numpy arrays into the plain pointers of include/rfast.h and back.  The functions carry the
names of the C entry points.  There is no fallback: if the shared library is missing, or no
CUDA device is present, the calls raise.
"""

from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librfast.so")

OK, EINVAL, EGRAPH, ESCHED, ENOMEM, ECUDA, ETIMEOUT, ESTATE = 0, -1, -2, -3, -4, -5, -6, -7
_ERRNAMES = {-1: "EINVAL", -2: "EGRAPH", -3: "ESCHED", -4: "ENOMEM", -5: "ECUDA", -6: "ETIMEOUT", -7: "ESTATE"}

MODEL_IDS = {"quad_diag": 0, "least_squares": 1, "softmax": 2, "mlp": 3, "logistic_sparse": 4}

STATE_X, STATE_Y, STATE_G_LAST, STATE_RHO_LATEST, STATE_RHO_BUF = 0, 1, 2, 3, 4
STATE_T_LOCAL, STATE_USED_TAU_V, STATE_USED_TAU_RHO, STATE_TAU_V_END, STATE_TAU_RHO_END, STATE_ROUND = 5, 6, 7, 8, 9, 10
Q_ROUND, Q_EVENTS_TOTAL, Q_EVENTS_RUN, Q_LAUNCHES, Q_BYTES_RUN, Q_V_SLOTS, Q_RHO_SLOTS = 0, 1, 2, 3, 4, 5, 6
Q_DEVICE_BYTES, Q_N_USED_TAU_V, Q_N_USED_TAU_RHO, Q_BYTES_TOTAL = 7, 8, 9, 10
Q_METHOD_BYTES_RUN, Q_METHOD_BYTES_TOTAL = 11, 12
STATE_V_LATEST, STATE_V_HELD, STATE_TAU_V, STATE_TAU_RHO = 11, 12, 13, 14
_FLOAT_VIEWS = (STATE_X, STATE_Y, STATE_G_LAST, STATE_RHO_LATEST, STATE_RHO_BUF, STATE_V_LATEST)
NOT_HELD = 1
GRAPH_R, GRAPH_C = 0, 1


class RFastError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"rfast: {_ERRNAMES.get(code, code)}: {msg}")
        self.code = code


class _Graph(C.Structure):
    _fields_ = [("n_edges", C.c_int32), ("rowptr", C.c_void_p), ("col", C.c_void_p),
                ("w", C.c_void_p), ("diag", C.c_void_p)]


class _Problem(C.Structure):
    _fields_ = [("n", C.c_int32), ("root", C.c_int32), ("p", C.c_int64), ("alpha", C.c_float),
                ("l2", C.c_float), ("G_R", _Graph), ("G_C", _Graph), ("model", C.c_int32),
                ("batch", C.c_int32), ("rows", C.c_int32), ("n_features", C.c_int32),
                ("n_classes", C.c_int32), ("n_hidden", C.c_int32),
                ("quad_d", C.c_void_p), ("quad_b", C.c_void_p), ("feat", C.c_void_p),
                ("target", C.c_void_p), ("label", C.c_void_p), ("sp_rowptr", C.c_void_p),
                ("sp_col", C.c_void_p), ("sp_val", C.c_void_p), ("x0", C.c_void_p),
                ("compensated", C.c_int32), ("tracker", C.c_int32)]


class _Schedule(C.Structure):
    _fields_ = [("K", C.c_int32), ("act_ptr", C.c_void_p), ("act_node", C.c_void_p),
                ("n_send_r", C.c_int64), ("send_r", C.c_void_p), ("n_send_c", C.c_int64),
                ("send_c", C.c_void_p), ("n_batch_idx", C.c_int64), ("batch_idx", C.c_void_p),
                ("alpha_round", C.c_void_p)]


_lib = None


def lib():
    """The loaded shared library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it first "
                               "(python -m paper_2307_11617_b200.build); there is no fallback path")
        L = C.CDLL(LIB_PATH)
        L.rfast_create.argtypes = [C.POINTER(_Problem), C.c_void_p, C.POINTER(C.c_void_p)]
        L.rfast_load_schedule.argtypes = [C.c_void_p, C.POINTER(_Schedule)]
        L.rfast_append_schedule.argtypes = [C.c_void_p, C.POINTER(_Schedule)]
        L.rfast_compile_append_check.argtypes = [C.POINTER(_Problem), C.POINTER(_Schedule), C.POINTER(_Schedule),
                                                 C.c_void_p, C.c_char_p, C.c_size_t]
        L.rfast_run.argtypes = [C.c_void_p, C.c_int32, C.c_int]
        L.rfast_read_state.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_size_t]
        L.rfast_reset.argtypes = [C.c_void_p]
        L.rfast_sync.argtypes = [C.c_void_p]
        L.rfast_query.argtypes = [C.c_void_p, C.c_int]
        L.rfast_query.restype = C.c_int64
        L.rfast_destroy.argtypes = [C.c_void_p]
        L.rfast_destroy.restype = None
        L.rfast_last_error.argtypes = [C.c_void_p]
        L.rfast_last_error.restype = C.c_char_p
        L.rfast_version.restype = C.c_char_p
        L.rfast_compile_host.argtypes = [C.POINTER(_Problem), C.POINTER(_Schedule)] + [C.c_void_p] * 5 + \
            [C.c_char_p, C.c_size_t]
        L.rfast_compile_digest.argtypes = [C.POINTER(_Problem), C.POINTER(_Schedule), C.POINTER(C.c_uint64), C.c_char_p, C.c_size_t]
        L.rfast_set_option.argtypes = [C.c_void_p, C.c_int, C.c_int64]
        L.rfast_checkpoint_size.argtypes = [C.c_void_p]
        L.rfast_checkpoint_size.restype = C.c_int64
        L.rfast_checkpoint_save.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t]
        L.rfast_checkpoint_load.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t]
        L.rfast_diagnostics.argtypes = [C.c_void_p, C.c_void_p, C.c_int32]
        L.rfast_seek.argtypes = [C.c_void_p, C.c_int32]
        L.rfast_snapshot.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.rfast_snapshot_wait.argtypes = [C.c_void_p]
        L.rfast_write_state.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_size_t]
        L.rfast_read_packet.argtypes = [C.c_void_p, C.c_int, C.c_int32, C.c_int32, C.c_void_p, C.c_size_t]
        L.rfast_write_packet.argtypes = [C.c_void_p, C.c_int, C.c_int32, C.c_int32, C.c_void_p, C.c_size_t]
        L.rfast_ls_gradient_static.argtypes = [C.c_void_p] * 4 + [C.c_int32, C.c_int32, C.c_float,
                                               C.c_void_p, C.c_char_p, C.c_size_t]
        _lib = L
    return _lib


def _arr(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _graph(g, keep):
    rowptr, col = _arr(g.rowptr, np.int32), _arr(g.col, np.int32)
    w, diag = _arr(g.w, np.float32), _arr(g.diag, np.float32)
    keep += [rowptr, col, w, diag]
    return _Graph(len(col), _ptr(rowptr), _ptr(col), _ptr(w), _ptr(diag))


def _problem(wl, keep):
    """wl: object with n, p, root, alpha, l2, G_R, G_C, model (name), batch, rows, dims, data, x0."""
    P = _Problem()
    P.n, P.root, P.p, P.alpha, P.l2 = int(wl.n), int(wl.root), int(wl.p), float(wl.alpha), float(wl.l2)
    P.G_R, P.G_C = _graph(wl.G_R, keep), _graph(wl.G_C, keep)
    P.model = MODEL_IDS[wl.model] if isinstance(wl.model, str) else int(wl.model)
    P.batch, P.rows = int(wl.batch), int(wl.rows)
    P.compensated = int(getattr(wl, "compensated", 0) or 0)     # False/True/2 -> 0/1/2
    P.tracker = int(getattr(wl, "tracker", 0) or 0)             # 0 running sums, 1 mass buckets
    dims = getattr(wl, "dims", {}) or {}
    P.n_features = int(dims.get("n_features", 0))
    P.n_classes = int(dims.get("n_classes", 0))
    P.n_hidden = int(dims.get("n_hidden", 0))
    data = getattr(wl, "data", {}) or {}
    spec = {"quad_d": ("d", np.float32), "quad_b": ("b", np.float32), "feat": ("feat", np.float32),
            "target": ("target", np.float32), "label": ("label", np.int32),
            "sp_rowptr": ("sp_rowptr", np.int64), "sp_col": ("sp_col", np.int32),
            "sp_val": ("sp_val", np.float32)}
    for field, (key, dt) in spec.items():
        if key in data and data[key] is not None:
            a = _arr(data[key], dt)
            keep.append(a)
            setattr(P, field, _ptr(a))
    if getattr(wl, "x0", None) is not None:
        a = _arr(wl.x0, np.float32)
        keep.append(a)
        P.x0 = _ptr(a)
    return P


def _schedule(s, keep):
    S = _Schedule()
    act_ptr, act_node = _arr(s.act_ptr, np.int32), _arr(s.act_node, np.int32)
    send_r, send_c = _arr(s.send_r, np.int8), _arr(s.send_c, np.int8)
    bidx = _arr(s.batch_idx, np.int32)
    keep += [act_ptr, act_node, send_r, send_c, bidx]
    S.K = int(s.K)
    S.act_ptr, S.act_node = _ptr(act_ptr), _ptr(act_node)
    S.n_send_r, S.send_r = len(send_r), _ptr(send_r)
    S.n_send_c, S.send_c = len(send_c), _ptr(send_c)
    S.n_batch_idx, S.batch_idx = len(bidx), _ptr(bidx)
    if getattr(s, "alpha_round", None) is not None:
        ar = _arr(s.alpha_round, np.float32)
        if len(ar) != int(s.K):
            raise ValueError("alpha_round must hold one step size per round")
        keep.append(ar)
        S.alpha_round = _ptr(ar)
    return S


def _check(rc, handle=None):
    if rc != OK:
        raise RFastError(rc, lib().rfast_last_error(handle).decode())


def rfast_version() -> str:
    return lib().rfast_version().decode()


def rfast_create(wl, cuda_stream: int = 0) -> int:
    """Returns an opaque handle.  cuda_stream: a cudaStream_t as an integer (0: default stream)."""
    keep = []
    P = _problem(wl, keep)
    h = C.c_void_p()
    _check(lib().rfast_create(C.byref(P), C.c_void_p(cuda_stream), C.byref(h)))
    return h.value


def rfast_load_schedule(handle, s) -> None:
    keep = []
    S = _schedule(s, keep)
    _check(lib().rfast_load_schedule(handle, C.byref(S)), handle)


def rfast_append_schedule(handle, more) -> None:
    keep = []
    S = _schedule(more, keep)
    _check(lib().rfast_append_schedule(handle, C.byref(S)), handle)


def rfast_run(handle, rounds: int, sync: bool = True) -> None:
    _check(lib().rfast_run(handle, int(rounds), 1 if sync else 0), handle)


def rfast_reset(handle) -> None:
    _check(lib().rfast_reset(handle), handle)


def rfast_sync(handle) -> None:
    _check(lib().rfast_sync(handle), handle)


def rfast_query(handle, what: int) -> int:
    v = lib().rfast_query(handle, int(what))
    if v < 0:
        _check(int(v), handle)
    return int(v)


def rfast_read_state(handle, which: int, shape, out=None) -> np.ndarray:
    """shape: the view's shape; float views are float32, integer views int32."""
    dt = np.float32 if which in _FLOAT_VIEWS else np.int32
    if out is None:
        out = np.empty(shape, dtype=dt)
    assert out.dtype == dt and out.flags.c_contiguous
    _check(lib().rfast_read_state(handle, int(which), _ptr(out), out.nbytes), handle)
    return out


def rfast_snapshot(handle, x_out: np.ndarray, y_out: np.ndarray) -> None:
    """x_out, y_out: C-contiguous float32 [n][p] host arrays (page-locked for an overlapped transfer)
    that must stay alive until rfast_snapshot_wait."""
    for a in (x_out, y_out):
        if a.dtype != np.float32 or not a.flags["C_CONTIGUOUS"]:
            raise ValueError("snapshot destinations must be C-contiguous float32 arrays")
    _check(lib().rfast_snapshot(handle, _ptr(x_out), _ptr(y_out)), handle)


def rfast_snapshot_wait(handle) -> None:
    _check(lib().rfast_snapshot_wait(handle), handle)


def rfast_seek(handle, rnd: int) -> None:
    _check(lib().rfast_seek(handle, int(rnd)), handle)


def rfast_write_state(handle, which: int, values) -> None:
    """values: the float view as an array (converted to contiguous float32)."""
    a = _arr(values, np.float32)
    _check(lib().rfast_write_state(handle, int(which), _ptr(a), a.nbytes), handle)


def rfast_read_packet(handle, graph: int, ident: int, stamp: int, p: int):
    """Payload (float32 [p]) of one packet version, or None when the engine does not hold it."""
    out = np.empty(int(p), dtype=np.float32)
    rc = lib().rfast_read_packet(handle, int(graph), int(ident), int(stamp), _ptr(out), out.nbytes)
    if rc == NOT_HELD:
        return None
    _check(rc, handle)
    return out


def rfast_write_packet(handle, graph: int, ident: int, stamp: int, values) -> bool:
    """True when the version is held and was written, False when the engine keeps no row for it."""
    a = _arr(values, np.float32)
    rc = lib().rfast_write_packet(handle, int(graph), int(ident), int(stamp), _ptr(a), a.nbytes)
    if rc == NOT_HELD:
        return False
    _check(rc, handle)
    return True


def rfast_destroy(handle) -> None:
    lib().rfast_destroy(handle)


def rfast_compile_host(wl, s):
    """Host-only schedule compilation (no device needed).  Returns a dict of int arrays."""
    keep = []
    P, S = _problem(wl, keep), _schedule(s, keep)
    indeg_r = np.diff(np.asarray(wl.G_R.rowptr)).astype(np.int64)
    indeg_c = np.diff(np.asarray(wl.G_C.rowptr)).astype(np.int64)
    nodes = np.clip(np.asarray(s.act_node, dtype=np.int64), 0, int(wl.n) - 1)   # bad ids are the library's to reject
    ev = len(nodes)
    used_v = np.empty(int(indeg_r[nodes].sum()), np.int32)
    used_r = np.empty(int(indeg_c[nodes].sum()), np.int32)
    v_ver = np.empty((ev, 3), np.int32)
    rho_ver = np.empty((len(s.send_c), 3), np.int32)
    counts = np.zeros(4, np.int64)
    err = C.create_string_buffer(512)
    rc = lib().rfast_compile_host(C.byref(P), C.byref(S), _ptr(used_v), _ptr(used_r), _ptr(v_ver),
                                  _ptr(rho_ver), _ptr(counts), err, 512)
    if rc != OK:
        raise RFastError(rc, err.value.decode())
    return {"used_tau_v": used_v, "used_tau_rho": used_r, "v_ver": v_ver, "rho_ver": rho_ver,
            "v_rows": int(counts[0]), "rho_rows": int(counts[1]), "events": int(counts[2]),
            "streams": int(counts[3])}


def rfast_compile_digest(wl, s) -> int:
    """One number for everything the compiled schedule drives the kernels with (host only)."""
    keep = []
    P, S = _problem(wl, keep), _schedule(s, keep)
    out = C.c_uint64(0)
    err = C.create_string_buffer(512)
    rc = lib().rfast_compile_digest(C.byref(P), C.byref(S), C.byref(out), err, 512)
    if rc != OK:
        raise RFastError(rc, err.value.decode())
    return int(out.value)


def rfast_compile_append_check(wl, first, more):
    """Host only: `first` loaded open-ended and `more` appended keeps every row of `first` in place
    and consumes the stamps of the whole schedule.  Returns the six row counts; raises otherwise."""
    keep = []
    P, S1, S2 = _problem(wl, keep), _schedule(first, keep), _schedule(more, keep)
    counts = np.zeros(6, np.int64)
    err = C.create_string_buffer(512)
    rc = lib().rfast_compile_append_check(C.byref(P), C.byref(S1), C.byref(S2), _ptr(counts), err, 512)
    if rc != OK:
        raise RFastError(rc, err.value.decode())
    return {"first": (int(counts[0]), int(counts[1])), "appended": (int(counts[2]), int(counts[3])),
            "whole": (int(counts[4]), int(counts[5]))}


OPT_PERSISTENT, OPT_GRAPHS, OPT_WAIT_LIMIT_MS, OPT_PHANTOM_ARRIVALS, OPT_ONE_PASS, OPT_CLUSTER_SIZE, OPT_OPEN_END = 0, 1, 2, 3, 4, 5, 6


def rfast_set_option(handle, option: int, value: int) -> None:
    _check(lib().rfast_set_option(handle, int(option), int(value)), handle)


def rfast_checkpoint_save(handle) -> np.ndarray:
    """The handle's complete state as an opaque byte array (see rfast_checkpoint_save in rfast.h)."""
    size = lib().rfast_checkpoint_size(handle)
    if size < 0:
        _check(int(size), handle)
    blob = np.empty(size, dtype=np.uint8)
    _check(lib().rfast_checkpoint_save(handle, _ptr(blob), blob.nbytes), handle)
    return blob


def rfast_checkpoint_load(handle, blob: np.ndarray) -> None:
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    _check(lib().rfast_checkpoint_load(handle, _ptr(blob), blob.nbytes), handle)


def rfast_diagnostics(handle, full: bool = True) -> dict:
    """Consensus error, norm of the mean iterate, conservation residual (Lemma 3) and its scale,
    tracker norm, all computed on the device in one pass over the state; with full=True also the
    full gradient, the merit function and the objective at the mean iterate (a pass over every
    row of every shard)."""
    n_out = 8 if full else 5
    out = np.full(8, np.nan, dtype=np.float64)
    _check(lib().rfast_diagnostics(handle, _ptr(out), n_out), handle)
    return {"consensus_error": out[0], "xbar_norm": out[1], "conservation_residual": out[2],
            "gradient_sum_max": out[3], "tracker_norm": out[4], "full_gradient_norm": out[5],
            "merit": out[6], "objective": out[7]}


STATIC_MAX_ROWS = 65536


def rfast_ls_gradient_static(d_feat: int, d_target: int, d_x: int, d_grad: int, rows: int,
                             n_features: int, l2: float = 0.0, cuda_stream: int = 0) -> None:
    """Full-shard least-squares gradient without any device allocation, for callers that may not
    allocate (a framework that owns all GPU memory, a loop that cannot afford cudaMalloc's
    device-wide synchronisation).  All four arguments are raw DEVICE addresses (integers) of
    caller-owned fp32 arrays: feat [rows][n_features], target [rows], x [n_features] in, grad
    [n_features] out.  Enqueued on cuda_stream; the caller synchronises.  At most
    STATIC_MAX_ROWS rows; calls that overlap on the GPU race on the shared built-in scratch."""
    err = C.create_string_buffer(256)
    rc = lib().rfast_ls_gradient_static(C.c_void_p(d_feat), C.c_void_p(d_target), C.c_void_p(d_x),
                                        C.c_void_p(d_grad), int(rows), int(n_features), float(l2),
                                        C.c_void_p(cuda_stream), err, 256)
    if rc != OK:
        raise RFastError(rc, err.value.decode())


class Engine:
    """Convenience wrapper owning one handle."""

    def __init__(self, wl, cuda_stream: int = 0):
        self.n, self.p = int(wl.n), int(wl.p)
        self.n_edges_c = len(wl.G_C.col)
        self.n_edges_r = len(wl.G_R.col)
        self.h = rfast_create(wl, cuda_stream)
        self.K = 0

    def load_schedule(self, s):
        rfast_load_schedule(self.h, s)
        self.K = int(s.K)

    def append_schedule(self, more):
        rfast_append_schedule(self.h, more)
        self.K += int(more.K)

    def run(self, rounds=None, sync=True):
        rfast_run(self.h, self.K - self.query(Q_ROUND) if rounds is None else rounds, sync)

    def reset(self):
        rfast_reset(self.h)

    def sync(self):
        rfast_sync(self.h)

    def query(self, what):
        return rfast_query(self.h, what)

    def read(self, which, out=None):
        n, p = self.n, self.p
        shape = {STATE_X: (n, p), STATE_Y: (n, p), STATE_G_LAST: (n, p),
                 STATE_RHO_LATEST: (self.n_edges_c, p), STATE_RHO_BUF: (self.n_edges_c, p),
                 STATE_T_LOCAL: (n,), STATE_TAU_V_END: (self.n_edges_r,),
                 STATE_TAU_RHO_END: (self.n_edges_c,), STATE_ROUND: (1,),
                 STATE_V_LATEST: (n, p), STATE_V_HELD: (n,), STATE_TAU_V: (self.n_edges_r,),
                 STATE_TAU_RHO: (self.n_edges_c,)}.get(which)
        if which == STATE_USED_TAU_V:
            shape = (self.query(Q_N_USED_TAU_V),)
        if which == STATE_USED_TAU_RHO:
            shape = (self.query(Q_N_USED_TAU_RHO),)
        return rfast_read_state(self.h, which, shape, out)

    def seek(self, rnd):
        rfast_seek(self.h, rnd)

    def write(self, which, values):
        rfast_write_state(self.h, which, values)

    def read_packet(self, graph, ident, stamp):
        return rfast_read_packet(self.h, graph, ident, stamp, self.p)

    def write_packet(self, graph, ident, stamp, values):
        return rfast_write_packet(self.h, graph, ident, stamp, values)

    def set_option(self, option, value):
        rfast_set_option(self.h, option, value)

    def checkpoint(self):
        return rfast_checkpoint_save(self.h)

    def restore(self, blob):
        rfast_checkpoint_load(self.h, blob)

    def snapshot(self, x_out, y_out):
        if x_out.shape != (self.n, self.p) or y_out.shape != (self.n, self.p):
            raise ValueError("snapshot destinations must be [n][p]")
        rfast_snapshot(self.h, x_out, y_out)

    def snapshot_wait(self):
        rfast_snapshot_wait(self.h)

    def diagnostics(self, full=True):
        return rfast_diagnostics(self.h, full)

    def close(self):
        if self.h:
            rfast_destroy(self.h)
            self.h = None

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

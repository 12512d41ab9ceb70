"""CPU oracle of the synchronous parameter-server step with backup workers.

TEST INFRASTRUCTURE ONLY: a plain fp64 restatement of Section 3 / Algorithm 4 of
"Revisiting Distributed Synchronous SGD" (arXiv 1604.00981), in C
(`sgdb_oracle.c`), wrapped here with ctypes and numpy.  It shares nothing with
the CUDA library and does not import it.  Only tests, the smoke check and the
CPU-baseline leg of the benchmark may use it.

Every function takes and returns numpy arrays; parameters and optimizer state are
fp64, gradients are fp32 arrays or uint16 arrays of bf16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sgdb_oracle.c")
_LIB = os.path.join(_HERE, "libsgdb_oracle.so")

OK, INVALID, INSUFFICIENT = 0, 1, 2
F32, BF16 = 0, 1
SGD, MOMENTUM, RMSPROP, ADAM, ADAGRAD = 0, 1, 2, 3, 4


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, no fast-math) into a shared object beside its source."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.run(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-o", tmp, _SRC, "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Opt(ctypes.Structure):
    _fields_ = [
        ("kind", ctypes.c_int32),
        ("lr", ctypes.c_double),
        ("momentum", ctypes.c_double),
        ("decay", ctypes.c_double),
        ("beta1", ctypes.c_double),
        ("beta2", ctypes.c_double),
        ("eps", ctypes.c_double),
        ("step", ctypes.c_int64),
    ]


@dataclass
class Opt:
    """Optimizer rule and hyper-parameters (see oracle_update in sgdb_oracle.c)."""

    kind: int = SGD
    lr: float = 0.1
    momentum: float = 0.0
    decay: float = 0.0
    beta1: float = 0.0
    beta2: float = 0.0
    eps: float = 0.0
    step: int = 1

    def _c(self) -> _Opt:
        return _Opt(self.kind, self.lr, self.momentum, self.decay, self.beta1, self.beta2, self.eps, self.step)


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        for name in (
            "oracle_select",
            "oracle_aggregate",
            "oracle_update",
            "oracle_step",
            "oracle_accumulate_arrival",
            "oracle_step_ema",
            "oracle_accumulate_arrival_ema",
            "oracle_select_deadline",
            "oracle_step_deadline",
            "oracle_accumulate_arrival_deadline",
            "oracle_accumulate_close",
            "oracle_select_grouped",
            "oracle_step_grouped",
        ):
            getattr(lib, name).restype = ctypes.c_int
        lib.oracle_ema.restype = None
        lib.oracle_learning_rate.restype = ctypes.c_double
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _grad(grad):
    """(array, dtype code) for an fp32 matrix or a uint16 matrix of bf16 bit patterns."""
    if grad.dtype == np.float32:
        return np.ascontiguousarray(grad), F32
    if grad.dtype == np.uint16:
        return np.ascontiguousarray(grad), BF16
    raise TypeError("gradients must be float32 or uint16 (bf16 bits), got %s" % grad.dtype)


def select(arrival, tags, t: int, N: int, b: int):
    """Section 3 / Algorithm 4: the first N gradients tagged t.  Returns (status, mask, order, n_valid)."""
    W = N + b
    arrival = np.ascontiguousarray(arrival, dtype=np.float32)
    tags = np.ascontiguousarray(tags, dtype=np.int32)
    assert arrival.shape == (W,) and tags.shape == (W,)
    mask = np.zeros(W, dtype=np.uint8)
    order = np.full(N, -1, dtype=np.int32)
    n_valid = ctypes.c_int32(0)
    rc = _load().oracle_select(
        _p(arrival), _p(tags), ctypes.c_int32(t), ctypes.c_int32(N), ctypes.c_int32(b),
        _p(mask), _p(order), ctypes.byref(n_valid),
    )
    return rc, mask, order, n_valid.value


def aggregate(grad, P: int, order, ld: int | None = None):
    """Mean of the rows named in `order` (Algorithm 4's sum over the kept set, divided by N), fp64 [P]."""
    g, dt = _grad(grad)
    ld = g.shape[1] if ld is None else ld
    order = np.ascontiguousarray(order, dtype=np.int32)
    mean = np.zeros(P, dtype=np.float64)
    rc = _load().oracle_aggregate(
        _p(g), ctypes.c_int(dt), ctypes.c_int64(P), ctypes.c_int64(ld), ctypes.c_int32(len(order)),
        _p(order), _p(mean),
    )
    assert rc == OK, rc
    return mean


def update(theta, s0, s1, mean, opt: Opt):
    """Apply the optimizer rule in place to fp64 theta / state arrays."""
    for a in (theta, s0, s1):
        assert a is None or (a.dtype == np.float64 and a.flags.c_contiguous)
    mean = np.ascontiguousarray(mean, dtype=np.float64)
    c = opt._c()
    rc = _load().oracle_update(_p(theta), _p(s0), _p(s1), _p(mean), ctypes.c_int64(len(theta)), ctypes.byref(c))
    assert rc == OK, rc


def step(grad, P: int, arrival, tags, t: int, N: int, b: int, theta, s0, s1, opt: Opt, ld: int | None = None):
    """One iteration of Algorithm 4 on fp64 theta/state (in place).  Returns (status, mask, order, n_valid)."""
    W = N + b
    g, dt = _grad(grad)
    ld = g.shape[1] if ld is None else ld
    arrival = np.ascontiguousarray(arrival, dtype=np.float32)
    tags = np.ascontiguousarray(tags, dtype=np.int32)
    for a in (theta, s0, s1):
        assert a is None or (a.dtype == np.float64 and a.flags.c_contiguous)
    mask = np.zeros(W, dtype=np.uint8)
    order = np.full(N, -1, dtype=np.int32)
    n_valid = ctypes.c_int32(0)
    c = opt._c()
    rc = _load().oracle_step(
        _p(g), ctypes.c_int(dt), ctypes.c_int64(P), ctypes.c_int64(ld), _p(arrival), _p(tags),
        ctypes.c_int32(t), ctypes.c_int32(N), ctypes.c_int32(b), _p(theta), _p(s0), _p(s1),
        ctypes.byref(c), _p(mask), _p(order), ctypes.byref(n_valid),
    )
    return rc, mask, order, n_valid.value


def ema(avg, theta, alpha: float) -> None:
    """avg <- alpha * avg + (1 - alpha) * theta, in place on the fp64 array avg (Section 1.1)."""
    assert avg.dtype == np.float64 and avg.flags.c_contiguous
    theta = np.ascontiguousarray(theta, dtype=np.float64)
    _load().oracle_ema(_p(avg), _p(theta), ctypes.c_int64(len(avg)), ctypes.c_double(alpha))


def step_ema(grad, P: int, arrival, tags, t: int, N: int, b: int, theta, s0, s1, opt: Opt, avg, alpha: float,
             ld: int | None = None):
    """One iteration of Algorithm 4 with its last line (the average of the pre-update parameters)."""
    W = N + b
    g, dt = _grad(grad)
    ld = g.shape[1] if ld is None else ld
    arrival = np.ascontiguousarray(arrival, dtype=np.float32)
    tags = np.ascontiguousarray(tags, dtype=np.int32)
    for a in (theta, s0, s1, avg):
        assert a is None or (a.dtype == np.float64 and a.flags.c_contiguous)
    mask = np.zeros(W, dtype=np.uint8)
    order = np.full(N, -1, dtype=np.int32)
    n_valid = ctypes.c_int32(0)
    c = opt._c()
    rc = _load().oracle_step_ema(
        _p(g), ctypes.c_int(dt), ctypes.c_int64(P), ctypes.c_int64(ld), _p(arrival), _p(tags),
        ctypes.c_int32(t), ctypes.c_int32(N), ctypes.c_int32(b), _p(theta), _p(s0), _p(s1),
        ctypes.byref(c), _p(avg), ctypes.c_double(alpha), _p(mask), _p(order), ctypes.byref(n_valid),
    )
    return rc, mask, order, n_valid.value


def learning_rate(gamma0: float, beta: float, t: int, N: int, T: float) -> float:
    """gamma0 * beta^(t N / (2 T)) (Appendix A.2, A.3)."""
    return float(_load().oracle_learning_rate(ctypes.c_double(gamma0), ctypes.c_double(beta), ctypes.c_int64(t),
                                              ctypes.c_int64(N), ctypes.c_double(T)))


def select_deadline(arrival, tags, t: int, deadline: float, n_min: int = 1):
    """Time-out rule: every gradient tagged t with arrival <= deadline.  Returns (status, mask, order[:n], n)."""
    arrival = np.ascontiguousarray(arrival, dtype=np.float32)
    tags = np.ascontiguousarray(tags, dtype=np.int32)
    W = len(arrival)
    mask = np.zeros(W, dtype=np.uint8)
    order = np.full(W, -1, dtype=np.int32)
    n = ctypes.c_int32(0)
    rc = _load().oracle_select_deadline(_p(arrival), _p(tags), ctypes.c_int32(t), ctypes.c_int32(W),
                                        ctypes.c_float(deadline), ctypes.c_int32(n_min), _p(mask), _p(order),
                                        ctypes.byref(n))
    return rc, mask, order[: n.value if rc == OK else 0], n.value


def step_deadline(grad, P: int, arrival, tags, t: int, deadline: float, n_min: int, theta, s0, s1, opt: Opt,
                  ld: int | None = None):
    """One iteration with the time-out rule on fp64 theta/state (in place).  Returns (status, mask, order[:n], n)."""
    g, dt = _grad(grad)
    ld = g.shape[1] if ld is None else ld
    arrival = np.ascontiguousarray(arrival, dtype=np.float32)
    tags = np.ascontiguousarray(tags, dtype=np.int32)
    W = len(arrival)
    for a in (theta, s0, s1):
        assert a is None or (a.dtype == np.float64 and a.flags.c_contiguous)
    mask = np.zeros(W, dtype=np.uint8)
    order = np.full(W, -1, dtype=np.int32)
    n = ctypes.c_int32(0)
    c = opt._c()
    rc = _load().oracle_step_deadline(
        _p(g), ctypes.c_int(dt), ctypes.c_int64(P), ctypes.c_int64(ld), _p(arrival), _p(tags), ctypes.c_int32(t),
        ctypes.c_int32(W), ctypes.c_float(deadline), ctypes.c_int32(n_min), _p(theta), _p(s0), _p(s1),
        ctypes.byref(c), _p(mask), _p(order), ctypes.byref(n),
    )
    return rc, mask, order[: n.value if rc == OK else 0], n.value


def new_server_state():
    """Fresh state of the arrival-by-arrival server: {|G|, gradients received, lowest open iteration}."""
    return np.zeros(3, dtype=np.int32)


def accumulate_arrival(row, row_tag: int, t: int, N: int, acc, state, theta, s0, s1, opt: Opt) -> int:
    """Algorithm 4's while loop for one received gradient.  Returns 0 dropped, 1 kept, 2 kept and updated."""
    r, dt = _grad(row)
    P = len(theta)
    assert acc.dtype == np.float64 and state.dtype == np.int32 and len(state) == 3
    outcome = ctypes.c_int32(-1)
    c = opt._c()
    rc = _load().oracle_accumulate_arrival(
        _p(r), ctypes.c_int(dt), ctypes.c_int32(row_tag), ctypes.c_int32(t), ctypes.c_int32(N),
        ctypes.c_int64(P), _p(acc), _p(state), _p(theta), _p(s0), _p(s1), ctypes.byref(c),
        ctypes.byref(outcome),
    )
    assert rc == OK, rc
    return outcome.value


def accumulate_arrival_ema(row, row_tag: int, t: int, N: int, acc, state, theta, s0, s1, opt: Opt, avg, alpha: float) -> int:
    """accumulate_arrival plus the parameter average, which moves only when the N-th gradient fires the update."""
    r, dt = _grad(row)
    P = len(theta)
    assert acc.dtype == np.float64 and state.dtype == np.int32 and len(state) == 3 and avg.dtype == np.float64
    outcome = ctypes.c_int32(-1)
    c = opt._c()
    rc = _load().oracle_accumulate_arrival_ema(
        _p(r), ctypes.c_int(dt), ctypes.c_int32(row_tag), ctypes.c_int32(t), ctypes.c_int32(N),
        ctypes.c_int64(P), _p(acc), _p(state), _p(theta), _p(s0), _p(s1), ctypes.byref(c), _p(avg),
        ctypes.c_double(alpha), ctypes.byref(outcome),
    )
    assert rc == OK, rc
    return outcome.value


def select_grouped(arrival, tags, group, t: int, M: int, N: int):
    """Two-level selection: the first N machine messages.  Returns (status, mask[W], group_order[N], order[:n_rows], n_valid)."""
    arrival = np.ascontiguousarray(arrival, dtype=np.float32)
    tags = np.ascontiguousarray(tags, dtype=np.int32)
    group = np.ascontiguousarray(group, dtype=np.int32)
    W = len(arrival)
    assert tags.shape == (W,) and group.shape == (W,)
    mask = np.zeros(W, dtype=np.uint8)
    group_order = np.full(N, -1, dtype=np.int32)
    order = np.full(W, -1, dtype=np.int32)
    n_rows, n_valid = ctypes.c_int32(0), ctypes.c_int32(0)
    rc = _load().oracle_select_grouped(_p(arrival), _p(tags), _p(group), ctypes.c_int32(t), ctypes.c_int32(W),
                                       ctypes.c_int32(M), ctypes.c_int32(N), _p(mask), _p(group_order), _p(order),
                                       ctypes.byref(n_rows), ctypes.byref(n_valid))
    return rc, mask, group_order, order[: n_rows.value if rc == OK else 0], n_valid.value


def step_grouped(grad, P: int, arrival, tags, group, t: int, M: int, N: int, theta, s0, s1, opt: Opt,
                 ld: int | None = None):
    """One server iteration over machine messages on fp64 theta/state (in place).
    Returns (status, mask[W], group_order[N], order[:n_rows], n_valid)."""
    g, dt = _grad(grad)
    ld = g.shape[1] if ld is None else ld
    arrival = np.ascontiguousarray(arrival, dtype=np.float32)
    tags = np.ascontiguousarray(tags, dtype=np.int32)
    group = np.ascontiguousarray(group, dtype=np.int32)
    W = len(arrival)
    for a in (theta, s0, s1):
        assert a is None or (a.dtype == np.float64 and a.flags.c_contiguous)
    mask = np.zeros(W, dtype=np.uint8)
    group_order = np.full(N, -1, dtype=np.int32)
    order = np.full(W, -1, dtype=np.int32)
    n_rows, n_valid = ctypes.c_int32(0), ctypes.c_int32(0)
    c = opt._c()
    rc = _load().oracle_step_grouped(
        _p(g), ctypes.c_int(dt), ctypes.c_int64(P), ctypes.c_int64(ld), _p(arrival), _p(tags), _p(group),
        ctypes.c_int32(t), ctypes.c_int32(W), ctypes.c_int32(M), ctypes.c_int32(N), _p(theta), _p(s0), _p(s1),
        ctypes.byref(c), _p(mask), _p(group_order), _p(order), ctypes.byref(n_rows), ctypes.byref(n_valid))
    return rc, mask, group_order, order[: n_rows.value if rc == OK else 0], n_valid.value


def accumulate_arrival_deadline(row, row_tag: int, row_arrival: float, t: int, deadline: float, acc, state) -> int:
    """Time-out rule, one received gradient: joins the set iff tagged t, t open, arrived by the deadline.  0 dropped, 1 added."""
    r, dt = _grad(row)
    assert acc.dtype == np.float64 and state.dtype == np.int32 and len(state) == 3
    outcome = ctypes.c_int32(-1)
    rc = _load().oracle_accumulate_arrival_deadline(
        _p(r), ctypes.c_int(dt), ctypes.c_int32(row_tag), ctypes.c_float(row_arrival), ctypes.c_int32(t),
        ctypes.c_float(deadline), ctypes.c_int64(len(acc)), _p(acc), _p(state), ctypes.byref(outcome))
    assert rc == OK, rc
    return outcome.value


def accumulate_close(t: int, n_min: int, acc, state, theta, s0, s1, opt: Opt, avg=None, alpha: float = 0.0):
    """The deadline of iteration t has passed.  Returns (status, outcome): outcome 2 = theta updated with the mean of the
    set, 0 = nothing done; status INSUFFICIENT (nothing changed) with fewer than n_min gradients in the set."""
    outcome = ctypes.c_int32(-1)
    c = opt._c()
    rc = _load().oracle_accumulate_close(
        ctypes.c_int32(t), ctypes.c_int32(n_min), ctypes.c_int64(len(theta)), _p(acc), _p(state), _p(theta), _p(s0), _p(s1),
        ctypes.byref(c), _p(avg), ctypes.c_double(alpha), ctypes.byref(outcome))
    return rc, outcome.value

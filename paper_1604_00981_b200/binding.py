"""ctypes binding of libsgdb.so: the same names and arguments as include/sgdb.h.

This layer only marshals arguments (tensor -> device pointer, current torch stream
-> cudaStream_t).  Every step of the path runs in the library's CUDA kernels; if
the library is missing the import fails: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsgdb.so")

SGDB_OK, SGDB_ERR_INVALID_ARG, SGDB_ERR_INSUFFICIENT, SGDB_ERR_CUDA, SGDB_ERR_UNSUPPORTED, SGDB_ERR_TIMEOUT = range(6)
SGDB_F32, SGDB_BF16 = 0, 1
SGDB_SGD, SGDB_MOMENTUM, SGDB_RMSPROP, SGDB_ADAM, SGDB_ADAGRAD = range(5)
SGDB_MAX_WORKERS = 1024
SGDB_MAX_SEGMENTS = 4096
_KINDS = {"sgd": SGDB_SGD, "momentum": SGDB_MOMENTUM, "rmsprop": SGDB_RMSPROP, "adam": SGDB_ADAM,
          "adagrad": SGDB_ADAGRAD}

EXPORTS = (
    "sgdb_select", "sgdb_aggregate", "sgdb_update", "sgdb_step", "sgdb_step_segmented",
    "sgdb_select_deadline", "sgdb_step_deadline", "sgdb_step_ema", "sgdb_ema", "sgdb_learning_rate", "sgdb_accumulate_arrival", "sgdb_accumulate_arrival_ema", "sgdb_step_host", "sgdb_step_host_workspace_bytes", "sgdb_step_host_static",
    "sgdb_select_grouped", "sgdb_step_grouped", "sgdb_step_segmented_ema", "sgdb_step_segmented_deadline",
    "sgdb_accumulate_arrival_deadline", "sgdb_accumulate_close", "sgdb_set_tuning", "sgdb_set_arrival_tuning", "sgdb_strerror", "sgdb_version",
    "sgdb_step_rows", "sgdb_step_rows_ordered", "sgdb_shard_range", "sgdb_enable_peer_access", "sgdb_selftest_bounded_wait", "sgdb_set_wait_limit_ns",
)
SGDB_STATIC_SCRATCH_BYTES = 8 << 20
SGDB_MAX_REPLICAS = 64
SGDB_SHARD_ALIGN = 64


class SgdbError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, sgdb_strerror(status), status))


class _COpt(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("lr", ctypes.c_float), ("momentum", ctypes.c_float),
                ("decay", ctypes.c_float), ("beta1", ctypes.c_float), ("beta2", ctypes.c_float),
                ("eps", ctypes.c_float), ("step", ctypes.c_int64)]


class CSegment(ctypes.Structure):
    """sgdb_segment_t: one tensor of a multi-tensor model (all device pointers)."""

    _fields_ = [("theta", ctypes.c_void_p), ("state0", ctypes.c_void_p), ("state1", ctypes.c_void_p),
                ("grad", ctypes.c_void_p), ("ld", ctypes.c_int64), ("len", ctypes.c_int64)]


@dataclass
class Opt:
    """sgdb_opt_t.  `kind` is "sgd" | "momentum" | "rmsprop" | "adam" | "adagrad" (or the enum value)."""

    kind: object = "sgd"
    lr: float = 0.1
    momentum: float = 0.0
    decay: float = 0.0
    beta1: float = 0.0
    beta2: float = 0.0
    eps: float = 0.0
    step: int = 1

    def _c(self) -> _COpt:
        kind = _KINDS[self.kind] if isinstance(self.kind, str) else int(self.kind)
        return _COpt(kind, self.lr, self.momentum, self.decay, self.beta1, self.beta2, self.eps, self.step)


def _load():
    if not os.path.exists(LIB_PATH):
        # not built yet: compile it now if the CUDA toolkit is here; there is nothing else to fall back to
        try:
            from . import build as _build

            _build.build()
        except Exception as e:
            raise ImportError(
                "libsgdb.so is not built (%s) and building it failed: %s. Run `python -m paper_1604_00981_b200.build`; "
                "this package has no CPU fallback." % (LIB_PATH, e))
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    sigs = {
        "sgdb_select": (i32, [vp, vp, i32, i32, i32, vp, vp, vp, vp]),
        "sgdb_aggregate": (i32, [vp, i32, i64, i64, i32, vp, vp, vp, vp]),
        "sgdb_update": (i32, [vp, vp, vp, vp, i64, ctypes.POINTER(_COpt), vp, vp]),
        "sgdb_step": (i32, [vp, i32, i64, i64, vp, vp, i32, i32, i32, vp, vp, vp, ctypes.POINTER(_COpt), vp, vp, vp, vp]),
        "sgdb_select_deadline": (i32, [vp, vp, i32, i32, ctypes.c_float, i32, vp, vp, vp, vp]),
        "sgdb_step_deadline": (i32, [vp, i32, i64, i64, vp, vp, i32, i32, ctypes.c_float, i32, vp, vp, vp,
                                     ctypes.POINTER(_COpt), vp, vp, vp, vp]),
        "sgdb_step_ema": (i32, [vp, i32, i64, i64, vp, vp, i32, i32, i32, vp, vp, vp, ctypes.POINTER(_COpt), vp,
                                ctypes.c_float, vp, vp, vp, vp]),
        "sgdb_ema": (i32, [vp, vp, i64, ctypes.c_float, vp, vp]),
        "sgdb_learning_rate": (ctypes.c_double, [ctypes.c_double, ctypes.c_double, i64, i64, ctypes.c_double]),
        "sgdb_step_segmented": (i32, [vp, i32, i32, vp, vp, i32, i32, i32, ctypes.POINTER(_COpt), vp, vp, vp, vp]),
        "sgdb_step_segmented_ema": (i32, [vp, vp, ctypes.c_float, i32, i32, vp, vp, i32, i32, i32, ctypes.POINTER(_COpt),
                                          vp, vp, vp, vp]),
        "sgdb_step_segmented_deadline": (i32, [vp, i32, i32, vp, vp, i32, i32, ctypes.c_float, i32, ctypes.POINTER(_COpt),
                                               vp, vp, vp, vp]),
        "sgdb_accumulate_arrival_deadline": (i32, [vp, i32, i32, ctypes.c_float, i32, ctypes.c_float, i64, vp, vp, vp, vp]),
        "sgdb_accumulate_close": (i32, [i32, i32, i64, vp, vp, vp, vp, vp, ctypes.POINTER(_COpt), vp, ctypes.c_float, vp, vp]),
        "sgdb_select_grouped": (i32, [vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp, vp]),
        "sgdb_step_grouped": (i32, [vp, i32, i64, i64, vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, ctypes.POINTER(_COpt),
                                    vp, vp, vp, vp, vp]),
        "sgdb_step_rows": (i32, [vp, i32, i64, vp, vp, i32, i32, i32, vp, vp, vp, ctypes.POINTER(_COpt), vp, i32,
                                 vp, vp, vp, vp]),
        "sgdb_step_rows_ordered": (i32, [vp, i32, i32, i64, i32, vp, vp, vp, vp, vp, ctypes.POINTER(_COpt), vp, i32, vp]),
        "sgdb_shard_range": (i32, [i64, i32, i32, ctypes.POINTER(i64), ctypes.POINTER(i64)]),
        "sgdb_accumulate_arrival": (i32, [vp, i32, i32, i32, i32, i64, vp, vp, vp, vp, vp, ctypes.POINTER(_COpt), vp, vp]),
        "sgdb_accumulate_arrival_ema": (i32, [vp, i32, i32, i32, i32, i64, vp, vp, vp, vp, vp, ctypes.POINTER(_COpt), vp,
                                              ctypes.c_float, vp, vp]),
        "sgdb_step_host": (i32, [vp, i32, i64, i64, vp, vp, i32, i32, i32, vp, vp, vp, ctypes.POINTER(_COpt),
                                 vp, vp, vp, vp, vp, sz, vp]),
        "sgdb_step_host_workspace_bytes": (sz, [i32, i64, i64, i32, i32]),
        "sgdb_step_host_static": (i32, [vp, i32, i64, i64, vp, vp, i32, i32, i32, vp, vp, vp, ctypes.POINTER(_COpt),
                                        vp, vp, vp, vp, vp]),
        "sgdb_selftest_bounded_wait": (i32, [i64, vp, vp]),
        "sgdb_enable_peer_access": (i32, [i32]),
        "sgdb_set_tuning": (i32, [i32, i32]),
        "sgdb_set_wait_limit_ns": (i32, [i64]),
        "sgdb_set_arrival_tuning": (i32, [i64, i32]),
        "sgdb_strerror": (ctypes.c_char_p, [i32]),
        "sgdb_version": (ctypes.c_int, []),
    }
    for name, (res, args) in sigs.items():
        fn = getattr(lib, name)  # AttributeError here means the library lacks a declared symbol
        fn.restype, fn.argtypes = res, args
    return lib


_lib = _load()


def _stream(stream=None) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


def _dev(x, dtype=None, name="tensor") -> int:
    """Device pointer of a CUDA tensor (None -> NULL)."""
    if x is None:
        return 0
    if not x.is_cuda or not x.is_contiguous():
        raise ValueError("%s must be a contiguous CUDA tensor" % name)
    if dtype is not None and x.dtype != dtype:
        raise ValueError("%s must have dtype %s, got %s" % (name, dtype, x.dtype))
    return x.data_ptr()


def _host(x, dtype=None, name="tensor") -> int:
    if x is None:
        return 0
    if x.is_cuda or not x.is_contiguous():
        raise ValueError("%s must be a contiguous host tensor" % name)
    if dtype is not None and x.dtype != dtype:
        raise ValueError("%s must have dtype %s, got %s" % (name, dtype, x.dtype))
    return x.data_ptr()


def _grad_dtype(g) -> int:
    if g.dtype == torch.float32:
        return SGDB_F32
    if g.dtype == torch.bfloat16:
        return SGDB_BF16
    raise ValueError("gradient rows must be float32 or bfloat16, got %s" % g.dtype)


def _check(status: int, where: str):
    if status != SGDB_OK:
        raise SgdbError(status, where)


def sgdb_strerror(status: int) -> str:
    return _lib.sgdb_strerror(int(status)).decode()


def sgdb_version() -> int:
    return int(_lib.sgdb_version())


def sgdb_selftest_bounded_wait(limit_ns: int, out, stream=None) -> None:
    """A wait for a barrier that nothing completes, with the kernels' own wait routine: out i32[3] receives
    {SGDB_ERR_TIMEOUT, nanoseconds waited, 1 if a second waiter was released by the give-up}."""
    _check(_lib.sgdb_selftest_bounded_wait(limit_ns, _dev(out, torch.int32, "out"), _stream(stream)),
           "sgdb_selftest_bounded_wait")


def sgdb_set_tuning(stages: int = 0, ctas_per_sm: int = 0) -> None:
    _check(_lib.sgdb_set_tuning(stages, ctas_per_sm), "sgdb_set_tuning")


def sgdb_set_wait_limit_ns(limit_ns: int = -1) -> None:
    """Patience of the waits inside the row-streaming kernels in nanoseconds (negative: the 2 s default)."""
    _check(_lib.sgdb_set_wait_limit_ns(limit_ns), "sgdb_set_wait_limit_ns")


def sgdb_set_arrival_tuning(resident_bytes: int = -1, blocks_per_sm: int = 0) -> None:
    _check(_lib.sgdb_set_arrival_tuning(resident_bytes, blocks_per_sm), "sgdb_set_arrival_tuning")


def sgdb_select(arrival, tags, t: int, N: int, b: int, mask, order, info, stream=None) -> None:
    """arrival f32[W], tags i32[W] -> mask u8[W], order i32[N], info i32[2] (all CUDA tensors)."""
    _check(_lib.sgdb_select(_dev(arrival, torch.float32, "arrival"), _dev(tags, torch.int32, "tags"), t, N, b,
                            _dev(mask, torch.uint8, "mask"), _dev(order, torch.int32, "order"),
                            _dev(info, torch.int32, "info"), _stream(stream)), "sgdb_select")


def sgdb_aggregate(grad, P: int, N: int, order, info, mean, ld: int | None = None, stream=None) -> None:
    """grad [W, ld] (f32 or bf16) -> mean f32[P] of the rows named in order[N]."""
    ld = grad.stride(0) if ld is None else ld
    _check(_lib.sgdb_aggregate(_dev(grad, None, "grad"), _grad_dtype(grad), P, ld, N,
                               _dev(order, torch.int32, "order"), _dev(info, torch.int32, "info"),
                               _dev(mean, torch.float32, "mean"), _stream(stream)), "sgdb_aggregate")


def sgdb_update(theta, state0, state1, mean, opt: Opt, info=None, P: int | None = None, stream=None) -> None:
    P = theta.numel() if P is None else P
    c = opt._c()
    _check(_lib.sgdb_update(_dev(theta, torch.float32, "theta"), _dev(state0, torch.float32, "state0"),
                            _dev(state1, torch.float32, "state1"), _dev(mean, torch.float32, "mean"), P,
                            ctypes.byref(c), _dev(info, torch.int32, "info"), _stream(stream)), "sgdb_update")


def sgdb_step(grad, P: int, arrival, tags, t: int, N: int, b: int, theta, state0, state1, opt: Opt,
              mask, order, info, ld: int | None = None, stream=None) -> None:
    """One fused iteration: select + mean of the kept rows + optimizer rule."""
    ld = grad.stride(0) if ld is None else ld
    c = opt._c()
    _check(_lib.sgdb_step(_dev(grad, None, "grad"), _grad_dtype(grad), P, ld,
                          _dev(arrival, torch.float32, "arrival"), _dev(tags, torch.int32, "tags"), t, N, b,
                          _dev(theta, torch.float32, "theta"), _dev(state0, torch.float32, "state0"),
                          _dev(state1, torch.float32, "state1"), ctypes.byref(c),
                          _dev(mask, torch.uint8, "mask"), _dev(order, torch.int32, "order"),
                          _dev(info, torch.int32, "info"), _stream(stream)), "sgdb_step")


def sgdb_select_deadline(arrival, tags, t: int, deadline: float, n_min: int, mask, order, info, stream=None) -> None:
    """Time-out rule: keep every gradient tagged t with arrival <= deadline.  order has W entries; info = {n, status}."""
    W = arrival.numel()
    _check(_lib.sgdb_select_deadline(_dev(arrival, torch.float32, "arrival"), _dev(tags, torch.int32, "tags"), t, W,
                                     deadline, n_min, _dev(mask, torch.uint8, "mask"),
                                     _dev(order, torch.int32, "order"), _dev(info, torch.int32, "info"),
                                     _stream(stream)), "sgdb_select_deadline")


def sgdb_step_deadline(grad, P: int, arrival, tags, t: int, deadline: float, n_min: int, theta, state0, state1,
                       opt: Opt, mask, order, info, ld: int | None = None, stream=None) -> None:
    """One fused iteration with the time-out rule: mean over the n gradients kept, then the optimizer rule."""
    ld = grad.stride(0) if ld is None else ld
    W = arrival.numel()
    c = opt._c()
    _check(_lib.sgdb_step_deadline(_dev(grad, None, "grad"), _grad_dtype(grad), P, ld,
                                   _dev(arrival, torch.float32, "arrival"), _dev(tags, torch.int32, "tags"), t, W,
                                   deadline, n_min, _dev(theta, torch.float32, "theta"),
                                   _dev(state0, torch.float32, "state0"), _dev(state1, torch.float32, "state1"),
                                   ctypes.byref(c), _dev(mask, torch.uint8, "mask"), _dev(order, torch.int32, "order"),
                                   _dev(info, torch.int32, "info"), _stream(stream)), "sgdb_step_deadline")


def sgdb_step_ema(grad, P: int, arrival, tags, t: int, N: int, b: int, theta, state0, state1, opt: Opt, ema,
                  alpha: float, mask, order, info, ld: int | None = None, stream=None) -> None:
    """sgdb_step plus avg <- alpha * avg + (1 - alpha) * theta(before the update), in the same launch."""
    ld = grad.stride(0) if ld is None else ld
    c = opt._c()
    _check(_lib.sgdb_step_ema(_dev(grad, None, "grad"), _grad_dtype(grad), P, ld,
                              _dev(arrival, torch.float32, "arrival"), _dev(tags, torch.int32, "tags"), t, N, b,
                              _dev(theta, torch.float32, "theta"), _dev(state0, torch.float32, "state0"),
                              _dev(state1, torch.float32, "state1"), ctypes.byref(c),
                              _dev(ema, torch.float32, "ema"), alpha, _dev(mask, torch.uint8, "mask"),
                              _dev(order, torch.int32, "order"), _dev(info, torch.int32, "info"), _stream(stream)),
           "sgdb_step_ema")


def sgdb_ema(ema, theta, alpha: float, info=None, P: int | None = None, stream=None) -> None:
    """avg <- alpha * avg + (1 - alpha) * theta on its own."""
    P = theta.numel() if P is None else P
    _check(_lib.sgdb_ema(_dev(ema, torch.float32, "ema"), _dev(theta, torch.float32, "theta"), P, alpha,
                         _dev(info, torch.int32, "info"), _stream(stream)), "sgdb_ema")


def sgdb_learning_rate(gamma0: float, beta: float, t: int, N: int, T: float) -> float:
    """gamma0 * beta^(t N / (2 T)): the paper's schedule (host computation)."""
    return float(_lib.sgdb_learning_rate(gamma0, beta, t, N, T))


def make_segment_table(segments, device) -> torch.Tensor:
    """Device table for sgdb_step_segmented from (theta, state0, state1, grad) tensor tuples.

    grad is [W, ld] with ld = grad.stride(0); len = theta.numel().  Returns a uint8 CUDA tensor
    holding the packed sgdb_segment_t array; the caller keeps the listed tensors alive.
    """
    arr = (CSegment * len(segments))()
    for i, (theta, s0, s1, grad) in enumerate(segments):
        arr[i] = CSegment(_dev(theta, torch.float32, "theta"), _dev(s0, torch.float32, "state0"),
                          _dev(s1, torch.float32, "state1"), grad.data_ptr(), grad.stride(0), theta.numel())
    raw = bytes(arr)
    host = torch.frombuffer(bytearray(raw), dtype=torch.uint8) if raw else torch.empty(0, dtype=torch.uint8)
    return host.to(device)


def sgdb_step_segmented(table, S: int, grad_dtype, arrival, tags, t: int, N: int, b: int, opt: Opt,
                        mask, order, info, stream=None) -> None:
    dt = SGDB_BF16 if grad_dtype == torch.bfloat16 else SGDB_F32
    c = opt._c()
    _check(_lib.sgdb_step_segmented(_dev(table, torch.uint8, "segment table"), S, dt,
                                    _dev(arrival, torch.float32, "arrival"), _dev(tags, torch.int32, "tags"),
                                    t, N, b, ctypes.byref(c), _dev(mask, torch.uint8, "mask"),
                                    _dev(order, torch.int32, "order"), _dev(info, torch.int32, "info"),
                                    _stream(stream)), "sgdb_step_segmented")


def make_pointer_table(tensors, device) -> torch.Tensor:
    """Device array of device pointers (int64 CUDA tensor) from a list of CUDA tensors; None -> NULL.
    The caller keeps the listed tensors alive."""
    return torch.tensor([0 if x is None else _dev(x, torch.float32, "tensor") for x in tensors], dtype=torch.int64).to(device)


def sgdb_step_segmented_ema(table, ema_table, alpha: float, S: int, grad_dtype, arrival, tags, t: int, N: int, b: int,
                            opt: Opt, mask, order, info, stream=None) -> None:
    """sgdb_step_segmented plus the per-tensor parameter averages (ema_table from make_pointer_table)."""
    dt = SGDB_BF16 if grad_dtype == torch.bfloat16 else SGDB_F32
    c = opt._c()
    _check(_lib.sgdb_step_segmented_ema(_dev(table, torch.uint8, "segment table"), _dev(ema_table, torch.int64, "ema table"),
                                        alpha, S, dt, _dev(arrival, torch.float32, "arrival"),
                                        _dev(tags, torch.int32, "tags"), t, N, b, ctypes.byref(c),
                                        _dev(mask, torch.uint8, "mask"), _dev(order, torch.int32, "order"),
                                        _dev(info, torch.int32, "info"), _stream(stream)), "sgdb_step_segmented_ema")


def sgdb_step_segmented_deadline(table, S: int, grad_dtype, arrival, tags, t: int, deadline: float, n_min: int, opt: Opt,
                                 mask, order, info, stream=None) -> None:
    """sgdb_step_segmented with the time-out rule; order has W entries, info = {n, status}."""
    dt = SGDB_BF16 if grad_dtype == torch.bfloat16 else SGDB_F32
    W = arrival.numel()
    c = opt._c()
    _check(_lib.sgdb_step_segmented_deadline(_dev(table, torch.uint8, "segment table"), S, dt,
                                             _dev(arrival, torch.float32, "arrival"), _dev(tags, torch.int32, "tags"),
                                             t, W, deadline, n_min, ctypes.byref(c), _dev(mask, torch.uint8, "mask"),
                                             _dev(order, torch.int32, "order"), _dev(info, torch.int32, "info"),
                                             _stream(stream)), "sgdb_step_segmented_deadline")


def sgdb_accumulate_arrival_deadline(row, row_tag: int, row_arrival: float, t: int, deadline: float, acc, counter, info,
                                     P: int | None = None, stream=None) -> None:
    """Time-out rule, one arriving gradient: joins the running sum iff tagged t, t open and arrived by the deadline."""
    P = acc.numel() if P is None else P
    _check(_lib.sgdb_accumulate_arrival_deadline(_dev(row, None, "row"), _grad_dtype(row), row_tag, row_arrival, t,
                                                 deadline, P, _dev(acc, torch.float32, "acc"),
                                                 _dev(counter, torch.int32, "counter"), _dev(info, torch.int32, "info"),
                                                 _stream(stream)), "sgdb_accumulate_arrival_deadline")


def sgdb_accumulate_close(t: int, n_min: int, acc, counter, theta, state0, state1, opt: Opt, info, ema=None,
                          alpha: float = 0.0, P: int | None = None, stream=None) -> None:
    """The deadline of iteration t has passed: update from the mean of the set if it holds at least n_min gradients."""
    P = theta.numel() if P is None else P
    c = opt._c()
    _check(_lib.sgdb_accumulate_close(t, n_min, P, _dev(acc, torch.float32, "acc"), _dev(counter, torch.int32, "counter"),
                                      _dev(theta, torch.float32, "theta"), _dev(state0, torch.float32, "state0"),
                                      _dev(state1, torch.float32, "state1"), ctypes.byref(c),
                                      _dev(ema, torch.float32, "ema"), alpha, _dev(info, torch.int32, "info"),
                                      _stream(stream)), "sgdb_accumulate_close")


def sgdb_select_grouped(arrival, tags, group, t: int, M: int, N: int, mask, group_order, order, info, stream=None) -> None:
    """Two-level selection: the first N machine messages.  mask u8[W], group_order i32[N], order i32[W], info i32[3]."""
    W = arrival.numel()
    _check(_lib.sgdb_select_grouped(_dev(arrival, torch.float32, "arrival"), _dev(tags, torch.int32, "tags"),
                                    _dev(group, torch.int32, "group"), t, W, M, N, _dev(mask, torch.uint8, "mask"),
                                    _dev(group_order, torch.int32, "group_order"), _dev(order, torch.int32, "order"),
                                    _dev(info, torch.int32, "info"), _stream(stream)), "sgdb_select_grouped")


def sgdb_step_grouped(grad, P: int, arrival, tags, group, t: int, M: int, N: int, theta, state0, state1, opt: Opt,
                      mask, group_order, order, info, ld: int | None = None, stream=None) -> None:
    """One fused iteration over machine messages: machines send the mean of their workers' rows, the first N
    messages are averaged, then the optimizer rule."""
    ld = grad.stride(0) if ld is None else ld
    W = arrival.numel()
    c = opt._c()
    _check(_lib.sgdb_step_grouped(_dev(grad, None, "grad"), _grad_dtype(grad), P, ld,
                                  _dev(arrival, torch.float32, "arrival"), _dev(tags, torch.int32, "tags"),
                                  _dev(group, torch.int32, "group"), t, W, M, N, _dev(theta, torch.float32, "theta"),
                                  _dev(state0, torch.float32, "state0"), _dev(state1, torch.float32, "state1"),
                                  ctypes.byref(c), _dev(mask, torch.uint8, "mask"),
                                  _dev(group_order, torch.int32, "group_order"), _dev(order, torch.int32, "order"),
                                  _dev(info, torch.int32, "info"), _stream(stream)), "sgdb_step_grouped")


def make_address_table(addresses, device) -> torch.Tensor:
    """Device array of device addresses (int64 CUDA tensor) from integers, e.g. tensor.data_ptr() plus a byte
    offset, or the address of a peer GPU's buffer mapped into this process.  The caller keeps the memory alive."""
    return torch.tensor([int(a) for a in addresses], dtype=torch.int64).to(device)


def sgdb_step_rows(rows, grad_dtype, length: int, arrival, tags, t: int, N: int, b: int, theta, state0, state1, opt: Opt,
                   replicas, mask, order, info, stream=None) -> None:
    """The fused step of one parameter server over its range of `length` columns: rows i64[W] holds the address of
    each worker's gradient at the range's first column (make_address_table), replicas i64[R] or None the addresses
    the new parameters are also stored to."""
    dt = SGDB_BF16 if grad_dtype == torch.bfloat16 else SGDB_F32
    R = 0 if replicas is None else replicas.numel()
    c = opt._c()
    _check(_lib.sgdb_step_rows(_dev(rows, torch.int64, "rows"), dt, length, _dev(arrival, torch.float32, "arrival"),
                               _dev(tags, torch.int32, "tags"), t, N, b, _dev(theta, torch.float32, "theta"),
                               _dev(state0, torch.float32, "state0"), _dev(state1, torch.float32, "state1"),
                               ctypes.byref(c), _dev(replicas, torch.int64, "replicas"), R,
                               _dev(mask, torch.uint8, "mask"), _dev(order, torch.int32, "order"),
                               _dev(info, torch.int32, "info"), _stream(stream)), "sgdb_step_rows")


def sgdb_step_rows_ordered(rows, grad_dtype, length: int, N: int, order, info, theta, state0, state1, opt: Opt,
                           replicas, stream=None) -> None:
    """sgdb_step_rows with the selection given: order i32[N] row ids in summation sequence, info i32[2] in/out."""
    dt = SGDB_BF16 if grad_dtype == torch.bfloat16 else SGDB_F32
    R = 0 if replicas is None else replicas.numel()
    c = opt._c()
    _check(_lib.sgdb_step_rows_ordered(_dev(rows, torch.int64, "rows"), rows.numel(), dt, length, N,
                                       _dev(order, torch.int32, "order"), _dev(info, torch.int32, "info"),
                                       _dev(theta, torch.float32, "theta"), _dev(state0, torch.float32, "state0"),
                                       _dev(state1, torch.float32, "state1"), ctypes.byref(c),
                                       _dev(replicas, torch.int64, "replicas"), R, _stream(stream)),
           "sgdb_step_rows_ordered")


def sgdb_shard_range(P: int, n_servers: int, j: int):
    """(first column, number of columns) of parameter server j out of n_servers over P columns (host computation)."""
    first, length = ctypes.c_int64(0), ctypes.c_int64(0)
    _check(_lib.sgdb_shard_range(P, n_servers, j, ctypes.byref(first), ctypes.byref(length)), "sgdb_shard_range")
    return int(first.value), int(length.value)


def sgdb_enable_peer_access(peer_device: int) -> None:
    """Kernels launched on the current device may then use the memory of peer_device (one-time set-up)."""
    _check(_lib.sgdb_enable_peer_access(int(peer_device)), "sgdb_enable_peer_access")


def sgdb_accumulate_arrival(row, row_tag: int, t: int, N: int, acc, counter, theta, state0, state1,
                            opt: Opt, info, P: int | None = None, stream=None) -> None:
    """One arriving gradient row (f32 or bf16 [P]); counter i32[4] is the server state, info i32[2] the outcome."""
    P = theta.numel() if P is None else P
    c = opt._c()
    _check(_lib.sgdb_accumulate_arrival(_dev(row, None, "row"), _grad_dtype(row), row_tag, t, N, P,
                                        _dev(acc, torch.float32, "acc"), _dev(counter, torch.int32, "counter"),
                                        _dev(theta, torch.float32, "theta"), _dev(state0, torch.float32, "state0"),
                                        _dev(state1, torch.float32, "state1"), ctypes.byref(c),
                                        _dev(info, torch.int32, "info"), _stream(stream)),
           "sgdb_accumulate_arrival")


def sgdb_accumulate_arrival_ema(row, row_tag: int, t: int, N: int, acc, counter, theta, state0, state1, opt: Opt, ema,
                                alpha: float, info, P: int | None = None, stream=None) -> None:
    """sgdb_accumulate_arrival that also moves the parameter average when the N-th gradient fires the update."""
    P = theta.numel() if P is None else P
    c = opt._c()
    _check(_lib.sgdb_accumulate_arrival_ema(_dev(row, None, "row"), _grad_dtype(row), row_tag, t, N, P,
                                            _dev(acc, torch.float32, "acc"), _dev(counter, torch.int32, "counter"),
                                            _dev(theta, torch.float32, "theta"), _dev(state0, torch.float32, "state0"),
                                            _dev(state1, torch.float32, "state1"), ctypes.byref(c),
                                            _dev(ema, torch.float32, "ema"), alpha, _dev(info, torch.int32, "info"),
                                            _stream(stream)), "sgdb_accumulate_arrival_ema")


def sgdb_step_host_workspace_bytes(grad_dtype, P: int, ld: int, N: int, b: int) -> int:
    dt = SGDB_BF16 if grad_dtype == torch.bfloat16 else SGDB_F32
    return int(_lib.sgdb_step_host_workspace_bytes(dt, P, ld, N, b))


def sgdb_step_host(h_grad, P: int, h_arrival, h_tags, t: int, N: int, b: int, theta, state0, state1, opt: Opt,
                   h_theta_out, h_mask, h_order, h_info, workspace, ld: int | None = None, stream=None) -> int:
    """sgdb_step with gradients, arrival times and tags in host memory; returns the status (0 or INSUFFICIENT)."""
    ld = h_grad.stride(0) if ld is None else ld
    c = opt._c()
    st = _lib.sgdb_step_host(_host(h_grad, None, "h_grad"), _grad_dtype(h_grad), P, ld,
                             _host(h_arrival, torch.float32, "h_arrival"), _host(h_tags, torch.int32, "h_tags"),
                             t, N, b, _dev(theta, torch.float32, "theta"), _dev(state0, torch.float32, "state0"),
                             _dev(state1, torch.float32, "state1"), ctypes.byref(c),
                             _host(h_theta_out, torch.float32, "h_theta_out"), _host(h_mask, torch.uint8, "h_mask"),
                             _host(h_order, torch.int32, "h_order"), _host(h_info, torch.int32, "h_info"),
                             _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream))
    if st not in (SGDB_OK, SGDB_ERR_INSUFFICIENT):
        raise SgdbError(st, "sgdb_step_host")
    return st


def sgdb_step_host_static(h_grad, P: int, h_arrival, h_tags, t: int, N: int, b: int, theta, state0, state1, opt: Opt,
                          h_theta_out, h_mask, h_order, h_info, ld: int | None = None, stream=None) -> int:
    """sgdb_step_host without a workspace argument, for callers that can neither supply device memory nor
    allocate any: the staging area is a fixed SGDB_STATIC_SCRATCH_BYTES array inside the library.  Sizes that
    do not fit raise SgdbError (SGDB_ERR_UNSUPPORTED).  Calls on one device share that array: do not overlap
    them.  Returns the status (0 or SGDB_ERR_INSUFFICIENT)."""
    ld = h_grad.stride(0) if ld is None else ld
    c = opt._c()
    st = _lib.sgdb_step_host_static(_host(h_grad, None, "h_grad"), _grad_dtype(h_grad), P, ld,
                                    _host(h_arrival, torch.float32, "h_arrival"), _host(h_tags, torch.int32, "h_tags"),
                                    t, N, b, _dev(theta, torch.float32, "theta"), _dev(state0, torch.float32, "state0"),
                                    _dev(state1, torch.float32, "state1"), ctypes.byref(c),
                                    _host(h_theta_out, torch.float32, "h_theta_out"),
                                    _host(h_mask, torch.uint8, "h_mask"), _host(h_order, torch.int32, "h_order"),
                                    _host(h_info, torch.int32, "h_info"), _stream(stream))
    if st not in (SGDB_OK, SGDB_ERR_INSUFFICIENT):
        raise SgdbError(st, "sgdb_step_host_static")
    return st

"""Shared helpers of the parity tests: error metric, tolerances, oracle/GPU drivers."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_1604_00981_b200 import workload as wl

# Tolerances stated for this path: max relative error against the fp64 oracle.
TOL_F32 = 1e-5
TOL_BF16 = 2e-3

OPTS = {
    "sgd": dict(kind="sgd", lr=0.1),
    "momentum": dict(kind="momentum", lr=0.01, momentum=0.9),
    "rmsprop": dict(kind="rmsprop", lr=0.045, decay=0.9, momentum=0.9, eps=1.0),
    "adam": dict(kind="adam", lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8),
    "adagrad": dict(kind="adagrad", lr=0.05, eps=1e-7),
}

_ORACLE_KIND = {"sgd": oracle.SGD, "momentum": oracle.MOMENTUM, "rmsprop": oracle.RMSPROP, "adam": oracle.ADAM,
                "adagrad": oracle.ADAGRAD}
STATES = {"sgd": 0, "momentum": 1, "rmsprop": 2, "adam": 2, "adagrad": 1}


def rel_err(x, y) -> float:
    """max_i |x_i - y_i| / max(|y_i|, rms(y)): relative error with a floor at the vector's rms, so that
    elements where a mean of zero-centred terms cancels to almost nothing do not dominate."""
    x = np.asarray(x, dtype=np.float64)
    y = np.asarray(y, dtype=np.float64)
    if y.size == 0:
        return 0.0
    floor = float(np.sqrt(np.mean(y * y)))
    denom = np.maximum(np.abs(y), floor if floor > 0 else 1.0)
    return float(np.max(np.abs(x - y) / denom))


def f32(x) -> float:
    """The value a Python float takes when the C ABI stores it as fp32."""
    return float(np.float32(x))


def oracle_opt(opt_kw: dict, step: int = 1) -> oracle.Opt:
    kw = {k: f32(v) for k, v in opt_kw.items() if k != "kind"}
    return oracle.Opt(kind=_ORACLE_KIND[opt_kw["kind"]], step=step, **kw)


def gpu_opt(opt_kw: dict, step: int = 1):
    from paper_1604_00981_b200 import binding

    return binding.Opt(step=step, **opt_kw)


def gpu_state(kind: str, P: int, device):
    n = STATES[kind]
    s0 = torch.zeros(P, dtype=torch.float32, device=device) if n >= 1 else None
    s1 = torch.zeros(P, dtype=torch.float32, device=device) if n >= 2 else None
    return s0, s1


def oracle_state(kind: str, P: int):
    n = STATES[kind]
    return (np.zeros(P) if n >= 1 else None), (np.zeros(P) if n >= 2 else None)


def selection_buffers(W: int, N: int, device):
    mask = torch.full((W,), 255, dtype=torch.uint8, device=device)
    order = torch.full((N,), -7, dtype=torch.int32, device=device)
    info = torch.full((2,), -7, dtype=torch.int32, device=device)
    return mask, order, info


def to_dev(a: np.ndarray, device) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def step_inputs(seed: int, t: int, W: int, N: int):
    return wl.arrivals(seed, t, W), wl.tags(seed, t, W, N)


def oracle_step_over_column_ranges(grad, P, arrival, tags, t, N, b, theta, s0, s1, opt, threads):
    """The oracle's step on [W, P] host rows, one unchanged oracle call per contiguous column range, each from its
    own thread (the oracle itself stays single-threaded; the path is separable by column).  Returns the list of
    (status, mask, order, n_valid) of the pieces."""
    from concurrent.futures import ThreadPoolExecutor

    flat = grad.reshape(-1)
    ld = grad.shape[1]
    edges = [P * k // threads for k in range(threads + 1)]
    pieces = [(edges[k], edges[k + 1]) for k in range(threads) if edges[k + 1] > edges[k]]

    def piece(r):
        c0, c1 = r
        return oracle.step(flat[c0:], c1 - c0, arrival, tags, t, N, b, theta[c0:c1], None if s0 is None else s0[c0:c1],
                           None if s1 is None else s1[c0:c1], opt, ld=ld)

    with ThreadPoolExecutor(max_workers=len(pieces)) as pool:
        return list(pool.map(piece, pieces))

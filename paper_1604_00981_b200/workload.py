"""Seeded synthetic inputs for the parameter-server step with backup workers.

This module only draws inputs: worker gradient rows, arrival times, iteration
tags, initial parameters, tensor lengths.  It holds none of the method's
arithmetic and imports neither the CUDA binding nor the CPU oracle, so both can
be fed the same bytes.

The inputs stand in for the workloads of "Revisiting Distributed Synchronous SGD"
(arXiv 1604.00981), whose models and datasets are not used here:
  * arrival times have a tight bulk and a long right tail, like the measured time
    to collect the k-th gradient (Section 3.1, the straggler figures);
  * a stale tag marks a gradient computed for the previous iteration, the only way
    Algorithm 4 meets a tag other than t;
  * W = N + b follows the paper's best split of 100 machines (N=96, b=4, Section 3.1)
    and its 53/106/212-worker runs (Section 4.2, Appendix A.3).

Small per-worker quantities come from numpy's Philox generator on the host; the
large gradient matrices are drawn with torch's seeded generator on the device
that will hold them (values differ between device types, never between runs).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

MASTER_SEED = 160400981

# stream ids keep the different kinds of draws independent of each other
_S_SCALE, _S_ARRIVAL, _S_TAG, _S_GRAD, _S_THETA, _S_SEGLEN = range(6)


@dataclass(frozen=True)
class Config:
    """One of the five seeded workloads."""

    name: str
    N: int
    b: int
    P: int  # total parameters (sum of segment lengths for the segmented workload)
    T: int  # steps
    grad_dtype: str  # "f32" or "bf16"
    opt: dict = field(default_factory=dict)  # kind + hyper-parameters
    segments: int = 0  # > 0: multi-tensor model with this many tensors
    seed: int = MASTER_SEED

    @property
    def W(self) -> int:
        return self.N + self.b


CONFIGS = {
    0: Config("c0_tiny_sgd", N=5, b=1, P=10_000, T=20, grad_dtype="f32",
              opt=dict(kind="sgd", lr=0.1), seed=MASTER_SEED + 0),
    1: Config("c1_inception_rmsprop", N=96, b=4, P=23_800_000, T=10, grad_dtype="f32",
              opt=dict(kind="rmsprop", lr=0.045, decay=0.9, momentum=0.9, eps=1.0), seed=MASTER_SEED + 1),
    2: Config("c2_segmented_momentum", N=50, b=4, P=0, T=3, grad_dtype="f32",
              opt=dict(kind="momentum", lr=0.01, momentum=0.9), segments=300, seed=MASTER_SEED + 2),
    3: Config("c3_large_bf16_adam", N=200, b=8, P=100_000_000, T=5, grad_dtype="bf16",
              opt=dict(kind="adam", lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8), seed=MASTER_SEED + 3),
    4: Config("c4_accumulate_rmsprop", N=96, b=4, P=23_800_000, T=2, grad_dtype="f32",
              opt=dict(kind="rmsprop", lr=0.045, decay=0.9, momentum=0.9, eps=1.0), seed=MASTER_SEED + 4),
}


def _rng(seed: int, stream: int, t: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(seed=np.random.SeedSequence([seed, stream, t + 1_000_000])))


def worker_scales(seed: int, W: int) -> np.ndarray:
    """Per-worker gradient standard deviation s_w ~ U[0.5, 2], fp32 [W]."""
    return _rng(seed, _S_SCALE).uniform(0.5, 2.0, size=W).astype(np.float32)


def arrivals(seed: int, t: int, W: int) -> np.ndarray:
    """Arrival time of each worker's gradient at step t: lognormal(0, 0.3), times 5 with probability 0.05."""
    g = _rng(seed, _S_ARRIVAL, t)
    a = g.lognormal(mean=0.0, sigma=0.3, size=W)
    slow = g.random(W) < 0.05
    return np.where(slow, 5.0 * a, a).astype(np.float32)


def tags(seed: int, t: int, W: int, N: int, max_draws: int = 1_000_000) -> np.ndarray:
    """Iteration tag per worker: t, or t-1 with probability 0.1; redrawn while fewer than N are current."""
    g = _rng(seed, _S_TAG, t)
    for _ in range(max_draws):
        stale = g.random(W) < 0.1
        tg = np.where(stale, t - 1, t).astype(np.int32)
        if int((tg == t).sum()) >= N:
            return tg
    raise ValueError("no draw with %d current tags among %d workers at a stale rate of 0.1" % (N, W))


def theta0(seed: int, P: int, device="cpu") -> torch.Tensor:
    """Initial parameters ~ N(0, 1), fp32 [P]."""
    gen = torch.Generator(device=device)
    gen.manual_seed(seed * 16 + _S_THETA)
    return torch.randn(P, dtype=torch.float32, device=device, generator=gen)


def grad_matrix(seed: int, t: int, W: int, P: int, scales, dtype: str = "f32", device="cpu",
                ld: int | None = None, out: torch.Tensor | None = None, pad_value: float = 0.0) -> torch.Tensor:
    """Gradient rows of step t: row w ~ N(0, s_w^2) per element, [W, ld] with ld >= P.

    dtype "bf16" rounds each fp32 draw to nearest-even bf16 (torch's conversion).
    Rows are drawn in blocks so that a bf16 matrix never needs a full fp32 copy.
    Columns P..ld-1, if any, are filled with `pad_value` (they are not part of the model).
    """
    ld = P if ld is None else ld
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    if out is None:
        out = torch.empty((W, ld), dtype=tdt, device=device)
    assert out.shape == (W, ld) and out.dtype == tdt
    gen = torch.Generator(device=device)
    gen.manual_seed((seed * 16 + _S_GRAD) * 1_000_003 + t)
    s = torch.as_tensor(np.asarray(scales, dtype=np.float32), device=device)
    rows_per_block = max(1, min(W, (256 << 20) // max(1, 4 * P)))
    for w0 in range(0, W, rows_per_block):
        w1 = min(W, w0 + rows_per_block)
        if tdt == torch.float32 and ld == P:
            blk = out[w0:w1]
            blk.normal_(generator=gen)
            blk.mul_(s[w0:w1, None])
        else:
            blk = torch.randn((w1 - w0, P), dtype=torch.float32, device=device, generator=gen)
            blk.mul_(s[w0:w1, None])
            out[w0:w1, :P] = blk.to(tdt)
            if ld > P:
                out[w0:w1, P:] = pad_value
    return out


def segment_lengths(seed: int, S: int = 300, lo: int = 64, hi: int = 1 << 21) -> np.ndarray:
    """Tensor lengths drawn log-uniformly in [lo, hi] elements, int64 [S]."""
    u = _rng(seed, _S_SEGLEN).uniform(np.log(lo), np.log(hi), size=S)
    return np.clip(np.floor(np.exp(u)).astype(np.int64), lo, hi)


def delivery_sequence(arrival: np.ndarray) -> np.ndarray:
    """Worker ids in the sequence their gradients are delivered: by arrival time, equal times by lower id.

    Workers whose gradient never arrives (non-finite time) are left out.
    """
    ids = np.argsort(np.asarray(arrival, dtype=np.float32), kind="stable")
    return ids[np.isfinite(np.asarray(arrival)[ids])].astype(np.int32)


def as_oracle_array(x: torch.Tensor) -> np.ndarray:
    """Host numpy view of a tensor: fp32 as float32, bf16 as uint16 bit patterns, ints unchanged."""
    x = x.detach().cpu().contiguous()
    if x.dtype == torch.bfloat16:
        return x.view(torch.int16).numpy().view(np.uint16)
    return x.numpy()

"""The seeded input generators: reproducible, and shaped as the workload recipe says."""
import numpy as np
import torch

from paper_1604_00981_b200 import workload as wl


def test_draws_are_reproducible_and_step_dependent():
    c = wl.CONFIGS[0]
    assert np.array_equal(wl.arrivals(c.seed, 3, c.W), wl.arrivals(c.seed, 3, c.W))
    assert not np.array_equal(wl.arrivals(c.seed, 3, c.W), wl.arrivals(c.seed, 4, c.W))
    assert np.array_equal(wl.tags(c.seed, 3, c.W, c.N), wl.tags(c.seed, 3, c.W, c.N))
    s = wl.worker_scales(c.seed, c.W)
    g1 = wl.grad_matrix(c.seed, 2, c.W, 500, s)
    g2 = wl.grad_matrix(c.seed, 2, c.W, 500, s)
    assert torch.equal(g1, g2) and not torch.equal(g1, wl.grad_matrix(c.seed, 3, c.W, 500, s))
    assert torch.equal(wl.theta0(c.seed, 100), wl.theta0(c.seed, 100))


def test_distributions():
    W = 20000
    a = wl.arrivals(wl.MASTER_SEED, 0, W).astype(np.float64)
    assert a.dtype == np.float64 and (a > 0).all()
    assert abs(np.median(a) - 1.0) < 0.03  # lognormal(0, .3) has median 1
    assert 0.03 < (a > 3.0).mean() < 0.07  # the x5 stragglers
    s = wl.worker_scales(wl.MASTER_SEED, W)
    assert s.min() >= 0.5 and s.max() <= 2.0 and abs(s.mean() - 1.25) < 0.02
    for t in range(5):
        tg = wl.tags(wl.MASTER_SEED, t, 100, 96)
        assert set(np.unique(tg)) <= {t - 1, t} and (tg == t).sum() >= 96
    scales = np.array([0.5, 1.0, 2.0], dtype=np.float32)
    g = wl.grad_matrix(1, 0, 3, 200_000, scales)
    assert np.allclose(g.std(dim=1).numpy(), scales, rtol=0.02)
    assert abs(float(g.mean())) < 0.01


def test_bf16_rows_are_round_to_nearest_of_the_fp32_draws_and_padding():
    scales = np.array([1.0, 1.5], dtype=np.float32)
    f = wl.grad_matrix(5, 1, 2, 1000, scales, dtype="f32", ld=1000 + 8)
    h = wl.grad_matrix(5, 1, 2, 1000, scales, dtype="bf16", ld=1000 + 8)
    assert h.dtype == torch.bfloat16 and h.shape == (2, 1008)
    assert torch.equal(f[:, :1000].to(torch.bfloat16), h[:, :1000])
    assert (h[:, 1000:] == 0).all() and (f[:, 1000:] == 0).all()
    bits = wl.as_oracle_array(h)
    assert bits.dtype == np.uint16
    back = (bits.astype(np.uint32) << 16).view(np.float32)
    assert np.array_equal(back, h.to(torch.float32).numpy())


def test_segment_lengths_and_delivery_sequence():
    L = wl.segment_lengths(wl.CONFIGS[2].seed)
    assert len(L) == 300 and L.min() >= 64 and L.max() <= 2 ** 21
    assert 30e6 < L.sum() < 100e6
    a = np.array([2.0, 1.0, np.inf, 1.0, 0.5], dtype=np.float32)
    assert wl.delivery_sequence(a).tolist() == [4, 1, 3, 0]


def test_impossible_tag_request_raises_instead_of_looping():
    import pytest

    with pytest.raises(ValueError):
        wl.tags(1, 0, 400, 400, max_draws=2000)  # all 400 current at a stale rate of 0.1: 0.9^400

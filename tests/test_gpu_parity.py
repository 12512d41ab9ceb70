"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element.

Selection (mask, order, counts) must match bit for bit.  Means, parameters and optimizer state must
match the fp64 oracle within 1e-5 (fp32 gradient rows) or 2e-3 (bf16 rows) in the metric of
helpers.rel_err.  Sizes span several 2048-column tiles and ragged tails.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import (OPTS, TOL_BF16, TOL_F32, f32, gpu_opt, gpu_state, oracle_opt, oracle_state, rel_err,
                     selection_buffers, step_inputs, to_dev)
from paper_1604_00981_b200 import workload as wl

pytestmark = pytest.mark.gpu

@pytest.fixture(scope="module")
def sgdb(cuda_device):
    from paper_1604_00981_b200 import binding

    return binding


# ------------------------------------------------------------------ selection


def _select_case(sgdb, dev, arrival, tags, t, N, b):
    W = N + b
    mask, order, info = selection_buffers(W, N, dev)
    sgdb.sgdb_select(to_dev(arrival, dev), to_dev(tags, dev), t, N, b, mask, order, info)
    rc, mask_o, order_o, n_valid = oracle.select(arrival, tags, t, N, b)
    info_h = info.cpu().tolist()
    assert info_h[0] == n_valid
    if rc == oracle.INSUFFICIENT:
        assert info_h[1] == sgdb.SGDB_ERR_INSUFFICIENT
        assert (mask.cpu() == 255).all() and (order.cpu() == -7).all()  # untouched
    else:
        assert info_h[1] == sgdb.SGDB_OK
        assert mask.cpu().numpy().tolist() == mask_o.tolist()
        assert order.cpu().numpy().tolist() == order_o.tolist()
    return rc


def test_select_bit_exact_random_and_special_values(sgdb, cuda_device):
    rng = np.random.default_rng(11)
    values = np.array([0.25, 0.5, 0.5, 1.0, 1.5, 2.0, 7.0, np.inf, np.nan, -0.0, 0.0, -1.0, -np.inf], np.float32)
    outcomes = set()
    for trial in range(150):
        W = int(rng.choice([1, 2, 3, 6, 31, 32, 33, 54, 64, 100, 208]))
        N = int(rng.integers(1, W + 1))
        if trial % 2:
            arrival = values[rng.integers(0, len(values), size=W)]
        else:
            arrival = rng.lognormal(0, 0.3, size=W).astype(np.float32)
            arrival[rng.integers(0, W, size=W // 4)] = 1.0
        t = int(rng.integers(0, 100))
        tags = np.where(rng.random(W) < 0.15, t - 1, t).astype(np.int32)
        tags[rng.random(W) < 0.05] = t + 1
        outcomes.add(_select_case(sgdb, cuda_device, arrival, tags, t, N, W - N))
    assert outcomes == {oracle.OK, oracle.INSUFFICIENT}


def test_select_maximum_width_and_workload_draws(sgdb, cuda_device):
    rng = np.random.default_rng(12)
    W = sgdb.SGDB_MAX_WORKERS
    arrival = rng.lognormal(0, 0.3, size=W).astype(np.float32)
    arrival[::7] = arrival[3]
    tags = np.where(rng.random(W) < 0.1, 4, 5).astype(np.int32)
    assert _select_case(sgdb, cuda_device, arrival, tags, 5, 700, W - 700) == oracle.OK
    assert _select_case(sgdb, cuda_device, arrival, np.full(W, 5, np.int32), 5, W, 0) == oracle.OK
    for cfg in wl.CONFIGS.values():
        for t in range(4):
            a, tg = step_inputs(cfg.seed, t, cfg.W, cfg.N)
            assert _select_case(sgdb, cuda_device, a, tg, t, cfg.N, cfg.b) == oracle.OK
    with pytest.raises(sgdb.SgdbError):
        _select_case(sgdb, cuda_device, np.zeros(1025, np.float32), np.zeros(1025, np.int32), 0, 1000, 25)


# ------------------------------------------------------------------ masked mean


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("P,pad", [(1, 0), (3, 0), (5, 3), (2047, 1), (2048, 0), (2049, 7), (4096, 0),
                                   (10_000, 0), (10_001, 0), (10_001, 3), (150_003, 5), (301_111, 9)])
def test_aggregate_matches_oracle(sgdb, cuda_device, dtype, P, pad):
    """pad chooses the row pitch: ld = P + pad; aligned and unaligned pitches take different load paths."""
    W, N, seed = 9, 6, 21
    ld = P + pad
    scales = wl.worker_scales(seed, W)
    grad = wl.grad_matrix(seed, 0, W, P, scales, dtype, cuda_device, ld=ld, pad_value=float("nan"))
    order_h = np.array([7, 2, 8, 0, 3, 5], dtype=np.int32)
    info = to_dev(np.array([N, 0], np.int32), cuda_device)
    mean = torch.full((P + 8,), 123.0, device=cuda_device)
    sgdb.sgdb_aggregate(grad, P, N, to_dev(order_h, cuda_device), info, mean, ld=ld)
    ref = oracle.aggregate(wl.as_oracle_array(grad), P, order_h, ld=ld)
    got = mean.cpu().numpy()
    assert (got[P:] == 123.0).all()  # nothing written past P
    assert rel_err(got[:P], ref) < (TOL_F32 if dtype == "f32" else TOL_BF16)
    # the device adds the kept rows one after another in fp32: reproduce that sum exactly
    rows = wl.as_oracle_array(grad.to(torch.float32))[:, :P]
    acc = np.zeros(P, np.float32)
    for w in order_h:
        acc = acc + rows[w]
    assert np.array_equal(got[:P], acc / np.float32(N))


def test_aggregate_error_within_the_sequential_sum_bound(sgdb, cuda_device):
    """A sequential fp32 sum of N terms is off by at most (N - 1) u sum|g_k| (u = 2^-24), the division adds
    one more rounding: every element of the device mean must sit inside that band around the fp64 mean."""
    dev = cuda_device
    c = wl.CONFIGS[1]
    W, N, P = c.W, c.N, 300_007
    grad = wl.grad_matrix(c.seed, 0, W, P, wl.worker_scales(c.seed, W), "f32", dev)
    arrival, tags = step_inputs(c.seed, 0, W, N)
    rc, _, order_o, _ = oracle.select(arrival, tags, 0, N, W - N)
    mean = torch.empty(P, device=dev)
    sgdb.sgdb_aggregate(grad, P, N, to_dev(order_o, dev), None, mean)
    rows = wl.as_oracle_array(grad)[order_o].astype(np.float64)
    ref = rows.mean(axis=0)
    u = 2.0 ** -24
    bound = ((N - 1) * u * np.abs(rows).sum(axis=0)) / N + u * np.abs(ref) + 1e-45
    err = np.abs(mean.cpu().numpy().astype(np.float64) - ref)
    assert (err <= bound).all()
    assert err.max() > 0  # it is an fp32 sum, not the oracle in disguise
    assert rel_err(mean.cpu().numpy(), ref) < TOL_F32 / 5


def test_aggregate_skipped_when_selection_failed(sgdb, cuda_device):
    P = 5000
    grad = torch.ones((3, P), device=cuda_device)
    mean = torch.full((P,), 7.0, device=cuda_device)
    info = to_dev(np.array([1, sgdb.SGDB_ERR_INSUFFICIENT], np.int32), cuda_device)
    sgdb.sgdb_aggregate(grad, P, 2, to_dev(np.array([0, 1], np.int32), cuda_device), info, mean)
    assert (mean.cpu() == 7.0).all()


# ------------------------------------------------------------------ optimizer rules


@pytest.mark.parametrize("kind", list(OPTS))
@pytest.mark.parametrize("P", [1, 7, 4096, 100_003])
def test_update_matches_oracle(sgdb, cuda_device, kind, P):
    rng = np.random.default_rng(31)
    theta = to_dev(rng.normal(size=P).astype(np.float32), cuda_device)
    s0, s1 = gpu_state(kind, P, cuda_device)
    th_o = theta.cpu().numpy().astype(np.float64)
    s0_o, s1_o = oracle_state(kind, P)
    for step in range(1, 5):
        mean = rng.normal(size=P).astype(np.float32) * 0.3
        sgdb.sgdb_update(theta, s0, s1, to_dev(mean, cuda_device), gpu_opt(OPTS[kind], step))
        oracle.update(th_o, s0_o, s1_o, mean.astype(np.float64), oracle_opt(OPTS[kind], step))
    assert rel_err(theta.cpu().numpy(), th_o) < TOL_F32
    if s0 is not None:
        assert rel_err(s0.cpu().numpy(), s0_o) < TOL_F32
    if s1 is not None:
        assert rel_err(s1.cpu().numpy(), s1_o) < TOL_F32


# ------------------------------------------------------------------ fused step, T-step trajectories


def _trajectory(sgdb, dev, W, N, P, T, dtype, opt_kw, seed, pad=0, check_every_step=True):
    kind = opt_kw["kind"]
    ld = P + pad
    scales = wl.worker_scales(seed, W)
    theta = wl.theta0(seed, P, dev)
    s0, s1 = gpu_state(kind, P, dev)
    th_o = theta.cpu().numpy().astype(np.float64)
    s0_o, s1_o = oracle_state(kind, P)
    mask, order, info = selection_buffers(W, N, dev)
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    for t in range(T):
        grad = wl.grad_matrix(seed, t, W, P, scales, dtype, dev, ld=ld, pad_value=float("nan"))
        arrival, tags = step_inputs(seed, t, W, N)
        sgdb.sgdb_step(grad, P, to_dev(arrival, dev), to_dev(tags, dev), t, N, W - N, theta, s0, s1,
                       gpu_opt(opt_kw, t + 1), mask, order, info, ld=ld)
        rc, mask_o, order_o, n_valid = oracle.step(wl.as_oracle_array(grad), P, arrival, tags, t, N, W - N,
                                                   th_o, s0_o, s1_o, oracle_opt(opt_kw, t + 1), ld=ld)
        assert rc == oracle.OK
        assert info.cpu().tolist() == [n_valid, 0]
        assert mask.cpu().numpy().tolist() == mask_o.tolist()
        assert order.cpu().numpy().tolist() == order_o.tolist()
        if check_every_step or t == T - 1:
            assert rel_err(theta.cpu().numpy(), th_o) < tol, t
    if s0 is not None:
        assert rel_err(s0.cpu().numpy(), s0_o) < tol
    if s1 is not None:
        assert rel_err(s1.cpu().numpy(), s1_o) < tol
    return theta, s0, s1


def test_config0_tiny_sgd_trajectory(sgdb, cuda_device):
    c = wl.CONFIGS[0]
    _trajectory(sgdb, cuda_device, c.W, c.N, c.P, c.T, c.grad_dtype, c.opt, c.seed)


@pytest.mark.parametrize("kind", list(OPTS))
@pytest.mark.parametrize("dtype,P,pad", [("f32", 70_001, 3), ("f32", 131_072, 0), ("bf16", 70_001, 7),
                                         ("bf16", 70_003, 0), ("f32", 70_001, 0)])
def test_fused_step_trajectories(sgdb, cuda_device, kind, dtype, P, pad):
    _trajectory(sgdb, cuda_device, 20, 16, P, 4, dtype, OPTS[kind], seed=41 + pad, pad=pad)


@pytest.mark.parametrize("N,b", [(1, 0), (1, 5), (2, 1), (3, 0)])
def test_few_kept_gradients(sgdb, cuda_device, N, b):
    """N = 1 returns the single earliest current gradient; odd and even N take different branches of the row loop."""
    _trajectory(sgdb, cuda_device, N + b, N, 20_011, 3, "f32", OPTS["momentum"], seed=43 + N + b)
    _trajectory(sgdb, cuda_device, N + b, N, 20_011, 2, "bf16", OPTS["sgd"], seed=44 + N + b, pad=5)


def test_config1_shape_reduced_columns(sgdb, cuda_device):
    """W=100, N=96, RMSProp with the Inception hyper-parameters, T=10, on a 1/100 column slice."""
    c = wl.CONFIGS[1]
    _trajectory(sgdb, cuda_device, c.W, c.N, 238_000, c.T, c.grad_dtype, c.opt, c.seed, check_every_step=False)


def test_config3_shape_reduced_columns(sgdb, cuda_device):
    """W=208, N=200, bf16 rows, Adam, T=5, on a 1/1000 column slice."""
    c = wl.CONFIGS[3]
    _trajectory(sgdb, cuda_device, c.W, c.N, 100_000, c.T, c.grad_dtype, c.opt, c.seed, check_every_step=False)


# ------------------------------------------------------------------ properties of the method


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_widest_server_1024_workers(sgdb, cuda_device, dtype):
    """The largest accepted W: 880 kept of 1024 (about 920 carry the current tag), a ragged vector."""
    _trajectory(sgdb, cuda_device, 1024, 880, 10_007, 2, dtype, OPTS["rmsprop"], seed=47, pad=1)


def test_empty_parameter_vector_is_a_selection_only(sgdb, cuda_device):
    dev = cuda_device
    W, N = 10, 8
    arrival, tags = step_inputs(49, 0, W, N)
    mask, order, info = selection_buffers(W, N, dev)
    grad = torch.zeros((W, 4), device=dev)
    theta = torch.zeros(4, device=dev)
    sgdb.sgdb_step(grad, 0, to_dev(arrival, dev), to_dev(tags, dev), 0, N, W - N, theta, None, None,
                   gpu_opt(OPTS["sgd"]), mask, order, info, ld=4)
    rc, mask_o, order_o, n_valid = oracle.select(arrival, tags, 0, N, W - N)
    assert info.cpu().tolist() == [n_valid, 0] and order.cpu().numpy().tolist() == order_o.tolist()
    assert mask.cpu().numpy().tolist() == mask_o.tolist() and (theta == 0).all()


def test_fused_equals_separate_calls_bitwise(sgdb, cuda_device):
    dev = cuda_device
    W, N, P, seed = 30, 24, 123_457, 51
    scales = wl.worker_scales(seed, W)
    for kind in OPTS:
        for dtype in ("f32", "bf16"):
            theta_a = wl.theta0(seed, P, dev)
            theta_b = theta_a.clone()
            sa = gpu_state(kind, P, dev)
            sb = gpu_state(kind, P, dev)
            mask_a, order_a, info_a = selection_buffers(W, N, dev)
            mask_b, order_b, info_b = selection_buffers(W, N, dev)
            mean = torch.empty(P, device=dev)
            for t in range(3):
                grad = wl.grad_matrix(seed, t, W, P, scales, dtype, dev)
                arrival, tags = step_inputs(seed, t, W, N)
                a_d, t_d = to_dev(arrival, dev), to_dev(tags, dev)
                opt = gpu_opt(OPTS[kind], t + 1)
                sgdb.sgdb_step(grad, P, a_d, t_d, t, N, W - N, theta_a, sa[0], sa[1], opt, mask_a, order_a, info_a)
                sgdb.sgdb_select(a_d, t_d, t, N, W - N, mask_b, order_b, info_b)
                sgdb.sgdb_aggregate(grad, P, N, order_b, info_b, mean)
                sgdb.sgdb_update(theta_b, sb[0], sb[1], mean, opt, info_b)
            assert torch.equal(theta_a, theta_b), (kind, dtype)
            assert torch.equal(order_a, order_b) and torch.equal(mask_a, mask_b)
            for x, y in zip(sa, sb):
                assert x is None or torch.equal(x, y)


def test_dropped_rows_never_reach_the_result(sgdb, cuda_device):
    """Rows of late or stale workers may hold anything, NaN included: the result has the same bits."""
    dev = cuda_device
    W, N, P, seed = 40, 33, 90_001, 61
    scales = wl.worker_scales(seed, W)
    grad = wl.grad_matrix(seed, 0, W, P, scales, "f32", dev)
    arrival, tags = step_inputs(seed, 0, W, N)
    tags[int(np.argmin(arrival))] = -1  # the earliest arrival is stale
    rc, mask_o, _, _ = oracle.select(arrival, tags, 0, N, W - N)
    assert rc == oracle.OK
    results = []
    for poison in (None, float("nan"), float("inf"), 1e30):
        g = grad.clone()
        if poison is not None:
            g[to_dev(mask_o == 0, dev)] = poison
        theta = wl.theta0(seed, P, dev)
        s0, s1 = gpu_state("rmsprop", P, dev)
        mask, order, info = selection_buffers(W, N, dev)
        sgdb.sgdb_step(g, P, to_dev(arrival, dev), to_dev(tags, dev), 0, N, W - N, theta, s0, s1,
                       gpu_opt(OPTS["rmsprop"]), mask, order, info)
        assert torch.isfinite(theta).all()
        results.append((theta, s0, s1))
    for th, s0, s1 in results[1:]:
        assert torch.equal(th, results[0][0]) and torch.equal(s0, results[0][1]) and torch.equal(s1, results[0][2])


def test_b0_is_plain_synchronous_minibatch_sgd(sgdb, cuda_device):
    """No backups, all tags current: theta - lr * (mean over every worker), a library mean in fp64."""
    dev = cuda_device
    W, P = 16, 50_000
    grad = wl.grad_matrix(71, 0, W, P, wl.worker_scales(71, W), "f32", dev)
    theta = wl.theta0(71, P, dev)
    ref = theta.double() - f32(0.1) * grad.double().mean(dim=0)
    mask, order, info = selection_buffers(W, W, dev)
    sgdb.sgdb_step(grad, P, to_dev(wl.arrivals(71, 0, W), dev), torch.zeros(W, dtype=torch.int32, device=dev),
                   0, W, 0, theta, None, None, gpu_opt(OPTS["sgd"]), mask, order, info)
    assert mask.cpu().all()
    assert rel_err(theta.cpu().numpy(), ref.cpu().numpy()) < TOL_F32


def test_insufficient_gradients_leave_parameters_untouched(sgdb, cuda_device):
    dev = cuda_device
    W, N, P = 10, 8, 30_000
    grad = torch.randn((W, P), device=dev)
    theta = torch.randn(P, device=dev)
    s0, s1 = torch.randn(P, device=dev), torch.randn(P, device=dev)
    before = (theta.clone(), s0.clone(), s1.clone())
    arrival = np.linspace(1, 2, W).astype(np.float32)
    arrival[0] = np.inf
    tags = np.array([3, 3, 3, 3, 3, 3, 3, 2, 2, 4], np.int32)  # 6 usable < N
    mask, order, info = selection_buffers(W, N, dev)
    sgdb.sgdb_step(grad, P, to_dev(arrival, dev), to_dev(tags, dev), 3, N, W - N, theta, s0, s1,
                   gpu_opt(OPTS["adam"]), mask, order, info)
    assert info.cpu().tolist() == [6, sgdb.SGDB_ERR_INSUFFICIENT]
    assert torch.equal(theta, before[0]) and torch.equal(s0, before[1]) and torch.equal(s1, before[2])
    assert (mask.cpu() == 255).all() and (order.cpu() == -7).all()


def test_outputs_stay_inside_their_buffers(sgdb, cuda_device):
    """Guard bands around every output keep their pattern (stands in for a memory checker)."""
    dev = cuda_device
    W, N, P, G = 12, 9, 10_001, 64
    canary = -12345.5

    def banded(n, dtype=torch.float32, fill=canary):
        buf = torch.full((n + 2 * G,), fill, dtype=dtype, device=dev)
        return buf, buf[G:G + n]

    grad = wl.grad_matrix(81, 0, W, P, wl.worker_scales(81, W), "f32", dev, ld=P + 3)
    bufs = [banded(P) for _ in range(3)]
    for _, view in bufs:
        view.zero_()
    mbuf, mask = banded(W, torch.uint8, 201)
    obuf, order = banded(N, torch.int32, -99)
    ibuf, info = banded(2, torch.int32, -99)
    arrival, tags = step_inputs(81, 0, W, N)
    sgdb.sgdb_step(grad, P, to_dev(arrival, dev), to_dev(tags, dev), 0, N, W - N, bufs[0][1], bufs[1][1], bufs[2][1],
                   gpu_opt(OPTS["rmsprop"]), mask, order, info, ld=P + 3)
    assert info.cpu().tolist()[1] == 0
    for buf, _ in bufs:
        assert (buf[:G] == canary).all() and (buf[-G:] == canary).all()
    assert (mbuf[:G] == 201).all() and (mbuf[-G:] == 201).all()
    assert (obuf[:G] == -99).all() and (obuf[-G:] == -99).all()
    assert (ibuf[:G] == -99).all() and (ibuf[-G:] == -99).all()


def test_run_to_run_bitwise_determinism_and_tuning_independence(sgdb, cuda_device):
    dev = cuda_device
    W, N, P, seed = 50, 44, 400_003, 91
    grad = wl.grad_matrix(seed, 0, W, P, wl.worker_scales(seed, W), "bf16", dev)
    arrival, tags = step_inputs(seed, 0, W, N)
    outs = []
    try:
        for stages, ctas in ((0, 0), (0, 0), (2, 1), (3, 1), (20, 1), (5, 3), (64, 8)):
            sgdb.sgdb_set_tuning(stages, ctas)
            theta = wl.theta0(seed, P, dev)
            s0, s1 = gpu_state("adam", P, dev)
            mask, order, info = selection_buffers(W, N, dev)
            sgdb.sgdb_step(grad, P, to_dev(arrival, dev), to_dev(tags, dev), 0, N, W - N, theta, s0, s1,
                           gpu_opt(OPTS["adam"]), mask, order, info)
            assert info.cpu().tolist()[1] == 0
            outs.append((theta, s0, s1))
    finally:
        sgdb.sgdb_set_tuning(0, 0)
    for o in outs[1:]:
        assert all(torch.equal(x, y) for x, y in zip(o, outs[0]))


def test_invalid_arguments_raise(sgdb, cuda_device):
    dev = cuda_device
    grad = torch.zeros((4, 100), device=dev)
    theta = torch.zeros(100, device=dev)
    mask, order, info = selection_buffers(4, 3, dev)
    a, tg = torch.zeros(4, device=dev), torch.zeros(4, dtype=torch.int32, device=dev)
    with pytest.raises(sgdb.SgdbError):  # ld < P
        sgdb.sgdb_step(grad, 100, a, tg, 0, 3, 1, theta, None, None, gpu_opt(OPTS["sgd"]), mask, order, info, ld=99)
    with pytest.raises(sgdb.SgdbError):  # momentum without its state
        sgdb.sgdb_step(grad, 100, a, tg, 0, 3, 1, theta, None, None, gpu_opt(OPTS["momentum"]), mask, order, info)
    with pytest.raises(sgdb.SgdbError):  # misaligned parameter pointer
        sgdb.sgdb_step(grad, 99, a, tg, 0, 3, 1, torch.zeros(101, device=dev)[1:100], None, None,
                       gpu_opt(OPTS["sgd"]), mask, order, info, ld=100)
    assert (theta == 0).all()

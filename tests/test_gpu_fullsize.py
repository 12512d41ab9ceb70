"""Parity at the full sizes of the five workloads, in the launch configuration the benchmark times.

The oracle cannot chew through 10-40 GB in seconds, but the path is separable by column: the oracle
runs on a sample of columns (random ones, the first and last, and tile borders) cut out of the very
matrices the GPU consumed, and the GPU's results are compared at those columns.  Whole-vector
properties that hold at any size are checked as well (bitwise agreement between the fused step and
the other entry points, untouched padding, finite results).
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import (TOL_BF16, TOL_F32, gpu_opt, gpu_state, oracle_opt, oracle_state, rel_err,
                     selection_buffers, step_inputs, to_dev)
from paper_1604_00981_b200 import workload as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sgdb(cuda_device):
    from paper_1604_00981_b200 import binding

    return binding


def _need_memory(dev, gigabytes):
    free, _ = torch.cuda.mem_get_info(dev)
    if free < gigabytes * 1e9:
        pytest.skip("needs %.0f GB of free device memory" % gigabytes)


def _sample_columns(P, rng, n=3000, tile=2048):
    cols = [rng.integers(0, P, size=min(n, P)), np.arange(min(16, P)), np.arange(max(0, P - 16), P)]
    for k in rng.integers(1, max(2, P // tile), size=8):
        cols.append(np.array([k * tile - 1, k * tile, min(P - 1, k * tile + 1)]))
    cols = np.unique(np.concatenate(cols))
    return cols[(cols >= 0) & (cols < P)].astype(np.int64)


def _flat_trajectory_sampled(sgdb, dev, cfg, T):
    W, N, P, kind = cfg.W, cfg.N, cfg.P, cfg.opt["kind"]
    rng = np.random.default_rng(cfg.seed)
    cols = _sample_columns(P, rng, tile=2048 if cfg.grad_dtype == "f32" else 4096)
    cols_d = to_dev(cols, dev)
    scales = wl.worker_scales(cfg.seed, W)
    theta = wl.theta0(cfg.seed, P, dev)
    s0, s1 = gpu_state(kind, P, dev)
    th_o = theta[cols_d].cpu().numpy().astype(np.float64)
    s0_o, s1_o = oracle_state(kind, len(cols))
    mask, order, info = selection_buffers(W, N, dev)
    grad = None
    for t in range(T):
        grad = wl.grad_matrix(cfg.seed, t, W, P, scales, cfg.grad_dtype, dev, out=grad)
        arrival, tags = step_inputs(cfg.seed, t, W, N)
        sgdb.sgdb_step(grad, P, to_dev(arrival, dev), to_dev(tags, dev), t, N, cfg.b, theta, s0, s1,
                       gpu_opt(cfg.opt, t + 1), mask, order, info)
        sample = wl.as_oracle_array(grad.index_select(1, cols_d))
        rc, mask_o, order_o, n_valid = oracle.step(sample, len(cols), arrival, tags, t, N, cfg.b, th_o, s0_o, s1_o,
                                                   oracle_opt(cfg.opt, t + 1))
        assert rc == oracle.OK and info.cpu().tolist() == [n_valid, 0]
        assert mask.cpu().numpy().tolist() == mask_o.tolist()
        assert order.cpu().numpy().tolist() == order_o.tolist()
    tol = TOL_F32 if cfg.grad_dtype == "f32" else TOL_BF16
    assert rel_err(theta[cols_d].cpu().numpy(), th_o) < tol
    assert rel_err(s0[cols_d].cpu().numpy(), s0_o) < tol
    assert rel_err(s1[cols_d].cpu().numpy(), s1_o) < tol
    assert bool(torch.isfinite(theta).all())
    return grad, theta, s0, s1, arrival, tags, T - 1


def test_config1_full_size(sgdb, cuda_device):
    """P = 23.8 M fp32, W = 100 (N = 96, b = 4), RMSProp, T = 10 steps; fused step vs oracle at sampled columns, then the
    separate select / aggregate / update calls against the fused step on the whole vector."""
    _need_memory(cuda_device, 12)
    dev, cfg = cuda_device, wl.CONFIGS[1]
    grad, theta, s0, s1, arrival, tags, t = _flat_trajectory_sampled(sgdb, dev, cfg, T=cfg.T)
    W, N, P = cfg.W, cfg.N, cfg.P
    th_f, s0_f, s1_f = theta.clone(), s0.clone(), s1.clone()
    mask, order, info = selection_buffers(W, N, dev)
    a_d, t_d = to_dev(arrival, dev), to_dev(tags, dev)
    opt = gpu_opt(cfg.opt, t + 2)
    sgdb.sgdb_step(grad, P, a_d, t_d, t, N, cfg.b, th_f, s0_f, s1_f, opt, mask, order, info)
    mean = torch.empty(P, device=dev)
    mask2, order2, info2 = selection_buffers(W, N, dev)
    sgdb.sgdb_select(a_d, t_d, t, N, cfg.b, mask2, order2, info2)
    sgdb.sgdb_aggregate(grad, P, N, order2, info2, mean)
    sgdb.sgdb_update(theta, s0, s1, mean, opt, info2)
    assert torch.equal(order, order2) and torch.equal(mask, mask2)
    assert torch.equal(theta, th_f) and torch.equal(s0, s0_f) and torch.equal(s1, s1_f)


def test_config1_full_size_every_column_against_the_oracle(sgdb, cuda_device):
    """Two fused steps at P = 23.8 M, W = 100 (N = 96, b = 4), RMSProp, in the launch configuration the benchmark
    times, and EVERY element of theta and of both state vectors compared with the oracle: the gradient matrix is
    copied back in column chunks and the oracle runs chunk by chunk (one call per column range and host thread)."""
    import os

    from helpers import oracle_step_over_column_ranges

    _need_memory(cuda_device, 12)
    dev, cfg = cuda_device, wl.CONFIGS[1]
    W, N, P, kind = cfg.W, cfg.N, cfg.P, cfg.opt["kind"]
    threads = max(1, len(os.sched_getaffinity(0)))
    scales = wl.worker_scales(cfg.seed, W)
    theta = wl.theta0(cfg.seed, P, dev)
    s0, s1 = gpu_state(kind, P, dev)
    th_o = theta.cpu().numpy().astype(np.float64)
    s0_o, s1_o = oracle_state(kind, P)
    mask, order, info = selection_buffers(W, N, dev)
    chunk = 2_000_000
    grad = None
    for t in range(2):
        grad = wl.grad_matrix(cfg.seed, t, W, P, scales, cfg.grad_dtype, dev, out=grad)
        arrival, tags = step_inputs(cfg.seed, t, W, N)
        sgdb.sgdb_step(grad, P, to_dev(arrival, dev), to_dev(tags, dev), t, N, cfg.b, theta, s0, s1,
                       gpu_opt(cfg.opt, t + 1), mask, order, info)
        for c0 in range(0, P, chunk):
            c1 = min(P, c0 + chunk)
            rows = wl.as_oracle_array(grad[:, c0:c1].contiguous())
            for rc, mask_o, order_o, n_valid in oracle_step_over_column_ranges(
                    rows, c1 - c0, arrival, tags, t, N, cfg.b, th_o[c0:c1], s0_o[c0:c1], s1_o[c0:c1],
                    oracle_opt(cfg.opt, t + 1), threads):
                assert rc == oracle.OK
            del rows
        assert info.cpu().tolist() == [n_valid, 0]
        assert mask.cpu().numpy().tolist() == mask_o.tolist() and order.cpu().numpy().tolist() == order_o.tolist()
    got = theta.cpu().numpy()
    assert rel_err(got, th_o) < TOL_F32
    assert rel_err(s0.cpu().numpy(), s0_o) < TOL_F32 and rel_err(s1.cpu().numpy(), s1_o) < TOL_F32
    # element by element as well, each against its own size with a floor far below the rms of the vector
    assert float(np.max(np.abs(got - th_o) / np.maximum(np.abs(th_o), 1e-2))) < 1e-4


def test_config3_full_size(sgdb, cuda_device):
    """P = 100 M, W = 208 (N = 200, b = 8), bf16 rows (41.6 GB), Adam, T = 5 steps."""
    _need_memory(cuda_device, 48)
    _flat_trajectory_sampled(sgdb, cuda_device, wl.CONFIGS[3], T=wl.CONFIGS[3].T)


def test_config2_full_size_segmented(sgdb, cuda_device):
    """300 tensors with log-uniform lengths in [64, 2^21], W = 54 (N = 50, b = 4), momentum SGD:
    one launch over the device table, which also keeps one parameter average per tensor, vs the oracle (small
    tensors whole, large ones at sampled columns) and vs one fused launch per tensor (bitwise, parameters and state)."""
    _need_memory(cuda_device, 20)
    dev, cfg = cuda_device, wl.CONFIGS[2]
    W, N, kind = cfg.W, cfg.N, cfg.opt["kind"]
    lengths = wl.segment_lengths(cfg.seed, cfg.segments)
    rng = np.random.default_rng(cfg.seed)
    scales = wl.worker_scales(cfg.seed, W)
    segs, samples = [], []
    for i, L in enumerate(int(x) for x in lengths):
        ld = (L + 3) // 4 * 4
        theta = wl.theta0(cfg.seed + i, L, dev)
        grad = wl.grad_matrix(cfg.seed + i, 0, W, L, scales, "f32", dev, ld=ld)
        segs.append((theta, torch.zeros(L, device=dev), None, grad))
        cols = np.arange(L) if L <= 4096 else _sample_columns(L, rng, n=256)
        samples.append(cols)
    twins = [(s[0].clone(), s[1].clone()) for s in segs]
    table = sgdb.make_segment_table(segs, dev)
    avgs = [s[0].clone() for s in segs]  # one parameter average per tensor, kept by the same launch
    ema_table = sgdb.make_pointer_table(avgs, dev)
    alpha = 0.875
    th_o = [segs[i][0][to_dev(samples[i], dev)].cpu().numpy().astype(np.float64) for i in range(len(segs))]
    v_o = [np.zeros(len(c)) for c in samples]
    avg_o = [x.copy() for x in th_o]
    mask, order, info = selection_buffers(W, N, dev)
    mask2, order2, info2 = selection_buffers(W, N, dev)
    for t in range(2):
        if t:
            for i, (theta, _, _, grad) in enumerate(segs):
                wl.grad_matrix(cfg.seed + i, t, W, theta.numel(), scales, "f32", dev, ld=grad.stride(0), out=grad)
        arrival, tags = step_inputs(cfg.seed, t, W, N)
        a_d, t_d = to_dev(arrival, dev), to_dev(tags, dev)
        sgdb.sgdb_step_segmented_ema(table, ema_table, alpha, len(segs), torch.float32, a_d, t_d, t, N, cfg.b,
                                     gpu_opt(cfg.opt, t + 1), mask, order, info)
        rc, mask_o, order_o, n_valid = oracle.select(arrival, tags, t, N, cfg.b)
        assert rc == oracle.OK and info.cpu().tolist() == [n_valid, 0]
        assert order.cpu().numpy().tolist() == order_o.tolist()
        for i, (theta, v, _, grad) in enumerate(segs):
            cols_d = to_dev(samples[i], dev)
            sample = wl.as_oracle_array(grad.index_select(1, cols_d))
            mean = oracle.aggregate(sample, len(samples[i]), order_o)
            oracle.ema(avg_o[i], th_o[i], alpha)  # the average takes in the parameters before the update
            oracle.update(th_o[i], v_o[i], None, mean, oracle_opt(cfg.opt, t + 1))
            if i % 10 == 0:  # one launch per tensor, every tenth tensor
                sgdb.sgdb_step(grad, theta.numel(), a_d, t_d, t, N, cfg.b, twins[i][0], twins[i][1], None,
                               gpu_opt(cfg.opt, t + 1), mask2, order2, info2, ld=grad.stride(0))
    got = np.concatenate([segs[i][0][to_dev(samples[i], dev)].cpu().numpy() for i in range(len(segs))])
    got_v = np.concatenate([segs[i][1][to_dev(samples[i], dev)].cpu().numpy() for i in range(len(segs))])
    assert rel_err(got, np.concatenate(th_o)) < TOL_F32
    assert rel_err(got_v, np.concatenate(v_o)) < TOL_F32
    got_avg = np.concatenate([avgs[i][to_dev(samples[i], dev)].cpu().numpy() for i in range(len(segs))])
    assert rel_err(got_avg, np.concatenate(avg_o)) < TOL_F32
    for i in range(0, len(segs), 10):
        assert torch.equal(segs[i][0], twins[i][0]) and torch.equal(segs[i][1], twins[i][1]), i


@pytest.mark.parametrize("b", [0, 2, 4, 8])
def test_config4_full_size_accumulate_on_arrival(sgdb, cuda_device, b):
    """P = 23.8 M fp32, N = 96, b swept: one iteration delivered row by row in arrival sequence;
    outcomes replayed by the oracle's arrival-by-arrival server, parameters compared at sampled columns
    with the oracle and on the whole vector with the fused step (bitwise)."""
    _need_memory(cuda_device, 14)
    dev, cfg = cuda_device, wl.CONFIGS[4]
    N, P, kind = cfg.N, cfg.P, cfg.opt["kind"]
    W = N + b
    seed = cfg.seed + b
    rng = np.random.default_rng(seed)
    cols = _sample_columns(P, rng)
    cols_d = to_dev(cols, dev)
    grad = wl.grad_matrix(seed, 0, W, P, wl.worker_scales(seed, W), "f32", dev)
    arrival, tags = step_inputs(seed, 0, W, N)
    theta = wl.theta0(seed, P, dev)
    theta_f = theta.clone()
    s0, s1 = gpu_state(kind, P, dev)
    sf = gpu_state(kind, P, dev)
    acc = torch.empty(P, device=dev)
    counter = torch.zeros(4, dtype=torch.int32, device=dev)
    info = torch.zeros(2, dtype=torch.int32, device=dev)
    th_o = theta[cols_d].cpu().numpy().astype(np.float64)
    s0_o, s1_o = oracle_state(kind, len(cols))
    acc_o, state_o = np.zeros(len(cols)), oracle.new_server_state()
    sample = wl.as_oracle_array(grad.index_select(1, cols_d))
    outcomes = []
    for w in wl.delivery_sequence(arrival):
        sgdb.sgdb_accumulate_arrival(grad[w], int(tags[w]), 0, N, acc, counter, theta, s0, s1, gpu_opt(cfg.opt), info)
        want = oracle.accumulate_arrival(sample[w], int(tags[w]), 0, N, acc_o, state_o, th_o, s0_o, s1_o,
                                         oracle_opt(cfg.opt))
        assert info.cpu().tolist()[0] == want
        outcomes.append(want)
    assert outcomes.count(2) == 1 and outcomes.count(1) == N - 1
    assert counter.cpu().tolist() == [0, len(outcomes), 0, 1]
    assert rel_err(theta[cols_d].cpu().numpy(), th_o) < TOL_F32
    assert rel_err(s0[cols_d].cpu().numpy(), s0_o) < TOL_F32
    mask, order, finfo = selection_buffers(W, N, dev)
    sgdb.sgdb_step(grad, P, to_dev(arrival, dev), to_dev(tags, dev), 0, N, b, theta_f, sf[0], sf[1], gpu_opt(cfg.opt),
                   mask, order, finfo)
    assert torch.equal(theta, theta_f) and torch.equal(s0, sf[0]) and torch.equal(s1, sf[1])


def test_config1_full_size_two_level(sgdb, cuda_device):
    """The C1 matrix with its 100 workers on 25 machines of 4 and the first 24 messages used: the one-launch
    two-level step against the oracle at sampled columns, three steps with a stale worker in each."""
    _need_memory(cuda_device, 12)
    dev, cfg = cuda_device, wl.CONFIGS[1]
    W, P, kind, M, N = cfg.W, cfg.P, cfg.opt["kind"], 25, 24
    group = (np.arange(W) // 4).astype(np.int32)
    rng = np.random.default_rng(cfg.seed + 7)
    cols = _sample_columns(P, rng)
    cols_d = to_dev(cols, dev)
    scales = wl.worker_scales(cfg.seed, W)
    theta = wl.theta0(cfg.seed, P, dev)
    s0, s1 = gpu_state(kind, P, dev)
    th_o = theta[cols_d].cpu().numpy().astype(np.float64)
    s0_o, s1_o = oracle_state(kind, len(cols))
    mask = torch.full((W,), 255, dtype=torch.uint8, device=dev)
    gorder = torch.full((N,), -7, dtype=torch.int32, device=dev)
    order = torch.full((W,), -7, dtype=torch.int32, device=dev)
    info = torch.full((3,), -7, dtype=torch.int32, device=dev)
    grad = None
    for t in range(3):
        grad = wl.grad_matrix(cfg.seed, t, W, P, scales, cfg.grad_dtype, dev, out=grad)
        arrival = wl.arrivals(cfg.seed, t, W)
        tags = np.full(W, t, np.int32)
        if t == 1:
            tags[int(rng.integers(0, W))] = t - 1  # its machine's message does not count: exactly 24 are left
        sgdb.sgdb_step_grouped(grad, P, to_dev(arrival, dev), to_dev(tags, dev), to_dev(group, dev), t, M, N, theta, s0, s1,
                               gpu_opt(cfg.opt, t + 1), mask, gorder, order, info)
        rc, mask_o, gorder_o, order_o, n_valid = oracle.step_grouped(
            wl.as_oracle_array(grad.index_select(1, cols_d)), len(cols), arrival, tags, group, t, M, N, th_o, s0_o, s1_o,
            oracle_opt(cfg.opt, t + 1))
        assert rc == oracle.OK and info.cpu().tolist() == [n_valid, 0, 4 * N]
        assert mask.cpu().numpy().tolist() == mask_o.tolist() and gorder.cpu().numpy().tolist() == gorder_o.tolist()
        assert order.cpu().numpy()[: 4 * N].tolist() == order_o.tolist()
    assert rel_err(theta[cols_d].cpu().numpy(), th_o) < TOL_F32
    assert rel_err(s0[cols_d].cpu().numpy(), s0_o) < TOL_F32 and rel_err(s1[cols_d].cpu().numpy(), s1_o) < TOL_F32
    assert bool(torch.isfinite(theta).all())


def test_config4_full_size_arrivals_with_time_out(sgdb, cuda_device):
    """P = 23.8 M, 100 workers, the time-out rule one gradient per call, then the close call: outcomes replayed by the
    oracle, parameters at sampled columns against the oracle and on the whole vector against the fused time-out step."""
    _need_memory(cuda_device, 14)
    dev, cfg = cuda_device, wl.CONFIGS[4]
    W, P, kind = cfg.W, cfg.P, cfg.opt["kind"]
    seed = cfg.seed + 31
    rng = np.random.default_rng(seed)
    cols = _sample_columns(P, rng)
    cols_d = to_dev(cols, dev)
    grad = wl.grad_matrix(seed, 0, W, P, wl.worker_scales(seed, W), "f32", dev)
    arrival, tags = step_inputs(seed, 0, W, 1)
    deadline = float(np.float32(1.5))
    theta = wl.theta0(seed, P, dev)
    theta_f = theta.clone()
    s0, s1 = gpu_state(kind, P, dev)
    sf = gpu_state(kind, P, dev)
    acc = torch.empty(P, device=dev)
    counter = torch.zeros(4, dtype=torch.int32, device=dev)
    info = torch.zeros(2, dtype=torch.int32, device=dev)
    th_o = theta[cols_d].cpu().numpy().astype(np.float64)
    s0_o, s1_o = oracle_state(kind, len(cols))
    acc_o, state_o = np.zeros(len(cols)), oracle.new_server_state()
    sample = wl.as_oracle_array(grad.index_select(1, cols_d))
    kept = 0
    for w in wl.delivery_sequence(arrival):
        sgdb.sgdb_accumulate_arrival_deadline(grad[w], int(tags[w]), float(arrival[w]), 0, deadline, acc, counter, info)
        want = oracle.accumulate_arrival_deadline(sample[w], int(tags[w]), float(arrival[w]), 0, deadline, acc_o, state_o)
        assert info.cpu().tolist()[0] == want
        kept += want
    assert 20 < kept < W and counter.cpu().tolist() == [kept, W, 0, 0]
    sgdb.sgdb_accumulate_close(0, 1, acc, counter, theta, s0, s1, gpu_opt(cfg.opt), info)
    rc, outcome = oracle.accumulate_close(0, 1, acc_o, state_o, th_o, s0_o, s1_o, oracle_opt(cfg.opt))
    assert rc == oracle.OK and outcome == 2 and info.cpu().tolist() == [2, kept] and counter.cpu().tolist() == [0, W, 0, 1]
    assert rel_err(theta[cols_d].cpu().numpy(), th_o) < TOL_F32 and rel_err(s0[cols_d].cpu().numpy(), s0_o) < TOL_F32
    mask, order, finfo = selection_buffers(W, W, dev)
    sgdb.sgdb_step_deadline(grad, P, to_dev(arrival, dev), to_dev(tags, dev), 0, deadline, 1, theta_f, sf[0], sf[1],
                            gpu_opt(cfg.opt), mask, order, finfo)
    assert finfo.cpu().tolist() == [kept, 0]
    assert torch.equal(theta, theta_f) and torch.equal(s0, sf[0]) and torch.equal(s1, sf[1])


def test_config3_full_size_every_column_against_the_oracle(sgdb, cuda_device):
    """One fused step at P = 100 M, W = 208 (N = 200, b = 8), bf16 rows, Adam, in the benchmark's launch
    configuration, and EVERY element of theta, m and v compared with the oracle: the 41.6 GB matrix comes back
    in column chunks and the oracle runs chunk by chunk, one call per column range and host thread."""
    import os

    from helpers import oracle_step_over_column_ranges

    _need_memory(cuda_device, 48)
    dev, cfg = cuda_device, wl.CONFIGS[3]
    W, N, P, kind = cfg.W, cfg.N, cfg.P, cfg.opt["kind"]
    threads = max(1, len(os.sched_getaffinity(0)))
    theta = wl.theta0(cfg.seed, P, dev)
    s0, s1 = gpu_state(kind, P, dev)
    th_o = theta.cpu().numpy().astype(np.float64)
    s0_o, s1_o = oracle_state(kind, P)
    mask, order, info = selection_buffers(W, N, dev)
    grad = wl.grad_matrix(cfg.seed, 0, W, P, wl.worker_scales(cfg.seed, W), cfg.grad_dtype, dev)
    arrival, tags = step_inputs(cfg.seed, 0, W, N)
    sgdb.sgdb_step(grad, P, to_dev(arrival, dev), to_dev(tags, dev), 0, N, cfg.b, theta, s0, s1, gpu_opt(cfg.opt, 1), mask,
                   order, info)
    chunk = 2_000_000
    for c0 in range(0, P, chunk):
        c1 = min(P, c0 + chunk)
        rows = wl.as_oracle_array(grad[:, c0:c1].contiguous())
        for rc, mask_o, order_o, n_valid in oracle_step_over_column_ranges(
                rows, c1 - c0, arrival, tags, 0, N, cfg.b, th_o[c0:c1], s0_o[c0:c1], s1_o[c0:c1], oracle_opt(cfg.opt, 1),
                threads):
            assert rc == oracle.OK
        del rows
    del grad
    assert info.cpu().tolist() == [n_valid, 0]
    assert mask.cpu().numpy().tolist() == mask_o.tolist() and order.cpu().numpy().tolist() == order_o.tolist()
    got = theta.cpu().numpy()
    assert rel_err(got, th_o) < TOL_BF16
    assert rel_err(s0.cpu().numpy(), s0_o) < TOL_BF16 and rel_err(s1.cpu().numpy(), s1_o) < TOL_BF16
    # far inside the bar stated for bf16 rows: the rows are exact inputs, what is left is the rounding of an fp32
    # sum of 200 terms (worst element of 100 M)
    assert rel_err(got, th_o) < 1e-4


def test_config2_full_size_every_element_against_the_oracle(sgdb, cuda_device):
    """One step over the 300-tensor table (56.7 M parameters, W = 54, N = 50, momentum SGD) and EVERY element of
    every tensor's parameters and momentum compared with the oracle's mean and update, tensor by tensor."""
    import os
    from concurrent.futures import ThreadPoolExecutor

    _need_memory(cuda_device, 20)
    dev, cfg = cuda_device, wl.CONFIGS[2]
    W, N = cfg.W, cfg.N
    lengths = wl.segment_lengths(cfg.seed, cfg.segments)
    scales = wl.worker_scales(cfg.seed, W)
    segs = []
    for i, L in enumerate(int(x) for x in lengths):
        ld = (L + 3) // 4 * 4
        segs.append((wl.theta0(cfg.seed + i, L, dev), torch.zeros(L, device=dev), None,
                     wl.grad_matrix(cfg.seed + i, 0, W, L, scales, "f32", dev, ld=ld)))
    before = [s[0].cpu().numpy().astype(np.float64) for s in segs]
    table = sgdb.make_segment_table(segs, dev)
    mask, order, info = selection_buffers(W, N, dev)
    arrival, tags = step_inputs(cfg.seed, 0, W, N)
    sgdb.sgdb_step_segmented(table, len(segs), torch.float32, to_dev(arrival, dev), to_dev(tags, dev), 0, N, cfg.b,
                             gpu_opt(cfg.opt, 1), mask, order, info)
    rc, mask_o, order_o, n_valid = oracle.select(arrival, tags, 0, N, cfg.b)
    assert rc == oracle.OK and info.cpu().tolist() == [n_valid, 0] and order.cpu().numpy().tolist() == order_o.tolist()

    def one_tensor(i):
        theta, v, _, grad = segs[i]
        L = theta.numel()
        mean = oracle.aggregate(wl.as_oracle_array(grad), L, order_o, ld=grad.stride(0))
        th_o, v_o = before[i], np.zeros(L)
        oracle.update(th_o, v_o, None, mean, oracle_opt(cfg.opt, 1))
        return theta.cpu().numpy(), th_o, v.cpu().numpy(), v_o

    with ThreadPoolExecutor(max_workers=max(1, len(os.sched_getaffinity(0)))) as pool:
        results = list(pool.map(one_tensor, range(len(segs))))
    got = np.concatenate([r[0] for r in results])
    want = np.concatenate([r[1] for r in results])
    assert got.size == int(lengths.sum())
    assert rel_err(got, want) < TOL_F32
    assert rel_err(np.concatenate([r[2] for r in results]), np.concatenate([r[3] for r in results])) < TOL_F32
    assert float(np.max(np.abs(got - want) / np.maximum(np.abs(want), 1e-2))) < 1e-4


def test_more_columns_than_a_32_bit_index_holds(sgdb, cuda_device):
    """P = 2^31 + 4099 columns (8.6 GB per fp32 vector), W = 3 (N = 2, b = 1), plain SGD: every column index, tile
    start and byte offset beyond 2^31 must be computed in 64 bits.  The fused step against the oracle at sampled
    columns (the first, the last, both sides of 2^31 and of 2^32 bytes); the separate calls, the rows-by-address
    step and the arrival-by-arrival server against the fused step on the whole vector, bit for bit."""
    _need_memory(cuda_device, 80)
    dev = cuda_device
    P, W, N, b, seed = (1 << 31) + 4099, 3, 2, 1, 977
    opt_kw = dict(kind="sgd", lr=0.1)
    rng = np.random.default_rng(seed)
    edges = np.concatenate([np.arange(e - 3, e + 3) for e in ((1 << 30), (1 << 31), (1 << 31) + 2048, P - 3)])
    cols = np.unique(np.concatenate([_sample_columns(P, rng, n=2000), edges[(edges >= 0) & (edges < P)]]))
    cols_d = to_dev(cols, dev)
    grad = wl.grad_matrix(seed, 0, W, P, wl.worker_scales(seed, W), "f32", dev)
    arrival = np.array([2.0, 1.0, 3.0], np.float32)
    tags = np.zeros(W, np.int32)
    a_d, t_d = to_dev(arrival, dev), to_dev(tags, dev)
    theta = wl.theta0(seed, P, dev)
    th_o = theta[cols_d].cpu().numpy().astype(np.float64)
    twin = theta.clone()
    mask, order, info = selection_buffers(W, N, dev)
    sgdb.sgdb_step(grad, P, a_d, t_d, 0, N, b, theta, None, None, gpu_opt(opt_kw), mask, order, info)
    rc, mask_o, order_o, n_valid = oracle.step(wl.as_oracle_array(grad.index_select(1, cols_d)), len(cols), arrival, tags, 0,
                                               N, b, th_o, None, None, oracle_opt(opt_kw))
    assert rc == oracle.OK and info.cpu().tolist() == [n_valid, 0] and order.cpu().numpy().tolist() == order_o.tolist()
    assert rel_err(theta[cols_d].cpu().numpy(), th_o) < TOL_F32
    # separate calls: the mean goes through memory
    mean = torch.empty(P, device=dev)
    sgdb.sgdb_aggregate(grad, P, N, order, info, mean)
    sgdb.sgdb_update(twin, None, None, mean, gpu_opt(opt_kw), info)
    assert torch.equal(twin, theta)
    # the arrival-by-arrival server, the running sum in the buffer that held the mean; rows in delivery sequence
    twin.copy_(wl.theta0(seed, P, dev))
    counter = torch.zeros(4, dtype=torch.int32, device=dev)
    ainfo = torch.zeros(2, dtype=torch.int32, device=dev)
    for w in wl.delivery_sequence(arrival):
        sgdb.sgdb_accumulate_arrival(grad[w], 0, 0, N, mean, counter, twin, None, None, gpu_opt(opt_kw), ainfo)
    assert counter.cpu().tolist() == [0, W, 0, 1] and torch.equal(twin, theta)
    # every row at its own address, two servers over two ranges, each storing into the other's copy as well
    del mean
    twin.copy_(wl.theta0(seed, P, dev))
    other = twin.clone()
    for j, copies in ((0, (twin, other)), (1, (other, twin))):
        first, n = sgdb.sgdb_shard_range(P, 2, j)
        rows = sgdb.make_address_table([grad[w].data_ptr() + first * 4 for w in range(W)], dev)
        push = sgdb.make_address_table([copies[1].data_ptr() + first * 4], dev)
        sgdb.sgdb_step_rows(rows, torch.float32, n, a_d, t_d, 0, N, b, copies[0][first:first + n], None, None, gpu_opt(opt_kw),
                            push, mask, order, info)
    assert torch.equal(twin, theta) and torch.equal(other, theta)

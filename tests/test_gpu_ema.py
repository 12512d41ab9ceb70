"""Parity of the fused parameter average (sgdb_step_ema), the stand-alone average (sgdb_ema) and the
learning-rate schedule with the oracle."""
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


@pytest.mark.parametrize("kind,dtype,P,pad,alpha", [("rmsprop", "f32", 70_001, 3, 0.9999), ("sgd", "f32", 5, 0, 0.5),
                                                    ("adam", "bf16", 70_003, 0, 0.9), ("momentum", "f32", 131_072, 0, 0.0),
                                                    ("rmsprop", "bf16", 40_001, 7, 1.0)])
def test_step_with_parameter_average(sgdb, cuda_device, kind, dtype, P, pad, alpha):
    dev = cuda_device
    W, N, T, seed = 20, 16, 5, 141
    ld = P + pad
    scales = wl.worker_scales(seed, W)
    theta = wl.theta0(seed, P, dev)
    avg = theta.clone()  # the average before the first iteration: theta(0)
    s0, s1 = gpu_state(kind, P, dev)
    twin = (theta.clone(), avg.clone()) + gpu_state(kind, P, dev)  # separate calls: sgdb_ema, then sgdb_step
    th_o = theta.cpu().numpy().astype(np.float64)
    avg_o = th_o.copy()
    s0_o, s1_o = oracle_state(kind, P)
    mask, order, info = selection_buffers(W, N, dev)
    mask2, order2, info2 = selection_buffers(W, N, dev)
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    for t in range(T):
        grad = wl.grad_matrix(seed, t, W, P, scales, dtype, dev, ld=ld, pad_value=float("nan"))
        arrival, tags = step_inputs(seed, t, W, N)
        a_d, t_d = to_dev(arrival, dev), to_dev(tags, dev)
        sgdb.sgdb_step_ema(grad, P, a_d, t_d, t, N, W - N, theta, s0, s1, gpu_opt(OPTS[kind], t + 1), avg, alpha,
                           mask, order, info, ld=ld)
        rc, mask_o, order_o, n_valid = oracle.step_ema(wl.as_oracle_array(grad), P, arrival, tags, t, N, W - N, th_o,
                                                       s0_o, s1_o, oracle_opt(OPTS[kind], t + 1), avg_o, f32(alpha), ld=ld)
        assert rc == oracle.OK and info.cpu().tolist() == [n_valid, 0]
        assert order.cpu().numpy().tolist() == order_o.tolist() and mask.cpu().numpy().tolist() == mask_o.tolist()
        sgdb.sgdb_ema(twin[1], twin[0], alpha)
        sgdb.sgdb_step(grad, P, a_d, t_d, t, N, W - N, twin[0], twin[2], twin[3], gpu_opt(OPTS[kind], t + 1),
                       mask2, order2, info2, ld=ld)
    assert rel_err(theta.cpu().numpy(), th_o) < tol
    assert rel_err(avg.cpu().numpy(), avg_o) < tol
    assert torch.equal(theta, twin[0]) and torch.equal(avg, twin[1])  # fused == separate, bit for bit


@pytest.mark.parametrize("kind,dtype", [("rmsprop", "f32"), ("adagrad", "bf16")])
def test_arrival_mode_with_parameter_average(sgdb, cuda_device, kind, dtype):
    """Row by row delivery: the average moves only in the launch that fires the update; results equal the fused
    sgdb_step_ema bit for bit and the oracle within tolerance."""
    dev = cuda_device
    N, b, P, T, seed, alpha = 9, 2, 40_003, 3, 211, 0.9
    W = N + b
    scales = wl.worker_scales(seed, W)
    theta = wl.theta0(seed, P, dev)
    avg = theta.clone()
    s0, s1 = gpu_state(kind, P, dev)
    fused = (theta.clone(), avg.clone()) + gpu_state(kind, P, dev)
    acc = torch.empty(P, device=dev)
    counter = torch.zeros(4, dtype=torch.int32, device=dev)
    info = torch.zeros(2, dtype=torch.int32, device=dev)
    th_o = theta.cpu().numpy().astype(np.float64)
    avg_o = th_o.copy()
    s0_o, s1_o = oracle_state(kind, P)
    acc_o, state_o = np.zeros(P), oracle.new_server_state()
    mask, order, finfo = selection_buffers(W, N, dev)
    for t in range(T):
        grad = wl.grad_matrix(seed, t, W, P, scales, dtype, dev)
        grad_h = wl.as_oracle_array(grad)
        arrival, tags = step_inputs(seed, t, W, N)
        for w in wl.delivery_sequence(arrival):
            before = avg.clone()
            sgdb.sgdb_accumulate_arrival_ema(grad[w], int(tags[w]), t, N, acc, counter, theta, s0, s1,
                                             gpu_opt(OPTS[kind], t + 1), avg, alpha, info)
            want = oracle.accumulate_arrival_ema(grad_h[w], int(tags[w]), t, N, acc_o, state_o, th_o, s0_o, s1_o,
                                                 oracle_opt(OPTS[kind], t + 1), avg_o, f32(alpha))
            assert info.cpu().tolist()[0] == want
            if want != 2:
                assert torch.equal(avg, before)  # the average waits for the update
        sgdb.sgdb_step_ema(grad, P, to_dev(arrival, dev), to_dev(tags, dev), t, N, b, fused[0], fused[2], fused[3],
                           gpu_opt(OPTS[kind], t + 1), fused[1], alpha, mask, order, finfo)
        assert torch.equal(theta, fused[0]) and torch.equal(avg, fused[1])
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    assert rel_err(theta.cpu().numpy(), th_o) < tol and rel_err(avg.cpu().numpy(), avg_o) < tol


def test_average_untouched_when_gradients_are_insufficient_and_bad_arguments(sgdb, cuda_device):
    dev = cuda_device
    W, N, P = 6, 5, 10_000
    grad = torch.randn((W, P), device=dev)
    theta, avg = torch.randn(P, device=dev), torch.randn(P, device=dev)
    before = (theta.clone(), avg.clone())
    mask, order, info = selection_buffers(W, N, dev)
    arrival = to_dev(np.arange(W, dtype=np.float32), dev)
    stale = to_dev(np.array([1, 1, 0, 0, 1, 1], np.int32), dev)
    sgdb.sgdb_step_ema(grad, P, arrival, stale, 1, N, 1, theta, None, None, gpu_opt(OPTS["sgd"]), avg, 0.5, mask, order, info)
    assert info.cpu().tolist() == [4, sgdb.SGDB_ERR_INSUFFICIENT]
    assert torch.equal(theta, before[0]) and torch.equal(avg, before[1])
    sgdb.sgdb_ema(avg, theta, 0.5, info)  # the separate call honours the same status word
    assert torch.equal(avg, before[1])
    for bad_alpha in (-0.1, 1.5, float("nan")):
        with pytest.raises(sgdb.SgdbError):
            sgdb.sgdb_step_ema(grad, P, arrival, stale, 1, N, 1, theta, None, None, gpu_opt(OPTS["sgd"]), avg, bad_alpha,
                               mask, order, info)
        with pytest.raises(sgdb.SgdbError):
            sgdb.sgdb_ema(avg, theta, bad_alpha)


def test_learning_rate_schedule_matches_oracle(sgdb):
    for gamma0, beta, t, N, T in [(4.5, 0.94, 0, 100, 40_000.0), (4.5, 0.94, 12_345, 100, 40_036.0),
                                  (0.045, 0.94, 777_777, 1, 40_036.0), (1e-4, 0.5, 3, 16, 12_500.0)]:
        assert sgdb.sgdb_learning_rate(gamma0, beta, t, N, T) == pytest.approx(oracle.learning_rate(gamma0, beta, t, N, T), rel=1e-14)
    assert np.isnan(sgdb.sgdb_learning_rate(1.0, 0.9, 1, 1, 0.0)) and np.isnan(sgdb.sgdb_learning_rate(1.0, 0.9, -1, 1, 5.0))


@pytest.mark.parametrize("kind,dtype,packed", [("rmsprop", "f32", False), ("adam", "bf16", True), ("sgd", "f32", True)])
def test_segmented_step_with_parameter_averages(sgdb, cuda_device, kind, dtype, packed):
    """The multi-tensor step keeps one average per tensor (Algorithm 4 runs its last line for every variable):
    against the oracle per tensor, and bit for bit against one sgdb_step_ema launch per (aligned) tensor.  One
    tensor has no average (NULL entry)."""
    dev = cuda_device
    W, N, T, seed, alpha = 12, 9, 3, 221, 0.75
    lengths = [1, 5, 64, 2047, 2048, 2049, 4100, 0, 30_001, 7, 12_288]
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    vec = 4 if dtype == "f32" else 8
    scales = wl.worker_scales(seed, W)
    total = sum(lengths)
    th_all = wl.theta0(seed, total, dev)
    avg_all = th_all.clone()
    st_all = [torch.zeros(total, device=dev), torch.zeros(total, device=dev)]
    n_state = {"sgd": 0, "rmsprop": 2, "adam": 2}[kind]
    segs, avgs, off = [], [], 0
    for i, L in enumerate(lengths):
        if packed:  # carved back to back out of shared buffers: most tensors are only element-aligned
            theta, avg = th_all[off:off + L], avg_all[off:off + L]
            s0, s1 = st_all[0][off:off + L], st_all[1][off:off + L]
            grad = wl.grad_matrix(seed + i, 0, W, L, scales, dtype, dev)
        else:
            theta = wl.theta0(seed + i, L, dev)
            avg = theta.clone()
            s0, s1 = torch.zeros(L, device=dev), torch.zeros(L, device=dev)
            grad = wl.grad_matrix(seed + i, 0, W, L, scales, dtype, dev, ld=(L + vec - 1) // vec * vec, pad_value=float("nan"))
        segs.append((theta, s0 if n_state >= 1 else None, s1 if n_state >= 2 else None, grad))
        avgs.append(None if i == 2 else avg)
        off += L
    twins = [tuple(None if x is None else x.clone() for x in (s[0], s[1], s[2], a)) for s, a in zip(segs, avgs)]
    th_o = [s[0].cpu().numpy().astype(np.float64) for s in segs]
    avg_o = [x.copy() for x in th_o]
    st_o = [oracle_state(kind, L) for L in lengths]
    table = sgdb.make_segment_table(segs, dev)
    ema_table = sgdb.make_pointer_table(avgs, dev)
    mask, order, info = selection_buffers(W, N, dev)
    mask2, order2, info2 = selection_buffers(W, N, dev)
    for t in range(T):
        if t:
            for i, (theta, _, _, grad) in enumerate(segs):
                if theta.numel():
                    wl.grad_matrix(seed + i, t, W, theta.numel(), scales, dtype, dev, ld=grad.stride(0), out=grad,
                                   pad_value=float("nan"))
        arrival, tags = step_inputs(seed, t, W, N)
        a_d, t_d = to_dev(arrival, dev), to_dev(tags, dev)
        sgdb.sgdb_step_segmented_ema(table, ema_table, alpha, len(segs), tdt, a_d, t_d, t, N, W - N,
                                     gpu_opt(OPTS[kind], t + 1), mask, order, info)
        rc, _, order_o, n_valid = oracle.select(arrival, tags, t, N, W - N)
        assert rc == oracle.OK and info.cpu().tolist() == [n_valid, 0] and order.cpu().numpy().tolist() == order_o.tolist()
        for i, (theta, s0, s1, grad) in enumerate(segs):
            L = theta.numel()
            if L == 0:
                continue
            rc, *_ = oracle.step_ema(wl.as_oracle_array(grad), L, arrival, tags, t, N, W - N, th_o[i], st_o[i][0], st_o[i][1],
                                     oracle_opt(OPTS[kind], t + 1), avg_o[i], f32(alpha), ld=grad.stride(0))
            assert rc == oracle.OK
            aligned = all(x is None or x.data_ptr() % 16 == 0 for x in (theta, s0, s1, grad, avgs[i]))
            if aligned and avgs[i] is not None:
                sgdb.sgdb_step_ema(grad, L, a_d, t_d, t, N, W - N, twins[i][0], twins[i][1], twins[i][2],
                                   gpu_opt(OPTS[kind], t + 1), twins[i][3], alpha, mask2, order2, info2, ld=grad.stride(0))
                assert torch.equal(theta, twins[i][0]) and torch.equal(avgs[i], twins[i][3]), (i, L)
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    for i, (theta, _, _, _) in enumerate(segs):
        L = theta.numel()
        if L == 0:
            continue
        scale = max(1.0, float(np.sqrt(np.mean(th_o[i] ** 2))))
        assert np.max(np.abs(theta.cpu().numpy() - th_o[i])) / scale < tol * 4, (i, L)
        if avgs[i] is not None:
            assert np.max(np.abs(avgs[i].cpu().numpy() - avg_o[i])) / scale < tol * 4, (i, L)
        if L >= 64:
            assert rel_err(theta.cpu().numpy(), th_o[i]) < tol
            if avgs[i] is not None:
                assert rel_err(avgs[i].cpu().numpy(), avg_o[i]) < tol
    if packed:  # the tensor without an average: its slot of the shared buffer still holds theta(0)
        start = sum(lengths[:2])
        assert torch.equal(avg_all[start:start + lengths[2]], wl.theta0(seed, total, dev)[start:start + lengths[2]])

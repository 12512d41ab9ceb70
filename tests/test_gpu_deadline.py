"""Parity of the time-out rule (sgdb_select_deadline, sgdb_step_deadline) with the oracle."""
import numpy as np
import pytest
import torch

import oracle
from helpers import (OPTS, TOL_BF16, TOL_F32, gpu_opt, gpu_state, oracle_opt, oracle_state, rel_err,
                     selection_buffers, step_inputs, to_dev)
from paper_1604_00981_b200 import workload as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sgdb(cuda_device):
    from paper_1604_00981_b200 import binding

    return binding


def test_deadline_selection_bit_exact(sgdb, cuda_device):
    dev = cuda_device
    rng = np.random.default_rng(151)
    values = np.array([0.25, 0.5, 0.5, 1.0, 1.5, 2.0, 7.0, np.inf, np.nan, -0.0, 0.0, -1.0, -np.inf], np.float32)
    outcomes = set()
    for trial in range(200):
        W = int(rng.choice([1, 2, 3, 6, 31, 32, 33, 54, 100, 208, 1024]))
        if trial % 2:
            arrival = values[rng.integers(0, len(values), size=W)]
        else:
            arrival = rng.lognormal(0, 0.3, size=W).astype(np.float32)
            arrival[rng.integers(0, W, size=W // 4)] = 1.0
        t = int(rng.integers(0, 50))
        tags = np.where(rng.random(W) < 0.15, t - 1, t).astype(np.int32)
        deadline = float(rng.choice([0.5, 0.9, 1.0, 1.2, 2.0, 100.0, np.inf, -2.0]))
        n_min = int(rng.integers(1, W + 1)) if trial % 3 == 0 else 1
        mask, order, info = selection_buffers(W, W, dev)
        sgdb.sgdb_select_deadline(to_dev(arrival, dev), to_dev(tags, dev), t, deadline, n_min, mask, order, info)
        rc, mask_o, order_o, n = oracle.select_deadline(arrival, tags, t, deadline, n_min)
        outcomes.add(rc)
        got = info.cpu().tolist()
        assert got[0] == n
        if rc == oracle.OK:
            assert got[1] == 0 and mask.cpu().numpy().tolist() == mask_o.tolist()
            assert order.cpu().numpy()[:n].tolist() == order_o.tolist()
            assert (order.cpu().numpy()[n:] == -7).all()  # entries past n are not written
        else:
            assert got[1] == sgdb.SGDB_ERR_INSUFFICIENT and (mask.cpu() == 255).all() and (order.cpu() == -7).all()
    assert outcomes == {oracle.OK, oracle.INSUFFICIENT}
    a, tg = torch.zeros(4, device=dev), torch.zeros(4, dtype=torch.int32, device=dev)
    mask, order, info = selection_buffers(4, 4, dev)
    for bad in (dict(deadline=float("nan"), n_min=1), dict(deadline=1.0, n_min=0), dict(deadline=1.0, n_min=5)):
        with pytest.raises(sgdb.SgdbError):
            sgdb.sgdb_select_deadline(a, tg, 0, bad["deadline"], bad["n_min"], mask, order, info)


@pytest.mark.parametrize("kind,dtype,P,pad", [("rmsprop", "f32", 70_001, 3), ("adam", "bf16", 70_003, 0),
                                              ("sgd", "f32", 131_072, 0), ("momentum", "bf16", 9, 0)])
def test_step_with_deadline_trajectory(sgdb, cuda_device, kind, dtype, P, pad):
    """The number of kept gradients changes from step to step with the drawn arrival times."""
    dev = cuda_device
    W, T, seed = 40, 5, 161
    ld = P + pad
    scales = wl.worker_scales(seed, W)
    theta = wl.theta0(seed, P, dev)
    s0, s1 = gpu_state(kind, P, dev)
    th_o = theta.cpu().numpy().astype(np.float64)
    s0_o, s1_o = oracle_state(kind, P)
    mask, order, info = selection_buffers(W, W, dev)
    counts = []
    for t in range(T):
        grad = wl.grad_matrix(seed, t, W, P, scales, dtype, dev, ld=ld, pad_value=float("nan"))
        arrival, tags = step_inputs(seed, t, W, 1)
        deadline = float(np.float32([1.0, 1.3, 0.8, 6.0, 1.1][t]))
        sgdb.sgdb_step_deadline(grad, P, to_dev(arrival, dev), to_dev(tags, dev), t, deadline, 1, theta, s0, s1,
                                gpu_opt(OPTS[kind], t + 1), mask, order, info, ld=ld)
        rc, mask_o, order_o, n = oracle.step_deadline(wl.as_oracle_array(grad), P, arrival, tags, t, deadline, 1,
                                                      th_o, s0_o, s1_o, oracle_opt(OPTS[kind], t + 1), ld=ld)
        assert rc == oracle.OK and info.cpu().tolist() == [n, 0]
        assert mask.cpu().numpy().tolist() == mask_o.tolist() and order.cpu().numpy()[:n].tolist() == order_o.tolist()
        counts.append(n)
    assert len(set(counts)) >= 3, counts
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    assert rel_err(theta.cpu().numpy(), th_o) < tol
    for x, y in ((s0, s0_o), (s1, s1_o)):
        assert x is None or rel_err(x.cpu().numpy(), y) < tol


def test_deadline_at_the_nth_arrival_is_the_first_n_rule_and_too_few_changes_nothing(sgdb, cuda_device):
    dev = cuda_device
    W, N, P, seed = 30, 24, 90_001, 171
    grad = wl.grad_matrix(seed, 0, W, P, wl.worker_scales(seed, W), "f32", dev)
    arrival, tags = step_inputs(seed, 0, W, N)
    rc, _, order_o, _ = oracle.select(arrival, tags, 0, N, W - N)
    deadline = float(arrival[order_o[-1]])  # the time the N-th kept gradient arrives
    assert (arrival[tags == 0] <= deadline).sum() == N  # no tie at the deadline in this draw
    th_a, th_b = wl.theta0(seed, P, dev), wl.theta0(seed, P, dev)
    sa, sb = gpu_state("rmsprop", P, dev), gpu_state("rmsprop", P, dev)
    mask_a, order_a, info_a = selection_buffers(W, N, dev)
    mask_b, order_b, info_b = selection_buffers(W, W, dev)
    a_d, t_d = to_dev(arrival, dev), to_dev(tags, dev)
    sgdb.sgdb_step(grad, P, a_d, t_d, 0, N, W - N, th_a, sa[0], sa[1], gpu_opt(OPTS["rmsprop"]), mask_a, order_a, info_a)
    sgdb.sgdb_step_deadline(grad, P, a_d, t_d, 0, deadline, 1, th_b, sb[0], sb[1], gpu_opt(OPTS["rmsprop"]), mask_b,
                            order_b, info_b)
    assert info_b.cpu().tolist() == [N, 0]
    assert torch.equal(th_a, th_b) and torch.equal(sa[0], sb[0]) and torch.equal(sa[1], sb[1])
    assert torch.equal(mask_a, mask_b) and torch.equal(order_a, order_b[:N])
    before = th_b.clone()
    sgdb.sgdb_step_deadline(grad, P, a_d, t_d, 0, deadline, N + 1, th_b, sb[0], sb[1], gpu_opt(OPTS["rmsprop"]), mask_b,
                            order_b, info_b)
    assert info_b.cpu().tolist() == [N, sgdb.SGDB_ERR_INSUFFICIENT] and torch.equal(th_b, before)

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


@pytest.mark.parametrize("kind,dtype", [("momentum", "f32"), ("rmsprop", "bf16")])
def test_segmented_step_with_deadline(sgdb, cuda_device, kind, dtype):
    """The time-out rule over a segment table: per tensor against the oracle's time-out step, and bit for bit
    against one sgdb_step_deadline launch per tensor."""
    dev = cuda_device
    W, T, seed = 24, 3, 231
    lengths = [3, 100, 2048, 4099, 0, 25_001, 8192]
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    vec = 4 if dtype == "f32" else 8
    scales = wl.worker_scales(seed, W)
    n_state = {"momentum": 1, "rmsprop": 2}[kind]
    segs = []
    for i, L in enumerate(lengths):
        grad = wl.grad_matrix(seed + i, 0, W, L, scales, dtype, dev, ld=(L + vec - 1) // vec * vec, pad_value=float("nan"))
        segs.append((wl.theta0(seed + i, L, dev), torch.zeros(L, device=dev), torch.zeros(L, device=dev) if n_state == 2 else None, grad))
    twins = [tuple(None if x is None else x.clone() for x in s[:3]) for s in segs]
    th_o = [s[0].cpu().numpy().astype(np.float64) for s in segs]
    st_o = [oracle_state(kind, L) for L in lengths]
    table = sgdb.make_segment_table(segs, dev)
    mask, order, info = selection_buffers(W, W, dev)
    mask2, order2, info2 = selection_buffers(W, W, dev)
    counts = []
    for t in range(T):
        if t:
            for i, (theta, _, _, grad) in enumerate(segs):
                if theta.numel():
                    wl.grad_matrix(seed + i, t, W, theta.numel(), scales, dtype, dev, ld=grad.stride(0), out=grad,
                                   pad_value=float("nan"))
        arrival, tags = step_inputs(seed, t, W, 1)
        deadline = float(np.float32([0.9, 1.4, 1.1][t]))
        a_d, t_d = to_dev(arrival, dev), to_dev(tags, dev)
        sgdb.sgdb_step_segmented_deadline(table, len(segs), tdt, a_d, t_d, t, deadline, 2, gpu_opt(OPTS[kind], t + 1),
                                          mask, order, info)
        rc, mask_o, order_o, n = oracle.select_deadline(arrival, tags, t, deadline, 2)
        assert rc == oracle.OK and info.cpu().tolist() == [n, 0]
        assert mask.cpu().numpy().tolist() == mask_o.tolist() and order.cpu().numpy()[:n].tolist() == order_o.tolist()
        counts.append(n)
        for i, (theta, s0, s1, grad) in enumerate(segs):
            L = theta.numel()
            if L == 0:
                continue
            rc, *_ = oracle.step_deadline(wl.as_oracle_array(grad), L, arrival, tags, t, deadline, 2, th_o[i], st_o[i][0],
                                          st_o[i][1], oracle_opt(OPTS[kind], t + 1), ld=grad.stride(0))
            assert rc == oracle.OK
            sgdb.sgdb_step_deadline(grad, L, a_d, t_d, t, deadline, 2, twins[i][0], twins[i][1], twins[i][2],
                                    gpu_opt(OPTS[kind], t + 1), mask2, order2, info2, ld=grad.stride(0))
            assert torch.equal(theta, twins[i][0]), (i, L)
    assert len(set(counts)) >= 2
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    for i, (theta, s0, _, _) in enumerate(segs):
        if theta.numel() >= 64:
            assert rel_err(theta.cpu().numpy(), th_o[i]) < tol and rel_err(s0.cpu().numpy(), st_o[i][0]) < tol
    # too few by the deadline: nothing moves
    before = [s[0].clone() for s in segs]
    sgdb.sgdb_step_segmented_deadline(table, len(segs), tdt, a_d, t_d, T - 1, -5.0, 1, gpu_opt(OPTS[kind]), mask, order, info)
    assert info.cpu().tolist() == [0, sgdb.SGDB_ERR_INSUFFICIENT]
    assert all(torch.equal(s[0], b) for s, b in zip(segs, before))


@pytest.mark.parametrize("kind,dtype,P", [("rmsprop", "f32", 70_001), ("adam", "bf16", 50_003), ("sgd", "f32", 6)])
def test_arrival_mode_with_deadline_and_close(sgdb, cuda_device, kind, dtype, P):
    """The time-out rule one gradient per call: rows in event order (those that arrive by the deadline, the close
    call, then the late ones), outcomes and counters against the oracle's replay, parameters, state and parameter
    average against the oracle and, bit for bit, against the fused sgdb_step_deadline."""
    dev = cuda_device
    W, T, seed, alpha = 16, 4, 241, 0.9
    scales = wl.worker_scales(seed, W)
    theta = wl.theta0(seed, P, dev)
    theta_f, avg = theta.clone(), theta.clone()
    s0, s1 = gpu_state(kind, P, dev)
    sf = gpu_state(kind, P, dev)
    acc = torch.full((P,), float("nan"), device=dev)
    counter = torch.zeros(4, dtype=torch.int32, device=dev)
    info = torch.zeros(2, dtype=torch.int32, device=dev)
    th_o = theta.cpu().numpy().astype(np.float64)
    avg_o = th_o.copy()
    s0_o, s1_o = oracle_state(kind, P)
    acc_o, state_o = np.zeros(P), oracle.new_server_state()
    mask, order, finfo = selection_buffers(W, W, dev)
    seen = 0
    for t in range(T):
        grad = wl.grad_matrix(seed, t, W, P, scales, dtype, dev)
        grad_h = wl.as_oracle_array(grad)
        arrival, tags = step_inputs(seed, t, W, 1)
        arrival[3] = np.inf  # a worker that died
        deadline = float(np.sort(arrival)[W // 2]) if t != 2 else -1.0  # iteration 2: nobody makes it
        n_min = 2
        ids = [int(w) for w in np.argsort(arrival, kind="stable")]
        early = [w for w in ids if arrival[w] <= np.float32(deadline)]
        late = [w for w in ids if not arrival[w] <= np.float32(deadline)]
        opt, opt_o = gpu_opt(OPTS[kind], t + 1), oracle_opt(OPTS[kind], t + 1)
        for w in early:
            sgdb.sgdb_accumulate_arrival_deadline(grad[w], int(tags[w]), float(arrival[w]), t, deadline, acc, counter, info)
            want = oracle.accumulate_arrival_deadline(grad_h[w], int(tags[w]), float(arrival[w]), t, deadline, acc_o, state_o)
            seen += 1
            assert info.cpu().tolist() == [want, int(state_o[0])]
            assert counter.cpu().tolist() == [int(state_o[0]), seen, 0, int(state_o[2])]
        sgdb.sgdb_accumulate_close(t, n_min, acc, counter, theta, s0, s1, opt, info, ema=avg, alpha=alpha)
        in_set = int(state_o[0])
        rc, outcome = oracle.accumulate_close(t, n_min, acc_o, state_o, th_o, s0_o, s1_o, opt_o, avg_o, alpha)
        assert info.cpu().tolist() == [outcome, in_set]
        assert (rc == oracle.OK) == (outcome == 2)
        assert counter.cpu().tolist() == [int(state_o[0]), seen, 0, int(state_o[2])]
        for w in late:  # after the close: dropped
            sgdb.sgdb_accumulate_arrival_deadline(grad[w], int(tags[w]), float(arrival[w]), t, deadline, acc, counter, info)
            want = oracle.accumulate_arrival_deadline(grad_h[w], int(tags[w]), float(arrival[w]), t, deadline, acc_o, state_o)
            seen += 1
            assert want == 0 and info.cpu().tolist()[0] == 0
        # the fused time-out step on the same inputs
        before = theta_f.clone()
        sgdb.sgdb_step_deadline(grad, P, to_dev(arrival, dev), to_dev(tags, dev), t, deadline, n_min, theta_f, sf[0], sf[1],
                                opt, mask, order, finfo)
        if outcome == 2:
            assert finfo.cpu().tolist() == [in_set, 0]
        else:
            assert finfo.cpu().tolist()[1] == sgdb.SGDB_ERR_INSUFFICIENT and torch.equal(theta_f, before)
            counter[0] = 0  # the test gives up on this iteration and moves on
            counter[3] = t + 1
            state_o[0], state_o[2] = 0, t + 1
        assert torch.equal(theta, theta_f)
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    for x, y in zip((s0, s1), sf):
        assert x is None or torch.equal(x, y)
    if P >= 64:
        assert rel_err(theta.cpu().numpy(), th_o) < tol and rel_err(avg.cpu().numpy(), avg_o) < tol
    else:
        assert np.max(np.abs(theta.cpu().numpy() - th_o)) < tol * 4

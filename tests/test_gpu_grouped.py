"""Two-level aggregation (machines combine their workers' gradients; the server keeps the first N messages):
the fused sgdb_step_grouped against the oracle and against the composition of existing calls."""
import numpy as np
import pytest
import torch

import oracle
from helpers import (OPTS, TOL_BF16, TOL_F32, gpu_opt, gpu_state, oracle_opt, oracle_state, rel_err, selection_buffers,
                     to_dev)
from paper_1604_00981_b200 import workload as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sgdb(cuda_device):
    from paper_1604_00981_b200 import binding

    return binding


def _buffers(W, N, dev):
    return (torch.full((W,), 255, dtype=torch.uint8, device=dev), torch.full((N,), -7, dtype=torch.int32, device=dev),
            torch.full((W,), -7, dtype=torch.int32, device=dev), torch.full((3,), -7, dtype=torch.int32, device=dev))


def _machines(rng, W, M, layout):
    if layout == "blocks":  # workers of a machine are neighbours, equal sizes where W divides
        return (np.arange(W) * M // W).astype(np.int32)
    if layout == "scattered":
        return rng.integers(0, M, size=W).astype(np.int32)
    return np.arange(W, dtype=np.int32) % M  # "striped"


def _special_arrivals(rng, W):
    values = np.array([0.25, 0.5, 0.5, 1.0, 1.5, 2.0, 7.0, -0.0, 0.0, -1.0, np.inf, np.nan, -np.inf], np.float32)
    return values[rng.integers(0, len(values), size=W)]


def test_grouped_selection_is_bit_exact(sgdb, cuda_device):
    """Selection alone on many random cases, special values included: every output word equals the oracle's, and
    nothing but the info words is written when the iteration cannot complete."""
    dev = cuda_device
    rng = np.random.default_rng(31)
    ok = short = 0
    for trial in range(300):
        W = int(rng.integers(1, 70)) if trial % 10 else int(rng.integers(900, 1025))
        M = int(rng.integers(1, min(W, 40) + 1)) if trial % 7 else W
        N = int(rng.integers(1, M + 1))
        group = _machines(rng, W, M, ("blocks", "scattered", "striped")[trial % 3])
        t = int(rng.integers(0, 4))
        if trial % 2:
            arrival = _special_arrivals(rng, W)
            tags = np.where(rng.random(W) < 0.05, t - 1, t).astype(np.int32)
        else:
            arrival = wl.arrivals(31 + trial, t, W)
            tags = np.where(rng.random(W) < 0.02, t + rng.choice([-1, 1], size=W), t).astype(np.int32)
        mask, gorder, order, info = _buffers(W, N, dev)
        sgdb.sgdb_select_grouped(to_dev(arrival, dev), to_dev(tags, dev), to_dev(group, dev), t, M, N, mask, gorder, order, info)
        rc, mask_o, gorder_o, order_o, n_valid = oracle.select_grouped(arrival, tags, group, t, M, N)
        if rc == oracle.OK:
            ok += 1
            assert info.cpu().tolist() == [n_valid, 0, len(order_o)]
            assert mask.cpu().numpy().tolist() == mask_o.tolist() and gorder.cpu().numpy().tolist() == gorder_o.tolist()
            assert order.cpu().numpy()[: len(order_o)].tolist() == order_o.tolist()
            assert (order.cpu().numpy()[len(order_o):] == -7).all()
        else:
            short += 1
            assert rc == oracle.INSUFFICIENT and info.cpu().tolist() == [n_valid, sgdb.SGDB_ERR_INSUFFICIENT, 0]
            assert (mask == 255).all() and (gorder == -7).all() and (order == -7).all()
    assert ok > 60 and short > 60


@pytest.mark.parametrize("kind,dtype,P,layout", [("rmsprop", "f32", 70_001, "blocks"), ("adam", "bf16", 100_003, "scattered"),
                                                 ("sgd", "f32", 4099, "striped"), ("momentum", "bf16", 8192, "blocks"),
                                                 ("adagrad", "f32", 33_333, "scattered"), ("sgd", "f32", 3, "blocks")])
def test_grouped_step_matches_oracle(sgdb, cuda_device, kind, dtype, P, layout):
    """T fused two-level steps against the oracle: selection bit-exact, parameters and state within tolerance.
    Rows of machines that are not used are poisoned with NaN: they must never be read."""
    dev = cuda_device
    W, M, N, T, seed = 26, 7, 5, 3, 151
    rng = np.random.default_rng(seed)
    group = _machines(rng, W, M, layout)
    scales = wl.worker_scales(seed, W)
    pad = 5 if dtype == "f32" else 0
    ld = P + pad
    theta = wl.theta0(seed, P, dev)
    s0, s1 = gpu_state(kind, P, dev)
    th_o = theta.cpu().numpy().astype(np.float64)
    s0_o, s1_o = oracle_state(kind, P)
    mask, gorder, order, info = _buffers(W, N, dev)
    g_d = to_dev(group, dev)
    for t in range(T):
        grad = wl.grad_matrix(seed, t, W, P, scales, dtype, dev, ld=ld, pad_value=float("nan"))
        arrival = wl.arrivals(seed, t, W)
        tags = np.full(W, t, np.int32)
        tags[rng.integers(0, W)] = t - 1  # one machine has a stale worker
        rc, mask_o, gorder_o, order_o, n_valid = oracle.step_grouped(wl.as_oracle_array(grad), P, arrival, tags, group, t, M, N,
                                                                     th_o, s0_o, s1_o, oracle_opt(OPTS[kind], t + 1), ld=ld)
        assert rc == oracle.OK
        grad[to_dev(np.flatnonzero(mask_o == 0), dev)] = float("nan")
        sgdb.sgdb_step_grouped(grad, P, to_dev(arrival, dev), to_dev(tags, dev), g_d, t, M, N, theta, s0, s1,
                               gpu_opt(OPTS[kind], t + 1), mask, gorder, order, info, ld=ld)
        assert info.cpu().tolist() == [n_valid, 0, len(order_o)]
        assert mask.cpu().numpy().tolist() == mask_o.tolist() and gorder.cpu().numpy().tolist() == gorder_o.tolist()
        assert order.cpu().numpy()[: len(order_o)].tolist() == order_o.tolist()
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    assert bool(torch.isfinite(theta).all())
    if P >= 64:
        assert rel_err(theta.cpu().numpy(), th_o) < tol
        for x, y in ((s0, s0_o), (s1, s1_o)):
            assert x is None or rel_err(x.cpu().numpy(), y) < tol
    else:
        assert np.max(np.abs(theta.cpu().numpy() - th_o)) < tol * 4


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_grouped_step_has_the_bits_of_the_composition(sgdb, cuda_device, dtype):
    """One sgdb_aggregate per kept machine (its workers in the order they were ready) followed by sgdb_step over
    the machines' means gives the same bits as the one-launch grouped step, for unequal machine sizes too."""
    dev = cuda_device
    W, M, N, P, seed, kind = 23, 6, 4, 50_001, 161, "rmsprop"
    rng = np.random.default_rng(seed)
    group = _machines(rng, W, M, "scattered")
    group[:M] = np.arange(M)  # every machine has a worker
    grad = wl.grad_matrix(seed, 0, W, P, wl.worker_scales(seed, W), dtype, dev)
    arrival = wl.arrivals(seed, 0, W)
    tags = np.zeros(W, np.int32)
    theta = wl.theta0(seed, P, dev)
    theta_c = theta.clone()
    s, sc = gpu_state(kind, P, dev), gpu_state(kind, P, dev)
    mask, gorder, order, info = _buffers(W, N, dev)
    sgdb.sgdb_step_grouped(grad, P, to_dev(arrival, dev), to_dev(tags, dev), to_dev(group, dev), 0, M, N, theta, s[0], s[1],
                           gpu_opt(OPTS[kind]), mask, gorder, order, info)
    assert info.cpu().tolist()[:2] == [M, 0]
    # the composition: every machine's message (an fp32 row), then the server step over the M messages
    ld = (P + 3) // 4 * 4
    sent = torch.full((M, ld), float("nan"), device=dev)
    arrival_m = np.array([arrival[group == g].max() for g in range(M)], np.float32)
    for g in range(M):
        ids = np.flatnonzero(group == g)
        ids = ids[np.argsort(arrival[ids], kind="stable")].astype(np.int32)
        ok = to_dev(np.array([len(ids), 0], np.int32), dev)
        sgdb.sgdb_aggregate(grad, P, len(ids), to_dev(ids, dev), ok, sent[g, :P])
    mask_m, order_m, info_m = selection_buffers(M, N, dev)
    sgdb.sgdb_step(sent, P, to_dev(arrival_m, dev), torch.zeros(M, dtype=torch.int32, device=dev), 0, N, M - N, theta_c,
                   sc[0], sc[1], gpu_opt(OPTS[kind]), mask_m, order_m, info_m, ld=ld)
    assert order_m.cpu().tolist() == gorder.cpu().tolist()
    assert torch.equal(theta, theta_c) and torch.equal(s[0], sc[0]) and torch.equal(s[1], sc[1])


def test_grouped_step_with_one_worker_per_machine_is_the_plain_step(sgdb, cuda_device):
    dev = cuda_device
    W, N, P, seed, kind = 40, 33, 80_001, 171, "adam"
    grad = wl.grad_matrix(seed, 0, W, P, wl.worker_scales(seed, W), "bf16", dev)
    arrival, tags = wl.arrivals(seed, 0, W), wl.tags(seed, 0, W, N)
    theta = wl.theta0(seed, P, dev)
    theta_p = theta.clone()
    s, sp = gpu_state(kind, P, dev), gpu_state(kind, P, dev)
    mask, gorder, order, info = _buffers(W, N, dev)
    a_d, t_d = to_dev(arrival, dev), to_dev(tags, dev)
    sgdb.sgdb_step_grouped(grad, P, a_d, t_d, torch.arange(W, dtype=torch.int32, device=dev), 0, W, N, theta, s[0], s[1],
                           gpu_opt(OPTS[kind]), mask, gorder, order, info)
    mask_p, order_p, info_p = selection_buffers(W, N, dev)
    sgdb.sgdb_step(grad, P, a_d, t_d, 0, N, W - N, theta_p, sp[0], sp[1], gpu_opt(OPTS[kind]), mask_p, order_p, info_p)
    assert info.cpu().tolist() == info_p.cpu().tolist() + [N]
    assert torch.equal(mask, mask_p) and torch.equal(gorder, order_p) and torch.equal(order[:N], order_p)
    assert torch.equal(theta, theta_p) and torch.equal(s[0], sp[0]) and torch.equal(s[1], sp[1])


def test_grouped_step_refusals_leave_everything_untouched(sgdb, cuda_device):
    dev = cuda_device
    W, M, N, P = 12, 4, 3, 5000
    group = (np.arange(W) // 3).astype(np.int32)
    grad = torch.ones((W, P), device=dev)
    theta = torch.zeros(P, device=dev)
    arrival = to_dev(np.arange(1, W + 1, dtype=np.float32), dev)
    tags = torch.zeros(W, dtype=torch.int32, device=dev)
    mask, gorder, order, info = _buffers(W, N, dev)
    opt = gpu_opt(OPTS["sgd"])
    # two machines have a stale worker: only two messages count
    stale = tags.clone()
    stale[0] = stale[4] = -1
    sgdb.sgdb_step_grouped(grad, P, arrival, stale, to_dev(group, dev), 0, M, N, theta, None, None, opt, mask, gorder, order, info)
    assert info.cpu().tolist() == [2, sgdb.SGDB_ERR_INSUFFICIENT, 0]
    assert (theta == 0).all() and (mask == 255).all() and (gorder == -7).all() and (order == -7).all()
    # a machine id out of range is reported by the device, nothing is touched
    bad = group.copy()
    bad[5] = M
    sgdb.sgdb_step_grouped(grad, P, arrival, tags, to_dev(bad, dev), 0, M, N, theta, None, None, opt, mask, gorder, order, info)
    assert info.cpu().tolist() == [0, sgdb.SGDB_ERR_INVALID_ARG, 0] and (theta == 0).all() and (mask == 255).all()
    # host-checkable arguments
    for kw in (dict(M=0), dict(N=M + 1), dict(N=0)):
        with pytest.raises(sgdb.SgdbError) as e:
            sgdb.sgdb_step_grouped(grad, P, arrival, tags, to_dev(group, dev), 0, kw.get("M", M), kw.get("N", N), theta, None,
                                   None, opt, mask, gorder, order, info)
        assert e.value.status == sgdb.SGDB_ERR_INVALID_ARG
    # P = 0 is a selection only; and a good call does move theta: 3 machines of constant-1 rows -> mean 1
    sgdb.sgdb_step_grouped(grad, 0, arrival, tags, to_dev(group, dev), 0, M, N, theta, None, None, opt, mask, gorder, order, info)
    assert info.cpu().tolist() == [4, 0, 9] and gorder.cpu().tolist() == [0, 1, 2]
    sgdb.sgdb_step_grouped(grad, P, arrival, tags, to_dev(group, dev), 0, M, N, theta, None, None, opt, mask, gorder, order, info)
    assert torch.equal(theta, torch.full((P,), -0.1, device=dev))


def test_grouped_step_mid_size_many_machines(sgdb, cuda_device):
    """The 100-worker split on 25 machines of 4 at a size of several waves of tiles, sampled columns against the oracle."""
    dev = cuda_device
    W, M, N, P, seed, kind = 100, 25, 24, 3_000_017, 181, "rmsprop"
    group = (np.arange(W) // 4).astype(np.int32)
    grad = wl.grad_matrix(seed, 0, W, P, wl.worker_scales(seed, W), "f32", dev)
    arrival, tags = wl.arrivals(seed, 0, W), np.zeros(W, np.int32)
    theta = wl.theta0(seed, P, dev)
    s0, s1 = gpu_state(kind, P, dev)
    cols = np.unique(np.concatenate([np.arange(16), np.arange(P - 16, P), np.random.default_rng(seed).integers(0, P, 2000)]))
    cols_d = to_dev(cols, dev)
    th_o = theta[cols_d].cpu().numpy().astype(np.float64)
    s0_o, s1_o = oracle_state(kind, len(cols))
    mask, gorder, order, info = _buffers(W, N, dev)
    sgdb.sgdb_step_grouped(grad, P, to_dev(arrival, dev), to_dev(tags, dev), to_dev(group, dev), 0, M, N, theta, s0, s1,
                           gpu_opt(OPTS[kind]), mask, gorder, order, info)
    rc, mask_o, gorder_o, order_o, n_valid = oracle.step_grouped(wl.as_oracle_array(grad.index_select(1, cols_d)), len(cols),
                                                                 arrival, tags, group, 0, M, N, th_o, s0_o, s1_o,
                                                                 oracle_opt(OPTS[kind]))
    assert rc == oracle.OK and info.cpu().tolist() == [n_valid, 0, 96]
    assert gorder.cpu().numpy().tolist() == gorder_o.tolist() and order.cpu().numpy()[:96].tolist() == order_o.tolist()
    assert rel_err(theta[cols_d].cpu().numpy(), th_o) < TOL_F32 and rel_err(s0[cols_d].cpu().numpy(), s0_o) < TOL_F32
    assert bool(torch.isfinite(theta).all())


@pytest.mark.parametrize("W,M,N", [(1024, 256, 200), (1000, 1000, 999), (37, 37, 37)])
def test_grouped_step_at_the_largest_counts(sgdb, cuda_device, W, M, N):
    """As many workers and machines as the library accepts (and every machine kept): selection words bit-exact,
    parameters within tolerance."""
    dev = cuda_device
    P, seed = 6000, 191
    rng = np.random.default_rng(seed + W)
    group = rng.permutation(np.arange(W) % M).astype(np.int32)
    grad = wl.grad_matrix(seed, 0, W, P, wl.worker_scales(seed, W), "f32", dev)
    arrival = wl.arrivals(seed, 0, W)
    arrival[: W // 8] = arrival[W // 8: 2 * (W // 8)]  # plenty of equal times
    tags = np.zeros(W, np.int32)
    theta = wl.theta0(seed, P, dev)
    th_o = theta.cpu().numpy().astype(np.float64)
    mask, gorder, order, info = _buffers(W, N, dev)
    sgdb.sgdb_step_grouped(grad, P, to_dev(arrival, dev), to_dev(tags, dev), to_dev(group, dev), 0, M, N, theta, None, None,
                           gpu_opt(OPTS["sgd"]), mask, gorder, order, info)
    rc, mask_o, gorder_o, order_o, n_valid = oracle.step_grouped(wl.as_oracle_array(grad), P, arrival, tags, group, 0, M, N,
                                                                 th_o, None, None, oracle_opt(OPTS["sgd"]))
    assert rc == oracle.OK and info.cpu().tolist() == [n_valid, 0, len(order_o)]
    assert mask.cpu().numpy().tolist() == mask_o.tolist() and gorder.cpu().numpy().tolist() == gorder_o.tolist()
    assert order.cpu().numpy()[: len(order_o)].tolist() == order_o.tolist()
    assert rel_err(theta.cpu().numpy(), th_o) < TOL_F32

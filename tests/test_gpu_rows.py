"""The step as one of several parameter servers runs it (Section 1.1: server j holds theta[j]): rows given by
address, a range of columns per server, the new parameters pushed to every replica.  One GPU stands in for
all of them here: the servers' launches run one after another on rows that all live in this GPU's memory
(no launch waits for another), which is enough to check every address, range and bit."""
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


def _esize(dtype):
    return 4 if dtype == "f32" else 2


def _scatter_rows(grad, P, shift_elems=0):
    """Every row of the matrix in a buffer of its own (what a server sees when each worker's gradient was received
    into separate memory); shift_elems moves each copy off the 16-byte grid."""
    bufs, addrs = [], []
    for w in range(grad.shape[0]):
        buf = torch.empty(P + 16, dtype=grad.dtype, device=grad.device)
        buf[shift_elems:shift_elems + P] = grad[w, :P]
        bufs.append(buf)
        addrs.append(buf.data_ptr() + shift_elems * grad.element_size())
    return bufs, addrs


@pytest.mark.parametrize("kind,dtype,P,shift", [("rmsprop", "f32", 70_001, 0), ("adam", "bf16", 100_003, 0),
                                                ("sgd", "f32", 4099, 1), ("momentum", "bf16", 8192, 3),
                                                ("adagrad", "f32", 33_333, 0), ("sgd", "bf16", 5, 0),
                                                ("rmsprop", "f32", 2048 * 3, 0)])
def test_rows_by_address_have_the_bits_of_the_matrix_step(sgdb, cuda_device, kind, dtype, P, shift):
    """One server owning every column, no replicas: the same selection words and the same bits as sgdb_step on the
    packed matrix, for rows on and off the 16-byte grid.  Dropped workers have no address at all."""
    dev = cuda_device
    W, N, T, seed = 19, 15, 3, 211
    scales = wl.worker_scales(seed, W)
    theta = wl.theta0(seed, P, dev)
    theta_m = theta.clone()
    s, sm = gpu_state(kind, P, dev), gpu_state(kind, P, dev)
    mask, order, info = selection_buffers(W, N, dev)
    mask_m, order_m, info_m = selection_buffers(W, N, dev)
    for t in range(T):
        grad = wl.grad_matrix(seed, t, W, P, scales, dtype, dev)
        arrival, tags = wl.arrivals(seed, t, W), wl.tags(seed, t, W, N)
        a_d, t_d = to_dev(arrival, dev), to_dev(tags, dev)
        sgdb.sgdb_step(grad, P, a_d, t_d, t, N, W - N, theta_m, sm[0], sm[1], gpu_opt(OPTS[kind], t + 1), mask_m, order_m,
                       info_m)
        bufs, addrs = _scatter_rows(grad, P, shift)
        for w in np.flatnonzero(mask_m.cpu().numpy() == 0):
            addrs[w] = 0
        rows = sgdb.make_address_table(addrs, dev)
        sgdb.sgdb_step_rows(rows, grad.dtype, P, a_d, t_d, t, N, W - N, theta, s[0], s[1], gpu_opt(OPTS[kind], t + 1), None,
                            mask, order, info)
        assert info.cpu().tolist() == info_m.cpu().tolist() and info.cpu().tolist()[1] == 0
        assert torch.equal(mask, mask_m) and torch.equal(order, order_m)
        assert torch.equal(theta, theta_m)
        for x, y in zip(s, sm):
            assert x is None or torch.equal(x, y)


@pytest.mark.parametrize("G,kind,dtype,P", [(2, "rmsprop", "f32", 300_007), (3, "adam", "bf16", 200_001), (8, "sgd", "f32", 1000),
                                            (8, "momentum", "f32", 123_457), (4, "adagrad", "bf16", 64 * 4)])
def test_servers_over_column_ranges_fill_every_replica(sgdb, cuda_device, G, kind, dtype, P):
    """G servers, each holding a full copy of theta for its workers and the state of its own range; the workers'
    rows are spread over the G memories.  After every server's launch each copy holds the parameters sgdb_step
    computes on one GPU, bit for bit, and the oracle agrees within tolerance."""
    dev = cuda_device
    W, N, T, seed = 22, 18, 3, 223
    es = _esize(dtype)
    scales = wl.worker_scales(seed, W)
    theta_1 = wl.theta0(seed, P, dev)
    copies = [theta_1.clone() for _ in range(G)]
    s1 = gpu_state(kind, P, dev)
    ranges = [sgdb.sgdb_shard_range(P, G, j) for j in range(G)]
    assert ranges[0][0] == 0 and sum(n for _, n in ranges) == P
    assert all(ranges[j][0] + ranges[j][1] == ranges[j + 1][0] for j in range(G - 1))
    states = [gpu_state(kind, max(n, 1), dev) for _, n in ranges]
    th_o = theta_1.cpu().numpy().astype(np.float64)
    s0_o, s1_o = oracle_state(kind, P)
    mask_1, order_1, info_1 = selection_buffers(W, N, dev)
    for t in range(T):
        grad = wl.grad_matrix(seed, t, W, P, scales, dtype, dev)
        arrival, tags = wl.arrivals(seed, t, W), wl.tags(seed, t, W, N)
        a_d, t_d = to_dev(arrival, dev), to_dev(tags, dev)
        sgdb.sgdb_step(grad, P, a_d, t_d, t, N, W - N, theta_1, s1[0], s1[1], gpu_opt(OPTS[kind], t + 1), mask_1, order_1,
                       info_1)
        rc, *_ = oracle.step(wl.as_oracle_array(grad), P, arrival, tags, t, N, W - N, th_o, s0_o, s1_o,
                             oracle_opt(OPTS[kind], t + 1))
        assert rc == oracle.OK
        # worker w's row lives in memory w % G: one buffer per memory, rows of full length on a 16-byte pitch
        ld = (P + 7) // 8 * 8
        held = []
        for g in range(G):
            part = grad[g::G]
            buf = torch.full((part.shape[0], ld), float("nan"), dtype=grad.dtype, device=dev)
            buf[:, :P] = part
            held.append(buf)
        for j, (first, n) in enumerate(ranges):
            rows = sgdb.make_address_table([held[w % G][w // G].data_ptr() + first * es for w in range(W)], dev)
            others = [copies[g].data_ptr() + first * 4 for g in range(G) if g != j]
            mask, order, info = selection_buffers(W, N, dev)
            sgdb.sgdb_step_rows(rows, grad.dtype, n, a_d, t_d, t, N, W - N, copies[j][first:first + n] if n else copies[j][:1],
                                states[j][0], states[j][1], gpu_opt(OPTS[kind], t + 1),
                                sgdb.make_address_table(others, dev), mask, order, info)
            assert info.cpu().tolist() == info_1.cpu().tolist()
            assert torch.equal(mask, mask_1) and torch.equal(order, order_1)
        for g in range(G):
            assert torch.equal(copies[g], theta_1), (t, g)
    for k in range(2):
        if s1[k] is not None:
            joined = torch.cat([states[j][k][:n] for j, (_, n) in enumerate(ranges)])
            assert torch.equal(joined, s1[k])
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    assert rel_err(copies[-1].cpu().numpy(), th_o) < tol
    if s0_o is not None:
        assert rel_err(s1[0].cpu().numpy(), s0_o) < tol


@pytest.mark.parametrize("dtype,kind", [("f32", "rmsprop"), ("bf16", "adam")])
def test_two_level_across_machines_has_the_bits_of_the_grouped_step(sgdb, cuda_device, dtype, kind):
    """Machines first combine their own workers' rows (sgdb_select over the machine's workers, sgdb_aggregate),
    then G servers take the kept machines' messages as rows, in the order sgdb_select_grouped gives: the bits of
    the one-launch sgdb_step_grouped.  A machine with a stale worker sends nothing and its buffer is never read."""
    dev = cuda_device
    W, M, N, P, G, seed = 23, 6, 4, 150_001, 3, 227
    group = (np.arange(W) * M // W).astype(np.int32)  # workers of a machine are neighbours: local order = global order
    ldg = (P + 7) // 8 * 8  # every row of the matrix starts on a 16-byte boundary
    grad = wl.grad_matrix(seed, 0, W, P, wl.worker_scales(seed, W), dtype, dev, ld=ldg, pad_value=float("nan"))
    arrival = wl.arrivals(seed, 0, W)
    tags = np.zeros(W, np.int32)
    tags[np.flatnonzero(group == 2)[0]] = -1
    a_d, t_d, g_d = to_dev(arrival, dev), to_dev(tags, dev), to_dev(group, dev)
    theta_1 = wl.theta0(seed, P, dev)
    copies = [theta_1.clone() for _ in range(G)]
    s1 = gpu_state(kind, P, dev)
    mask_1 = torch.full((W,), 255, dtype=torch.uint8, device=dev)
    gorder_1 = torch.full((N,), -7, dtype=torch.int32, device=dev)
    order_1 = torch.full((W,), -7, dtype=torch.int32, device=dev)
    info_1 = torch.full((3,), -7, dtype=torch.int32, device=dev)
    sgdb.sgdb_step_grouped(grad, P, a_d, t_d, g_d, 0, M, N, theta_1, s1[0], s1[1], gpu_opt(OPTS[kind]), mask_1, gorder_1,
                           order_1, info_1, ld=ldg)
    assert info_1.cpu().tolist()[:2] == [M - 1, 0]
    # stage 1, on every machine: the mean of its workers' rows, if all of them are current
    ld = (P + 3) // 4 * 4
    sent = torch.full((M, ld), float("nan"), device=dev)
    for m in range(M):
        ids = np.flatnonzero(group == m)
        mk, od, inf = selection_buffers(len(ids), len(ids), dev)
        sgdb.sgdb_select(a_d[ids[0]:ids[-1] + 1], t_d[ids[0]:ids[-1] + 1], 0, len(ids), 0, mk, od, inf)
        sgdb.sgdb_aggregate(grad[ids[0]:ids[-1] + 1], P, len(ids), od, inf, sent[m, :P], ld=ldg)
    assert bool(torch.isnan(sent[2]).all())
    # stage 2, on every server: the selection over machines, then the kept messages as rows
    ranges = [sgdb.sgdb_shard_range(P, G, j) for j in range(G)]
    states = [gpu_state(kind, n, dev) for _, n in ranges]
    for j, (first, n) in enumerate(ranges):
        mask = torch.full((W,), 255, dtype=torch.uint8, device=dev)
        gorder = torch.full((N,), -7, dtype=torch.int32, device=dev)
        order = torch.full((W,), -7, dtype=torch.int32, device=dev)
        info = torch.full((3,), -7, dtype=torch.int32, device=dev)
        sgdb.sgdb_select_grouped(a_d, t_d, g_d, 0, M, N, mask, gorder, order, info)
        rows = sgdb.make_address_table([sent[m].data_ptr() + first * 4 for m in range(M)], dev)
        others = sgdb.make_address_table([copies[g].data_ptr() + first * 4 for g in range(G) if g != j], dev)
        sgdb.sgdb_step_rows_ordered(rows, torch.float32, n, N, gorder, info, copies[j][first:first + n], states[j][0],
                                    states[j][1], gpu_opt(OPTS[kind]), others)
        assert info.cpu().tolist() == info_1.cpu().tolist() and torch.equal(gorder, gorder_1)
    for g in range(G):
        assert torch.equal(copies[g], theta_1)
    for k in range(2):
        assert torch.equal(torch.cat([states[j][k] for j in range(G)]), s1[k])


def test_rows_refusals_leave_everything_untouched(sgdb, cuda_device):
    dev = cuda_device
    W, N, P = 6, 4, 5000
    grad = torch.ones((W, P), device=dev)
    addrs = [grad[w].data_ptr() for w in range(W)]
    theta = torch.zeros(P, device=dev)
    copy = torch.zeros(P, device=dev)
    arrival = to_dev(np.arange(1, W + 1, dtype=np.float32), dev)
    tags = torch.zeros(W, dtype=torch.int32, device=dev)
    opt = gpu_opt(OPTS["sgd"])
    reps = sgdb.make_address_table([copy.data_ptr()], dev)
    mask, order, info = selection_buffers(W, N, dev)

    def run(rows_list, replicas=reps, tags_d=tags):
        sgdb.sgdb_step_rows(sgdb.make_address_table(rows_list, dev), torch.float32, P, arrival, tags_d, 0, N, W - N, theta, None,
                            None, opt, replicas, mask, order, info)
        return info.cpu().tolist()

    # a kept worker without an address, or with one that is not a multiple of the element size: reported by the
    # device, nothing touched (the selection words are the selection's business and are written)
    for bad in (0, addrs[1] + 2):
        assert run([addrs[0], bad] + addrs[2:]) == [W, sgdb.SGDB_ERR_INVALID_ARG]
        assert (theta == 0).all() and (copy == 0).all()
    # a replica without an address
    assert run(addrs, sgdb.make_address_table([copy.data_ptr(), 0], dev)) == [W, sgdb.SGDB_ERR_INVALID_ARG]
    assert (theta == 0).all() and (copy == 0).all()
    # the two slowest workers are dropped: they need no address
    assert run(addrs[:N] + [0, 0]) == [W, 0]
    assert torch.equal(theta, torch.full((P,), -0.1, device=dev)) and torch.equal(copy, theta)
    # too few current gradients: nothing moves
    theta.zero_(), copy.zero_()
    stale = tags.clone()
    stale[:3] = -1
    assert run(addrs, tags_d=stale) == [3, sgdb.SGDB_ERR_INSUFFICIENT]
    assert (theta == 0).all() and (copy == 0).all()
    # given selection: a row id outside [0, W) is reported, a status that is already bad means "do nothing"
    rows = sgdb.make_address_table(addrs, dev)
    for ids, word, expect in (([0, 1, 2, W], 0, sgdb.SGDB_ERR_INVALID_ARG), ([0, 1, 2, -1], 0, sgdb.SGDB_ERR_INVALID_ARG),
                              ([0, 1, 2, 3], sgdb.SGDB_ERR_INSUFFICIENT, sgdb.SGDB_ERR_INSUFFICIENT)):
        inf = to_dev(np.array([N, word], np.int32), dev)
        sgdb.sgdb_step_rows_ordered(rows, torch.float32, P, N, to_dev(np.array(ids, np.int32), dev), inf, theta, None, None,
                                    opt, reps)
        assert inf.cpu().tolist() == [N, expect] and (theta == 0).all() and (copy == 0).all()
    # host-checkable arguments
    many = sgdb.make_address_table([copy.data_ptr()] * (sgdb.SGDB_MAX_REPLICAS + 1), dev)
    for call in (lambda: sgdb.sgdb_step_rows(rows, torch.float32, -1, arrival, tags, 0, N, W - N, theta, None, None, opt, None,
                                             mask, order, info),
                 lambda: sgdb.sgdb_step_rows(rows, torch.float32, P, arrival, tags, 0, 0, W, theta, None, None, opt, None, mask,
                                             order, info),
                 lambda: sgdb.sgdb_step_rows(rows, torch.float32, P, arrival, tags, 0, N, W - N, theta, None, None, opt, many,
                                             mask, order, info),
                 lambda: sgdb.sgdb_step_rows(rows, torch.float32, P, arrival, tags, 0, N, W - N, theta[1:], None, None, opt, None,
                                             mask, order, info),
                 lambda: sgdb.sgdb_step_rows(rows, torch.float32, P, arrival, tags, 0, N, W - N, theta, None, None,
                                             gpu_opt(OPTS["momentum"]), None, mask, order, info),
                 lambda: sgdb.sgdb_step_rows_ordered(rows, torch.float32, P, W + 1, order, info, theta, None, None, opt, None)):
        with pytest.raises(sgdb.SgdbError) as e:
            call()
        assert e.value.status == sgdb.SGDB_ERR_INVALID_ARG
    assert (theta == 0).all()
    # an empty range is a selection only
    mask, order, info = selection_buffers(W, N, dev)
    sgdb.sgdb_step_rows(rows, torch.float32, 0, arrival, tags, 0, N, W - N, theta, None, None, opt, None, mask, order, info)
    assert info.cpu().tolist() == [W, 0] and order.cpu().tolist() == [0, 1, 2, 3]


def test_rows_mid_size_four_servers(sgdb, cuda_device):
    """The 100-worker split over four servers at a size of several waves of tiles per server: the one-GPU step's bits
    in every copy, and sampled columns against the oracle."""
    dev = cuda_device
    W, N, P, G, seed, kind = 100, 96, 3_000_017, 4, 229, "rmsprop"
    grad = wl.grad_matrix(seed, 0, W, P, wl.worker_scales(seed, W), "f32", dev, ld=P + 3, pad_value=float("nan"))
    arrival, tags = wl.arrivals(seed, 0, W), wl.tags(seed, 0, W, N)
    a_d, t_d = to_dev(arrival, dev), to_dev(tags, dev)
    theta_1 = wl.theta0(seed, P, dev)
    cols = np.unique(np.concatenate([np.arange(16), np.arange(P - 16, P), np.random.default_rng(seed).integers(0, P, 2000)]))
    cols_d = to_dev(cols, dev)
    th_o = theta_1[cols_d].cpu().numpy().astype(np.float64)
    s0_o, s1_o = oracle_state(kind, len(cols))
    copies = [theta_1.clone() for _ in range(G)]
    s1 = gpu_state(kind, P, dev)
    mask_1, order_1, info_1 = selection_buffers(W, N, dev)
    sgdb.sgdb_step(grad, P, a_d, t_d, 0, N, W - N, theta_1, s1[0], s1[1], gpu_opt(OPTS[kind]), mask_1, order_1, info_1,
                   ld=P + 3)
    ranges = [sgdb.sgdb_shard_range(P, G, j) for j in range(G)]
    states = [gpu_state(kind, n, dev) for _, n in ranges]
    for j, (first, n) in enumerate(ranges):
        rows = sgdb.make_address_table([grad[w].data_ptr() + first * 4 for w in range(W)], dev)
        others = sgdb.make_address_table([copies[g].data_ptr() + first * 4 for g in range(G) if g != j], dev)
        mask, order, info = selection_buffers(W, N, dev)
        sgdb.sgdb_step_rows(rows, torch.float32, n, a_d, t_d, 0, N, W - N, copies[j][first:first + n], states[j][0], states[j][1],
                            gpu_opt(OPTS[kind]), others, mask, order, info)
        assert info.cpu().tolist() == info_1.cpu().tolist() and torch.equal(order, order_1)
    for g in range(G):
        assert torch.equal(copies[g], theta_1)
    rc, *_ = oracle.step(wl.as_oracle_array(grad.index_select(1, cols_d)), len(cols), arrival, tags, 0, N, W - N, th_o, s0_o,
                         s1_o, oracle_opt(OPTS[kind]))
    assert rc == oracle.OK
    assert rel_err(copies[0][cols_d].cpu().numpy(), th_o) < TOL_F32
    assert torch.equal(torch.cat([states[j][0] for j in range(G)]), s1[0])


def test_peer_access_set_up_call(sgdb, cuda_device):
    """The set-up call for a peer's memory: the current device itself needs nothing, a device that does not exist is
    refused; with a second device present, enabling twice is fine."""
    sgdb.sgdb_enable_peer_access(torch.cuda.current_device())
    for bad in (-1, torch.cuda.device_count()):
        with pytest.raises(sgdb.SgdbError) as e:
            sgdb.sgdb_enable_peer_access(bad)
        assert e.value.status == sgdb.SGDB_ERR_INVALID_ARG
    if torch.cuda.device_count() > 1:
        other = (torch.cuda.current_device() + 1) % torch.cuda.device_count()
        try:
            sgdb.sgdb_enable_peer_access(other)
            sgdb.sgdb_enable_peer_access(other)
        except sgdb.SgdbError as e:
            assert e.status == sgdb.SGDB_ERR_UNSUPPORTED


def test_rows_at_the_largest_counts(sgdb, cuda_device):
    """As many workers and as many copies of theta as the library accepts: W = 1024 rows by address (N = 1000 kept),
    64 replicas; the bits of sgdb_step in theta and in every replica."""
    dev = cuda_device
    W, N, P, R, seed = sgdb.SGDB_MAX_WORKERS, 1000, 6000, sgdb.SGDB_MAX_REPLICAS, 233
    grad = wl.grad_matrix(seed, 0, W, P, wl.worker_scales(seed, W), "f32", dev)
    arrival = wl.arrivals(seed, 0, W)
    arrival[: W // 8] = arrival[W // 8: 2 * (W // 8)]  # plenty of equal times
    tags = np.zeros(W, np.int32)
    tags[np.random.default_rng(seed).choice(W, size=10, replace=False)] = -1  # ten stragglers of the previous iteration
    a_d, t_d = to_dev(arrival, dev), to_dev(tags, dev)
    theta_1 = wl.theta0(seed, P, dev)
    theta = theta_1.clone()
    s1, s = gpu_state("adam", P, dev), gpu_state("adam", P, dev)
    mask_1, order_1, info_1 = selection_buffers(W, N, dev)
    sgdb.sgdb_step(grad, P, a_d, t_d, 0, N, W - N, theta_1, s1[0], s1[1], gpu_opt(OPTS["adam"]), mask_1, order_1, info_1)
    copies = torch.zeros((R, P), device=dev)
    rows = sgdb.make_address_table([grad[w].data_ptr() for w in range(W)], dev)
    push = sgdb.make_address_table([copies[r].data_ptr() for r in range(R)], dev)
    mask, order, info = selection_buffers(W, N, dev)
    sgdb.sgdb_step_rows(rows, torch.float32, P, a_d, t_d, 0, N, W - N, theta, s[0], s[1], gpu_opt(OPTS["adam"]), push, mask,
                        order, info)
    assert info.cpu().tolist() == info_1.cpu().tolist() and info_1.cpu().tolist()[1] == 0
    assert torch.equal(order, order_1) and torch.equal(mask, mask_1)
    assert torch.equal(theta, theta_1) and torch.equal(s[0], s1[0]) and torch.equal(s[1], s1[1])
    assert all(torch.equal(copies[r], theta_1) for r in range(R))

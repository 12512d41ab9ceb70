"""Parity of the multi-tensor step, the arrival-by-arrival mode and the host-buffer step with the oracle."""
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


# ------------------------------------------------------------------ multi-tensor (segment table)


def _make_model(dev, lengths, W, kind, dtype, seed, packed):
    """Tensors of the given lengths.  packed=False: every tensor has its own allocation and a row pitch
    padded to 16 bytes.  packed=True: parameters, state and gradients of all tensors are carved out of
    shared buffers back to back, so most tensors start at an address that is only element-aligned."""
    scales = wl.worker_scales(seed, W)
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    vec = 4 if dtype == "f32" else 8
    segs = []
    total = int(sum(lengths))
    if packed:
        th_all = wl.theta0(seed, total, dev)
        s_all = [torch.zeros(total, device=dev) for _ in range(2)]
        g_all = torch.empty(W * total, dtype=tdt, device=dev)
    off = 0
    for i, L in enumerate(int(x) for x in lengths):
        if packed:
            theta = th_all[off:off + L]
            s0, s1 = s_all[0][off:off + L], s_all[1][off:off + L]
            grad = g_all[W * off:W * (off + L)].view(W, L)
            wl.grad_matrix(seed + i, 0, W, L, scales, dtype, dev, out=grad)
        else:
            theta = wl.theta0(seed + i, L, dev)
            s0, s1 = torch.zeros(L, device=dev), torch.zeros(L, device=dev)
            ld = (L + vec - 1) // vec * vec
            grad = wl.grad_matrix(seed + i, 0, W, L, scales, dtype, dev, ld=ld, pad_value=float("nan"))
        n = {"sgd": 0, "momentum": 1, "rmsprop": 2, "adam": 2, "adagrad": 1}[kind]
        segs.append((theta, s0 if n >= 1 else None, s1 if n >= 2 else None, grad))
        off += L
    return segs, scales


def _regen(segs, scales, seed, t, W, dtype, dev, packed):
    for i, (theta, _, _, grad) in enumerate(segs):
        L = theta.numel()
        if L == 0:
            continue
        if packed:
            wl.grad_matrix(seed + i, t, W, L, scales, dtype, dev, out=grad)
        else:
            wl.grad_matrix(seed + i, t, W, L, scales, dtype, dev, ld=grad.stride(0), out=grad, pad_value=float("nan"))


@pytest.mark.parametrize("packed", [False, True])
@pytest.mark.parametrize("kind,dtype", [("momentum", "f32"), ("adam", "bf16"), ("sgd", "f32"), ("rmsprop", "bf16"),
                                        ("adagrad", "f32")])
def test_segmented_step_matches_oracle_and_per_tensor_launches(sgdb, cuda_device, kind, dtype, packed):
    dev = cuda_device
    W, N, T, seed = 14, 11, 3, 101
    rng = np.random.default_rng(seed)
    # log-uniform lengths like the 300-tensor workload, scaled down; plus the awkward ones
    lengths = np.floor(np.exp(rng.uniform(np.log(1), np.log(30_000), size=60))).astype(np.int64).tolist()
    lengths += [1, 2, 3, 4, 5, 7, 8, 2047, 2048, 2049, 4096, 4097, 0, 6145]
    segs, scales = _make_model(dev, lengths, W, kind, dtype, seed, packed)
    twins = [tuple(None if x is None else x.clone() for x in s[:3]) for s in segs]  # per-tensor launches
    th_o = [s[0].cpu().numpy().astype(np.float64) for s in segs]
    st_o = [oracle_state(kind, len(x)) for x in th_o]
    table = sgdb.make_segment_table(segs, dev)
    mask, order, info = selection_buffers(W, N, dev)
    mask2, order2, info2 = selection_buffers(W, N, dev)
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    for t in range(T):
        if t:
            _regen(segs, scales, seed, t, W, dtype, dev, packed)
        arrival, tags = step_inputs(seed, t, W, N)
        a_d, t_d = to_dev(arrival, dev), to_dev(tags, dev)
        sgdb.sgdb_step_segmented(table, len(segs), tdt, a_d, t_d, t, N, W - N, gpu_opt(OPTS[kind], t + 1),
                                 mask, order, info)
        rc, mask_o, order_o, n_valid = oracle.select(arrival, tags, t, N, W - N)
        assert rc == oracle.OK and info.cpu().tolist() == [n_valid, 0]
        assert order.cpu().numpy().tolist() == order_o.tolist() and mask.cpu().numpy().tolist() == mask_o.tolist()
        for i, (theta, s0, s1, grad) in enumerate(segs):
            L = theta.numel()
            if L == 0:
                continue
            aligned = all(x is None or x.data_ptr() % 16 == 0 for x in (theta, s0, s1, grad))
            if aligned:  # the flat call wants 16-byte aligned bases; compare bit for bit where it applies
                sgdb.sgdb_step(grad, L, a_d, t_d, t, N, W - N, twins[i][0], twins[i][1], twins[i][2],
                               gpu_opt(OPTS[kind], t + 1), mask2, order2, info2, ld=grad.stride(0))
                assert torch.equal(theta, twins[i][0]), (i, L)
            mean = oracle.aggregate(wl.as_oracle_array(grad), L, order_o, ld=grad.stride(0))
            oracle.update(th_o[i], st_o[i][0], st_o[i][1], mean, oracle_opt(OPTS[kind], t + 1))
    for i, (theta, s0, s1, _) in enumerate(segs):
        if theta.numel() == 0:
            continue
        # tiny tensors: compare against the model-wide scale, not the tensor's own rms
        scale = max(1.0, float(np.sqrt(np.mean(th_o[i] ** 2))))
        assert np.max(np.abs(theta.cpu().numpy() - th_o[i])) / scale < tol * 4, (i, theta.numel())
        if theta.numel() >= 64:
            assert rel_err(theta.cpu().numpy(), th_o[i]) < tol, (i, theta.numel())
            if s0 is not None:
                assert rel_err(s0.cpu().numpy(), st_o[i][0]) < tol
            if s1 is not None:
                assert rel_err(s1.cpu().numpy(), st_o[i][1]) < tol


def test_segmented_edge_cases(sgdb, cuda_device):
    dev = cuda_device
    W, N = 4, 3
    mask, order, info = selection_buffers(W, N, dev)
    a_d = to_dev(np.array([1, 2, 3, 4], np.float32), dev)
    t_d = torch.zeros(W, dtype=torch.int32, device=dev)
    # an empty table is a selection only
    empty = torch.empty(0, dtype=torch.uint8, device=dev)
    keep = torch.zeros(48, dtype=torch.uint8, device=dev)
    sgdb.sgdb_step_segmented(keep, 0, torch.float32, a_d, t_d, 0, N, 1, gpu_opt(OPTS["sgd"]), mask, order, info)
    assert info.cpu().tolist() == [4, 0] and order.cpu().tolist() == [0, 1, 2]
    del empty
    with pytest.raises(sgdb.SgdbError) as e:
        sgdb.sgdb_step_segmented(keep, sgdb.SGDB_MAX_SEGMENTS + 1, torch.float32, a_d, t_d, 0, N, 1,
                                 gpu_opt(OPTS["sgd"]), mask, order, info)
    assert e.value.status == sgdb.SGDB_ERR_UNSUPPORTED
    # a segment without the state its rule needs is skipped and reported, never dereferenced
    th = [torch.zeros(5000, device=dev) for _ in range(3)]
    vel = [torch.zeros(5000, device=dev), None, torch.zeros(5000, device=dev)]
    gr = [torch.ones((W, 5000), device=dev) for _ in range(3)]
    table = sgdb.make_segment_table([(th[i], vel[i], None, gr[i]) for i in range(3)], dev)
    sgdb.sgdb_step_segmented(table, 3, torch.float32, a_d, t_d, 0, N, 1, gpu_opt(dict(kind="momentum", lr=1.0, momentum=0.5)),
                             mask, order, info)
    assert info.cpu().tolist() == [4, sgdb.SGDB_ERR_INVALID_ARG]
    assert (th[0] == -1).all() and (th[1] == 0).all() and (th[2] == -1).all()
    # entries the kernel must not touch: a pointer that is not aligned to its element, rows that overlap (ld < len)
    raw = torch.zeros(4 * 5000 + 16, dtype=torch.uint8, device=dev)
    # (torch refuses misaligned views, so the entries are built by hand)
    good = [torch.zeros(5000, device=dev) for _ in range(3)]
    entries = (sgdb.CSegment * 3)()
    entries[0] = sgdb.CSegment(good[0].data_ptr(), 0, 0, gr[0].data_ptr(), 5000, 5000)
    entries[1] = sgdb.CSegment(raw.data_ptr() + 2, 0, 0, gr[1].data_ptr(), 5000, 5000)          # theta at a 2-byte offset
    entries[2] = sgdb.CSegment(good[2].data_ptr(), 0, 0, gr[2].data_ptr(), 4999, 5000)          # ld < len
    table = torch.frombuffer(bytearray(bytes(entries)), dtype=torch.uint8).to(dev)
    sgdb.sgdb_step_segmented(table, 3, torch.float32, a_d, t_d, 0, N, 1, gpu_opt(dict(kind="sgd", lr=1.0)), mask, order, info)
    assert info.cpu().tolist() == [4, sgdb.SGDB_ERR_INVALID_ARG]
    assert (good[0] == -1).all() and (raw == 0).all() and (good[2] == 0).all()
    # the largest table, every tensor tiny
    S = sgdb.SGDB_MAX_SEGMENTS
    theta = torch.zeros(S * 3, device=dev)
    grad = torch.ones((S, W, 3), device=dev)
    segs = [(theta[3 * i:3 * i + 3], None, None, grad[i]) for i in range(S)]
    table = sgdb.make_segment_table(segs, dev)
    sgdb.sgdb_step_segmented(table, S, torch.float32, a_d, t_d, 0, N, 1, gpu_opt(dict(kind="sgd", lr=0.5)),
                             mask, order, info)
    assert info.cpu().tolist() == [4, 0]
    assert (theta == -0.5).all()


# ------------------------------------------------------------------ arrival by arrival


@pytest.mark.parametrize("kind,dtype,P,b", [("rmsprop", "f32", 100_003, 0), ("rmsprop", "f32", 100_003, 2),
                                            ("rmsprop", "f32", 65_536, 4), ("rmsprop", "f32", 100_003, 8),
                                            ("adam", "bf16", 50_001, 3), ("sgd", "f32", 5, 1),
                                            ("momentum", "bf16", 4099, 2), ("adagrad", "f32", 30_001, 2)])
def test_accumulate_on_arrival(sgdb, cuda_device, kind, dtype, P, b):
    """Rows are delivered one per call in arrival sequence, stale rows and late rows included.  Outcomes
    and counts match the oracle's replay of Algorithm 4; parameters match the oracle within tolerance
    and the fused step bit for bit."""
    dev = cuda_device
    N, T, seed = 12, 3, 111 + b
    W = N + b
    scales = wl.worker_scales(seed, W)
    theta = wl.theta0(seed, P, dev)
    theta_f = theta.clone()
    s0, s1 = gpu_state(kind, P, dev)
    sf = gpu_state(kind, P, dev)
    acc = torch.full((P,), float("nan"), device=dev)  # needs no clearing by the caller
    counter = torch.zeros(4, dtype=torch.int32, device=dev)
    info = torch.zeros(2, dtype=torch.int32, device=dev)
    th_o = theta.cpu().numpy().astype(np.float64)
    s0_o, s1_o = oracle_state(kind, P)
    acc_o, state_o = np.zeros(P), oracle.new_server_state()
    mask, order, finfo = selection_buffers(W, N, dev)
    seen = 0
    late = None
    for t in range(T):
        grad = wl.grad_matrix(seed, t, W, P, scales, dtype, dev)
        grad_h = wl.as_oracle_array(grad)
        arrival, tags = step_inputs(seed, t, W, N + 0)
        stale = int(np.argsort(arrival, kind="stable")[1])
        if b >= 2 and int((tags == t).sum()) - int(tags[stale] == t) >= N:
            tags[stale] = t - 1  # an early arrival that is stale
        opt, opt_o = gpu_opt(OPTS[kind], t + 1), oracle_opt(OPTS[kind], t + 1)
        deliveries = [(grad[w], grad_h[w], int(tags[w])) for w in wl.delivery_sequence(arrival)]
        if late is not None:
            deliveries.insert(1, late)  # a straggler of the previous iteration turns up now
        outcomes = []
        for row, row_h, tag in deliveries:
            sgdb.sgdb_accumulate_arrival(row, tag, t, N, acc, counter, theta, s0, s1, opt, info)
            want = oracle.accumulate_arrival(row_h, tag, t, N, acc_o, state_o, th_o, s0_o, s1_o, opt_o)
            seen += 1
            got = info.cpu().tolist()
            assert got[0] == want
            c = counter.cpu().tolist()
            assert c[0] == state_o[0] and c[1] == seen == state_o[1] and c[2] == 0 and c[3] == state_o[2]
            assert got[1] == (N if want == 2 else state_o[0])
            outcomes.append(want)
        assert outcomes.count(2) == 1 and outcomes.count(1) == N - 1
        assert all(o == 0 for o in outcomes[outcomes.index(2) + 1:])  # the slowest are dropped when they arrive
        sgdb.sgdb_step(grad, P, to_dev(arrival, dev), to_dev(tags, dev), t, N, b, theta_f, sf[0], sf[1], opt,
                       mask, order, finfo)
        assert torch.equal(theta, theta_f)
        late = (grad[int(order[-1])].clone(), grad_h[int(order[-1])].copy(), t)
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    assert rel_err(theta.cpu().numpy(), th_o) < tol
    for x, y in ((s0, s0_o), (s1, s1_o)):
        assert x is None or rel_err(x.cpu().numpy(), y) < tol
    for x, y in zip((s0, s1), sf):
        assert x is None or torch.equal(x, y)


@pytest.mark.parametrize("side_stream", [False, True])
@pytest.mark.parametrize("kind,dtype,P", [("rmsprop", "f32", 3_000_001), ("adam", "bf16", 5_000_008)])
def test_arrivals_enqueued_back_to_back_without_host_reads(sgdb, cuda_device, kind, dtype, P, side_stream):
    """Whole iterations are enqueued call after call with nothing read back in between, so consecutive launches
    really follow each other on the device (each launch may be set up while its predecessor still runs; its
    grid is larger than one wave).  Stale rows, rows arriving after the update and a straggler of the previous
    iteration are in the sequence.  At the end: parameters, state and the parameter average equal the fused
    step's bit for bit, and the server counters equal the oracle's replay of the same sequence."""
    dev = cuda_device
    N, b, T, seed, alpha = 10, 3, 3, 141, 0.99
    W = N + b
    scales = wl.worker_scales(seed, W)
    theta = wl.theta0(seed, P, dev)
    theta_f, avg, avg_f = theta.clone(), theta.clone(), theta.clone()
    s0, s1 = gpu_state(kind, P, dev)
    sf = gpu_state(kind, P, dev)
    acc = torch.full((P,), float("nan"), device=dev)
    counter = torch.zeros(4, dtype=torch.int32, device=dev)
    info = torch.zeros(2, dtype=torch.int32, device=dev)
    cols = np.unique(np.concatenate([np.arange(8), np.arange(P - 8, P), np.random.default_rng(seed).integers(0, P, 500)]))
    cols_d = to_dev(cols, dev)
    th_o = theta[cols_d].cpu().numpy().astype(np.float64)
    avg_o = th_o.copy()
    s0_o, s1_o = oracle_state(kind, len(cols))
    acc_o, state_o = np.zeros(len(cols)), oracle.new_server_state()
    stream = torch.cuda.Stream() if side_stream else torch.cuda.current_stream()
    grads, plans = [], []
    for t in range(T):  # all inputs first: nothing below this loop touches the host between launches
        grad = wl.grad_matrix(seed, t, W, P, scales, dtype, dev)
        arrival, tags = step_inputs(seed, t, W, N)
        seq = wl.delivery_sequence(arrival)
        if int((tags == t).sum()) - int(tags[seq[1]] == t) >= N:
            tags[seq[1]] = t - 1  # an early arrival that is stale
        grads.append(grad)
        plans.append((arrival, tags, [int(w) for w in seq]))
    torch.cuda.synchronize()
    seen, last_outcome = 0, None
    with torch.cuda.stream(stream):
        for t in range(T):
            arrival, tags, seq = plans[t]
            opt = gpu_opt(OPTS[kind], t + 1)
            deliveries = [(grads[t][w], int(tags[w])) for w in seq]
            if t > 0:  # the gradient the previous iteration dropped last turns up now, tagged t - 1
                deliveries.insert(2, (grads[t - 1][plans[t - 1][2][-1]], t - 1))
            for row, tag in deliveries:
                sgdb.sgdb_accumulate_arrival_ema(row, tag, t, N, acc, counter, theta, s0, s1, opt, avg, alpha, info)
                seen += 1
    stream.synchronize()
    # the oracle's replay of the same sequence (on sampled columns: the bookkeeping does not depend on the data)
    for t in range(T):
        arrival, tags, seq = plans[t]
        sample = wl.as_oracle_array(grads[t].index_select(1, cols_d))
        deliveries = [(sample[w], int(tags[w])) for w in seq]
        if t > 0:
            prev = wl.as_oracle_array(grads[t - 1].index_select(1, cols_d))
            deliveries.insert(2, (prev[plans[t - 1][2][-1]], t - 1))
        outcomes = []
        for row, tag in deliveries:
            last_outcome = oracle.accumulate_arrival_ema(row, tag, t, N, acc_o, state_o, th_o, s0_o, s1_o,
                                                         oracle_opt(OPTS[kind], t + 1), avg_o, alpha)
            outcomes.append(last_outcome)
        assert outcomes.count(2) == 1 and outcomes.count(1) == N - 1
    assert counter.cpu().tolist() == [int(state_o[0]), seen, 0, int(state_o[2])] == [0, seen, 0, T]
    assert info.cpu().tolist() == [last_outcome, int(state_o[0])]
    # the fused step on the same inputs
    mask, order, finfo = selection_buffers(W, N, dev)
    for t in range(T):
        arrival, tags, _ = plans[t]
        sgdb.sgdb_step_ema(grads[t], P, to_dev(arrival, dev), to_dev(tags, dev), t, N, b, theta_f, sf[0], sf[1],
                           gpu_opt(OPTS[kind], t + 1), avg_f, alpha, mask, order, finfo)
        assert finfo.cpu().tolist()[1] == 0
    assert torch.equal(theta, theta_f) and torch.equal(avg, avg_f)
    for x, y in zip((s0, s1), sf):
        assert x is None or torch.equal(x, y)
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    assert rel_err(theta[cols_d].cpu().numpy(), th_o) < tol and rel_err(avg[cols_d].cpu().numpy(), avg_o) < tol


def test_arriving_row_must_be_element_aligned(sgdb, cuda_device):
    """A row address that is not a multiple of the element size is refused on the host; nothing is launched."""
    import ctypes

    dev = cuda_device
    P = 1000
    raw = torch.zeros(4 * P + 16, dtype=torch.uint8, device=dev)
    acc, theta = torch.zeros(P, device=dev), torch.zeros(P, device=dev)
    counter = torch.zeros(4, dtype=torch.int32, device=dev)
    info = torch.zeros(2, dtype=torch.int32, device=dev)
    c = gpu_opt(OPTS["sgd"])._c()
    for dt, offset, want in ((sgdb.SGDB_F32, 2, sgdb.SGDB_ERR_INVALID_ARG), (sgdb.SGDB_BF16, 1, sgdb.SGDB_ERR_INVALID_ARG),
                             (sgdb.SGDB_F32, 4, sgdb.SGDB_OK), (sgdb.SGDB_BF16, 2, sgdb.SGDB_OK)):
        st = sgdb._lib.sgdb_accumulate_arrival(raw.data_ptr() + offset, dt, 0, 0, 4, P, acc.data_ptr(), counter.data_ptr(),
                                               theta.data_ptr(), 0, 0, ctypes.byref(c), info.data_ptr(), 0)
        assert st == want
    torch.cuda.synchronize()
    assert counter.cpu().tolist()[1] == 2  # only the two aligned rows were seen


@pytest.mark.parametrize("kind,dtype", [("sgd", "f32"), ("rmsprop", "bf16")])
def test_asynchronous_server_is_arrival_mode_with_n_equal_one(sgdb, cuda_device, kind, dtype):
    """Algorithm 2 (the asynchronous parameter server) applies each gradient as it arrives.  That is the
    arrival-by-arrival call with N = 1; gradients come from a delay queue, i.e. each was "computed" several
    updates ago (simulated staleness), which changes nothing in what the server computes."""
    dev = cuda_device
    P, K, seed = 60_001, 12, 181
    scales = wl.worker_scales(seed, K)
    rows = wl.grad_matrix(seed, 0, K, P, scales, dtype, dev)
    rows_h = wl.as_oracle_array(rows)
    theta = wl.theta0(seed, P, dev)
    s0, s1 = gpu_state(kind, P, dev)
    th_o = theta.cpu().numpy().astype(np.float64)
    s0_o, s1_o = oracle_state(kind, P)
    acc = torch.empty(P, device=dev)
    counter = torch.zeros(4, dtype=torch.int32, device=dev)
    info = torch.zeros(2, dtype=torch.int32, device=dev)
    queue = list(np.random.default_rng(seed).permutation(K))  # the order in which stale gradients surface
    for step, w in enumerate(queue):
        sgdb.sgdb_accumulate_arrival(rows[w], step, step, 1, acc, counter, theta, s0, s1, gpu_opt(OPTS[kind], step + 1), info)
        assert info.cpu().tolist() == [2, 1]
        mean = oracle.aggregate(rows_h, P, np.array([w], np.int32))  # the gradient itself
        oracle.update(th_o, s0_o, s1_o, mean, oracle_opt(OPTS[kind], step + 1))
    assert counter.cpu().tolist() == [0, K, 0, K]
    assert rel_err(theta.cpu().numpy(), th_o) < (TOL_F32 if dtype == "f32" else TOL_BF16)


def test_two_level_aggregation_by_composition(sgdb, cuda_device):
    """The paper's conclusion mentions combining the gradients of workers that share a machine before they
    are sent.  With equal groups that is sgdb_aggregate per machine (its mean is what the machine sends,
    when its slowest worker is done) followed by the server step over machines; the result is the mean over
    all workers of the kept machines."""
    dev = cuda_device
    machines, per, keep, P, seed = 6, 4, 5, 50_001, 201
    W = machines * per
    grad = wl.grad_matrix(seed, 0, W, P, wl.worker_scales(seed, W), "f32", dev)
    arrival_w = wl.arrivals(seed, 0, W)
    arrival_m = arrival_w.reshape(machines, per).max(axis=1)
    tags_m = np.zeros(machines, np.int32)
    ld = (P + 3) // 4 * 4  # machine rows start on 16-byte boundaries
    sent = torch.zeros((machines, ld), device=dev)
    ok = to_dev(np.array([per, 0], np.int32), dev)
    for m in range(machines):
        ids = to_dev(np.arange(m * per, (m + 1) * per, dtype=np.int32), dev)
        sgdb.sgdb_aggregate(grad, P, per, ids, ok, sent[m, :P])
    theta = wl.theta0(seed, P, dev)
    th_o = theta.cpu().numpy().astype(np.float64)
    mask, order, info = selection_buffers(machines, keep, dev)
    sgdb.sgdb_step(sent, P, to_dev(arrival_m, dev), to_dev(tags_m, dev), 0, keep, machines - keep, theta, None, None,
                   gpu_opt(OPTS["sgd"]), mask, order, info, ld=ld)
    rc, mask_o, order_o, _ = oracle.select(arrival_m, tags_m, 0, keep, machines - keep)
    assert rc == oracle.OK and order.cpu().numpy().tolist() == order_o.tolist()
    workers = np.concatenate([np.arange(m * per, (m + 1) * per) for m in order_o]).astype(np.int32)
    mean = oracle.aggregate(wl.as_oracle_array(grad), P, workers)  # flat mean over the 20 workers of the kept machines
    oracle.update(th_o, None, None, mean, oracle_opt(OPTS["sgd"]))
    assert rel_err(theta.cpu().numpy(), th_o) < TOL_F32


def test_checkpoint_and_resume_is_bit_identical(sgdb, cuda_device):
    """All state lives in the caller's buffers (parameters, optimizer state, accumulator, server counters):
    copying them out in the middle of an iteration and carrying on from the copies changes no bit."""
    dev = cuda_device
    N, b, P, seed, kind = 10, 2, 30_001, 191, "adam"
    W = N + b
    scales = wl.worker_scales(seed, W)

    def fresh():
        return dict(theta=wl.theta0(seed, P, dev), s0=torch.zeros(P, device=dev), s1=torch.zeros(P, device=dev),
                    acc=torch.zeros(P, device=dev), counter=torch.zeros(4, dtype=torch.int32, device=dev))

    def deliver(st, t, ids, grad, tags):
        info = torch.zeros(2, dtype=torch.int32, device=dev)
        for w in ids:
            sgdb.sgdb_accumulate_arrival(grad[w], int(tags[w]), t, N, st["acc"], st["counter"], st["theta"], st["s0"],
                                         st["s1"], gpu_opt(OPTS[kind], t + 1), info)

    straight, resumed = fresh(), fresh()
    for t in range(3):
        grad = wl.grad_matrix(seed, t, W, P, scales, "bf16", dev)
        arrival, tags = step_inputs(seed, t, W, N)
        ids = wl.delivery_sequence(arrival).tolist()
        deliver(straight, t, ids, grad, tags)
        deliver(resumed, t, ids[:5], grad, tags)  # stop in the middle of the iteration ...
        saved = {k: v.cpu().clone() for k, v in resumed.items()}
        resumed = {k: v.to(dev) for k, v in saved.items()}  # ... and carry on from the copies, in new buffers
        deliver(resumed, t, ids[5:], grad, tags)
    for k in straight:
        assert torch.equal(straight[k], resumed[k]), k
    assert straight["counter"].cpu().tolist() == [0, 3 * W, 0, 3]


# ------------------------------------------------------------------ gradients in host memory


@pytest.mark.parametrize("dtype,P,pad,pinned", [("f32", 70_001, 0, True), ("bf16", 70_001, 5, False), ("f32", 3, 0, False)])
def test_step_with_host_gradients(sgdb, cuda_device, dtype, P, pad, pinned):
    dev = cuda_device
    W, N, T, seed, kind = 18, 15, 3, 121, "rmsprop"
    ld = P + pad
    scales = wl.worker_scales(seed, W)
    theta = wl.theta0(seed, P, dev)
    theta_d = theta.clone()
    s0, s1 = gpu_state(kind, P, dev)
    sd = gpu_state(kind, P, dev)
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    ws = torch.empty(sgdb.sgdb_step_host_workspace_bytes(tdt, P, ld, N, W - N), dtype=torch.uint8, device=dev)
    h_theta = torch.empty(P, dtype=torch.float32)
    h_mask = torch.empty(W, dtype=torch.uint8)
    h_order = torch.empty(N, dtype=torch.int32)
    h_info = torch.empty(2, dtype=torch.int32)
    mask, order, info = selection_buffers(W, N, dev)
    for t in range(T):
        grad = wl.grad_matrix(seed, t, W, P, scales, dtype, dev, ld=ld)
        h_grad = grad.cpu()
        if pinned:
            h_grad = h_grad.pin_memory()
        arrival, tags = step_inputs(seed, t, W, N)
        st = sgdb.sgdb_step_host(h_grad, P, torch.from_numpy(arrival), torch.from_numpy(tags), t, N, W - N,
                                 theta, s0, s1, gpu_opt(OPTS[kind], t + 1), h_theta, h_mask, h_order, h_info, ws,
                                 ld=ld)
        assert st == 0
        sgdb.sgdb_step(grad, P, to_dev(arrival, dev), to_dev(tags, dev), t, N, W - N, theta_d, sd[0], sd[1],
                       gpu_opt(OPTS[kind], t + 1), mask, order, info, ld=ld)
        assert torch.equal(theta, theta_d) and torch.equal(h_theta, theta.cpu())
        assert torch.equal(h_order, order.cpu()) and torch.equal(h_mask, mask.cpu())
        assert h_info.tolist() == info.cpu().tolist()
    # too few current gradients: reported as the return value, nothing changes
    tags = np.full(W, 99, np.int32)
    before = theta.clone()
    st = sgdb.sgdb_step_host(h_grad, P, torch.from_numpy(arrival), torch.from_numpy(tags), 5, N, W - N, theta, s0, s1,
                             gpu_opt(OPTS[kind]), h_theta, h_mask, h_order, h_info, ws, ld=ld)
    assert st == sgdb.SGDB_ERR_INSUFFICIENT and torch.equal(theta, before)
    with pytest.raises(sgdb.SgdbError):  # workspace too small
        sgdb.sgdb_step_host(h_grad, P, torch.from_numpy(arrival), torch.from_numpy(tags), 5, N, W - N, theta, s0, s1,
                            gpu_opt(OPTS[kind]), h_theta, h_mask, h_order, h_info, ws[:256], ld=ld)

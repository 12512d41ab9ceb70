"""Child processes of the multi-server tests (one process per parameter server).  Not collected by pytest."""
from __future__ import annotations

import ctypes
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
for p in (ROOT, os.path.join(ROOT, "tests")):
    if p not in sys.path:
        sys.path.insert(0, p)


def _init(rank: int, world: int, port: int) -> None:
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)


def _f32_at(address: int, n: int) -> np.ndarray:
    return np.ctypeslib.as_array((ctypes.c_float * n).from_address(address)) if n else np.zeros(0, np.float32)


def cpu_servers(rank: int, world: int, port: int, P: int, W: int, N: int, T: int, kind: str) -> None:
    """Host memory stands in for device memory and the oracle for the kernel: what is under test is the plumbing --
    ranges, workers per machine, the addresses exchanged between processes, the fences.  The stand-in reads the
    rows and writes the copies through the very addresses the CUDA launch would be given."""
    import torch.multiprocessing as mp

    mp.set_sharing_strategy("file_system")
    _init(rank, world, port)
    import oracle
    from helpers import OPTS, oracle_opt, oracle_state
    from paper_1604_00981_b200 import servers
    from paper_1604_00981_b200 import workload as wl

    b, seed = W - N, 331

    def stand_in(server, t, arrival, tags, update):
        n = server.len
        if n == 0:  # a server without columns has nothing to pull, update or push
            return
        rows = np.stack([_f32_at(a, n) for a in server.row_addr])
        rc, *_ = oracle.step(np.ascontiguousarray(rows), n, arrival.numpy(), tags.numpy(), t, N, b, server.master,
                             server.master_s0, server.master_s1, oracle_opt(OPTS[kind], update))
        assert rc == oracle.OK
        new = server.master.astype(np.float32)
        server.my_theta().numpy()[:n] = new
        for a in server.replica_addr:
            _f32_at(a, n)[:] = new

    srv = servers.ServerGroup(P, W, N, b, torch.float32, OPTS[kind], "cpu", launch=stand_in)
    plan = srv.plan
    assert plan.G == world and sum(n for _, n in plan.ranges) == P
    theta0 = wl.theta0(seed, P)
    srv.theta[:P] = theta0
    srv.master = theta0.numpy()[srv.first:srv.first + srv.len].astype(np.float64)
    srv.master_s0, srv.master_s1 = oracle_state(kind, srv.len)
    # the same iteration computed in one piece, for comparison
    th_o = theta0.numpy().astype(np.float64)
    s0_o, s1_o = oracle_state(kind, P)
    scales = wl.worker_scales(seed, W)
    for t in range(T):
        grad = wl.grad_matrix(seed, t, W, P, scales, "f32")
        arrival, tags = wl.arrivals(seed, t, W), wl.tags(seed, t, W, N)
        mine = plan.workers_of(rank)
        srv.grads[:len(mine), :P] = grad[mine.start:mine.stop]
        srv.step(t, torch.from_numpy(arrival), torch.from_numpy(tags), update=t + 1)
        rc, *_ = oracle.step(grad.numpy(), P, arrival, tags, t, N, b, th_o, s0_o, s1_o, oracle_opt(OPTS[kind], t + 1))
        assert rc == oracle.OK
        got = srv.theta[:P].numpy()
        assert np.array_equal(got, th_o.astype(np.float32)), (rank, t, float(np.max(np.abs(got - th_o))))
    dist.barrier()
    dist.destroy_process_group()


def gpu_servers(rank: int, world: int, port: int, P: int, W: int, N: int, T: int, kind: str, dtype: str) -> None:
    """Two servers as two processes on ONE GPU (no launch waits for another; the fences are host barriers): the
    real exchange of device addresses between processes and the real kernel.  Every copy of theta must hold the
    bits of the one-GPU sgdb_step, and of sgdb_step_grouped for the two-level form."""
    _init(rank, world, port)
    from helpers import OPTS, gpu_opt, gpu_state, selection_buffers, to_dev
    from paper_1604_00981_b200 import binding as sgdb
    from paper_1604_00981_b200 import servers
    from paper_1604_00981_b200 import workload as wl

    dev = torch.device("cuda:0")
    b, seed = W - N, 337
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    srv = servers.ServerGroup(P, W, N, b, tdt, OPTS[kind], dev)
    two = servers.ServerGroup(P, W, N, b, tdt, OPTS[kind], dev)
    plan = srv.plan
    theta_1 = wl.theta0(seed, P, dev)
    theta_2 = theta_1.clone()
    srv.theta[:P] = theta_1
    two.theta[:P] = theta_1
    s1, s2 = gpu_state(kind, P, dev), gpu_state(kind, P, dev)
    mask_1, order_1, info_1 = selection_buffers(W, N, dev)
    scales = wl.worker_scales(seed, W)
    M = world
    groups = to_dev(np.array(plan.groups(), np.int32), dev)
    for t in range(T):
        grad = wl.grad_matrix(seed, t, W, P, scales, dtype, dev)
        arrival, tags = wl.arrivals(seed, t, W), wl.tags(seed, t, W, N)
        a_d, t_d = to_dev(arrival, dev), to_dev(tags, dev)
        mine = plan.workers_of(rank)
        for s in (srv, two):
            s.grads[:len(mine), :P] = grad[mine.start:mine.stop]
        # workers are all current in the two-level run: every machine's message counts, the later one is dropped
        now = torch.full((W,), t, dtype=torch.int32, device=dev)
        srv.step(t, a_d, t_d, update=t + 1)
        two.step_two_level(t, a_d, now, M - 1, update=t + 1)
        sgdb.sgdb_step(grad, P, a_d, t_d, t, N, b, theta_1, s1[0], s1[1], gpu_opt(OPTS[kind], t + 1), mask_1, order_1, info_1)
        gm = torch.zeros(W, dtype=torch.uint8, device=dev)
        go = torch.zeros(M - 1, dtype=torch.int32, device=dev)
        od = torch.zeros(W, dtype=torch.int32, device=dev)
        gi = torch.zeros(3, dtype=torch.int32, device=dev)
        sgdb.sgdb_step_grouped(grad, P, a_d, now, groups, t, M, M - 1, theta_2, s2[0], s2[1], gpu_opt(OPTS[kind], t + 1), gm, go,
                               od, gi)
        torch.cuda.synchronize()
        assert srv.info[:2].cpu().tolist() == info_1.cpu().tolist() and info_1.cpu().tolist()[1] == 0, (rank, t)
        assert torch.equal(srv.order[:N], order_1) and torch.equal(srv.mask, mask_1)
        assert torch.equal(srv.theta[:P], theta_1), (rank, t, "one row per worker")
        assert two.info.cpu().tolist() == gi.cpu().tolist() and gi.cpu().tolist()[1] == 0, (rank, t)
        assert torch.equal(two.theta[:P], theta_2), (rank, t, "one row per machine")
    for k in range(2):
        if s1[k] is not None:
            mine_state = (srv.state0, srv.state1)[k][:srv.len]
            assert torch.equal(mine_state, s1[k][srv.first:srv.first + srv.len])
    dist.barrier()
    dist.destroy_process_group()

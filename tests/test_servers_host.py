"""Host side of the several-GPUs form (one process per parameter server): who holds which columns and workers,
the addresses handed to the kernel, and -- as two gloo ranks on the CPU -- the exchange of buffers between
processes and the fences, with host memory standing in for device memory and the oracle for the kernel."""
import socket

import numpy as np
import pytest
import torch

from paper_1604_00981_b200 import servers


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("P,W,G", [(23_800_000, 100, 8), (1000, 6, 4), (63, 5, 2), (0, 3, 3), (100_000_000, 208, 8), (4096, 1, 1)])
def test_plan_covers_every_column_and_worker_once(P, W, G):
    plan = servers.make_plan(P, W, G)
    assert len(plan.ranges) == G and plan.ranges[0][0] == 0
    end = 0
    for first, n in plan.ranges:
        assert first == end and n >= 0 and (first % 64 == 0 or first == P)
        end = first + n
    assert end == P
    seen = [w for g in range(G) for w in plan.workers_of(g)]
    assert seen == list(range(W))
    for w in range(W):
        g = plan.machine_of(w)
        assert 0 <= g < G and plan.workers_of(g)[plan.local_index(w)] == w
    assert plan.groups() == [plan.machine_of(w) for w in range(W)]


def test_addresses_point_at_the_first_column_of_each_range():
    """Checked on real host buffers: reading `len` elements at every row address gives exactly the server's
    columns of that worker's row, and the replica addresses are the other copies' same columns."""
    import ctypes

    P, W, G = 1000, 7, 3
    plan = servers.make_plan(P, W, G)
    ld = 1008
    full = np.arange(W * P, dtype=np.float32).reshape(W, P)
    held = []
    for g in range(G):
        ws = plan.workers_of(g)
        buf = np.full((max(len(ws), 1), ld), -1.0, np.float32)
        buf[:len(ws), :P] = full[ws.start:ws.stop]
        held.append(buf)
    copies = [np.zeros(P, np.float32) for _ in range(G)]
    for j in range(G):
        first, n = plan.ranges[j]
        rows = servers.row_addresses(plan, j, [b.ctypes.data for b in held], ld * 4, 4)
        assert len(rows) == W
        for w, a in enumerate(rows):
            got = np.ctypeslib.as_array((ctypes.c_float * n).from_address(a))
            assert np.array_equal(got, full[w, first:first + n])
        reps = servers.replica_addresses(plan, j, [c.ctypes.data for c in copies])
        assert len(reps) == G - 1
        for a in reps:
            np.ctypeslib.as_array((ctypes.c_float * n).from_address(a))[:] = j + 1
        copies[j][first:first + n] = j + 1
    for c in copies:
        for j, (first, n) in enumerate(plan.ranges):
            assert (c[first:first + n] == j + 1).all()


@pytest.mark.parametrize("G,P,W,N,kind", [(2, 5000, 7, 5, "rmsprop"), (2, 333, 4, 4, "adam"), (3, 1000, 7, 6, "momentum"),
                                          (3, 100, 5, 4, "sgd"), (4, 777, 3, 2, "adagrad")])
def test_servers_as_gloo_ranks(G, P, W, N, kind):
    """G processes, G parameter servers (uneven numbers of workers per machine, a machine without workers, a
    server without columns among the cases): after every iteration each process's copy of theta equals the
    iteration computed in one piece."""
    import torch.multiprocessing as mp

    import servers_child

    mp.spawn(servers_child.cpu_servers, args=(G, _free_port(), P, W, N, 3, kind), nprocs=G, join=True)

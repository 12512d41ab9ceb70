"""Two parameter servers as two processes (the several-GPUs form of the step, Section 1.1), both on the one GPU
there is: device addresses really cross between processes and the real kernel pulls rows from and pushes
parameters to the other process's memory.  No launch waits for another, so sharing one GPU is safe."""
import socket

import pytest

pytestmark = pytest.mark.gpu


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("P,W,N,kind,dtype", [(300_007, 22, 18, "rmsprop", "f32"), (100_003, 9, 8, "adam", "bf16"),
                                              (64, 5, 4, "sgd", "f32")])  # the last: the second server has no columns
def test_two_servers_as_two_processes_on_one_gpu(cuda_device, P, W, N, kind, dtype):
    import torch.multiprocessing as mp

    import servers_child

    mp.spawn(servers_child.gpu_servers, args=(2, _free_port(), P, W, N, 3, kind, dtype), nprocs=2, join=True)

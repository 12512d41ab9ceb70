"""sgdb_step_host_static: the host-buffer step for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is not an option (all device memory already belongs to
another component's pool, or allocation is forbidden inside their serving loop).  For them the library
carries a fixed staging array.  This test calls that entry point through the C ABI twice in a row and
checks every output against sgdb_step_host, which uses a caller-supplied workspace; the two must agree
within the tolerance of the other parity tests (they are in fact the same bits).  It also checks what the
entry point is for: the amount of free device memory is the same before and after the second call.  The file sorts last so
that a run that stops at the first failure has already run everything else; it also passes on its own.
"""
import numpy as np
import pytest
import torch

from helpers import OPTS, TOL_BF16, TOL_F32, gpu_opt, gpu_state, rel_err, step_inputs
from paper_1604_00981_b200 import workload as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sgdb(cuda_device):
    from paper_1604_00981_b200 import binding

    return binding


def _host_outputs(W, N, P):
    return (torch.empty(P, dtype=torch.float32), torch.empty(W, dtype=torch.uint8),
            torch.empty(N, dtype=torch.int32), torch.empty(2, dtype=torch.int32))


@pytest.mark.parametrize("dtype,P,pad", [("f32", 70_001, 3), ("bf16", 150_000, 0)])
def test_static_scratch_step_matches_workspace_step_on_two_calls(sgdb, cuda_device, dtype, P, pad):
    dev = cuda_device
    W, N, seed, kind = 18, 15, 131, "rmsprop"
    ld = P + pad
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    need = sgdb.sgdb_step_host_workspace_bytes(tdt, P, ld, N, W - N)
    assert 0 < need <= sgdb.SGDB_STATIC_SCRATCH_BYTES
    ws = torch.empty(need, dtype=torch.uint8, device=dev)
    scales = wl.worker_scales(seed, W)
    theta_a = wl.theta0(seed, P, dev)
    theta_b = theta_a.clone()
    sa, sb = gpu_state(kind, P, dev), gpu_state(kind, P, dev)
    out_a, out_b = _host_outputs(W, N, P), _host_outputs(W, N, P)
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    for t in range(2):  # two calls in a row share the built-in array; the second must not see the first
        h_grad = wl.grad_matrix(seed, t, W, P, scales, dtype, "cpu", ld=ld)
        arrival, tags = step_inputs(seed, t, W, N)
        args = (h_grad, P, torch.from_numpy(arrival), torch.from_numpy(tags), t, N, W - N)
        opt_a = gpu_opt(OPTS[kind], t + 1)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info(dev)[0]
        st_a = sgdb.sgdb_step_host_static(*args, theta_a, sa[0], sa[1], opt_a, *out_a, ld=ld)
        free_after = torch.cuda.mem_get_info(dev)[0]
        if t > 0:  # the first call on a device may make the driver load the library's code; later calls take nothing
            assert free_after == free_before, "the call without a workspace changed the free device memory"
        st_b = sgdb.sgdb_step_host(*args, theta_b, sb[0], sb[1], gpu_opt(OPTS[kind], t + 1), *out_b, ws, ld=ld)
        assert st_a == st_b == 0
        assert torch.equal(out_a[1], out_b[1]) and torch.equal(out_a[2], out_b[2])  # mask, order
        assert out_a[3].tolist() == out_b[3].tolist()
        assert rel_err(out_a[0].numpy(), out_b[0].numpy()) < tol
        assert rel_err(theta_a.cpu().numpy(), theta_b.cpu().numpy()) < tol
        for x, y in zip(sa, sb):
            assert rel_err(x.cpu().numpy(), y.cpu().numpy()) < tol
    assert torch.equal(theta_a, theta_b)  # same kernels, same order of additions


def test_static_scratch_step_refuses_sizes_beyond_its_array(sgdb, cuda_device):
    dev = cuda_device
    W, N, P = 18, 15, 200_000  # 18 rows x 200000 x 4 B = 14.4 MB > 8 MiB
    assert sgdb.sgdb_step_host_workspace_bytes(torch.float32, P, P, N, W - N) > sgdb.SGDB_STATIC_SCRATCH_BYTES
    theta = torch.zeros(P, device=dev)
    out = _host_outputs(W, N, P)
    with pytest.raises(sgdb.SgdbError) as e:
        sgdb.sgdb_step_host_static(torch.zeros((W, P)), P, torch.ones(W), torch.zeros(W, dtype=torch.int32), 0, N,
                                   W - N, theta, None, None, gpu_opt(OPTS["sgd"]), *out)
    assert e.value.status == sgdb.SGDB_ERR_UNSUPPORTED
    assert (theta == 0).all()

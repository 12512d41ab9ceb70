"""Every wait inside the row-streaming kernels is bounded and ends in SGDB_ERR_TIMEOUT instead of hanging the
device.  A correct run never gets there, so the same wait routine is exercised on a barrier that nothing will
ever complete, with limits of at most a few milliseconds; the kernel ends normally and the context stays usable."""
import pytest
import torch

from helpers import OPTS, gpu_opt, selection_buffers

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sgdb(cuda_device):
    from paper_1604_00981_b200 import binding

    return binding


def test_a_wait_that_nothing_completes_gives_up_and_reports_it(sgdb, cuda_device):
    dev = cuda_device
    sgdb.sgdb_selftest_bounded_wait(0, torch.zeros(3, dtype=torch.int32, device=dev))  # loads the kernel
    torch.cuda.synchronize()
    for limit_ns in (0, 200_000, 3_000_000):
        out = torch.full((3,), -7, dtype=torch.int32, device=dev)
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        sgdb.sgdb_selftest_bounded_wait(limit_ns, out)
        stop.record()
        torch.cuda.synchronize()
        status, waited_ns, released = out.cpu().tolist()
        assert status == sgdb.SGDB_ERR_TIMEOUT
        assert released == 1, "the second waiter must leave through the abort flag, not through its own limit"
        assert limit_ns <= waited_ns < limit_ns + 1_000_000
        assert start.elapsed_time(stop) < limit_ns * 1e-6 + 20.0  # milliseconds: nowhere near the kernels' 2 s limit
    # limits that would hold the device for long are refused on the host
    out = torch.zeros(3, dtype=torch.int32, device=dev)
    for bad in (-1, 100_000_001):
        with pytest.raises(sgdb.SgdbError) as e:
            sgdb.sgdb_selftest_bounded_wait(bad, out)
        assert e.value.status == sgdb.SGDB_ERR_INVALID_ARG
    # the context is as usable as before: a fused step right after
    W, N, P = 6, 4, 10_000
    grad = torch.ones((W, P), device=dev)
    theta = torch.zeros(P, device=dev)
    arrival = torch.arange(1, W + 1, dtype=torch.float32, device=dev)
    tags = torch.zeros(W, dtype=torch.int32, device=dev)
    mask, order, info = selection_buffers(W, N, dev)
    sgdb.sgdb_step(grad, P, arrival, tags, 0, N, W - N, theta, None, None, gpu_opt(OPTS["sgd"]), mask, order, info)
    assert info.cpu().tolist() == [W, 0] and torch.equal(theta, torch.full((P,), -0.1, device=dev))


def test_the_step_gives_up_cleanly_when_its_waits_have_no_patience(sgdb, cuda_device):
    """The product kernel itself with a patience of zero: the first wait whose data is not there yet gives up, the
    block waits for the copies it still has in flight and the kernel ends normally with SGDB_ERR_TIMEOUT.  Nothing
    is broken on purpose: every copy goes to a valid address and lands.  Afterwards, with the default patience back,
    the same step gives the bits it always gives: no later block found stray bytes in its shared memory."""
    dev = cuda_device
    W, N, P = 12, 10, 1_500_000
    gen = torch.Generator(device=dev)
    gen.manual_seed(5)
    grad = torch.randn((W, P), device=dev, generator=gen)
    arrival = torch.arange(1, W + 1, dtype=torch.float32, device=dev)
    tags = torch.zeros(W, dtype=torch.int32, device=dev)
    opt = gpu_opt(OPTS["rmsprop"])

    def run():
        theta = torch.zeros(P, device=dev)
        s0, s1 = torch.zeros(P, device=dev), torch.zeros(P, device=dev)
        mask, order, info = selection_buffers(W, N, dev)
        sgdb.sgdb_step(grad, P, arrival, tags, 0, N, W - N, theta, s0, s1, opt, mask, order, info)
        torch.cuda.synchronize()
        return theta, s0, s1, info.cpu().tolist()

    want = run()
    assert want[3] == [W, 0]
    gave_up = 0
    try:
        sgdb.sgdb_set_wait_limit_ns(0)
        for _ in range(5):
            status = run()[3][1]
            gave_up += status == sgdb.SGDB_ERR_TIMEOUT
    finally:
        sgdb.sgdb_set_wait_limit_ns(-1)
    assert gave_up == 5, "with no patience every launch meets a wait whose data is not there yet"
    for _ in range(3):
        got = run()
        assert got[3] == [W, 0]
        assert torch.equal(got[0], want[0]) and torch.equal(got[1], want[1]) and torch.equal(got[2], want[2])
    with pytest.raises(sgdb.SgdbError):
        sgdb.sgdb_set_wait_limit_ns(11_000_000_000)

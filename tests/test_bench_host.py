"""Host-side logic of bench.py, without a GPU: the reference arm's JSON line, and the multi-rank path
(max over ranks, rank 0 alone prints) with two gloo ranks on CPU."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                          "--warmup", "1", "--columns", "40000"], capture_output=True, text=True, check=True).stdout
    lines = [l for l in out.splitlines() if l.strip()]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["unit"] == "GB/s" and line["higher_is_better"] is True
    assert line["steps"] == 2 and line["warmup"] == 1 and line["value"] > 0 and line["ms_per_step"] > 0
    cpu = line["cpu_baseline"]
    assert cpu["kind"] == "oracle" and cpu["cores"] == len(os.sched_getaffinity(0)) and cpu["nproc"] == os.cpu_count()
    assert isinstance(cpu["cpu_model"], str) and cpu["cpu_model"] and cpu["full_P"] is True
    assert cpu["single_thread"]["cores"] == 1 and cpu["single_thread"]["value"] > 0
    assert cpu["value"] == line["value"] == line["e2e"]["value"]
    # both arms describe the workload with the same keys
    assert set(line["config"]) == {"workload", "P", "W", "N", "b", "optimizer", "grad_dtype", "sharding", "l2"}
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["config"]["workload"].startswith("c1_") and "model" not in line["config"]
    assert line["vs_baseline"] is None and line["gpu_launches"] == 0


def test_reference_arm_under_torchrun_only_rank0_prints():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29631", os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference",
           "--steps", "1", "--warmup", "0", "--columns", "20000"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and json.loads(lines[0])["n_gpus"] == 2


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_step, ms_e2e = (1.5, 100.0) if rank == 0 else (2.0, 90.0)  # rank 1 is the slower one in the timed region
    got = bench.max_over_ranks(dist, [ms_step, ms_e2e], torch.device("cpu"))
    with open(os.path.join(out_dir, "rank%d.json" % rank), "w") as f:
        json.dump(got, f)
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_rate_with_two_gloo_ranks(tmp_path):
    mp.spawn(_rank_main, args=(2, 29641, str(tmp_path)), nprocs=2, join=True)
    for rank in range(2):
        assert json.load(open(tmp_path / ("rank%d.json" % rank))) == [2.0, 100.0]
    sys.path.insert(0, ROOT)
    import bench

    # two shards, each moving 8 GB in the slowest rank's 2 ms step: 8 TB/s for the job
    assert bench.whole_job_rate(2, 8e9, 2.0) == 8000.0
    assert bench.max_over_ranks(None, [1.0, 2.0], None) == [1.0, 2.0]


def test_column_ranges_cover_every_column_once():
    sys.path.insert(0, ROOT)
    import bench

    for P, parts in ((10, 3), (7, 16), (23_800_000, 48), (1, 1)):
        pieces = bench.column_ranges(P, parts)
        assert pieces[0][0] == 0 and pieces[-1][1] == P and len(pieces) <= parts
        assert all(a[1] == b[0] for a, b in zip(pieces, pieces[1:])) and all(c1 > c0 for c0, c1 in pieces)


def test_oracle_split_over_threads_equals_one_call():
    """The all-cores leg of the CPU baseline calls the unchanged oracle step once per column range; the pieces
    together must give exactly what one call over all columns gives."""
    sys.path.insert(0, ROOT)
    import numpy as np

    import bench
    import oracle
    from paper_1604_00981_b200 import workload as wl

    cfg = wl.CONFIGS[1]
    P, W, N = 10_007, cfg.W, cfg.N
    grad = wl.as_oracle_array(wl.grad_matrix(cfg.seed, 0, W, P, wl.worker_scales(cfg.seed, W), "f32", "cpu"))
    arrival, tags = wl.arrivals(cfg.seed, 0, W), wl.tags(cfg.seed, 0, W, N)
    opt = oracle.Opt(kind=oracle.RMSPROP, lr=0.045, decay=0.9, momentum=0.9, eps=1.0)
    whole = [np.ones(P), np.zeros(P), np.zeros(P)]
    rc, *_ = oracle.step(grad, P, arrival, tags, 0, N, cfg.b, *whole, opt)
    assert rc == oracle.OK
    split = [np.ones(P), np.zeros(P), np.zeros(P)]
    flat = grad.reshape(-1)
    for c0, c1 in bench.column_ranges(P, 5):
        rc, *_ = oracle.step(flat[c0:], c1 - c0, arrival, tags, 0, N, cfg.b, *(a[c0:c1] for a in split), opt, ld=P)
        assert rc == oracle.OK
    for a, b in zip(whole, split):
        assert np.array_equal(a, b)
    sec, gbs = bench.oracle_run(cfg.__class__(**{**cfg.__dict__, "P": P}), grad, P, steps=1, warmup=0, threads=3)
    assert sec > 0 and gbs > 0

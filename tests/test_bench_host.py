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
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] == 1
    assert line["cpu_baseline"]["value"] == line["value"] == line["e2e"]["value"]
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

#!/usr/bin/env python
"""Benchmark of the fused N-of-(N+b) aggregate + update step (sgdb_step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl native|reference]

A step is one pass of the whole path over one batch of synthetic input: select the first N of the
N+b gradients, average them, apply RMSProp with momentum.  The workload is the Inception-v3-sized
one: P = 23.8 M fp32 parameters, W = 100 (N = 96, b = 4).  Prints one JSON line.

value     gradient bytes read per second (N * P * 4 per step), inputs resident in HBM
e2e       the same metric through sgdb_step_host: gradients, arrival times and tags start in pinned
          host memory, the updated parameters are read back, all inside the timed region
roofline  algorithmic bytes of a step (gradient rows + parameters and state read and written) over
          the measured step time, against the measured HBM copy bandwidth of this machine
With --gpus N > 1 (under torchrun) every rank is one parameter-server shard holding its own P
columns; there is no data-path collective, and the value is the sum over ranks over the slowest rank.
--impl reference times the CPU oracle on a bounded column sample of the same workload.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_1604_00981_b200 import workload as wl

METRIC = "N-of-(N+b) aggregate+update: gradient GB/s read"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0  # earlier measurement on this machine, used only when MEASURED_PEAKS.json is absent
NOMINAL_HBM_GBS = 8000.0

# DRAM traffic of one fused-step launch from an ncu capture (dram__bytes_read.sum + dram__bytes_write.sum),
# as bytes per algorithmic byte; valid only for the kernel sources whose digest is recorded with it.
NCU_TRAFFIC = {"src_digest": "f559b579ce14cf57", "dram_bytes_per_algorithmic_byte": 0.9948}


def kernel_source_digest() -> str:
    """Digest of the device code the fused step runs: the shared device header, and the kernel file up to
    the end of the row-streaming kernel (selection prologue included)."""
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_1604_00981_b200", "csrc")
    with open(os.path.join(csrc, "sgdb_device.cuh"), "rb") as f:
        h.update(f.read())
    with open(os.path.join(csrc, "sgdb_kernels.cuh"), "rb") as f:
        text = f.read()
    end = text.find(b"// ====================================================================== update from a mean")
    h.update(text if end < 0 else text[:end])
    return h.hexdigest()[:16]


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = str(index)
        try:  # name the GPU by UUID: nvidia-smi's indices need not match CUDA's device order
            self.index = "GPU-" + str(torch.cuda.get_device_properties(index).uuid)
        except Exception:
            pass
        self.proc = None
        self.lines = []

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.index, "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def __exit__(self, *exc):
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            self.thread.join(timeout=2)

    def summary(self):
        sm, smax, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(smax)), "reasons": sorted(reasons),
                "samples": len(sm)}


def oracle_sample_run(cfg, P_sample: int, steps: int, warmup: int, seed_shift: int = 0):
    """Times the CPU oracle, as it stands, on the first P_sample columns of the workload.
    Returns (seconds per step, gradient GB/s)."""
    import oracle

    W, N = cfg.W, cfg.N
    scales = wl.worker_scales(cfg.seed, W)
    grad = wl.as_oracle_array(wl.grad_matrix(cfg.seed + seed_shift, 0, W, P_sample, scales, cfg.grad_dtype, "cpu"))
    theta = wl.theta0(cfg.seed, P_sample, "cpu").numpy().astype(np.float64)
    s0, s1 = np.zeros(P_sample), np.zeros(P_sample)
    hyper = {k: float(np.float32(v)) for k, v in cfg.opt.items() if k != "kind"}
    kind = {"sgd": oracle.SGD, "momentum": oracle.MOMENTUM, "rmsprop": oracle.RMSPROP, "adam": oracle.ADAM,
            "adagrad": oracle.ADAGRAD}[cfg.opt["kind"]]
    times = []
    for t in range(warmup + steps):
        arrival, tags = wl.arrivals(cfg.seed, t, W), wl.tags(cfg.seed, t, W, N)
        t0 = time.perf_counter()
        rc, *_ = oracle.step(grad, P_sample, arrival, tags, t, N, cfg.b, theta, s0, s1,
                             oracle.Opt(kind=kind, step=t + 1, **hyper))
        dt = time.perf_counter() - t0
        assert rc == oracle.OK
        if t >= warmup:
            times.append(dt)
    sec = float(np.mean(times))
    esize = 4 if cfg.grad_dtype == "f32" else 2
    return sec, N * P_sample * esize / sec / 1e9


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    P_sample = cfg.P // 4
    sec, gbs = oracle_sample_run(cfg, P_sample, args.steps, args.warmup)
    sample = "first %d of %d columns (1/4), all %d rows, %d steps, single thread" % (P_sample, cfg.P, cfg.W, args.steps)
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "P": cfg.P, "W": cfg.W, "N": cfg.N, "b": cfg.b, "optimizer": cfg.opt["kind"],
                   "grad_dtype": cfg.grad_dtype, "sample": sample},
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


N_STATE = {"sgd": 0, "momentum": 1, "rmsprop": 2, "adam": 2, "adagrad": 1}
N_SETS = 16  # arrival/tag draws rotate, so the kept set differs from step to step


def selection_sets(cfg, dev):
    arr = [torch.from_numpy(wl.arrivals(cfg.seed, t, cfg.W)).to(dev) for t in range(N_SETS)]
    tag = [torch.from_numpy(wl.tags(cfg.seed, t, cfg.W, cfg.N) - t).to(dev) for t in range(N_SETS)]  # relative to t = 0
    return arr, tag


def selection_outputs(W, N, dev):
    return (torch.zeros(W, dtype=torch.uint8, device=dev), torch.zeros(N, dtype=torch.int32, device=dev),
            torch.zeros(2, dtype=torch.int32, device=dev))


def setup_flat(cfg, dev, sgdb, seed, ema=False, deadline=None):
    """Workloads with one flat parameter vector (tiny SGD, Inception-sized RMSProp, large bf16 Adam)."""
    W, N, b, P = cfg.W, cfg.N, cfg.b, cfg.P
    scales = wl.worker_scales(cfg.seed, W)
    grad = wl.grad_matrix(seed, 0, W, P, scales, cfg.grad_dtype, dev)
    theta = wl.theta0(seed, P, dev)
    n_state = N_STATE[cfg.opt["kind"]]
    s0 = torch.zeros(P, device=dev) if n_state >= 1 else None
    s1 = torch.zeros(P, device=dev) if n_state >= 2 else None
    mask, order, info = selection_outputs(W, N, dev)
    arr_d, tag_d = selection_sets(cfg, dev)
    opt = sgdb.Opt(**cfg.opt)

    avg = theta.clone() if ema else None
    kept_mean = float(N)
    if deadline is not None:  # time-out rule: the number of kept rows differs from draw to draw
        order = torch.zeros(W, dtype=torch.int32, device=dev)
        kept = [int(((wl.arrivals(cfg.seed, t, W) <= np.float32(deadline)) & (wl.tags(cfg.seed, t, W, N) == t)).sum())
                for t in range(N_SETS)]
        kept_mean = float(np.mean(kept))

    def step(i):
        opt.step = i + 1
        if deadline is not None:
            sgdb.sgdb_step_deadline(grad, P, arr_d[i % N_SETS], tag_d[i % N_SETS], 0, deadline, 1, theta, s0, s1, opt,
                                    mask, order, info)
        elif ema:  # the step plus the running average of the parameters (last line of the server's loop)
            sgdb.sgdb_step_ema(grad, P, arr_d[i % N_SETS], tag_d[i % N_SETS], 0, N, b, theta, s0, s1, opt, avg, 0.9999,
                               mask, order, info)
        else:
            sgdb.sgdb_step(grad, P, arr_d[i % N_SETS], tag_d[i % N_SETS], 0, N, b, theta, s0, s1, opt, mask, order, info)

    def check():
        assert info.cpu().tolist()[1] == 0, "a step reported a device-side error"
        assert bool(torch.isfinite(theta).all()) and (avg is None or bool(torch.isfinite(avg).all()))

    def graph_replay():
        """Launch-bound sizes: the same steps captured once in a CUDA graph and replayed, so that the host's
        per-call cost (Python, ctypes, launch) is out of the picture."""
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for i in range(3):
                step(i)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for i in range(N_SETS):
                step(i)
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        for _ in range(20):
            graph.replay()
        stop.record()
        torch.cuda.synchronize()
        return {"cuda_graph_replay_us_per_step": 1e3 * start.elapsed_time(stop) / (20 * N_SETS)}

    def separate_calls():
        """The same step as three calls (select, aggregate into a mean vector, update from it)."""
        mean = torch.empty(P, device=dev)

        def separate_step(i):
            opt.step = i + 1
            sgdb.sgdb_select(arr_d[i % N_SETS], tag_d[i % N_SETS], 0, N, b, mask, order, info)
            sgdb.sgdb_aggregate(grad, P, N, order, info, mean)
            sgdb.sgdb_update(theta, s0, s1, mean, opt, info)

        ms = time_steps(separate_step, 10, 3)
        moved = grad_bytes + 2 * (1 + n_state) * P * 4 + 2 * P * 4  # the mean is written and read back
        return {"separate_calls_ms_per_step": ms, "separate_calls_total_gbs": moved / (ms * 1e-3) / 1e9,
                "separate_calls_launches_per_step": 3}

    grad_bytes = int(kept_mean * P * grad.element_size())
    state = dict(grad=grad, theta=theta, s0=s0, s1=s1, opt=opt)
    total = grad_bytes + 2 * (1 + n_state) * P * 4 + (2 * P * 4 if ema else 0)
    return dict(step=step, check=check, grad_bytes=grad_bytes, total_bytes=total,
                launches_per_step=1, kernel="stream_rows_kernel<%s, %s>%s (the step is this one launch)"
                % (cfg.grad_dtype, cfg.opt["kind"], " + parameter average" if ema else ""), state=state,
                extra={"parameter_average": True} if ema else
                ({"deadline_s": deadline, "mean_rows_kept": kept_mean} if deadline is not None else
                 (graph_replay if P * W <= 1_000_000 else separate_calls)))


def setup_segmented(cfg, dev, sgdb, seed):
    """300 tensors of log-uniform length, one launch over a device-side segment table."""
    W, N, b = cfg.W, cfg.N, cfg.b
    scales = wl.worker_scales(cfg.seed, W)
    lengths = wl.segment_lengths(cfg.seed, cfg.segments)
    n_state = N_STATE[cfg.opt["kind"]]
    segs = []
    for i, L in enumerate(int(x) for x in lengths):
        ld = (L + 3) // 4 * 4
        segs.append((wl.theta0(seed + i, L, dev), torch.zeros(L, device=dev) if n_state >= 1 else None,
                     torch.zeros(L, device=dev) if n_state >= 2 else None,
                     wl.grad_matrix(seed + i, 0, W, L, scales, cfg.grad_dtype, dev, ld=ld)))
    table = sgdb.make_segment_table(segs, dev)
    mask, order, info = selection_outputs(W, N, dev)
    arr_d, tag_d = selection_sets(cfg, dev)
    opt = sgdb.Opt(**cfg.opt)
    P = int(lengths.sum())

    def step(i):
        opt.step = i + 1
        sgdb.sgdb_step_segmented(table, len(segs), segs[0][3].dtype, arr_d[i % N_SETS], tag_d[i % N_SETS], 0, N, b,
                                 opt, mask, order, info)

    def per_tensor_step(i):
        opt.step = i + 1
        for theta, s0, s1, grad in segs:
            sgdb.sgdb_step(grad, theta.numel(), arr_d[i % N_SETS], tag_d[i % N_SETS], 0, N, b, theta, s0, s1, opt,
                           mask, order, info, ld=grad.stride(0))

    def check():
        assert info.cpu().tolist()[1] == 0
        assert all(bool(torch.isfinite(sg[0]).all()) for sg in segs[:20])

    def extra():
        ms = time_steps(per_tensor_step, 5, 2)
        return {"one_launch_per_tensor_ms_per_step": ms, "tensors": len(segs), "total_parameters": P}

    grad_bytes = N * P * segs[0][3].element_size()
    return dict(step=step, check=check, grad_bytes=grad_bytes, total_bytes=grad_bytes + 2 * (1 + n_state) * P * 4,
                launches_per_step=1, kernel="stream_rows_kernel<%s, %s> over a %d-entry segment table"
                % (cfg.grad_dtype, cfg.opt["kind"], len(segs)), state=dict(segs=segs, table=table), extra=extra, P=P)


def setup_arrivals(cfg, dev, sgdb, seed):
    """Accumulate-on-arrival: a step is one whole iteration, W calls in arrival sequence (N accepted, b dropped)."""
    N, P = cfg.N, cfg.P
    n_state = N_STATE[cfg.opt["kind"]]
    b_max = 8
    scales = wl.worker_scales(cfg.seed, N + b_max)
    grad = wl.grad_matrix(seed, 0, N + b_max, P, scales, cfg.grad_dtype, dev)
    theta = wl.theta0(seed, P, dev)
    s0, s1 = torch.zeros(P, device=dev), torch.zeros(P, device=dev)
    acc = torch.empty(P, device=dev)
    counter = torch.zeros(4, dtype=torch.int32, device=dev)
    info = torch.zeros(2, dtype=torch.int32, device=dev)
    opt = sgdb.Opt(**cfg.opt)
    sequences = {bb: [int(w) for w in wl.delivery_sequence(wl.arrivals(cfg.seed + bb, 0, N + bb))] for bb in (0, 2, 4, 8)}
    iteration = [0]

    def make_step(bb):
        def step(i):
            t = iteration[0]
            opt.step = t + 1
            for w in sequences[bb]:  # every tag is current; the last bb arrivals come after the update fired
                sgdb.sgdb_accumulate_arrival(grad[w], t, t, N, acc, counter, theta, s0, s1, opt, info)
            iteration[0] = t + 1
        return step

    def check():
        c = counter.cpu().tolist()
        assert c[0] == 0 and c[2] == 0 and c[3] == iteration[0], c
        assert bool(torch.isfinite(theta).all())

    def extra():
        out = {}
        for bb in (0, 2, 8):
            ms = time_steps(make_step(bb), 5, 2)
            out["b=%d" % bb] = {"ms_per_step": ms, "calls_per_step": N + bb}
        return {"b_sweep": out, "bytes_per_accepted_arrival": P * 12}

    esize = grad.element_size()
    grad_bytes = N * P * esize
    # first accepted row: read row, write acc; middle rows: read row + acc, write acc; N-th: read row + acc + theta
    # + state, write theta + state
    total = grad_bytes + (N - 1) * P * 4 + (N - 1) * P * 4 + 2 * (1 + n_state) * P * 4
    return dict(step=make_step(cfg.b), check=check, grad_bytes=grad_bytes, total_bytes=total,
                launches_per_step=N + cfg.b, kernel="accumulate_arrival_kernel<%s, %s>, %d launches per step"
                % (cfg.grad_dtype, cfg.opt["kind"], N + cfg.b), state=dict(grad=grad), extra=extra)


def max_over_ranks(dist, values, device):
    """Element-wise maximum of `values` over all ranks (the slowest rank sets the job's time)."""
    if dist is None:
        return list(values)
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_rate(world: int, bytes_per_rank_step: float, ms_per_step: float) -> float:
    """GB/s of the whole job: every rank moves bytes_per_rank_step in the (slowest rank's) step time."""
    return world * bytes_per_rank_step / (ms_per_step * 1e-3) / 1e9


def time_steps(step, steps, warmup):
    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for i in range(steps):
        step(warmup + i)
    stop.record()
    torch.cuda.synchronize()
    return start.elapsed_time(stop) / steps


def run_native(args, cfg):
    from paper_1604_00981_b200 import binding as sgdb

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    seed = cfg.seed + 1000 * rank  # every rank is its own parameter-server shard
    if cfg.segments:
        wk = setup_segmented(cfg, dev, sgdb, seed)
    elif cfg.name.startswith("c4"):
        wk = setup_arrivals(cfg, dev, sgdb, seed)
    else:
        wk = setup_flat(cfg, dev, sgdb, seed, ema=args.ema, deadline=args.deadline)
    step = wk["step"]

    for i in range(args.warmup):
        step(i)
    barrier()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local_rank) as clocks:
        barrier()
        start.record()
        for i in range(args.steps):
            step(args.warmup + i)
        stop.record()
        barrier()
    ms_total = start.elapsed_time(stop)
    wk["check"]()
    extra = wk["extra"]() if callable(wk["extra"]) else wk["extra"]

    # ---- end to end: gradients start in pinned host memory, new parameters are read back
    flat = not cfg.segments and not cfg.name.startswith("c4")
    if args.no_e2e or args.ema or args.deadline is not None or not flat or cfg.W * cfg.P * (4 if cfg.grad_dtype == "f32" else 2) > 16e9:
        return finish(args, cfg, wk, extra, dist, dev, rank, world, ms_total, None, 0, clocks)
    W, N, b, P = cfg.W, cfg.N, cfg.b, cfg.P
    st = wk["state"]
    grad, theta, s0, s1, opt = st["grad"], st["theta"], st["s0"], st["s1"], st["opt"]
    e2e_steps = max(1, min(args.steps, 3))
    ws = torch.empty(sgdb.sgdb_step_host_workspace_bytes(grad.dtype, P, P, N, b), dtype=torch.uint8, device=dev)
    h_grad = torch.empty((W, P), dtype=grad.dtype, pin_memory=True)
    h_grad.copy_(grad)
    del grad, st["grad"]
    h_theta = torch.empty(P, dtype=torch.float32, pin_memory=True)
    h_mask = torch.empty(W, dtype=torch.uint8, pin_memory=True)
    h_order = torch.empty(N, dtype=torch.int32, pin_memory=True)
    h_info = torch.empty(2, dtype=torch.int32, pin_memory=True)
    h_arr = [torch.from_numpy(wl.arrivals(cfg.seed, t, W)).pin_memory() for t in range(N_SETS)]
    h_tag = [torch.from_numpy(wl.tags(cfg.seed, t, W, N) - t).pin_memory() for t in range(N_SETS)]

    def host_step(i):
        opt.step = i + 1
        status = sgdb.sgdb_step_host(h_grad, P, h_arr[i % N_SETS], h_tag[i % N_SETS], 0, N, b, theta, s0, s1, opt,
                                     h_theta, h_mask, h_order, h_info, ws)
        assert status == 0

    host_step(0)
    barrier()
    e_start, e_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e_start.record()
    for i in range(e2e_steps):
        host_step(1 + i)
    e_stop.record()
    barrier()
    e2e_ms = e_start.elapsed_time(e_stop)
    return finish(args, cfg, wk, extra, dist, dev, rank, world, ms_total, e2e_ms, e2e_steps, clocks)


def finish(args, cfg, wk, extra, dist, dev, rank, world, ms_total, e2e_ms, e2e_steps, clocks):
    W, N, b = cfg.W, cfg.N, cfg.b
    P = wk.get("P", cfg.P)
    grad_bytes, total_bytes = wk["grad_bytes"], wk["total_bytes"]
    esize = 4 if cfg.grad_dtype == "f32" else 2
    ms_total, e2e_max = max_over_ranks(dist, [ms_total, e2e_ms or 0.0], dev)
    e2e_ms = e2e_max if e2e_ms is not None else None
    ms_per_step = ms_total / args.steps
    value = whole_job_rate(world, grad_bytes, ms_per_step)
    total_gbs_per_gpu = total_bytes / (ms_per_step * 1e-3) / 1e9
    e2e = None
    if e2e_ms is not None:
        e2e = {"value": whole_job_rate(world, grad_bytes, e2e_ms / e2e_steps), "unit": UNIT,
               "h2d_bytes_per_step": N * P * esize + W * 8, "d2h_bytes_per_step": P * 4 + W + N * 4 + 16,
               "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps}

    if rank == 0:
        peak, peak_kind = measured_hbm_peak()
        digest = kernel_source_digest()
        traffic = None
        if (cfg.name == "c1_inception_rmsprop" and not args.ema and args.deadline is None and NCU_TRAFFIC["src_digest"] == digest
                and NCU_TRAFFIC["dram_bytes_per_algorithmic_byte"] is not None):
            traffic = NCU_TRAFFIC["dram_bytes_per_algorithmic_byte"] * total_bytes
        cpu = None
        if world == 1 and not args.no_cpu_baseline and cfg.name.startswith("c1"):
            P_sample = P // 4
            sec, gbs = oracle_sample_run(cfg, P_sample, steps=25, warmup=1)
            cpu = {"value": gbs, "unit": UNIT, "cores": 1, "kind": "oracle",
                   "sample": "first %d of %d columns (1/4), all %d rows, 25 steps of %.2f s, single thread"
                             % (P_sample, P, W, sec)}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": cfg.name, "P": P, "W": W, "N": N, "b": b, "optimizer": cfg.opt["kind"],
                       "grad_dtype": cfg.grad_dtype, "sharding": "one parameter-server column shard of P per GPU",
                       "l2": ("inputs larger than L2 (126 MB): %.3f GB of gradient rows and %.1f MB of parameters and "
                              "state per step" % (grad_bytes / 1e9, (total_bytes - grad_bytes) / 2e6))
                             if total_bytes > 4 * 126e6 else
                             "inputs fit in L2 (%.0f KB per step): a launch-bound workload, read its step time only"
                             % (total_bytes / 1e3)},
            "step_us": ms_per_step * 1e3,
            "total_gbs_per_gpu": total_gbs_per_gpu,
            "pct_of_nominal_8tbs": 100.0 * total_gbs_per_gpu / NOMINAL_HBM_GBS,
            "roofline": {"bound": "hbm", "achieved": total_gbs_per_gpu, "peak": peak, "unit": "GB/s",
                         "frac": total_gbs_per_gpu / peak, "traffic": traffic, "peak_source": peak_kind,
                         "kernel": wk["kernel"], "algorithmic_bytes_per_step": total_bytes},
            "e2e": e2e,
            "gpu_launches": wk["launches_per_step"] * args.steps,
            "clocks": clocks.summary(),
            "cpu_baseline": cpu,
        }
        if extra:
            line["extra"] = extra
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["native", "reference"], default="native")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing leg")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--workload", choices=["c0", "c1", "c2", "c3", "c4"], default="c1",
                    help="c1 (default) is the benchmark workload; the others time the remaining seeded workloads")
    ap.add_argument("--ema", action="store_true",
                    help="flat workloads: also keep the exponential moving average of the parameters (sgdb_step_ema)")
    ap.add_argument("--deadline", type=float, default=None,
                    help="flat workloads: time-out rule (sgdb_step_deadline) with this deadline in seconds")
    ap.add_argument("--columns", type=int, default=0,
                    help="override P with a smaller column count (profiler captures); not the benchmark workload")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "native":
        args.warmup = 3
    cfg = wl.CONFIGS[{"c0": 0, "c1": 1, "c2": 2, "c3": 3, "c4": 4}[args.workload]]
    if args.columns > 0:
        import dataclasses

        cfg = dataclasses.replace(cfg, P=args.columns, name=cfg.name + "_columns_%d" % args.columns)
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_native(args, cfg)


if __name__ == "__main__":
    main()

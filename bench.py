#!/usr/bin/env python
"""Benchmark of the fused N-of-(N+b) aggregate + update step (sgdb_step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl native|reference]

A step is one pass of the whole path over one batch of synthetic input: select the first N of the
N+b gradients, average them, apply RMSProp with momentum.  The headline workload is the
Inception-v3-sized one: P = 23.8 M fp32 parameters, W = 100 (N = 96, b = 4).  Prints one JSON line.

value     gradient bytes read per second (N * P * 4 per step), inputs resident in HBM
e2e       the same metric through sgdb_step_host: gradients, arrival times and tags start in pinned
          host memory, the updated parameters are read back, all inside the timed region
roofline  algorithmic bytes of a step (gradient rows + parameters and state read and written) over
          the measured step time, against the measured HBM copy bandwidth of this machine
extra     (one GPU, default workload) the spread of single-step times, a sustained run of at least
          two seconds with the clocks seen, the same step as three separate calls, its variants (with
          the parameter average, with the time-out rule, two-level), and the other four seeded
          workloads: tiny SGD, 300-tensor segmented, bf16 rows + Adam, arrival by arrival
With --gpus N > 1 (under torchrun) every rank is one parameter-server shard holding its own P
columns; there is no data-path collective, and the value is the sum over ranks over the slowest rank.
--impl reference times the CPU oracle on the same workload (all host cores, column ranges split
over threads; the single-thread figure beside it).
"""
from __future__ import annotations

import argparse
import gc
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

# DRAM traffic of one full-size fused-step launch in steady state from an ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum, caches left alone), as bytes per algorithmic byte; valid only for the kernel sources whose
# digest is recorded with it.
NCU_TRAFFIC = {"src_digest": "26cc691490d24e95", "dram_bytes_per_algorithmic_byte": 0.9891}


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
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap,power.draw")

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
        sm, smax, power, reasons = [], [], [], set()
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
            try:
                power.append(float(parts[6]))
            except (IndexError, ValueError):
                pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        out = {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(smax)), "reasons": sorted(reasons),
               "samples": len(sm)}
        if power:
            out["power_w_max"] = float(max(power))
        return out


# ====================================================================== the CPU oracle as a baseline


def cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def host_cores() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def column_ranges(P: int, parts: int):
    """[c0, c1) ranges that split P columns into `parts` nearly equal contiguous pieces (empty ones left out)."""
    edges = [P * k // parts for k in range(parts + 1)]
    return [(edges[k], edges[k + 1]) for k in range(parts) if edges[k + 1] > edges[k]]


def _oracle_kind(cfg):
    import oracle

    return {"sgd": oracle.SGD, "momentum": oracle.MOMENTUM, "rmsprop": oracle.RMSPROP, "adam": oracle.ADAM,
            "adagrad": oracle.ADAGRAD}[cfg.opt["kind"]]


def oracle_run(cfg, grad: np.ndarray, P_used: int, steps: int, warmup: int, threads: int):
    """Times the CPU oracle, as it stands, on the first P_used columns of `grad` ([W, ld] host array).

    threads == 1: one call of the oracle's step per iteration.  threads > 1: the column range is split into
    contiguous pieces and each piece is one call of the same, unchanged oracle step from its own Python
    thread (the foreign call releases the interpreter lock); every piece redoes the selection, as every
    parameter-server shard would.  Returns (seconds per step, gradient GB/s)."""
    import oracle
    from concurrent.futures import ThreadPoolExecutor

    W, N = cfg.W, cfg.N
    ld = grad.shape[1]
    flat = grad.reshape(-1)
    theta = np.random.default_rng(cfg.seed).standard_normal(P_used)
    s0, s1 = np.zeros(P_used), np.zeros(P_used)
    hyper = {k: float(np.float32(v)) for k, v in cfg.opt.items() if k != "kind"}
    kind = _oracle_kind(cfg)
    pieces = column_ranges(P_used, threads)

    def piece(c0, c1, t, arrival, tags):
        rc, *_ = oracle.step(flat[c0:], c1 - c0, arrival, tags, t, N, cfg.b, theta[c0:c1], s0[c0:c1], s1[c0:c1],
                             oracle.Opt(kind=kind, step=t + 1, **hyper), ld=ld)
        return rc

    times = []
    with ThreadPoolExecutor(max_workers=len(pieces)) as pool:
        for t in range(warmup + steps):
            arrival, tags = wl.arrivals(cfg.seed, t, W), wl.tags(cfg.seed, t, W, N)
            t0 = time.perf_counter()
            if len(pieces) == 1:
                rcs = [piece(0, P_used, t, arrival, tags)]
            else:
                rcs = list(pool.map(lambda r: piece(r[0], r[1], t, arrival, tags), pieces))
            dt = time.perf_counter() - t0
            assert all(rc == oracle.OK for rc in rcs)
            if t >= warmup:
                times.append(dt)
    sec = float(np.mean(times))
    esize = grad.dtype.itemsize
    return sec, N * P_used * esize / sec / 1e9


def cpu_baseline(cfg, grad: np.ndarray, P: int, all_steps: int, single_steps: int, warmup: int = 1):
    """The oracle on all host cores over the first P columns, and on one core over the first quarter of them."""
    cores = host_cores()
    sec_all, gbs_all = oracle_run(cfg, grad, P, all_steps, warmup, cores)
    P_single = max(1, P // 4)
    sec_one, gbs_one = oracle_run(cfg, grad, P_single, single_steps, warmup, 1)
    full = P == cfg.P
    return {
        "value": gbs_all, "unit": UNIT, "cores": cores, "kind": "oracle", "nproc": os.cpu_count(),
        "cpu_model": cpu_model(), "ms_per_step": sec_all * 1e3, "full_P": full,
        "sample": "%s %d columns, all %d rows, %d steps of %.2f s, %d threads each on its own column range"
                  % ("all" if full else "first", P, cfg.W, all_steps, sec_all, cores),
        "single_thread": {"value": gbs_one, "unit": UNIT, "cores": 1, "ms_per_step": sec_one * 1e3,
                          "sample": "first %d of %d columns (1/4), all %d rows, %d steps of %.2f s"
                                    % (P_single, cfg.P, cfg.W, single_steps, sec_one)},
    }


def workload_config(cfg, P, grad_bytes, total_bytes):
    """The `config` object of the JSON line; both arms print the same one."""
    return {"workload": cfg.name, "P": P, "W": cfg.W, "N": cfg.N, "b": cfg.b, "optimizer": cfg.opt["kind"],
            "grad_dtype": cfg.grad_dtype, "sharding": "one parameter-server column shard of P per GPU",
            "l2": ("inputs larger than L2 (126 MB): %.3f GB of gradient rows and %.1f MB of parameters and "
                   "state per step" % (grad_bytes / 1e9, (total_bytes - grad_bytes) / 2e6))
                  if total_bytes > 4 * 126e6 else
                  "inputs fit in L2 (%.0f KB per step): a launch-bound workload, read its step time only"
                  % (total_bytes / 1e3)}


def flat_bytes(cfg, P):
    esize = 4 if cfg.grad_dtype == "f32" else 2
    grad_bytes = cfg.N * P * esize
    return grad_bytes, grad_bytes + 2 * (1 + N_STATE[cfg.opt["kind"]]) * P * 4


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    P = cfg.P
    grad = wl.as_oracle_array(wl.grad_matrix(cfg.seed, 0, cfg.W, P, wl.worker_scales(cfg.seed, cfg.W), cfg.grad_dtype, "cpu"))
    cores = host_cores()
    sec, gbs = oracle_run(cfg, grad, P, args.steps, args.warmup, cores)
    sec_one, gbs_one = oracle_run(cfg, grad, max(1, P // 4), max(1, min(args.steps, 3)), min(args.warmup, 1), 1)
    grad_bytes, total_bytes = flat_bytes(cfg, P)
    sample = "all %d columns, all %d rows, %d steps, %d threads each on its own column range" % (P, cfg.W, args.steps, cores)
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg, P, grad_bytes, total_bytes),
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": cores, "kind": "oracle", "nproc": os.cpu_count(),
                         "cpu_model": cpu_model(), "full_P": True, "sample": sample,
                         "single_thread": {"value": gbs_one, "unit": UNIT, "cores": 1, "ms_per_step": sec_one * 1e3,
                                           "sample": "first %d of %d columns (1/4)" % (max(1, P // 4), P)}},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ====================================================================== the five workloads on the GPU

N_STATE = {"sgd": 0, "momentum": 1, "rmsprop": 2, "adam": 2, "adagrad": 1}
N_SETS = 16  # arrival/tag draws rotate, so the kept set differs from step to step


def it(i: int) -> int:
    """The iteration number a step passes to the library: 0, 1, 0, 1, ...  Consecutive iterations differ in
    parity, as the iterations of a real server do (the kernels walk through the columns in alternating directions),
    and draw i % N_SETS carries the tags of iteration it(i) (N_SETS is even)."""
    return i & 1


def selection_sets(cfg, dev):
    arr = [torch.from_numpy(wl.arrivals(cfg.seed, t, cfg.W)).to(dev) for t in range(N_SETS)]
    tag = [torch.from_numpy(wl.tags(cfg.seed, t, cfg.W, cfg.N) - t + it(t)).to(dev) for t in range(N_SETS)]
    return arr, tag


def selection_outputs(W, N, dev):
    return (torch.zeros(W, dtype=torch.uint8, device=dev), torch.zeros(N, dtype=torch.int32, device=dev),
            torch.zeros(2, dtype=torch.int32, device=dev))


def time_steps(step, steps, warmup):
    """Mean milliseconds per step over `steps` steps between one pair of CUDA events."""
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


def time_each_step(step, steps, warmup):
    """Milliseconds of every single step: an event before the first step and one after each."""
    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    marks[0].record()
    for i in range(steps):
        step(warmup + i)
        marks[i + 1].record()
    torch.cuda.synchronize()
    return [marks[i].elapsed_time(marks[i + 1]) for i in range(steps)]


def spread(ms_list):
    a = np.asarray(ms_list, dtype=np.float64)
    return {"steps": int(a.size), "min_ms": float(a.min()), "median_ms": float(np.median(a)),
            "p95_ms": float(np.percentile(a, 95)), "max_ms": float(a.max())}


def rates(total_bytes, grad_bytes, ms):
    """Throughput figures of one step time against the measured and the nominal HBM peak."""
    peak, kind = measured_hbm_peak()
    total = total_bytes / (ms * 1e-3) / 1e9
    return {"step_us": ms * 1e3, "gradient_gbs": grad_bytes / (ms * 1e-3) / 1e9, "total_gbs": total,
            "frac_of_%s_peak" % kind: total / peak, "pct_of_nominal_8tbs": 100.0 * total / NOMINAL_HBM_GBS,
            "algorithmic_bytes_per_step": total_bytes}


def setup_flat(cfg, dev, sgdb, seed, ema=False, deadline=None, machines=0):
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

    if machines:  # two-level: worker w runs on machine w * machines // W; as many machines are kept as hold N workers
        group = torch.from_numpy((np.arange(W) * machines // W).astype(np.int32)).to(dev)
        n_machines = max(1, N * machines // W)
        group_order = torch.zeros(n_machines, dtype=torch.int32, device=dev)
        order = torch.zeros(W, dtype=torch.int32, device=dev)
        info = torch.zeros(3, dtype=torch.int32, device=dev)
        tag_d = [torch.full((W,), it(k), dtype=torch.int32, device=dev) for k in range(N_SETS)]  # every worker current
        kept_mean = n_machines * W / machines  # exact when the machines are equally large

    def step(i):
        opt.step = i + 1
        if machines:
            sgdb.sgdb_step_grouped(grad, P, arr_d[i % N_SETS], tag_d[i % N_SETS], group, it(i), machines, n_machines, theta, s0,
                                   s1, opt, mask, group_order, order, info)
        elif deadline is not None:
            sgdb.sgdb_step_deadline(grad, P, arr_d[i % N_SETS], tag_d[i % N_SETS], it(i), deadline, 1, theta, s0, s1, opt,
                                    mask, order, info)
        elif ema:  # the step plus the running average of the parameters (last line of the server's loop)
            sgdb.sgdb_step_ema(grad, P, arr_d[i % N_SETS], tag_d[i % N_SETS], it(i), N, b, theta, s0, s1, opt, avg, 0.9999,
                               mask, order, info)
        else:
            sgdb.sgdb_step(grad, P, arr_d[i % N_SETS], tag_d[i % N_SETS], it(i), N, b, theta, s0, s1, opt, mask, order, info)

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
            sgdb.sgdb_select(arr_d[i % N_SETS], tag_d[i % N_SETS], it(i), N, b, mask, order, info)
            sgdb.sgdb_aggregate(grad, P, N, order, info, mean)
            sgdb.sgdb_update(theta, s0, s1, mean, opt, info)

        ms = time_steps(separate_step, 10, 3)
        moved = grad_bytes + 2 * (1 + n_state) * P * 4 + 2 * P * 4  # the mean is written and read back
        return {"separate_calls_ms_per_step": ms, "separate_calls_total_gbs": moved / (ms * 1e-3) / 1e9,
                "separate_calls_launches_per_step": 3}

    def variants():
        """The other forms of the fused step on the same matrix: with the parameter average, with the time-out
        rule, and two-level (workers on machines of 4).  Each 20 steps after 3 warm-up steps."""
        esize = grad.element_size()
        state_bytes = 2 * (1 + n_state) * P * 4
        out = {}
        avg_v = theta.clone()

        def ema_step(i):
            opt.step = i + 1
            sgdb.sgdb_step_ema(grad, P, arr_d[i % N_SETS], tag_d[i % N_SETS], it(i), N, b, theta, s0, s1, opt, avg_v, 0.9999,
                               mask, order, info)

        ms = time_steps(ema_step, 20, 3)
        out["parameter_average"] = rates(N * P * esize + state_bytes + 2 * P * 4, N * P * esize, ms)
        del avg_v
        dl = 1.6
        order_w = torch.zeros(W, dtype=torch.int32, device=dev)
        kept = float(np.mean([int(((wl.arrivals(cfg.seed, t, W) <= np.float32(dl)) & (wl.tags(cfg.seed, t, W, N) == t)).sum())
                              for t in range(N_SETS)]))

        def deadline_step(i):
            opt.step = i + 1
            sgdb.sgdb_step_deadline(grad, P, arr_d[i % N_SETS], tag_d[i % N_SETS], it(i), dl, 1, theta, s0, s1, opt, mask,
                                    order_w, info)

        ms = time_steps(deadline_step, 20 - 20 % N_SETS + N_SETS, 3)  # whole rotations of the draws: the kept count varies
        out["deadline_1.6s"] = dict(rates(int(kept * P * esize) + state_bytes, int(kept * P * esize), ms), mean_rows_kept=kept)
        if W % 4 == 0:
            m_all = W // 4
            m_kept = N // 4
            group = torch.from_numpy((np.arange(W) // 4).astype(np.int32)).to(dev)
            group_order = torch.zeros(m_kept, dtype=torch.int32, device=dev)
            info3 = torch.zeros(3, dtype=torch.int32, device=dev)
            current = [torch.full((W,), par, dtype=torch.int32, device=dev) for par in (0, 1)]

            def grouped_step(i):
                opt.step = i + 1
                sgdb.sgdb_step_grouped(grad, P, arr_d[i % N_SETS], current[it(i)], group, it(i), m_all, m_kept, theta, s0, s1, opt,
                                       mask, group_order, order_w, info3)

            ms = time_steps(grouped_step, 20, 3)
            assert info3.cpu().tolist() == [m_all, 0, 4 * m_kept]
            out["two_level"] = dict(rates(4 * m_kept * P * esize + state_bytes, 4 * m_kept * P * esize, ms),
                                    machines=m_all, machines_kept=m_kept, rows_used=4 * m_kept)
        # the step as parameter servers run it (rows given by address): one server owning every column, then
        # eight servers over eight ranges, each pushing its new parameters into the seven other copies of theta --
        # the launches of an 8-GPU job, run one after another on this one GPU
        rows_all = sgdb.make_address_table([grad[w].data_ptr() for w in range(W)], dev)

        def rows_step(i):
            opt.step = i + 1
            sgdb.sgdb_step_rows(rows_all, grad.dtype, P, arr_d[i % N_SETS], tag_d[i % N_SETS], it(i), N, b, theta, s0, s1, opt, None,
                                mask, order, info)

        ms = time_steps(rows_step, 20, 3)
        out["rows_by_address"] = rates(N * P * esize + state_bytes, N * P * esize, ms)
        G = 8
        free, _ = torch.cuda.mem_get_info(dev)
        if free > (G + 2) * P * 4 + (1 << 30):
            copies = [theta] + [theta.clone() for _ in range(G - 1)]
            ranges = [sgdb.sgdb_shard_range(P, G, j) for j in range(G)]
            row_tables = [sgdb.make_address_table([grad[w].data_ptr() + first * esize for w in range(W)], dev)
                          for first, _ in ranges]
            push_tables = [sgdb.make_address_table([copies[g].data_ptr() + first * 4 for g in range(G) if g != j], dev)
                           for j, (first, _) in enumerate(ranges)]
            cut = lambda x, first, n: None if x is None else x[first:first + n]

            def servers_step(i):
                opt.step = i + 1
                for j, (first, n) in enumerate(ranges):
                    sgdb.sgdb_step_rows(row_tables[j], grad.dtype, n, arr_d[i % N_SETS], tag_d[i % N_SETS], it(i), N, b,
                                        cut(copies[j], first, n), cut(s0, first, n), cut(s1, first, n), opt, push_tables[j],
                                        mask, order, info)

            ms = time_steps(servers_step, 20, 3)
            assert all(torch.equal(c, copies[0]) for c in copies[1:]), "the copies of theta differ"
            pushed = (G - 1) * P * 4
            out["eight_servers_on_one_gpu"] = dict(rates(N * P * esize + state_bytes + pushed, N * P * esize, ms), servers=G,
                                                   launches_per_step=G, pushed_bytes_per_step=pushed)
            # the same eight GPUs with two-level aggregation: each machine first writes the mean of its own workers'
            # rows (all eight do, none knows yet whether its message will be used), then every server takes the
            # first seven messages as rows; 32 small launches per step on this one GPU
            M, m_kept, per = G, G - 1, -(-W // G)
            bounds = [(min(W, m * per), min(W, (m + 1) * per)) for m in range(M)]
            if all(hi > lo for lo, hi in bounds) and free > (2 * G + 2) * P * 4 + (1 << 30):
                messages = torch.empty((M, P), device=dev)
                message_tables = [sgdb.make_address_table([messages[m].data_ptr() + first * 4 for m in range(M)], dev)
                                  for first, _ in ranges]
                group = torch.from_numpy(np.repeat(np.arange(M), per)[:W].astype(np.int32)).to(dev)
                current = torch.zeros(W, dtype=torch.int32, device=dev)
                l_mask = torch.zeros(per, dtype=torch.uint8, device=dev)
                l_order = torch.zeros(per, dtype=torch.int32, device=dev)
                l_info = torch.zeros(2, dtype=torch.int32, device=dev)
                g_order = torch.zeros(m_kept, dtype=torch.int32, device=dev)
                g_info = torch.zeros(3, dtype=torch.int32, device=dev)

                def machines_step(i):
                    opt.step = i + 1
                    arr = arr_d[i % N_SETS]
                    for m, (lo, hi) in enumerate(bounds):
                        sgdb.sgdb_select(arr[lo:hi], current[lo:hi], 0, hi - lo, 0, l_mask, l_order, l_info)
                        sgdb.sgdb_aggregate(grad[lo:hi], P, hi - lo, l_order, l_info, messages[m])
                    for j, (first, n) in enumerate(ranges):
                        sgdb.sgdb_select_grouped(arr, current, group, 0, M, m_kept, mask, g_order, order_w, g_info)
                        sgdb.sgdb_step_rows_ordered(message_tables[j], torch.float32, n, m_kept, g_order, g_info,
                                                    cut(copies[j], first, n), cut(s0, first, n), cut(s1, first, n), opt,
                                                    push_tables[j])

                ms = time_steps(machines_step, 20, 3)
                assert g_info.cpu().tolist()[:2] == [M, 0]
                assert all(torch.equal(c, copies[0]) for c in copies[1:]), "the copies of theta differ"
                moved = W * P * esize + M * P * 4 + m_kept * P * 4 + state_bytes + pushed
                out["eight_machines_two_level_on_one_gpu"] = dict(
                    rates(moved, W * P * esize, ms), machines=M, machines_kept=m_kept, launches_per_step=4 * G,
                    rows_crossing_between_gpus_per_step=m_kept, pushed_bytes_per_step=pushed)
                del messages, message_tables
            del copies, row_tables, push_tables
        assert info.cpu().tolist()[1] == 0 and bool(torch.isfinite(theta).all())
        return out

    grad_bytes = int(kept_mean * P * grad.element_size())
    state = dict(grad=grad, theta=theta, s0=s0, s1=s1, opt=opt)
    total = grad_bytes + 2 * (1 + n_state) * P * 4 + (2 * P * 4 if ema else 0)
    return dict(step=step, check=check, grad_bytes=grad_bytes, total_bytes=total,
                launches_per_step=1, variants=variants,
                kernel="stream_rows_kernel<%s, %s>%s (the step is this one launch)"
                % (cfg.grad_dtype, cfg.opt["kind"], " + parameter average" if ema else
                   (", two-level: %d machines, %d kept" % (machines, n_machines) if machines else "")), state=state,
                extra={"parameter_average": True} if ema else {"machines": machines, "machines_kept": n_machines,
                                                               "rows_used": kept_mean} if machines else
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
        sgdb.sgdb_step_segmented(table, len(segs), segs[0][3].dtype, arr_d[i % N_SETS], tag_d[i % N_SETS], it(i), N, b,
                                 opt, mask, order, info)

    def per_tensor_step(i):
        opt.step = i + 1
        for theta, s0, s1, grad in segs:
            sgdb.sgdb_step(grad, theta.numel(), arr_d[i % N_SETS], tag_d[i % N_SETS], it(i), N, b, theta, s0, s1, opt,
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

    esize = grad.element_size()
    grad_bytes = N * P * esize
    # first accepted row: read row, write acc; middle rows: read row + acc, write acc; N-th: read row + acc + theta
    # + state, write theta + state
    total = grad_bytes + (N - 1) * P * 4 + (N - 1) * P * 4 + 2 * (1 + n_state) * P * 4

    def extra():
        out = {}
        for bb in (0, 2, 4, 8):
            ms = time_steps(make_step(bb), 5, 2)
            out["b=%d" % bb] = {"ms_per_iteration": ms, "calls_per_iteration": N + bb, "us_per_call": 1e3 * ms / (N + bb),
                                "us_per_accepted_arrival": 1e3 * ms / N,
                                "total_gbs": total / (ms * 1e-3) / 1e9}
        # the batched fused step on the same rows, for comparison
        mask, order, finfo = selection_outputs(N + 4, N, dev)
        arr = torch.from_numpy(wl.arrivals(cfg.seed + 4, 0, N + 4)).to(dev)
        tag = [torch.full((N + 4,), par, dtype=torch.int32, device=dev) for par in (0, 1)]

        def batched(i):
            opt.step = i + 1
            sgdb.sgdb_step(grad[: N + 4], P, arr, tag[it(i)], it(i), N, 4, theta, s0, s1, opt, mask, order, finfo)

        ms = time_steps(batched, 10, 3)
        return {"b_sweep": out, "bytes_per_accepted_arrival": P * 12, "batched_fused_step_ms": ms,
                "batched_fused_step_total_gbs": (grad_bytes + 2 * (1 + n_state) * P * 4) / (ms * 1e-3) / 1e9}

    return dict(step=make_step(cfg.b), check=check, grad_bytes=grad_bytes, total_bytes=total,
                launches_per_step=N + cfg.b, kernel="accumulate_arrival_kernel<%s, %s>, %d launches per step"
                % (cfg.grad_dtype, cfg.opt["kind"], N + cfg.b), state=dict(grad=grad), extra=extra)


def setup_workload(cfg, dev, sgdb, seed, ema=False, deadline=None, machines=0):
    if cfg.segments:
        return setup_segmented(cfg, dev, sgdb, seed)
    if cfg.name.startswith("c4"):
        return setup_arrivals(cfg, dev, sgdb, seed)
    return setup_flat(cfg, dev, sgdb, seed, ema=ema, deadline=deadline, machines=machines)


def other_workload(index, dev, sgdb, steps, warmup):
    """One of the other seeded workloads, timed on its own: its step time and rates plus the comparison it names."""
    cfg = wl.CONFIGS[index]
    wk = setup_workload(cfg, dev, sgdb, cfg.seed)
    ms = time_each_step(wk["step"], steps, warmup) if index != 0 else [time_steps(wk["step"], steps, warmup)]
    wk["check"]()
    out = {"workload": cfg.name, "P": wk.get("P", cfg.P), "W": cfg.W, "N": cfg.N, "b": cfg.b,
           "optimizer": cfg.opt["kind"], "grad_dtype": cfg.grad_dtype, "kernel": wk["kernel"],
           "launches_per_step": wk["launches_per_step"]}
    out.update(rates(wk["total_bytes"], wk["grad_bytes"], float(np.median(ms))))
    if index == 0:  # 280 KB per step: everything sits in L2, only the time per call means something
        out = {k: v for k, v in out.items() if not (k.startswith("frac_of") or k.startswith("pct_of") or k.endswith("_gbs"))}
        out["per_call_us_from_python"] = out["step_us"]
    else:
        out["spread"] = spread(ms)
    extra = wk["extra"]() if callable(wk["extra"]) else wk["extra"]
    if extra:
        out.update(extra)
    return out


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


def release_device_memory():
    gc.collect()
    torch.cuda.empty_cache()


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
    wk = setup_workload(cfg, dev, sgdb, seed, ema=args.ema, deadline=args.deadline, machines=args.machines)
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
    extra = dict(extra) if extra else {}

    headline = (world == 1 and cfg.name == "c1_inception_rmsprop" and not args.ema and args.deadline is None
                and not args.machines)
    if headline and not args.only_headline:
        # ---- spread of single steps, then a sustained run: the server runs for hours, not for 30 ms
        each = time_each_step(step, args.spread_steps, 3)
        extra["per_step"] = spread(each)
        ms_guess = float(np.median(each))
        n_sustained = max(args.steps, int(np.ceil(args.sustain_seconds * 1e3 / ms_guess)))
        with ClockSampler(local_rank) as sustained_clocks:
            ms_sustained = time_steps(step, n_sustained, 3)
        sc = sustained_clocks.summary()
        sustained = {"steps": n_sustained, "seconds": ms_sustained * n_sustained * 1e-3, "ms_per_step": ms_sustained,
                     "clocks": sc}
        sustained.update({k: v for k, v in rates(wk["total_bytes"], wk["grad_bytes"], ms_sustained).items()
                          if k != "algorithmic_bytes_per_step"})
        if sc.get("sm_mhz"):
            sustained["step_us_times_sm_mhz"] = ms_sustained * 1e3 * sc["sm_mhz"]
        extra["sustained"] = sustained
        wk["check"]()
        extra["variants"] = wk["variants"]()

    # ---- end to end: gradients start in pinned host memory, new parameters are read back
    flat = not cfg.segments and not cfg.name.startswith("c4")
    e2e_ms, e2e_steps, h_grad = None, 0, None
    if not (args.no_e2e or args.ema or args.deadline is not None or args.machines or not flat
            or cfg.W * cfg.P * (4 if cfg.grad_dtype == "f32" else 2) > 16e9):
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
        h_tag = [torch.from_numpy(wl.tags(cfg.seed, t, W, N) - t + it(t)).pin_memory() for t in range(N_SETS)]

        def host_step(i):
            opt.step = i + 1
            status = sgdb.sgdb_step_host(h_grad, P, h_arr[i % N_SETS], h_tag[i % N_SETS], it(i), N, b, theta, s0, s1, opt,
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
        del ws

    # ---- the CPU oracle on this machine's host cores, on the very bytes the GPU consumed
    cpu = None
    if world == 1 and not args.no_cpu_baseline and cfg.name.startswith("c1"):
        if h_grad is None:
            h_grad = wk["state"]["grad"].cpu()
        cpu = cpu_baseline(cfg, wl.as_oracle_array(h_grad), cfg.P, all_steps=args.cpu_steps, single_steps=4)
    del h_grad

    # ---- the other four seeded workloads, one after the other (each frees its memory before the next)
    if headline and not args.only_headline:
        del wk["state"], step
        wk["step"] = wk["check"] = wk["extra"] = wk["variants"] = None
        release_device_memory()
        others = {}
        for index, name, steps in ((0, "c0", 200), (2, "c2", 20), (3, "c3", 10), (4, "c4", 5)):
            free, _ = torch.cuda.mem_get_info(dev)
            need = {0: 1e9, 2: 16e9, 3: 46e9, 4: 12e9}[index]
            if free < need:
                others[name] = {"skipped": "needs %.0f GB of free device memory, %.0f GB free" % (need / 1e9, free / 1e9)}
                continue
            others[name] = other_workload(index, dev, sgdb, steps, 3)
            release_device_memory()
        extra["workloads"] = others

    finish(args, cfg, wk, extra, dist, dev, rank, world, ms_total, e2e_ms, e2e_steps, clocks, cpu)


def run_servers(args, cfg):
    """The several-GPUs form, one process per parameter server (`--servers`): the workers' gradient rows are whole
    rows spread over the GPUs' memories, GPU j updates its range of columns in one launch that pulls the kept rows
    from wherever they live and pushes the new parameters into every GPU's copy.  P is the whole model whatever the
    number of GPUs (strong scaling); what bounds it beyond one GPU is the link, not HBM."""
    import torch.distributed as dist

    from paper_1604_00981_b200 import binding as sgdb
    from paper_1604_00981_b200 import servers

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29531")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    else:  # a group of one needs no device collective: nothing crosses, the fences have nobody to wait for
        dist.init_process_group("gloo", rank=0, world_size=1)
    W, N, b, P = cfg.W, cfg.N, cfg.b, cfg.P
    tdt = torch.float32 if cfg.grad_dtype == "f32" else torch.bfloat16
    srv = servers.ServerGroup(P, W, N, b, tdt, cfg.opt, dev)
    mine = srv.plan.workers_of(rank)
    scales = wl.worker_scales(cfg.seed, W)
    if len(mine):
        wl.grad_matrix(cfg.seed + 1000 * rank, 0, len(mine), P, scales[mine.start:mine.stop], cfg.grad_dtype, dev,
                       ld=srv.grads.stride(0), out=srv.grads[:len(mine)])
    srv.theta[:P] = wl.theta0(cfg.seed, P, dev)
    arr_d, tag_d = selection_sets(cfg, dev)

    def step(i):
        srv.step(it(i), arr_d[i % N_SETS], tag_d[i % N_SETS], update=i + 1)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

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
    ms_total = max_over_ranks(dist if world > 1 else None, [start.elapsed_time(stop)], dev)[0]
    assert srv.info[:2].cpu().tolist()[1] == 0 and bool(torch.isfinite(srv.theta).all())
    if rank == 0:
        esize = 4 if cfg.grad_dtype == "f32" else 2
        ms = ms_total / args.steps
        grad_bytes = N * P * esize
        first, n = srv.plan.ranges[0]
        # per GPU and step: its columns of the kept rows, theta and state of its range read and written, its range
        # stored into the other copies; of the rows, (G - 1) / G arrive over the link on average
        per_gpu = N * n * esize + 2 * (1 + N_STATE[cfg.opt["kind"]]) * n * 4 + (world - 1) * n * 4
        link = N * n * esize * (world - 1) / world
        hbm_peak, peak_kind = measured_hbm_peak()
        if world == 1:
            roof = {"bound": "hbm", "achieved": per_gpu / (ms * 1e-3) / 1e9, "peak": hbm_peak, "unit": "GB/s",
                    "peak_source": peak_kind}
        else:
            roof = {"bound": "nvlink", "achieved": link / (ms * 1e-3) / 1e9, "peak": 770.0, "unit": "GB/s",
                    "peak_source": "peer copy measured on this pool, per direction"}
        roof.update({"frac": roof["achieved"] / roof["peak"], "traffic": None,
                     "kernel": "stream_rows_kernel<%s, %s, rows by address>, one launch per GPU and step" % (cfg.grad_dtype, cfg.opt["kind"]),
                     "algorithmic_bytes_per_step": per_gpu, "link_bytes_per_step": link})
        config = workload_config(cfg, P, grad_bytes, grad_bytes + 2 * (1 + N_STATE[cfg.opt["kind"]]) * P * 4)
        config["sharding"] = ("%d parameter servers, one per GPU: columns split in %d ranges, workers' rows spread over the "
                              "GPUs, no collective (pull + push inside the one launch, fences between)" % (world, world))
        print(json.dumps({
            "metric": METRIC, "value": grad_bytes / (ms * 1e-3) / 1e9, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
            "dtype": cfg.grad_dtype, "data": "synthetic", "config": config, "step_us": ms * 1e3, "roofline": roof,
            "e2e": None, "gpu_launches": args.steps, "clocks": clocks.summary(), "cpu_baseline": None}), flush=True)
    dist.destroy_process_group()


def finish(args, cfg, wk, extra, dist, dev, rank, world, ms_total, e2e_ms, e2e_steps, clocks, cpu):
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
        if (cfg.name == "c1_inception_rmsprop" and not args.ema and args.deadline is None and not args.machines and NCU_TRAFFIC["src_digest"] == digest
                and NCU_TRAFFIC["dram_bytes_per_algorithmic_byte"] is not None):
            traffic = NCU_TRAFFIC["dram_bytes_per_algorithmic_byte"] * total_bytes
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": cfg.grad_dtype, "data": "synthetic",
            "config": workload_config(cfg, P, grad_bytes, total_bytes),
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
    ap.add_argument("--only-headline", action="store_true",
                    help="skip the spread, the sustained run and the other four workloads (profiling runs)")
    ap.add_argument("--workload", choices=["c0", "c1", "c2", "c3", "c4"], default="c1",
                    help="c1 (default) is the benchmark workload; the others time the remaining seeded workloads")
    ap.add_argument("--ema", action="store_true",
                    help="flat workloads: also keep the exponential moving average of the parameters (sgdb_step_ema)")
    ap.add_argument("--deadline", type=float, default=None,
                    help="flat workloads: time-out rule (sgdb_step_deadline) with this deadline in seconds")
    ap.add_argument("--machines", type=int, default=0,
                    help="flat workloads: two-level aggregation (sgdb_step_grouped) with the workers spread over this many machines")
    ap.add_argument("--servers", action="store_true",
                    help="flat workloads: one process per parameter server over the WHOLE model (rows pulled from and "
                         "parameters pushed to the other GPUs inside the one launch); default is one independent column "
                         "shard per GPU")
    ap.add_argument("--columns", type=int, default=0,
                    help="override P with a smaller column count (profiler captures); not the benchmark workload")
    ap.add_argument("--rows", type=int, default=0,
                    help="override N, the number of gradients used per step (profiler captures); not the benchmark workload")
    ap.add_argument("--spread-steps", type=int, default=200, help="single steps timed one by one for the spread")
    ap.add_argument("--sustain-seconds", type=float, default=2.0, help="length of the sustained run")
    ap.add_argument("--cpu-steps", type=int, default=5, help="steps of the all-cores oracle leg")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "native":
        args.warmup = 3
    cfg = wl.CONFIGS[{"c0": 0, "c1": 1, "c2": 2, "c3": 3, "c4": 4}[args.workload]]
    if args.columns > 0:
        import dataclasses

        cfg = dataclasses.replace(cfg, P=args.columns, name=cfg.name + "_columns_%d" % args.columns)
    if args.rows > 0:
        import dataclasses

        cfg = dataclasses.replace(cfg, N=args.rows, name=cfg.name + "_rows_%d" % args.rows)
    if args.impl == "reference":
        run_reference(args, cfg)
    elif args.servers:
        run_servers(args, cfg)
    else:
        run_native(args, cfg)


if __name__ == "__main__":
    main()

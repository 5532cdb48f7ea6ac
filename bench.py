#!/usr/bin/env python
"""Benchmark of the coded tree aggregation on B200.

A step is one cr_aggregate call (encode of every consumed node, masked decode at every level,
root recovery) on one batch of straggler masks over synthetic partition gradients that are already
resident in HBM.  The default workload is the large-gradient configuration (n=5, L=2, s=2,
d=2^24, 270 slots = 17.3 GB, exactly two stragglers per sibling group); `--workload` selects the
others.  Prints one JSON line (see README of the repo for the keys).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--impl reference]

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica on its own
GPU -- the path has no exchange step -- and rank 0 reports the sum of units over the slowest rank's
time.  `--impl reference` times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1902_01981_b200 import inputs  # noqa: E402

METRIC = "CR aggregation GB/s (fraction of HBM peak) and coded iterations/sec"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0

TRAFFIC_TABLE = os.path.join(ROOT, "profiles", "ncu_dram_traffic.txt")
KERNEL_SOURCES = [os.path.join(ROOT, "paper_1902_01981_b200", "csrc", f) for f in ("cr_kernels.cu", "cr_tc.cu")]


def kernel_source_digest() -> str:
    """Short digest of the kernel sources: a DRAM-traffic figure taken under ncu is quoted only for the
    very sources it was measured on."""
    import hashlib
    h = hashlib.sha256()
    for path in KERNEL_SOURCES:
        with open(path, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(workload: str, dtype: str, d: int, kernel: str):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of `kernel` on `workload`, from the table of
    ncu captures under profiles/ (one line per capture: workload, dtype, captured d, kernel as the library
    names it, DRAM bytes per launch at the captured d, digest of the kernel sources, summary file).  The
    captures are small cases; traffic grows in proportion to d, so the figure is scaled by d / captured d.
    None when there is no capture, when another kernel served the call, or when the kernel sources have
    changed since the capture."""
    try:
        rows = [ln.split("|") for ln in open(TRAFFIC_TABLE) if ln.strip() and not ln.startswith("#")]
    except OSError:
        return None
    digest = kernel_source_digest()
    for r in rows:
        r = [c.strip() for c in r]
        if len(r) >= 7 and r[0] == workload and r[1] == dtype and r[3] == kernel and r[5] == digest:
            return {"bytes": float(r[4]) * d / float(r[2]), "captured_d": int(r[2]), "summary": r[6],
                    "note": "ncu capture of a small case, scaled by d / captured d"}
    return None


def peak_hbm():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------- multi-rank plumbing

def combine_ranks(elapsed_s: float, units: float, world: int, dist=None, device=None):
    """Whole-job figure: total units of all ranks over the slowest rank's time."""
    if world == 1 or dist is None:
        return elapsed_s, units
    import torch
    t = torch.tensor([elapsed_s], dtype=torch.float64, device=device)
    u = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples while the timed region runs."""
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def wait_first_sample(self, limit_s: float = 3.0):
        """Blocks until nvidia-smi has written its first line (it takes a moment to start)."""
        t0 = time.time()
        while self.proc is not None and time.time() - t0 < limit_s:
            if os.path.getsize(self.file.name) > 0:
                return
            time.sleep(0.05)

    def stop(self, window=None):
        """Median SM clock and the throttle reasons seen; `window` = (t0, t1) in time.time() seconds
        keeps only the samples taken inside it (all samples if none fall inside)."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        import datetime
        rows = []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file.read().splitlines():
            cols = [c.strip() for c in line.split(",")]
            if len(cols) < 9:
                continue
            try:
                stamp = datetime.datetime.strptime(cols[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((stamp, float(cols[1]), float(cols[2]), float(cols[3]),
                             [n for n, v in zip(names, cols[5:9]) if v.lower().startswith("active")]))
            except ValueError:
                continue
        self.file.close()
        os.unlink(self.file.name)
        inside = [r for r in rows if window and window[0] <= r[0] <= window[1]]
        use = inside or rows
        if use:
            reasons = sorted({n for r in use for n in r[4]})
            out.update(sm_mhz=float(np.median([r[1] for r in use])), sm_max_mhz=float(max(r[2] for r in use)),
                       power_w=float(np.median([r[3] for r in use])), reasons=reasons, samples=len(use),
                       samples_in_timed_region=len(inside))
        return out


class L2Flush:
    """Pushes the workload's data out of L2 between timed steps: writes one 256 MB buffer (twice the L2),
    then reads a second one.  The read pass matters: after the write alone L2 is left full of dirty lines,
    and the timed launch that follows would pay for their write-back (it shows as DRAM write traffic
    inside a read-only kernel)."""

    def __init__(self, torch, device):
        self.torch = torch
        self.wbuf = torch.empty(256 << 20, dtype=torch.uint8, device=device)
        self.rbuf = torch.zeros(64 << 20, dtype=torch.int32, device=device)
        self.sink = torch.zeros((), dtype=torch.int64, device=device)

    def __call__(self, i: int):
        self.wbuf.fill_(i & 0xff)
        self.torch.sum(self.rbuf, (0,), out=self.sink)


# ----------------------------------------------------------------------------- CPU oracle legs

def oracle_sample(cfg, d_sample: int, steps: int, warmup: int, G=None, threads: int = 1):
    """Times the CPU oracle, as it stands, on `d_sample` columns of the workload (the array G
    [P, d_sample] if given, else freshly drawn ones).  With threads > 1 the columns are cut into chunks
    and the oracle's CR.Execute runs on the chunks side by side (a thread pool; NumPy releases the
    interpreter lock inside its array operations) -- the oracle's code is the same either way.
    Returns (seconds per step, algorithmic bytes per step, results of the last step, masks used)."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import cr_oracle as O
    from oracle import cr_setup
    code, local, _ = cr_setup.setup(cfg)
    batch = cfg.get("batch", 1)
    if G is None:
        G = inputs.partition_gradients(cfg["P"], d_sample, cfg["seed"], cfg.get("std", 1.0))
    masks = inputs.straggler_masks(cfg["n"], cfg["L"], cfg["s"], (steps + warmup) * batch, cfg["mask_seed"],
                                   cfg.get("exactly_s", False)).reshape(steps + warmup, batch, -1)
    m = len(local[0])
    threads = max(1, min(threads, d_sample // 1024))
    bounds = np.linspace(0, d_sample, 4 * threads + 1).astype(int) if threads > 1 else None
    chunks = [np.ascontiguousarray(G[:, a:b]) for a, b in zip(bounds[:-1], bounds[1:])] if threads > 1 else None
    pool = ThreadPoolExecutor(threads) if threads > 1 else None

    def execute_all(mk):
        if pool is None:
            return O.execute(code, local, G, mk)
        return np.concatenate(list(pool.map(lambda c: O.execute(code, local, c, mk), chunks)))

    times, nbytes, last = [], [], None
    for it in range(steps + warmup):
        t0 = time.perf_counter()
        last = [execute_all(masks[it, b]) for b in range(batch)]
        dt = time.perf_counter() - t0
        if it >= warmup:
            times.append(dt)
            union = set()
            for b in range(batch):
                union |= set(O.used_nodes(code, masks[it, b]))
            nbytes.append(4 * d_sample * (m * len(union) + batch))
    if pool is not None:
        pool.shutdown()
    return float(np.mean(times)), float(np.mean(nbytes)), last, masks[-1]


def calibrated_columns(cfg, steps: int, seconds: float, max_cols: int, threads: int = 1) -> int:
    """Largest power-of-two column count (>= 4096, <= max_cols) for which `steps` oracle steps take
    about `seconds` on `threads` threads, from one timed single-thread step on 4096 columns (taken as if
    the threads scaled perfectly: the sample then errs on the short side)."""
    sec, _, _, _ = oracle_sample(cfg, 4096, 1, 0)
    cols = 4096
    while cols * 2 <= max_cols and sec * (cols * 2 / 4096.0) * steps / threads <= seconds:
        cols *= 2
    return cols


def blas_threads() -> int:
    """Threads NumPy's BLAS uses for a matrix product (1 if that cannot be told)."""
    try:
        from threadpoolctl import threadpool_info
        return max([int(i.get("num_threads", 1)) for i in threadpool_info() if i.get("user_api") == "blas"] or [1])
    except Exception:
        return 1


def host_threads() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def run_reference(args, cfg):
    """The oracle as the reference arm: same metric and unit, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # bounded sample: calibrate the oracle on 4096 columns, then size the sample for about a minute
    cores = host_threads()
    d_sample = calibrated_columns(cfg, args.steps + args.warmup, 60.0, min(args.ref_columns, cfg["d"]), cores)
    sec, nbytes, _, _ = oracle_sample(cfg, d_sample, args.steps, args.warmup, threads=cores)
    value = nbytes / sec / 1e9
    sample = (f"first {d_sample} of {cfg['d']} columns, every step a fresh straggler pattern, NumPy fp64, "
              f"column chunks on {cores} threads")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(args.workload, cfg, None),
        "iterations_per_s": 1.0 / sec,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def oracle_regression_sample(workload, cfg, steps, warmup, seconds):
    """Times the oracle's gradient-descent step on a regression workload: per step the fp64 partial
    gradients of a bounded sample of the partitions (the definition, once per partition), CR.Execute over
    all of them under a fresh straggler pattern, and the model update.  The sample is sized from the first
    full gradient pass so that all steps take about `seconds`.
    Returns (seconds per step, algorithmic bytes per step, description of the sample)."""
    from oracle import cr_oracle as O
    from oracle import cr_setup
    code, local, _ = cr_setup.setup(cfg)
    n, L, s, P, d, rows = cfg["n"], cfg["L"], cfg["s"], cfg["P"], cfg["d"], cfg["rows"]
    logistic = cfg["kind"] == "logistic"
    if logistic:
        X, y, _ = inputs.logistic_partitions(P, rows, d, cfg["seed"], cfg["x_std"])
    else:
        X, y, _ = inputs.linreg_partitions(P, rows, d, cfg["seed"], cfg["x_std"], cfg["noise_std"])
    grad = O.partial_gradient_logistic if logistic else O.partial_gradient_linreg
    N, m = O.num_nodes(n, L), len(local[0])
    w = np.zeros(d, dtype=np.float32)
    total = steps + warmup
    masks = inputs.straggler_masks(n, L, s, total, cfg.get("mask_seed", 1))
    lr_eff = cfg["lr"] if workload == "cfg1" else cfg["lr"] / P
    t0 = time.perf_counter()
    G = np.stack([grad(X[p], y[p], w) for p in range(P)])
    per_partition = (time.perf_counter() - t0) / P
    sampled = int(min(P, max(1, seconds / total / per_partition)))
    times, nbytes = [], []
    for it in range(total):
        t0 = time.perf_counter()
        for p in range(sampled):
            q = (it * sampled + p) % P
            G[q] = grad(X[q], y[q], w)
        g = O.execute(code, local, G, masks[it])
        w = (w.astype(np.float64) - lr_eff * g).astype(np.float32)
        dt = time.perf_counter() - t0
        if it >= warmup:
            times.append(dt)
            # the workload's own count: every (node, slot) item reads its partition; scaled to the sample
            nbytes.append(4.0 * rows * d * N * m * sampled / P + 4.0 * d * (m * len(O.used_nodes(code, masks[it])) + 1))
    sample = (f"gradients of {sampled} of {P} partitions per step (each computed once, not once per slot), "
              f"aggregation of all {P}, {steps} steps, NumPy fp64")
    return float(np.mean(times)), float(np.mean(nbytes)), sample


def regression_workload_name(workload, cfg):
    return (f"{workload}: {'logistic' if cfg['kind'] == 'logistic' else 'linear'} regression n={cfg['n']} L={cfg['L']} "
            f"s={cfg['s']} P={cfg['P']} rows={cfg['rows']} d={cfg['d']}")


def run_reference_regression(args, cfg):
    """The oracle as the reference arm of a regression workload (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    sec, nbytes, sample = oracle_regression_sample(args.workload, cfg, args.steps, args.warmup, 60.0)
    value = nbytes / sec / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": regression_workload_name(args.workload, cfg)},
        "iterations_per_s": 1.0 / sec,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                         "sample": sample + "; the matrix products run on NumPy's BLAS threads (the count given), CR.Execute on one"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- our arm

def workload_config(name, cfg, extra):
    out = {"workload": f"{name}: n={cfg['n']} L={cfg['L']} s={cfg['s']} code={cfg['code']} P={cfg['P']} "
                       f"d={cfg['d']} batch={cfg.get('batch', 1)}",
           "l2": "inputs larger than L2 (no flush needed)" if cfg["d"] * 4 * cfg["P"] > 126e6 else "L2 flushed between steps (256 MB written, then 256 MB read)",
           "parallelism": "independent replicas (no exchange step)"}
    if extra:
        out.update(extra)
    return out


CODE_IDS = {"printed_3_1": "CR_CODE_PAPER_3_1", "cyclic": "CR_CODE_CYCLIC_RANDOM", "repetition": "CR_CODE_FRACTIONAL_REPETITION"}


class AggregateSetup:
    """An aggregation workload resident on one GPU: plan, slot buffer, output, straggler patterns."""

    def __init__(self, torch, B, cfg, dtype, dev, seed_offset=0, patterns=256):
        self.torch, self.B, self.cfg, self.dev = torch, B, cfg, dev
        self.is_int = dtype == "int32"
        self.plan = B.cr_plan_create(cfg["n"], cfg["L"], cfg["s"], cfg["P"], cfg["d"], code=getattr(B, CODE_IDS[cfg["code"]]),
                                     dtype=B.CR_I32 if self.is_int else B.CR_F32, seed=0, device=dev.index or 0)
        self.N, self.m, self.groups = B.cr_plan_num_nodes(self.plan), B.cr_plan_load(self.plan), B.cr_plan_num_groups(self.plan)
        self.d, self.batch = cfg["d"], cfg.get("batch", 1)
        self.tdtype = torch.int32 if self.is_int else torch.float32
        # synthetic inputs: one vector per partition on the host, replicated into the slots on the device
        if self.is_int:
            self.G_parts = inputs.integer_gradients(cfg["P"], self.d, cfg["seed"] + seed_offset, cfg.get("int_bound", 1 << 10))
        else:
            self.G_parts = inputs.partition_gradients(cfg["P"], self.d, cfg["seed"] + seed_offset, cfg.get("std", 1.0))
        part = torch.from_numpy(B.slot_partitions(self.plan).astype(np.int64).reshape(-1)).to(dev)
        parts_dev = torch.from_numpy(self.G_parts).to(dev)
        self.G_slots = torch.empty((self.N * self.m, self.d), dtype=self.tdtype, device=dev)
        step_rows = max(1, (1 << 30) // (4 * self.d))
        for r0 in range(0, self.N * self.m, step_rows):
            torch.index_select(parts_dev, 0, part[r0:r0 + step_rows], out=self.G_slots[r0:r0 + step_rows])
        del parts_dev
        self.out = torch.zeros((self.batch, self.d), dtype=self.tdtype, device=dev)
        self.total = patterns                       # distinct straggler patterns, cycled over the steps
        self.masks = inputs.straggler_masks(cfg["n"], cfg["L"], cfg["s"], self.total * self.batch, cfg["mask_seed"],
                                            cfg.get("exactly_s", False)).reshape(self.total, self.batch, self.groups)
        self.step_bytes = [B.cr_aggregate_bytes(self.plan, self.masks[i])[0] for i in range(self.total)]
        self.need_flush = self.d * 4 * cfg["P"] <= 126e6
        self.flush = L2Flush(torch, dev) if self.need_flush else None
        self.stream = torch.cuda.current_stream()

    def timed(self, flags, steps, warmup, ws=None, dist=None, first=0):
        """`steps` calls of cr_aggregate, a CUDA-event pair around each on the launching stream.
        Returns (seconds per step [steps], seconds of the whole region on the device, host window)."""
        torch, B = self.torch, self.B
        starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        stops = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        for i in range(warmup):
            B.cr_aggregate(self.plan, self.G_slots, self.masks[(first + i) % self.total], self.out, flags, ws, self.stream)
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()
        t0 = time.time()
        n0 = B.cr_plan_launch_count(self.plan)
        for i in range(steps):
            if self.flush is not None:
                self.flush(i)
            starts[i].record(self.stream)
            B.cr_aggregate(self.plan, self.G_slots, self.masks[(first + warmup + i) % self.total], self.out, flags, ws, self.stream)
            stops[i].record(self.stream)
        torch.cuda.synchronize()
        t1 = time.time()
        self.launches = B.cr_plan_launch_count(self.plan) - n0
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()
        per = np.array([a.elapsed_time(b) for a, b in zip(starts, stops)]) * 1e-3
        span = starts[0].elapsed_time(stops[-1]) * 1e-3
        return per, (span if self.flush is None else float(per.sum())), (t0, t1)

    def bytes_of(self, steps, warmup, first=0):
        return float(sum(self.step_bytes[(first + warmup + i) % self.total] for i in range(steps)))

    def host_cost_us(self, flags, calls=200):
        """Host time of one call with the stream idle (median over `calls`): the direct form, which expands
        the masks, and the form with a schedule made beforehand, given plain addresses."""
        torch, B = self.torch, self.B
        sched = B.cr_schedule_create(self.plan, self.masks[0], flags)
        g, o, st = self.G_slots.data_ptr(), self.out.data_ptr(), self.stream.cuda_stream
        direct, scheduled = [], []
        for i in range(calls):
            torch.cuda.synchronize()
            t0 = time.perf_counter_ns()
            B.cr_aggregate(self.plan, self.G_slots, self.masks[0], self.out, flags, None, self.stream)
            t1 = time.perf_counter_ns()
            torch.cuda.synchronize()
            t2 = time.perf_counter_ns()
            B.cr_aggregate_scheduled(self.plan, g, sched, o, (0, 0), st)
            t3 = time.perf_counter_ns()
            direct.append(t1 - t0)
            scheduled.append(t3 - t2)
        torch.cuda.synchronize()
        B.cr_schedule_destroy(sched)
        # what the binding itself costs: a call through ctypes that does nothing on the device
        trivial = []
        for i in range(calls):
            t0 = time.perf_counter_ns()
            B.cr_plan_launch_count(self.plan)
            trivial.append(time.perf_counter_ns() - t0)
        return {"cr_aggregate": float(np.median(direct)) * 1e-3, "cr_aggregate_scheduled": float(np.median(scheduled)) * 1e-3,
                "ctypes_call_that_launches_nothing": float(np.median(trivial)) * 1e-3,
                "note": "host clock around the call through the Python binding, stream idle, median of %d" % calls}

    def graph_replay_ms(self, flags, reps=100):
        """Device time of one scheduled call replayed as a CUDA graph (one fixed pattern): the launch-bound
        end of the table without the host in the loop."""
        torch, B = self.torch, self.B
        sched = B.cr_schedule_create(self.plan, self.masks[0], flags)
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                B.cr_aggregate_scheduled(self.plan, self.G_slots, sched, self.out, None, torch.cuda.current_stream())
            for _ in range(3):
                graph.replay()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            tt = []
            for i in range(reps):
                if self.flush is not None:
                    self.flush(i)
                a.record()
                graph.replay()
                b.record()
                torch.cuda.synchronize()
                tt.append(a.elapsed_time(b))
            return float(np.median(tt))
        finally:
            B.cr_schedule_destroy(sched)

    def parity_on_sample(self, cols, flags, patterns=2):
        """The GPU result on the first `cols` columns against the CPU oracle for the last straggler patterns:
        worst relative L2 error (fp32) or exact equality (int32)."""
        from oracle import cr_oracle as O
        from oracle import cr_setup
        torch, B = self.torch, self.B
        code, local, _ = cr_setup.setup(self.cfg)
        mk = self.masks[self.total - 1]
        B.cr_aggregate(self.plan, self.G_slots, mk, self.out, flags, None, self.stream)
        torch.cuda.synchronize()
        got = self.out[:, :cols].cpu().numpy()
        G = np.ascontiguousarray(self.G_parts[:, :cols])
        picks = sorted(set(np.linspace(0, self.batch - 1, min(patterns, self.batch)).astype(int).tolist()))
        if self.is_int:
            exact = G.astype(np.int64).sum(0)
            ok = all(np.array_equal(got[b].astype(np.int64), exact) and
                     np.array_equal(O.execute_integer(code, local, G, mk[b]), exact) for b in picks)
            return {"bit_exact_on_sample": bool(ok), "columns": cols, "patterns": len(picks)}
        worst = 0.0
        for b in picks:
            want = O.execute(code, local, G, mk[b])
            worst = max(worst, float(np.linalg.norm(got[b].astype(np.float64) - want) / np.linalg.norm(want)))
        return {"gpu_rel_l2_on_sample": worst, "columns": cols, "patterns": len(picks)}

    def close(self):
        self.B.cr_plan_destroy(self.plan)
        del self.G_slots, self.out, self.G_parts
        self.flush = None
        self.torch.cuda.empty_cache()


def other_aggregate(torch, B, dev, name, dtype, steps, overrides=None):
    """One more workload measured in the same process: value, time, kernel, parity against the oracle on a
    column sample.  Kept short; the headline region is not touched."""
    cfg = dict(inputs.CONFIGS[name])
    cfg.update(overrides or {})
    ws = AggregateSetup(torch, B, cfg, dtype, dev, patterns=min(64, steps + 3))
    try:
        per, wall, _ = ws.timed(B.CR_AGG_FUSED, steps, 3)
        kernel = B.cr_plan_last_kernel(ws.plan)
        nbytes = ws.bytes_of(steps, 3)
        assert B.cr_plan_device_status(ws.plan) == B.CR_OK, "a device-side wait timed out"
        peak, peak_kind = peak_hbm()
        value = nbytes / wall / 1e9
        out = {"workload": workload_config(name, cfg, None)["workload"], "dtype": "int32" if ws.is_int else "f32",
               "value": value, "unit": UNIT, "ms_per_step": wall / steps * 1e3, "median_launch_ms": float(np.median(per)) * 1e3,
               "steps": steps, "kernel": kernel,
               "algorithmic_bytes_per_step": nbytes / steps, "frac": value / peak, "peak_kind": f"of {peak_kind}",
               "l2": "flushed between steps" if ws.need_flush else "inputs larger than L2"}
        out.update(ws.parity_on_sample(min(cfg["d"], 1 << 15), B.CR_AGG_FUSED))
        return out
    finally:
        ws.close()


def other_regression(torch, B, name, steps):
    """cfg3-like regression step measured in the same process: partial gradients of every slot, fused aggregation,
    model update; the aggregated gradient of the last step checked against the oracle's (fp64 partial gradients
    from the definition, then CR.Execute)."""
    from oracle import cr_oracle as O
    from oracle import cr_setup
    cfg = dict(inputs.CONFIGS[name])
    n, L, s, P, d, rows = cfg["n"], cfg["L"], cfg["s"], cfg["P"], cfg["d"], cfg["rows"]
    plan = B.cr_plan_create(n, L, s, P, d, code=getattr(B, CODE_IDS[cfg["code"]]), device=0)
    try:
        N, m = B.cr_plan_num_nodes(plan), B.cr_plan_load(plan)
        logistic = cfg["kind"] == "logistic"
        loss = B.CR_LOSS_LOGISTIC if logistic else B.CR_LOSS_SQUARED
        X, y, _ = (inputs.logistic_partitions(P, rows, d, cfg["seed"], cfg["x_std"]) if logistic else
                   inputs.linreg_partitions(P, rows, d, cfg["seed"], cfg["x_std"], cfg["noise_std"]))
        X_dev, y_dev = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda()
        w_dev = torch.zeros(d, device="cuda")
        G_slots = torch.zeros((N, m, d), device="cuda")
        ws = torch.empty(max(16, B.cr_partial_gradients_workspace_bytes(plan, rows)), dtype=torch.uint8, device="cuda")
        out = torch.zeros((1, d), device="cuda")
        masks = inputs.straggler_masks(n, L, s, steps + 3, cfg.get("mask_seed", 1))
        lr_eff = cfg["lr"] / P
        flush = L2Flush(torch, "cuda") if X.nbytes <= 126e6 else None
        stream = torch.cuda.current_stream()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
        w_before = None
        for i in range(steps + 3):
            if i >= 3:
                if flush is not None:
                    flush(i)
                ev[i - 3][0].record(stream)
            if i == steps + 2:
                w_before = w_dev.clone()
            B.cr_partial_gradients_loss(plan, loss, X_dev, y_dev, rows, w_dev, G_slots, ws, stream)
            if i >= 3:
                ev[i - 3][1].record(stream)
            B.cr_aggregate(plan, G_slots, masks[i], out, B.CR_AGG_FUSED, None, stream)
            w_dev.sub_(out[0], alpha=lr_eff)
            if i >= 3:
                ev[i - 3][2].record(stream)
        torch.cuda.synchronize()
        t_grad = np.array([e[0].elapsed_time(e[1]) for e in ev]) * 1e-3
        t_step = np.array([e[0].elapsed_time(e[2]) for e in ev]) * 1e-3
        grad_bytes = 4.0 * rows * d * N * m
        agg_bytes = float(np.mean([B.cr_aggregate_bytes(plan, masks[i])[0] for i in range(3, steps + 3)]))
        peak, peak_kind = peak_hbm()
        # parity of the last step's aggregated gradient
        code, local, _ = cr_setup.setup(cfg)
        w_h = w_before.cpu().numpy()
        grad = O.partial_gradient_logistic if logistic else O.partial_gradient_linreg
        G_parts = np.stack([grad(X[p], y[p], w_h) for p in range(P)])
        want = O.execute(code, local, G_parts, masks[steps + 2])
        got = out[0].cpu().numpy().astype(np.float64)
        value = (grad_bytes + agg_bytes) / float(t_step.mean()) / 1e9
        traffic = ncu_traffic(name, "f32", d, "partial gradients")
        res = {"workload": regression_workload_name(name, cfg), "dtype": "f32", "value": value, "unit": UNIT,
               "ms_per_step": float(t_step.mean()) * 1e3, "gradient_ms": float(t_grad.mean()) * 1e3, "steps": steps,
               "kernel": "partial gradients (one pass) + " + B.cr_plan_last_kernel(plan),
               "algorithmic_bytes_per_step": grad_bytes + agg_bytes, "frac": value / peak, "peak_kind": f"of {peak_kind}",
               "gradient_GBs_algorithmic": grad_bytes / float(t_grad.mean()) / 1e9,
               "l2": "flushed between steps" if flush is not None else "inputs larger than L2",
               "gpu_rel_l2_of_aggregated_gradient": float(np.linalg.norm(got - want) / np.linalg.norm(want))}
        if traffic:
            res["gradient_dram_frac"] = traffic["bytes"] / float(t_grad.mean()) / 1e9 / peak
            res["gradient_dram_note"] = ("DRAM bytes of an ncu capture over time over peak: slots that hold the same partition "
                                         "share its rows through L2, so DRAM sees less than the algorithmic bytes")
        return res
    finally:
        B.cr_plan_destroy(plan)
        torch.cuda.empty_cache()


def run_ours(args, cfg):
    import torch
    from paper_1902_01981_b200 import binding as B
    from paper_1902_01981_b200 import build as cr_build

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        cr_build.build()
    if dist is not None:
        dist.barrier()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)

    ws0 = AggregateSetup(torch, B, cfg, args.dtype, dev, seed_offset=rank, patterns=min(args.steps + args.warmup, 256))
    plan, is_int, d, batch, N, m = ws0.plan, ws0.is_int, ws0.d, ws0.batch, ws0.N, ws0.m
    if args.tune:
        B.cr_plan_tune(plan, *[int(x) for x in args.tune.split(",")])
    if args.share or args.e_buffers:
        B.cr_plan_tune_batch(plan, args.share, args.e_buffers)

    # ---- the timed region: K steps of the fused kernel
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid).replace("GPU-", "")
    except Exception:
        gpu_id = local_rank
    sampler = ClockSampler(gpu_id)
    sampler.wait_first_sample()
    per, wall, window = ws0.timed(B.CR_AGG_FUSED, args.steps, args.warmup, dist=dist)
    launches = ws0.launches
    timed_kernel = B.cr_plan_last_kernel(plan)
    clocks = sampler.stop(window)
    assert B.cr_plan_device_status(plan) == B.CR_OK, "a device-side wait timed out"
    # device time of the K steps: first start event to last stop event on the launching stream (with
    # an L2 flush between steps: the sum of the per-step intervals, which leaves the flushes out)
    elapsed = float(wall)
    units = ws0.bytes_of(args.steps, args.warmup)
    elapsed_all, units_all = combine_ranks(elapsed, units, world, dist, dev)
    value = units_all / elapsed_all / 1e9

    # ---- a sustained leg of the same call, long enough for the clock samples to fall inside it (the
    # K-step region above can be shorter than one sampling period); rank 0 only
    sustained = None
    if rank == 0 and not args.no_sustained and world == 1:
        s_steps = int(min(20000, max(args.steps, np.ceil(args.sustain_seconds / max(float(per.mean()), 1e-6)))))
        sampler2 = ClockSampler(gpu_id)
        sampler2.wait_first_sample()
        per2, wall2, window2 = ws0.timed(B.CR_AGG_FUSED, s_steps, 3)
        clocks2 = sampler2.stop(window2)
        bytes2 = ws0.bytes_of(s_steps, 3)
        sustained = {"value": bytes2 / wall2 / 1e9, "unit": UNIT, "steps": s_steps, "seconds": wall2,
                     "ms_per_step": wall2 / s_steps * 1e3, "clocks": clocks2,
                     "ms_times_sm_mhz": (wall2 / s_steps * 1e3) * (clocks2.get("sm_mhz") or 0.0)}
        if not clocks.get("samples_in_timed_region"):
            clocks["note"] = ("the timed region is shorter than the sampling period: these samples lie around it; "
                              "the sustained leg carries samples taken inside its own region")

    # ---- comparators on the same slots (rank 0 only, outside the timed region)
    extras = {}
    host_cost = None
    if rank == 0 and not args.no_extras:
        ksteps = min(args.steps, 50)
        bytes_k = ws0.bytes_of(ksteps, args.warmup) / ksteps
        for name, flags in (("fused_plain_loads", B.CR_AGG_FUSED_LDG), ("uncoded_sum_same_bytes", B.CR_AGG_UNCODED_SUM)):
            p2, _, _ = ws0.timed(flags, ksteps, args.warmup)
            extras[name] = {"GB/s": bytes_k / float(p2.mean()) / 1e9, "ms_per_step": float(p2.mean()) * 1e3}
        nws = B.cr_aggregate_workspace_bytes(plan, batch, B.CR_AGG_UNFUSED)
        free, _ = torch.cuda.mem_get_info()
        if nws < free - (2 << 30):
            wsb = torch.empty(nws, dtype=torch.uint8, device=dev)
            p2, _, _ = ws0.timed(B.CR_AGG_UNFUSED, min(ksteps, 5), args.warmup, ws=wsb)
            extras["unfused_per_level"] = {"GB/s": bytes_k / float(p2.mean()) / 1e9, "ms_per_step": float(p2.mean()) * 1e3}
            del wsb
        host_cost = ws0.host_cost_us(B.CR_AGG_FUSED)
        try:    # short launches: the same call captured once in a CUDA graph and replayed
            host_cost["graph_replay_ms"] = ws0.graph_replay_ms(B.CR_AGG_FUSED)
        except Exception as exc:
            host_cost["graph_replay_ms"] = None
            host_cost["graph_replay_unavailable"] = repr(exc)[:200]
            torch.cuda.synchronize()

    # ---- end to end through the host-buffer entry point: H2D of the slots and D2H of the result
    # inside the timed region
    e2e = None
    if not args.no_e2e:
        e2e_steps = max(1, min(args.e2e_steps, args.steps))
        host_slots = torch.empty((N * m, d), dtype=ws0.tdtype, pin_memory=True)
        host_slots.copy_(ws0.G_slots)
        host_out = torch.empty((batch, d), dtype=ws0.tdtype, pin_memory=True)
        torch.cuda.synchronize()
        B.cr_aggregate_host(plan, host_slots, ws0.masks[0], host_out, ws0.G_slots, ws0.out, B.CR_AGG_FUSED, None, ws0.stream)
        if dist is not None:
            dist.barrier()
        t0 = time.perf_counter()
        for i in range(e2e_steps):
            B.cr_aggregate_host(plan, host_slots, ws0.masks[(args.warmup + i) % ws0.total], host_out, ws0.G_slots, ws0.out,
                                B.CR_AGG_FUSED, None, ws0.stream)
        torch.cuda.synchronize()
        e2e_elapsed = time.perf_counter() - t0
        e2e_units = ws0.bytes_of(e2e_steps, args.warmup)
        e2e_elapsed, e2e_units = combine_ranks(e2e_elapsed, e2e_units, world, dist, dev)
        e2e = {"value": e2e_units / e2e_elapsed / 1e9, "unit": UNIT,
               # cr_aggregate_host sends the slots of the consumed nodes only (stragglers are not waited for)
               "h2d_bytes_per_step": int(e2e_units / e2e_steps / world - batch * d * 4 + ws0.masks[0].nbytes),
               "d2h_bytes_per_step": int(batch * d * 4),
               "steps": e2e_steps, "ms_per_step": e2e_elapsed / e2e_steps * 1e3}
        del host_slots

    if rank == 0:
        peak, peak_kind = peak_hbm()
        avg_launch = float(per.mean())
        avg_bytes = units / args.steps
        achieved = avg_bytes / avg_launch / 1e9
        dtype_name = "int32" if is_int else "f32"
        traffic = ncu_traffic(args.workload, dtype_name, d, timed_kernel) if not (args.tune or args.tree) else None
        roofline = {"bound": "hbm", "kernel": timed_kernel, "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                    "frac_note": "the peak is a measured copy (read + write); a read-mostly stream can exceed it slightly",
                    "frac_of_nominal_8TBs": achieved / 8000.0,
                    "traffic": traffic["bytes"] if traffic else None, "traffic_source": traffic,
                    "algorithmic_bytes_per_launch": avg_bytes,
                    "avg_launch_ms": avg_launch * 1e3, "best_launch_ms": float(per.min()) * 1e3}
        cpu = None
        if not args.no_cpu_baseline and not is_int:
            cores = host_threads()
            d_sample = calibrated_columns(cfg, args.cpu_steps + 1, 15.0, min(d, args.cpu_columns), cores)
            sec, nbytes, last, last_masks = oracle_sample(cfg, d_sample, args.cpu_steps, 1,
                                                          np.ascontiguousarray(ws0.G_parts[:, :d_sample]), threads=cores)
            cpu = {"value": nbytes / sec / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
                   "sample": f"first {d_sample} of {d} columns, {args.cpu_steps} steps, NumPy fp64, column chunks on {cores} threads",
                   "ms_per_step_on_sample": sec * 1e3}
            # by-product: the GPU result for the same masks on those columns against the oracle
            B.cr_aggregate(plan, ws0.G_slots, last_masks, ws0.out, B.CR_AGG_FUSED, None, ws0.stream)
            torch.cuda.synchronize()
            got = ws0.out[:, :d_sample].cpu().numpy().astype(np.float64)
            worst = max(float(np.linalg.norm(got[b] - last[b]) / np.linalg.norm(last[b])) for b in range(batch))
            cpu["gpu_rel_l2_on_sample"] = worst
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": elapsed_all / args.steps * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": dtype_name, "data": "synthetic",
            "config": workload_config(args.workload, cfg, None),
            "iterations_per_s": world * args.steps / elapsed_all,
            "patterns_per_s": world * args.steps * batch / elapsed_all,
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches),
            "clocks": clocks, "sustained": sustained, "comparators": extras, "host_us_per_call": host_cost,
            "slots_gb": N * m * d * 4 / 1e9, "tune": args.tune or "auto",
        }
    ws0.close()
    # ---- the other workloads of the results table, measured in the same process (default run, one GPU)
    if rank == 0 and world == 1 and args.others and not (args.tune or args.tree or args.d or args.batch):
        others = []
        for name, dtype, steps, over in (("cfg5", "f32", 8, None), ("cfg5", "int32", 8, None), ("cfg2", "f32", 100, None),
                                         ("cfg_tree12", "f32", 20, None),
                                         ("cfg_tree12", "f32", 20, {"batch": 64, "d": 1 << 20}), ("cfg_cnn", "f32", 100, None)):
            if name == args.workload and dtype == args.dtype and not over:
                continue
            others.append(other_aggregate(torch, B, dev, name, dtype, steps, over))
        others.append(other_regression(torch, B, "cfg3", 20))
        line["other_workloads"] = others
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def run_linreg(args, cfg):
    """End-to-end gradient-descent step of a linear-regression workload (cfg1, cfg3): partial gradients of
    every node's slots, fused aggregation under a fresh straggler pattern, model update.  One GPU."""
    import torch
    from paper_1902_01981_b200 import binding as B
    from paper_1902_01981_b200 import build as cr_build
    cr_build.build()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(0)
    code_id = {"printed_3_1": B.CR_CODE_PAPER_3_1, "cyclic": B.CR_CODE_CYCLIC_RANDOM,
               "repetition": B.CR_CODE_FRACTIONAL_REPETITION}[cfg["code"]]
    n, L, s, P, d, rows = cfg["n"], cfg["L"], cfg["s"], cfg["P"], cfg["d"], cfg["rows"]
    plan = B.cr_plan_create(n, L, s, P, d, code=code_id, device=0)
    if args.tune_gradients:
        B.cr_plan_tune_gradients(plan, *[int(x) for x in args.tune_gradients.split(",")])
    if args.item_order:
        B.cr_plan_tune_items(plan, args.item_order, 0)
    N, m, groups = B.cr_plan_num_nodes(plan), B.cr_plan_load(plan), B.cr_plan_num_groups(plan)
    logistic = cfg["kind"] == "logistic"
    loss = B.CR_LOSS_LOGISTIC if logistic else B.CR_LOSS_SQUARED
    if logistic:
        X, y, w_star = inputs.logistic_partitions(P, rows, d, cfg["seed"], cfg["x_std"])
    else:
        X, y, w_star = inputs.linreg_partitions(P, rows, d, cfg["seed"], cfg["x_std"], cfg["noise_std"])
    X_dev, y_dev = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda()
    E_coded = torch.zeros((N, d), device="cuda")
    coded = args.coded and d % 4 == 0 and d <= 8192
    w_dev = torch.zeros(d, device="cuda")
    G_slots = torch.zeros((N, m, d), device="cuda")
    ws = torch.empty(max(16, B.cr_partial_gradients_workspace_bytes(plan, rows)), dtype=torch.uint8, device="cuda")
    out = torch.zeros((1, d), device="cuda")
    total = min(args.steps + args.warmup, 256)
    masks = inputs.straggler_masks(n, L, s, total, cfg.get("mask_seed", 1))
    lr_eff = cfg["lr"] if args.workload == "cfg1" else cfg["lr"] / P
    flush = L2Flush(torch, "cuda") if X.nbytes <= 126e6 else None
    stream = torch.cuda.current_stream()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]

    def step(i, events=None):
        if events:
            events[0].record(stream)
        if coded:
            B.cr_coded_gradients(plan, loss, X_dev, y_dev, rows, w_dev, E_coded, stream)
        else:
            B.cr_partial_gradients_loss(plan, loss, X_dev, y_dev, rows, w_dev, G_slots, ws, stream)
        if events:
            events[1].record(stream)
        if coded:
            B.cr_aggregate(plan, E_coded, masks[i % total], out, B.CR_AGG_FUSED | B.CR_AGG_FROM_CODED, None, stream)
        else:
            B.cr_aggregate(plan, G_slots, masks[i % total], out, B.CR_AGG_FUSED, None, stream)
        w_dev.sub_(out[0], alpha=lr_eff)
        if events:
            events[2].record(stream)

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.wait_first_sample()
    n0 = B.cr_plan_launch_count(plan)
    t0 = time.time()
    for i in range(args.steps):
        if flush is not None:
            flush(i)
        step(args.warmup + i, ev[i])
    torch.cuda.synchronize()
    t1 = time.time()
    launches = B.cr_plan_launch_count(plan) - n0
    clocks = sampler.stop((t0, t1))
    t_grad = np.array([e[0].elapsed_time(e[1]) for e in ev]) * 1e-3
    t_step = np.array([e[0].elapsed_time(e[2]) for e in ev]) * 1e-3
    elapsed = float(t_step.sum())
    # algorithmic bytes: every (node, slot) reads its partition once; the aggregation reads the consumed slots
    grad_bytes = 4.0 * rows * d * N * m
    agg_bytes = float(np.mean([B.cr_aggregate_bytes(plan, masks[i])[0] for i in range(total)]))
    step_bytes = grad_bytes + agg_bytes
    peak, peak_kind = peak_hbm()
    achieved = grad_bytes / float(t_grad.mean()) / 1e9
    w_final = w_dev.cpu().numpy()
    # end to end: the data set stays resident (it does not change between steps); the model goes up from
    # pinned host memory and the aggregated gradient comes back, every step, and the host applies the update
    e2e = None
    if not args.no_e2e:
        e2e_steps = max(1, min(args.steps, 50))
        w_host = torch.zeros(d, pin_memory=True)
        g_host = torch.zeros(d, pin_memory=True)
        t0 = time.perf_counter()
        for i in range(e2e_steps):
            w_dev.copy_(w_host, non_blocking=True)
            step(i)
            g_host.copy_(out[0], non_blocking=True)
            torch.cuda.synchronize()
            w_host.sub_(g_host, alpha=lr_eff)
        e2e_sec = (time.perf_counter() - t0) / e2e_steps
        e2e = {"value": step_bytes / e2e_sec / 1e9, "unit": UNIT, "h2d_bytes_per_step": int(4 * d + masks[0].nbytes),
               "d2h_bytes_per_step": int(4 * d), "steps": e2e_steps, "ms_per_step": e2e_sec * 1e3}
    # The same step as one CUDA graph (gradients, aggregation with a schedule made beforehand, model update),
    # replayed: what a launch-bound step costs once the host is out of the loop.  A graph bakes its arguments
    # in, so every replay runs the straggler pattern of the schedule it was captured with.
    graph_leg = None
    if not args.no_extras:
        try:
            agg_flags = (B.CR_AGG_FUSED | B.CR_AGG_FROM_CODED) if coded else B.CR_AGG_FUSED
            sched = B.cr_schedule_create(plan, masks[0], agg_flags)
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                cs = torch.cuda.current_stream()
                if coded:
                    B.cr_coded_gradients(plan, loss, X_dev, y_dev, rows, w_dev, E_coded, cs)
                else:
                    B.cr_partial_gradients_loss(plan, loss, X_dev, y_dev, rows, w_dev, G_slots, ws, cs)
                B.cr_aggregate_scheduled(plan, E_coded if coded else G_slots, sched, out, None, cs)
                w_dev.sub_(out[0], alpha=lr_eff)
            w_keep = w_dev.clone()
            reps = max(20, min(args.steps, 200))
            for _ in range(3):
                graph.replay()
            torch.cuda.synchronize()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            if flush is None:
                g0.record()
                for _ in range(reps):
                    graph.replay()
                g1.record()
                torch.cuda.synchronize()
                graph_ms = g0.elapsed_time(g1) / reps
            else:   # data that fit L2 are flushed before every replay, each timed by itself
                tt = []
                for i in range(reps):
                    flush(i)
                    g0.record()
                    graph.replay()
                    g1.record()
                    torch.cuda.synchronize()
                    tt.append(g0.elapsed_time(g1))
                graph_ms = float(np.mean(tt))
            w_dev.copy_(w_keep)
            B.cr_schedule_destroy(sched)
            graph_leg = {"ms_per_step": graph_ms, "iterations_per_s": 1e3 / graph_ms, "replays": reps,
                         "note": "one CUDA graph per step (gradient kernels, scheduled aggregation, update), one fixed straggler pattern"}
        except Exception as exc:   # a capture that the runtime refuses is reported, not fatal
            graph_leg = {"unavailable": repr(exc)[:200]}
            torch.cuda.synchronize()
    cpu = None
    if not args.no_cpu_baseline:
        sec, nbytes, sample = oracle_regression_sample(args.workload, cfg, args.cpu_steps, 1, 15.0)
        cpu = {"value": nbytes / sec / 1e9, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
               "sample": sample + "; the matrix products run on NumPy's BLAS threads (the count given), CR.Execute on one",
               "ms_per_step_on_sample": sec * 1e3}
    traffic = ncu_traffic(args.workload, "f32", d, "partial gradients") if not args.tune_gradients else None
    line = {
        "metric": METRIC, "value": step_bytes * args.steps / elapsed / 1e9, "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": elapsed / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{args.workload}: {'logistic' if logistic else 'linear'} regression n={n} L={L} s={s} "
                               f"P={P} rows={rows} d={d}, step = "
                               + ("coded gradients of all N nodes (slot gradients never written)" if coded
                                  else "partial gradients of all N*m slots") + " + fused aggregation + model update",
                   "l2": "inputs larger than L2 (no flush needed)" if flush is None else "L2 flushed between steps (256 MB written, then 256 MB read)"},
        "iterations_per_s": args.steps / elapsed,
        "roofline": {"bound": "hbm", "kernel": "partial gradients", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "frac_note": "algorithmic bytes count every (node, slot) item reading its partition; items that hold the "
                                  "same partition share its rows through L2, so this fraction can exceed 1 (see dram_frac)",
                     "traffic": traffic["bytes"] if traffic else None, "traffic_source": traffic,
                     "dram_frac": (traffic["bytes"] / float(t_grad.mean()) / 1e9 / peak) if traffic else None,
                     "algorithmic_bytes_per_launch": grad_bytes, "avg_launch_ms": float(t_grad.mean()) * 1e3,
                     "aggregate_ms": float((t_step - t_grad).mean()) * 1e3},
        "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks, "graph_replay": graph_leg,
        "normalized_error_rate": float(np.sum((w_final - w_star) ** 2) / np.sum(w_star ** 2)),
    }
    print(json.dumps(line), flush=True)
    B.cr_plan_destroy(plan)


def run_multi(args, cfg):
    """Partial gradients of --models K models in one pass over a regression workload (tensor-core path),
    timed beside K passes of the single-model kernel.  One GPU; X is rounded to TF32-representable values."""
    import torch
    from paper_1902_01981_b200 import binding as B
    from paper_1902_01981_b200 import build as cr_build
    cr_build.build()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(0)
    code_id = {"printed_3_1": B.CR_CODE_PAPER_3_1, "cyclic": B.CR_CODE_CYCLIC_RANDOM,
               "repetition": B.CR_CODE_FRACTIONAL_REPETITION}[cfg["code"]]
    n, L, s, P, d, rows, K = cfg["n"], cfg["L"], cfg["s"], cfg["P"], cfg["d"], cfg["rows"], args.models
    plan = B.cr_plan_create(n, L, s, P, d, code=code_id, device=0)
    N, m = B.cr_plan_num_nodes(plan), B.cr_plan_load(plan)
    logistic = cfg["kind"] == "logistic"
    loss = B.CR_LOSS_LOGISTIC if logistic else B.CR_LOSS_SQUARED
    if logistic:
        X, y, _ = inputs.logistic_partitions(P, rows, d, cfg["seed"], cfg["x_std"])
    else:
        X, y, _ = inputs.linreg_partitions(P, rows, d, cfg["seed"], cfg["x_std"], cfg["noise_std"])
    X = inputs.tf32_representable(X)
    W = inputs.model_matrix(K, d, cfg["seed"] + 1)
    X_dev, y_dev, W_dev = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda(), torch.from_numpy(W).cuda()
    G = torch.zeros((K, N, m, d), device="cuda")
    ws = torch.empty(B.cr_partial_gradients_multi_workspace_bytes(plan, rows), dtype=torch.uint8, device="cuda")
    ws1 = torch.empty(max(16, B.cr_partial_gradients_workspace_bytes(plan, rows)), dtype=torch.uint8, device="cuda")
    flush = L2Flush(torch, "cuda") if X.nbytes <= 126e6 else None
    stream = torch.cuda.current_stream()

    def timed(fn, steps):
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(steps)]
        for i in range(steps):
            if flush is not None:
                flush(i)
            ev[i][0].record(stream)
            fn()
            ev[i][1].record(stream)
        torch.cuda.synchronize()
        return np.array([e[0].elapsed_time(e[1]) for e in ev]) * 1e-3

    def multi():
        B.cr_partial_gradients_multi(plan, loss, X_dev, y_dev, rows, W_dev, K, G, ws, None, stream)

    def singles():
        for k in range(K):
            B.cr_partial_gradients_loss(plan, loss, X_dev, y_dev, rows, W_dev[k], G[k], ws1, stream)

    steps = min(args.steps, 50)
    timed(multi, args.warmup)
    sampler = ClockSampler(0)
    sampler.wait_first_sample()
    n0 = B.cr_plan_launch_count(plan)
    t0 = time.time()
    t_multi = timed(multi, steps)
    t1 = time.time()
    launches = B.cr_plan_launch_count(plan) - n0
    clocks = sampler.stop((t0, t1))
    B.cr_plan_device_status(plan)
    timed(singles, 1)
    t_single = timed(singles, max(1, steps // 10))
    # algorithmic bytes: each (node, slot) item reads its partition once per contraction and writes K gradients
    items = N * m
    nbytes = 4.0 * items * (2.0 * rows * d + K * d)
    flops = 2.0 * 2.0 * rows * d * K * items
    peak, peak_kind = peak_hbm()
    sec = float(t_multi.mean())
    achieved = nbytes / sec / 1e9
    line = {
        "metric": METRIC, "value": achieved, "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": args.warmup,
        "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "tf32",
        "data": "synthetic",
        "config": {"workload": f"{args.workload}: partial gradients of K={K} models, n={n} L={L} s={s} P={P} rows={rows} "
                               f"d={d} ({items} slot items), X TF32-representable",
                   "l2": "inputs larger than L2 (no flush needed)" if flush is None else "L2 flushed between steps (256 MB written, then 256 MB read)"},
        "roofline": {"bound": "hbm", "kernel": "cr_tc_residual_kernel + cr_tc_gradient_kernel", "achieved": achieved,
                     "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "traffic": None, "algorithmic_bytes_per_launch": nbytes, "avg_launch_ms": sec * 1e3,
                     "tensor_tflops": flops / sec / 1e12},
        "k_single_model_passes_ms": float(t_single.mean()) * 1e3,
        "speedup_over_single_model_passes": float(t_single.mean()) / sec,
        "cpu_baseline": None, "e2e": None, "gpu_launches": int(launches), "clocks": clocks,
    }
    print(json.dumps(line), flush=True)
    B.cr_plan_destroy(plan)


def apply_tree_override(cfg, text):
    """`--tree n,L,s,code[,c]`: replaces the tree of a workload; P becomes c times the smallest partition
    count that the tree splits into whole chunks at every level."""
    f = text.split(",")
    n, L, s_ = int(f[0]), int(f[1]), int(f[2])
    quantum = sum(n ** l * (s_ + 1) ** (L - l) for l in range(1, L + 1))
    cfg.update(n=n, L=L, s=s_, code=f[3], P=quantum * (int(f[4]) if len(f) > 4 else 1))
    return cfg


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=list(inputs.CONFIGS))
    ap.add_argument("--dtype", default="f32", choices=["f32", "int32"])
    ap.add_argument("--d", type=int, default=0, help="override the gradient length (profiling on a small case)")
    ap.add_argument("--tree", default="", help="override the tree of the workload: n,L,s,code[,c] with code in "
                    "printed_3_1|cyclic|repetition and P = c times the smallest partition count the tree allows")
    ap.add_argument("--batch", type=int, default=0, help="aggregation workloads: straggler patterns per call")
    ap.add_argument("--rows", type=int, default=0, help="regression workloads: override the rows per partition")
    ap.add_argument("--tune", default="", help="consumer_warps,stages,ctas_per_sm,rows_per_box (0 = auto)")
    ap.add_argument("--tune-gradients", default="", help="regression workloads: block_kb,stages,cluster of the one-pass "
                    "gradient kernel (0 = auto)")
    ap.add_argument("--share", type=int, default=0, help="batches: messages shared by the patterns: 0 built-in choice, "
                    "1 never, 2 whenever possible")
    ap.add_argument("--e-buffers", type=int, default=0, help="batches: buffers of coded gradients in shared memory (1, 2)")
    ap.add_argument("--item-order", type=int, default=0, help="regression workloads: launch order of the (node, slot) items: "
                    "1 by node then slot, 2 grouped by partition (0: built-in choice)")
    ap.add_argument("--coded", action="store_true", help="regression workloads: gradient + encode in one kernel")
    ap.add_argument("--models", type=int, default=0, help="regression workloads: gradients of K models per pass (1..32)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-sustained", action="store_true", help="skip the sustained leg of the headline call")
    ap.add_argument("--sustain-seconds", type=float, default=2.0)
    ap.add_argument("--others", dest="others", action="store_true", default=None,
                    help="also measure the other workloads of the results table (default for the plain cfg4 run)")
    ap.add_argument("--no-others", dest="others", action="store_false")
    ap.add_argument("--no-extras", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-columns", type=int, default=1 << 21)
    ap.add_argument("--cpu-steps", type=int, default=8)
    ap.add_argument("--ref-columns", type=int, default=1 << 21)
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.others is None:
        args.others = args.workload == "cfg4" and not (args.no_extras or args.no_e2e or args.no_cpu_baseline)
    cfg = dict(inputs.CONFIGS[args.workload])
    if args.d:
        cfg["d"] = args.d
    if args.tree:
        apply_tree_override(cfg, args.tree)
    if args.batch and cfg["kind"] == "aggregate":
        cfg["batch"] = args.batch
    if args.rows and "rows" in cfg:
        cfg["rows"] = args.rows
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus != world and world > 1:
        args.gpus = world
    if cfg["kind"] in ("linreg", "logistic"):
        if args.impl == "reference":
            run_reference_regression(args, cfg)
        elif args.models:
            run_multi(args, cfg)
        else:
            run_linreg(args, cfg)
    elif args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()

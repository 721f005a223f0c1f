#!/usr/bin/env python
"""Benchmark of the gradient-compression hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

One step = one pass of the whole hot path over one fresh synthetic gradient per worker:
gc_compress (fold, select, compact, residual write-back) for each of the W workers, then
gc_decompress_accumulate of the W sparse sets into the dense fp32 sum.  The default workload
is the 110M-element BERT-base-shaped configuration (the one the throughput target is quoted
on).  Prints ONE JSON line.

`--impl reference` times the CPU oracle (as it stands) on a bounded sample of the same
workload on the host cores; with N > 1 ranks only rank 0 does that.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2104_01981_b200 import synth

METRIC = "gradient_GB_per_s_compressed_and_aggregated"
UNIT = "GB/s"
NOMINAL_HBM = 8.0e12          # the metric's "8 TB/s HBM roofline"
N_INPUT_SETS = 3              # distinct gradients cycled through (each far larger than L2)


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


def min_bytes(n: int, k: int, W: int, grad_bytes: int = 4):
    """Algorithmic bytes of one step: compress (grad_bytes + 8) n + 8k per worker, decode 4n + 8*W*k."""
    compress = ((grad_bytes + 8) * n + 8 * k) * W
    decode = 4 * n + 8 * k * W
    return compress, decode


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, path: str):
        self.path = path
        self.proc = None
        try:
            self.f = open(path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        for line in open(self.path):
            p = [x.strip() for x in line.split(",")]
            if len(p) < 8:
                continue
            try:
                sm.append(float(p[0])); mx.append(float(p[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                               p[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons),
                       samples=len(sm))
        return out


# --------------------------------------------------------------------------- CPU oracle legs
CPU_SAMPLE_ELEMENTS = 1 << 26        # one sample size for `cpu_baseline` and for `--impl reference`


def oracle_sample_inputs(w: synth.Workload, sample_n: int, n_grads: int = 2, worker: int = 0):
    """(sizes, ks, gradients) of the bounded sample the CPU oracle is timed on: the first `sample_n`
    elements of the workload's flat gradient (layer-wise workloads: whole tensors up to that)."""
    import oracle
    oracle.build()
    sizes = [min(sample_n, w.total_n)] if len(w.sizes) == 1 else None
    if sizes is None:                       # layer-wise workloads: keep whole tensors up to sample_n
        sizes, acc = [], 0
        for s in w.sizes:
            if acc + s > sample_n and sizes:
                break
            sizes.append(s); acc += s
    n = sum(sizes)
    ks = [oracle.k_from_density(s, w.density) for s in sizes]
    grads = [synth.gradient(w, worker, s, device="cpu")[:n].numpy().copy() for s in range(n_grads)]
    return sizes, ks, grads


def oracle_sample_run(w: synth.Workload, sample_n: int, steps: int, warmup: int, inputs=None):
    """Times the CPU oracle, one thread, on the sample (same density, one worker, compress + decode
    per step).  Returns (elements, k, seconds per timed step)."""
    import oracle
    sizes, ks, grads = inputs or oracle_sample_inputs(w, sample_n)
    n = sum(sizes)
    r = np.zeros(n, np.float32)
    out = np.empty(n, np.float32)
    times = []
    for it in range(warmup + steps):
        g = grads[it % len(grads)]
        t0 = time.perf_counter()
        idx, val = oracle.topk_compress_tensors(sizes, ks, g, r)
        oracle.decode_accumulate([(idx, val)], out, True)
        dt = time.perf_counter() - t0
        if it >= warmup:
            times.append(dt)
    return n, sum(ks), times


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def oracle_threads_run(w: synth.Workload, sample_n: int, steps: int, warmup: int, max_threads: int = 32,
                       inputs=None):
    """The same oracle step on one thread per simulated worker, all at once: every thread owns one
    worker's sample (its own gradient window, residual and dense buffer) and calls the oracle as it
    stands; the library calls run outside the interpreter lock.  Returns (threads, elements per
    thread, wall seconds of the timed steps)."""
    import threading
    import oracle
    sizes, ks, grads = inputs or oracle_sample_inputs(w, sample_n, n_grads=2)
    n = sum(sizes)
    threads = max(1, min(host_cores(), max_threads))
    try:
        import psutil
        room = int(psutil.virtual_memory().available * 0.5 // (8 * 4 * n))     # g, r, out + the oracle's index arrays
        threads = max(1, min(threads, room))
    except Exception:
        pass
    state = [(np.zeros(n, np.float32), np.empty(n, np.float32)) for _ in range(threads)]
    gate = threading.Barrier(threads + 1)

    def body(t: int):
        r, out = state[t]
        for it in range(warmup + steps):
            if it == warmup:
                gate.wait()
            g = grads[(it + t) % len(grads)]
            idx, val = oracle.topk_compress_tensors(sizes, ks, g, r)
            oracle.decode_accumulate([(idx, val)], out, True)
        gate.wait()

    th = [threading.Thread(target=body, args=(t,)) for t in range(threads)]
    for x in th:
        x.start()
    gate.wait()
    t0 = time.perf_counter()
    gate.wait()
    dt = time.perf_counter() - t0
    for x in th:
        x.join()
    return threads, n, dt


def cpu_baseline(w: synth.Workload, steps: int = 8, warmup: int = 1, with_threads: bool = True):
    """The `cpu_baseline` object: the oracle on one thread, and on one thread per worker."""
    inputs = oracle_sample_inputs(w, CPU_SAMPLE_ELEMENTS)
    sn, sk, times = oracle_sample_run(w, CPU_SAMPLE_ELEMENTS, steps, warmup, inputs)
    cpu = {"value": 4.0 * sn * len(times) / sum(times) / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
           "cores_available": host_cores(),
           "sample": f"first {sn} elements of the workload gradient, k={sk}, {len(times)} steps after {warmup} "
                     f"warm-up, compress + decode, single thread"}
    if with_threads:
        nth, tn, dt = oracle_threads_run(w, CPU_SAMPLE_ELEMENTS, 3, 1, inputs=inputs)
        cpu["multi_thread"] = {"value": 4.0 * tn * nth * 3 / dt / 1e9, "unit": UNIT, "cores": nth,
                               "sample": f"{nth} threads (one per simulated worker, each on its own {tn}-element "
                                         f"sample, residual and dense buffer), 3 steps after 1 warm-up"}
    return cpu


def run_reference(args, w: synth.Workload, rank: int):
    if rank != 0:
        return
    n, k, times = oracle_sample_run(w, CPU_SAMPLE_ELEMENTS, args.steps, args.warmup)
    t = sum(times)
    value = 4.0 * n * len(times) / t / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "config": {"workload": w.name, "mode": "topk", "grad_dtype": "f32", "elements": w.total_n,
                                         "density": w.density, "workers": w.workers, "tensors": len(w.sizes)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "cores_available": host_cores(),
                         "sample": f"first {n} elements of the workload gradient per step, k={k}, "
                                   f"compress + decode, single thread"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- ranks
def reduce_max_over_ranks(values, world: int, device) -> list:
    """Replicas only: every rank runs the same workload on its own GPU and the job's time is the
    slowest rank's.  Returns the element-wise maximum over ranks (identity for one rank)."""
    if world <= 1:
        return list(values)
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    t = torch.nan_to_num(t, nan=-1.0)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return [float("nan") if x < 0 else x for x in t.tolist()]


def whole_job_value(n: int, workers: int, world: int, steps: int, ms: float) -> float:
    """Gradient GB/s of the whole job: bytes of gradient all ranks consumed / slowest rank's time."""
    return 4.0 * n * workers * world * steps / (ms * 1e-3) / 1e9


def profile_traffic(name: str):
    """DRAM bytes of one launch as an ncu capture measured them: the `dram_bytes_per_launch = N` line
    of the summary under profiles/ (None when the summary or the line is missing)."""
    import re
    path = os.path.join(ROOT, "profiles", name)
    try:
        m = re.search(r"^dram_bytes_per_launch\s*=\s*(\d+)", open(path).read(), re.M)
        return (float(m.group(1)), "profiles/" + name) if m else (None, None)
    except OSError:
        return None, None


# --------------------------------------------------------------------------- GPU arm
class Rig:
    """Buffers of one (workload, mode) on one GPU and the calls of one step."""

    def __init__(self, api, w: synth.Workload, mode_name: str, dev: str, device_index: int, input_sets: int,
                 seed_worker0: int = 0, grad_dtype: str = "f32", path: str = "auto"):
        self.api, self.w = api, w
        self.mode = api.GC_THRESHOLD if mode_name == "threshold" else api.GC_TOPK
        self.plan = api.Plan(w.sizes, w.density, mode=self.mode, device=device_index)
        if path != "auto":
            self.plan.set_option(api.GC_OPT_PATH, {"exact": api.GC_PATH_EXACT, "staged": api.GC_PATH_STAGED}[path])
        # the bench owns its workspaces and nothing else writes to them between calls
        self.plan.set_option(api.GC_OPT_WORKSPACE_PRIVATE, 1)
        self.n, self.k, self.W = self.plan.total_n, self.plan.total_cap, w.workers
        n, W = self.n, self.W
        self.stream = torch.cuda.current_stream()
        # inputs resident in HBM before the timed region: `sets` gradients per worker slot, cycled;
        # each is far larger than the 126 MB L2 (or, for the small workloads, the set of buffers a
        # step touches is), so no explicit flush is needed
        self.sets = max(1, min(input_sets, int(24e9 // (4 * n * W)) or 1))
        self.grads = [[synth.gradient(w, wk + seed_worker0, s, device=dev) for s in range(self.sets)]
                      for wk in range(W)]
        self.bf16 = grad_dtype == "bf16"
        if self.bf16:                            # the gradient arrives as bfloat16 (gc_compress_bf16)
            self.grads = [[g.to(torch.bfloat16) for g in gs] for gs in self.grads]
        self.do_compress = self.plan.compress_bf16 if self.bf16 else self.plan.compress
        self.resid = [torch.zeros(n, dtype=torch.float32, device=dev) for _ in range(W)]
        self.outs = [self.plan.alloc_outputs() for _ in range(W)]
        self.ws = self.plan.alloc_workspace()
        self.dense = torch.empty(n, dtype=torch.float32, device=dev)
        self.thr = self.mode == api.GC_THRESHOLD          # threshold mode: variable counts travel with the pairs
        self.cnts = [o[2] for o in self.outs] if self.thr else None
        self.idx, self.val = [o[0] for o in self.outs], [o[1] for o in self.outs]
        # several workers: one gc_compress_workers call per step (own workspace per worker; the
        # library shares launches among them where the plan allows it, else it loops itself)
        self.workers_call = W > 1 and not self.bf16
        self.wss = [self.ws] + [self.plan.alloc_workspace() for _ in range(W - 1)] if self.workers_call else None

    def compress_only(self, i: int):
        if self.workers_call:
            self.plan.compress_workers([gs[i % self.sets] for gs in self.grads], self.resid, self.idx, self.val,
                                       self.cnts, self.wss, self.stream)
            return
        self.compress_separate(i)

    def compress_separate(self, i: int):
        for wk in range(self.W):
            o = self.outs[wk]
            self.do_compress(self.grads[wk][i % self.sets], self.resid[wk], o[0], o[1], o[2] if self.thr else None,
                             self.ws, self.stream)

    def decode_only(self, i: int):
        self.plan.decompress_accumulate(self.idx, self.val, self.cnts, self.dense, True, self.ws, self.stream)

    def step(self, i: int):
        self.compress_only(i)
        self.decode_only(i)

    def check(self):
        worst = self.api.GC_OK
        for ws in (self.wss or [self.ws]):
            st, det = self.plan.last_status(ws)
            if st not in (self.api.GC_OK, self.api.GC_W_TRUNCATED):
                raise RuntimeError(f"device status {st} (detail {det}) after the timed region")
            worst = max(worst, st)
        return worst


class Timer:
    """K-step loops timed with CUDA events on the launching stream, a barrier and a synchronize on
    both sides of every loop, the slowest rank's time per loop.  A loop is repeated until about
    `min_total_ms` of device time have passed (so that clock samples land under load); the
    reported time is the median loop."""

    def __init__(self, stream, world: int, dev, min_total_ms: float = 1000.0):
        self.stream, self.world, self.dev, self.min_total_ms = stream, world, dev, min_total_ms
        self.e0, self.e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def barrier(self):
        if self.world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    def one_loop(self, fn, steps: int, first: int = 0) -> float:
        self.barrier()
        self.e0.record(self.stream)
        for i in range(steps):
            fn(first + i)
        self.e1.record(self.stream)
        self.barrier()
        return reduce_max_over_ranks([self.e0.elapsed_time(self.e1)], self.world, self.dev)[0]

    def loops(self, fn, steps: int, first: int = 0, max_loops: int = 400, min_loops: int = 3):
        """Returns the per-loop times (ms), every rank the same list."""
        t = [self.one_loop(fn, steps, first)]
        want = int(min(max_loops, max(min_loops, -(-self.min_total_ms // max(t[0], 1e-3)))))
        while len(t) < want:
            t.append(self.one_loop(fn, steps, first))
        return t


def spread(times, steps):
    """(median, min, max) of the loop times, per step."""
    return statistics.median(times) / steps, min(times) / steps, max(times) / steps


def run_gpu(args, w: synth.Workload, rank: int, world: int, local_rank: int):
    from paper_2104_01981_b200 import api
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    api.lib()                                    # no fallback: raises when libgc.so is missing
    rig = Rig(api, w, args.mode, dev, local_rank, args.input_sets, 100 * rank, args.grad_dtype, args.path)
    plan, n, k, W, sets, stream = rig.plan, rig.n, rig.k, rig.W, rig.sets, rig.stream
    tm = Timer(stream, world, dev, args.min_loop_ms)
    res = {}

    for i in range(args.warmup):
        rig.step(i)
    tm.barrier()
    sampler = ClockSampler(local_rank, os.path.join(tempfile.gettempdir(), f"gc_bench_clocks_{os.getpid()}.csv")) \
        if rank == 0 else None
    # ---- timed region 1: device-resident inputs, K steps per loop (the headline value)
    launches0 = plan.launches()
    res["plain"] = tm.loops(rig.step, args.steps, args.warmup)
    res["launches_per_loop"] = (plan.launches() - launches0) // len(res["plain"])
    # ---- timed region 1b: the same loop once more with per-kernel events on (the kernel table)
    plan.profile_enable(args.steps * (8 * W + 8))
    res["with_events"] = tm.one_loop(rig.step, args.steps, args.warmup)
    res["per_kernel"] = plan.profile_read()
    plan.profile_enable(0)
    rig.check()
    res["counters"] = plan.last_counters(rig.ws)
    res["phase_us"] = plan.last_phase_times(rig.ws)
    # ---- timed regions 1c/1d: the two halves on their own
    res["compress"] = tm.loops(rig.compress_only, args.steps, args.warmup)
    res["decode"] = tm.loops(rig.decode_only, args.steps, args.warmup)
    res["clocks"] = sampler.stop() if sampler else None          # sampled across the loops above
    # ---- timed region 1e: decode with momentum SGD fused behind it (top-k lists only)
    res["apply"] = None
    if not rig.thr:
        param = torch.zeros(n, device=dev)
        vel = torch.zeros(n, device=dev)

        def apply_only(i: int):
            plan.decompress_apply_momentum(rig.idx, rig.val, None, param, vel, 0.01, 0.9, 1.0 / W, rig.ws, stream)

        for i in range(3):
            apply_only(i)
        res["apply"] = tm.one_loop(apply_only, args.steps) / args.steps
        del param, vel

    # ---- timed region 2: end to end through the host-buffer entry point
    res["e2e_steps"], res["e2e"] = 0, float("nan")
    if not (args.no_e2e or args.grad_dtype == "bf16" or rig.thr):
        e2e_steps = max(3, min(args.steps, 10))
        host_g = [torch.empty(n, dtype=torch.float32).pin_memory() for _ in range(2)]
        for j in range(2):
            host_g[j].copy_(rig.grads[0][j % sets])
        host_idx = torch.empty(max(k, 1), dtype=torch.int32).pin_memory()
        host_val = torch.empty(max(k, 1), dtype=torch.float32).pin_memory()
        staging = [torch.empty(n, dtype=torch.float32, device=dev) for _ in range(2)]      # alternated: the next copy
        call = [0]                                                                         # overlaps this compress

        def e2e_step(i: int):
            for wk in range(W):
                plan.compress_host(host_g[i % 2], staging[call[0] % 2], rig.resid[wk], rig.outs[wk][0], rig.outs[wk][1],
                                   None, host_idx, host_val, rig.ws, stream)
                call[0] += 1
            plan.decompress_accumulate(rig.idx, rig.val, None, rig.dense, True, rig.ws, stream)

        for i in range(2):
            e2e_step(i)
        res["e2e"] = tm.one_loop(e2e_step, e2e_steps)
        res["e2e_steps"] = e2e_steps
        del host_g, staging
    # ---- the other workloads, each timed the same way with fewer steps (rank 0 only: replicas)
    others = {}
    if args.configs == "all" and rank == 0 and args.grad_dtype == "f32" and args.path == "auto":
        del rig.grads, rig.resid, rig.dense
        torch.cuda.empty_cache()
        peak, _ = measured_peak_gbs()
        for cfg, mode in ((0, "topk"), (1, "topk"), (3, "topk"), (3, "threshold"), (4, "topk")):
            if cfg == w.config_id and mode == args.mode:
                continue
            others[f"c{cfg + 1}_{mode}"] = bench_other(api, cfg, mode, dev, local_rank, peak, args)
    _report(args, w, rank, world, dev, plan, n, k, W, sets, res, others)


def bench_other(api, cfg: int, mode: str, dev: str, device_index: int, peak: float, args):
    """One of the other workloads: compress per worker, decode and whole step by CUDA events."""
    w = synth.workload(cfg)
    rig = Rig(api, w, mode, dev, device_index, args.input_sets)
    n, k, W = rig.n, rig.k, rig.W
    tm = Timer(rig.stream, 1, dev, min_total_ms=300.0)
    steps = max(3, min(args.steps, int(200.0 / max(0.02, 12.0 * n * W / 5e9))))      # about 0.2 s per loop
    for i in range(3):
        rig.step(i)
    t_step, t_lo, t_hi = spread(tm.loops(rig.step, steps, 3), steps)
    t_c = spread(tm.loops(rig.compress_only, steps, 3), steps)[0]
    t_d = spread(tm.loops(rig.decode_only, steps, 3), steps)[0]
    t_sep = spread(tm.loops(rig.compress_separate, steps, 3), steps)[0] if rig.workers_call else None
    st = rig.check()
    counters = rig.plan.last_counters(rig.ws)
    sent = k
    if rig.thr:                                   # pairs actually sent by the last step (the lists are not full)
        T = len(w.sizes)
        sent = int(sum(int(c[:T].sum().item()) for c in rig.cnts) / W)
    cb, db = 12.0 * n + 8.0 * sent, 4.0 * n + 8.0 * sent * W
    out = {
        "workload": w.name, "mode": mode, "elements": n, "workers": W, "tensors": len(w.sizes), "steps_per_loop": steps,
        "pairs_per_worker": sent, "capacity_per_worker": k,
        "compress_us_per_worker": 1e3 * t_c / W, "decode_us": 1e3 * t_d, "ms_per_step": t_step,
        "compress_call": "gc_compress_workers (one call per step)" if rig.workers_call else "gc_compress",
        "compress_us_per_worker_separate_calls": None if t_sep is None else 1e3 * t_sep / W,
        "ms_per_step_min_max": [t_lo, t_hi],
        "gradient_GB_per_s": 4.0 * n * W / (t_step * 1e-3) / 1e9,
        "compress_frac_of_8TBs": cb / NOMINAL_HBM / (t_c / W * 1e-3),
        "compress_frac_of_measured": cb / (peak * 1e9) / (t_c / W * 1e-3),
        "decode_frac_of_8TBs": db / NOMINAL_HBM / (t_d * 1e-3),
        "decode_frac_of_measured": db / (peak * 1e9) / (t_d * 1e-3),
        "path_counters": {"candidates_last_step": counters[0], "candidate_overflow": counters[1],
                          "tensors_redone": counters[2], "status": st},
        "input_sets": rig.sets,
    }
    del rig
    torch.cuda.empty_cache()
    return out


def _report(args, w, rank, world, dev, plan, n, k, W, sets, res, others):
    if rank != 0:
        return
    per_kernel, counters, clocks = res["per_kernel"], res["counters"], res["clocks"]
    ms_step, ms_lo, ms_hi = spread(res["plain"], args.steps)
    ms_compress = spread(res["compress"], args.steps)[0]
    ms_decode = spread(res["decode"], args.steps)[0]
    e2e_steps, ms_e2e = res["e2e_steps"], res["e2e"]
    grad_bytes_step = 4.0 * n * W * world
    value = whole_job_value(n, W, world, 1, ms_step)
    cb, db = min_bytes(n, k, W, 2 if args.grad_dtype == "bf16" else 4)
    t_step = ms_step * 1e-3
    peak, peak_src = measured_peak_gbs()

    # dominant kernel: largest share of the per-kernel event time
    tot_ms = sum(v[0] for v in per_kernel.values()) or 1.0
    breakdown = {name: {"ms_per_launch": v[0] / v[1], "launches": v[1], "share": v[0] / tot_ms}
                 for name, v in per_kernel.items()}
    dom = max(per_kernel.items(), key=lambda kv: kv[1][0])[0]
    alg_bytes = {"fold_hist": 12.0 * n, "hist_refine": 4.0 * n, "compact": 4.0 * n + 8.0 * k,
                 "decode_clear": 4.0 * n, "decode_add": 8.0 * k, "fold_cand": 12.0 * n, "compress_fused": 12.0 * n + 8.0 * k,
                 "threshold_emit": 12.0 * n + 4.0 * k, "decode_tiles": 4.0 * n + 8.0 * k * W}
    # a compress launch may serve several workers (gc_compress_workers): its bytes are theirs together
    fused_per_step = per_kernel.get("compress_fused", (0.0, 0))[1] / args.steps
    workers_per_launch = W / fused_per_step if fused_per_step else 1.0
    alg_bytes["compress_fused"] *= workers_per_launch
    dom_ms = breakdown[dom]["ms_per_launch"]
    achieved = alg_bytes.get(dom, 12.0 * n) / (dom_ms * 1e-3) / 1e9
    # DRAM bytes of one launch of the dominant kernel as ncu measured them (read from the summary)
    prof = {("c3_bert_base_110m_student_t", "topk", "compress_fused"): "k_topk_single_c3_bert110m.md",
            ("c3_bert_base_110m_student_t", "threshold", "compress_fused"): "k_threshold_single_c3_bert110m.md",
            ("c2_resnet50_layerwise", "topk", "compress_fused"): "k_topk_multi_c2_resnet50.md",
            ("c4_resnet50_8workers", "topk", "compress_fused"): "k_topk_workers_c4_resnet50_8workers.md",
            ("c4_resnet50_8workers", "threshold", "compress_fused"): "k_threshold_workers_c4_resnet50_8workers.md",
            }.get((w.name, args.mode, dom) if args.grad_dtype == "f32" else None)
    ncu_traffic, ncu_src = profile_traffic(prof) if prof else (None, None)

    # CPU baseline: the oracle on a bounded sample of the same workload
    cpu = None if args.no_cpu_baseline else cpu_baseline(w)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "mode": args.mode, "grad_dtype": args.grad_dtype, "elements": n, "k": k, "density": w.density, "workers": W,
                   "tensors": len(w.sizes), "input_sets": sets,
                   "l2": "inputs larger than L2 (no flush): each gradient and residual is %d MB" % (4 * n >> 20)},
        "timing": {"what": "the K-step loop (barrier + synchronize on both sides, CUDA events on the launching stream) "
                           "is repeated until about one second of device time has passed; ms_per_step is the median loop",
                   "loops": len(res["plain"]), "ms_per_step_min": ms_lo, "ms_per_step_max": ms_hi,
                   "timed_region_ms_per_loop": ms_step * args.steps},
        "elements_per_s": n * W * world / t_step,
        "hbm_frac_of_8TBs": {"step": (cb + db) / NOMINAL_HBM / t_step,
                             "min_bytes_compress": cb, "min_bytes_decode": db,
                             "compress_only": cb / NOMINAL_HBM / (ms_compress * 1e-3),
                             "compress_ms_per_step": ms_compress,
                             "decode_only": db / NOMINAL_HBM / (ms_decode * 1e-3),
                             "decode_ms_per_step": ms_decode},
        "ms_per_step_with_kernel_events": res["with_events"] / args.steps,
        "kernels": breakdown,
        "roofline": {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": ncu_traffic, "peak_source": peak_src,
                     "traffic_source": ncu_src,
                     "algorithmic_bytes_per_launch": alg_bytes.get(dom),
                     "workers_per_launch": workers_per_launch if dom == "compress_fused" else None},
        "cpu_baseline": cpu,
        "e2e": None if not e2e_steps else {"value": grad_bytes_step * e2e_steps / (ms_e2e * 1e-3) / 1e9, "unit": UNIT,
                "h2d_bytes_per_step": 4 * n * W, "d2h_bytes_per_step": 8 * k * W,
                "ms_per_step": ms_e2e / e2e_steps, "steps": e2e_steps,
                "what": "gc_compress_host: pinned host gradient -> device (two staging buffers alternate, the copy "
                        "runs on the plan's copy stream), compress, pairs -> pinned host; decode stays on the device"},
        "fused_phase_us_last_step": [round(x, 2) for x in res["phase_us"]],
        "gpu_launches": res["launches_per_loop"],
        "path_counters": {"candidates_last_step": counters[0], "candidate_overflow": counters[1],
                          "tensors_redone": counters[2], "k": k},
        "clocks": clocks,
    }
    if res.get("apply"):
        ab = 16 * n + 8 * k * W                    # read and write parameter and velocity, read the pairs
        line["fused_decode_momentum"] = {"ms_per_call": res["apply"], "bytes": ab,
                                         "GB_per_s": ab / (res["apply"] * 1e-3) / 1e9,
                                         "frac_of_measured_peak": ab / (res["apply"] * 1e-3) / 1e9 / peak}
    if others:
        line["configs"] = others
    print(json.dumps(line))


# --------------------------------------------------------------------------- erasure-coded embedding tables
def run_ecrm(args, rank: int, world: int, local_rank: int):
    """Second workload (`--workload ecrm`): the server-side work of erasure-coded embedding-table
    training on one GPU that plays data server and parity host.  A step = optimizer on the m rows
    a batch touched (differences out) + the parity host adding them; the encoder, the full-shard
    decoder and degraded reads are timed beside it.  Prints its own JSON line."""
    from paper_2104_01981_b200 import ecrm
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    n_rows, p_rows, m, dim, k = args.ecrm_rows, args.ecrm_rows // 4, args.ecrm_batch, 128, 4
    peak, peak_src = measured_peak_gbs()
    entry = synth.ecrm_tables(n_rows, dim, 1, seed=1, device=dev)[0]
    state = torch.zeros(n_rows, dim, device=dev)
    p_entry = torch.zeros(p_rows, dim, device=dev)
    p_state = torch.zeros(p_rows, dim, device=dev)
    sets = []
    for sidx in range(4):                                  # distinct batches cycled through (each 0.5 GB: larger than L2)
        rows, g = synth.ecrm_batch(n_rows, m, dim, seed=10 + sidx, device="cpu")
        prow = torch.from_numpy((rows.numpy().view(np.uint32) % np.uint32(p_rows)).astype(np.uint32).view(np.int32))
        # parity rows must be distinct inside one call: keep the first occurrence of each
        _, first = np.unique(prow.numpy(), return_index=True)
        keep = torch.from_numpy(np.sort(first))
        sets.append((rows[keep].to(dev), g[keep].to(dev), prow[keep].to(dev)))
    m_eff = min(s[0].numel() for s in sets)
    sets = [(r[:m_eff].contiguous(), g[:m_eff].contiguous(), pr[:m_eff].contiguous()) for r, g, pr in sets]
    de = torch.empty(m_eff, dim, device=dev)
    ds = torch.empty(m_eff, dim, device=dev)
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        for i in range(args.warmup):
            fn(i)
        barrier()
        e0.record(stream)
        for i in range(steps):
            fn(args.warmup + i)
        e1.record(stream)
        barrier()
        return e0.elapsed_time(e1)

    def step(i):
        rows, g, prow = sets[i % len(sets)]
        ecrm.rows_step(ecrm.ECRM_MOMENTUM, rows, g, entry, state, 0.01, 0.9, de, ds, None, stream)
        ecrm.parity_add(prow, de, ds, p_entry, p_state, None, stream)

    def only_step(i):
        rows, g, _ = sets[i % len(sets)]
        ecrm.rows_step(ecrm.ECRM_MOMENTUM, rows, g, entry, state, 0.01, 0.9, de, ds, None, stream)

    def only_add(i):
        ecrm.parity_add(sets[i % len(sets)][2], de, ds, p_entry, p_state, None, stream)

    def fused_step(i):
        rows, g, prow = sets[i % len(sets)]
        ecrm.rows_step_parity(ecrm.ECRM_MOMENTUM, rows, prow, g, entry, state, p_entry, p_state, 0.01, 0.9, None, stream)

    clocks = ClockSampler(local_rank, os.path.join(tempfile.gettempdir(), f"gc_clocks_ecrm_{rank}.csv"))
    ms = timed(step, args.steps)
    ms_fused = timed(fused_step, args.steps)
    ms_step = timed(only_step, args.steps)
    ms_add = timed(only_add, args.steps)
    # encoder / decoder over whole shards (k = 4 shards of 1 GiB), degraded reads of m rows
    shard_n = min(n_rows, 2 * 1024 * 1024) * dim
    shards = [entry.view(-1)[:shard_n]] + [torch.randn(shard_n, device=dev) for _ in range(k - 1)]
    parity = torch.empty(shard_n, device=dev)
    out = torch.empty(shard_n, device=dev)
    n_cd = max(3, args.steps // 10)
    ms_enc = timed(lambda i: ecrm.encode(shards, parity, stream), n_cd)
    ms_dec = timed(lambda i: ecrm.decode(shards[1:], parity, out, stream), n_cd)
    rd_rows = (sets[0][0].view(torch.int32) % (shard_n // dim)).contiguous()
    rd_out = torch.empty(m_eff, dim, device=dev)
    sh2 = [x.view(-1, dim) for x in shards]
    ms_rd = timed(lambda i: ecrm.degraded_read(rd_rows, None, sh2[1:], parity.view(-1, dim), rd_out, None, stream), n_cd)
    clk = clocks.stop()
    ms, ms_step, ms_add, ms_enc, ms_dec, ms_rd, ms_fused = reduce_max_over_ranks(
        [ms, ms_step, ms_add, ms_enc, ms_dec, ms_rd, ms_fused], world, dev)
    if rank != 0:
        return
    row_b = dim * 4
    bytes_step = m_eff * (7 * row_b + 4)          # g, e, s read; e, s, de, ds written; row number
    bytes_add = m_eff * (6 * row_b + 4)           # de, ds read; parity entry and state read + written
    upd_gbs = (bytes_step + bytes_add) * world * args.steps / (ms * 1e-3) / 1e9
    step_gbs = bytes_step / (ms_step / args.steps * 1e-3) / 1e9
    cpu = None
    if not args.no_cpu_baseline:
        from oracle import ecrm_oracle as eo
        srows, sg, sprow = (t[:20000].cpu() for t in sets[0])
        he, hs = entry[:].cpu().numpy(), np.zeros((n_rows, dim), np.float32)
        hp, hps = np.zeros((p_rows, dim), np.float32), np.zeros((p_rows, dim), np.float32)
        t0 = time.perf_counter()
        d1, d2 = eo.rows_step(eo.MOMENTUM, srows.numpy().view(np.uint32), sg.numpy(), he, hs, 0.01, 0.9)
        eo.parity_add(sprow.numpy().view(np.uint32), d1, d2, hp, hps)
        dt = time.perf_counter() - t0
        cpu = {"value": 20000 * (13 * row_b + 8) / dt / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle",
               "sample": "20000 rows of one batch: optimizer step + parity add, numpy row by row"}
    line = {
        "metric": "ecrm_update_traffic_GB_per_s", "value": upd_gbs, "unit": "GB/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "ecrm_embedding_rows", "rows": n_rows, "parity_rows": p_rows, "dim": dim,
                   "rows_per_batch": m_eff, "optimizer": "momentum", "k": k,
                   "l2": "four batches of 0.5 GB cycled; tables of several GB (no flush)"},
        "rows_per_s": m_eff * world * args.steps / (ms * 1e-3),
        "kernels": {
            "rows_step": {"ms_per_launch": ms_step / args.steps, "GB_per_s": step_gbs},
            "rows_step_parity_fused": {"ms_per_launch": ms_fused / args.steps,
                                       "bytes": m_eff * (9 * row_b + 8),     # g, e, s, pe, ps read; e, s, pe, ps written
                                       "GB_per_s": m_eff * (9 * row_b + 8) / (ms_fused / args.steps * 1e-3) / 1e9,
                                       "rows_per_s": m_eff * world * args.steps / (ms_fused * 1e-3),
                                       "what": "ecrm_rows_step_parity: the same update when data and parity shard share the "
                                               "GPU (the differences stay in registers)"},
            "parity_add": {"ms_per_launch": ms_add / args.steps,
                           "GB_per_s": bytes_add / (ms_add / args.steps * 1e-3) / 1e9},
            "encode_k4": {"ms_per_launch": ms_enc / n_cd, "GB_per_s": (k + 1) * 4 * shard_n / (ms_enc / n_cd * 1e-3) / 1e9},
            "decode_k4": {"ms_per_launch": ms_dec / n_cd, "GB_per_s": (k + 1) * 4 * shard_n / (ms_dec / n_cd * 1e-3) / 1e9},
            "degraded_read_k4": {"ms_per_launch": ms_rd / n_cd,
                                 "GB_per_s": m_eff * ((k + 1) * row_b + 4) / (ms_rd / n_cd * 1e-3) / 1e9},
        },
        "roofline": {"bound": "hbm", "kernel": "rows_step", "achieved": step_gbs, "peak": peak, "unit": "GB/s",
                     "frac": step_gbs / peak, "traffic": m_eff * 3430.4, "peak_source": peak_src,
                     "traffic_source": "profiles/k_ecrm_rows_step_2m_rows_dim128.md (3430 B per row, scaled by rows)",
                     "algorithmic_bytes_per_launch": bytes_step},
        "cpu_baseline": cpu, "e2e": None, "gpu_launches": 2 * args.steps, "clocks": clk,
    }
    print(json.dumps(line))



# --------------------------------------------------------------------------- multi-GPU aggregation
def run_exchange(args, w: synth.Workload, rank: int, world: int, local_rank: int):
    """Third workload (`--workload exchange`): every rank is ONE worker.  A step = compress this
    rank's gradient into its exchange block, one NCCL all-gather of the blocks, decode of the
    `world` gathered lists in rank order.  At one GPU the group has one rank (the collective is
    a local copy inside NCCL).  Prints its own JSON line."""
    from paper_2104_01981_b200 import api, exchange
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    api.lib()
    mode = api.GC_THRESHOLD if args.mode == "threshold" else api.GC_TOPK
    plan = api.Plan(w.sizes, w.density, mode=mode, device=local_rank)
    n, k = plan.total_n, plan.total_cap
    stream = torch.cuda.current_stream()
    ex = exchange.PairExchange.for_plan(plan)
    sets = max(1, min(args.input_sets, int(24e9 // (4 * n)) or 1))
    grads = [synth.gradient(w, 100 * rank, s, device=dev) for s in range(sets)]
    resid = torch.zeros(n, dtype=torch.float32, device=dev)
    ws = plan.alloc_workspace()
    dense = torch.empty(n, dtype=torch.float32, device=dev)
    oi, ov, oc = ex.outputs()
    thr = mode == api.GC_THRESHOLD

    def do_compress(i):
        plan.compress(grads[i % sets], resid, oi, ov, oc if thr else None, ws, stream)

    def do_gather(i):
        ex.all_gather()

    def do_decode(i):
        ex.decode(plan, dense, True, ws, stream)

    def step(i):
        do_compress(i); do_gather(i); do_decode(i)

    def barrier():
        torch.distributed.barrier()
        torch.cuda.synchronize()

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn):
        barrier()
        e0.record(stream)
        for i in range(args.steps):
            fn(args.warmup + i)
        e1.record(stream)
        barrier()
        return e0.elapsed_time(e1)

    for i in range(args.warmup):
        step(i)
    launches0 = plan.launches()
    sampler = ClockSampler(local_rank, os.path.join("/tmp", f"gc_bench_clocks_{os.getpid()}.csv")) \
        if rank == 0 else None
    ms = timed(step)
    launches = plan.launches() - launches0
    legs = [timed(do_compress), timed(do_gather), timed(do_decode)]
    clocks = sampler.stop() if sampler else None
    st, det = plan.last_status(ws)
    if st not in (api.GC_OK, api.GC_W_TRUNCATED):
        raise RuntimeError(f"device status {st} (detail {det}) after the timed region")
    ms, *legs = reduce_max_over_ranks([ms] + legs, world, dev)
    if rank != 0:
        return
    peak, peak_src = measured_peak_gbs()
    t_step = ms * 1e-3 / args.steps
    wire = ex.bytes_on_wire_per_rank()
    line = {
        "metric": METRIC, "value": whole_job_value(n, 1, world, args.steps, ms), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name + "_exchange", "mode": args.mode, "elements": n, "k": k, "density": w.density,
                   "workers": world, "workers_per_rank": 1, "tensors": len(w.sizes), "input_sets": sets,
                   "collective": "all_gather_into_tensor (NCCL) of one fixed-size block per rank",
                   "l2": f"inputs larger than L2 (no flush): each gradient and residual is {4 * n / 1e6:.0f} MB"},
        "legs_ms_per_step": {"compress": legs[0] / args.steps, "all_gather": legs[1] / args.steps,
                             "decode": legs[2] / args.steps},
        "exchange": {"block_bytes": 4 * ex.layout.words, "bytes_received_per_rank": wire,
                     "all_gather_GB_per_s_per_rank": (wire / (legs[1] * 1e-3 / args.steps) / 1e9) if wire else None},
        "roofline": {"bound": "hbm", "kernel": "step (compress + decode of `world` lists)",
                     "achieved": (12.0 * n + 8.0 * k + 4.0 * n + 8.0 * k * world) / t_step / 1e9, "peak": peak,
                     "unit": "GB/s", "frac": (12.0 * n + 8.0 * k + 4.0 * n + 8.0 * k * world) / t_step / 1e9 / peak,
                     "traffic": None, "peak_source": peak_src},
        "cpu_baseline": None, "e2e": None, "gpu_launches": launches, "clocks": clocks,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- decode sweep
def run_decode_sweep(args, w: synth.Workload, rank: int, world: int, local_rank: int):
    """Fourth workload (`--workload decode`): gc_decompress_accumulate alone on W seeded sparse sets
    shaped like the workload's top-k output (a flat tensor of the workload's size and density), for
    every W in --decode-workers and each of the two tiled decode kernels.  Prints its own JSON line."""
    from paper_2104_01981_b200 import api
    if rank != 0:
        return
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    api.lib()
    n = w.total_n
    plan = api.Plan([n], w.density, device=local_rank)
    k = plan.total_cap
    ws = plan.alloc_workspace()
    dense = torch.empty(n, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    peak, peak_src = measured_peak_gbs()
    Ws = [int(x) for x in args.decode_workers.split(",")]
    idx, val = [], []
    for wk in range(max(Ws)):
        i, v = synth.sparse_set([n], [k], 4000 + wk)
        idx.append(torch.from_numpy(i.view(np.int32)).to(dev)); val.append(torch.from_numpy(v).to(dev))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    routes = {"auto": api.GC_DECODE_AUTO, "narrow": api.GC_DECODE_NARROW, "wide": api.GC_DECODE_WIDE}
    rows = []
    for W in Ws:
        row = {"workers": W, "bytes": 4 * n + 8 * k * W}
        for name, code in routes.items():
            plan.set_option(api.GC_OPT_DECODE_ROUTE, code)
            for _ in range(max(args.warmup, 3)):
                plan.decompress_accumulate(idx[:W], val[:W], None, dense, True, ws, stream)
            torch.cuda.synchronize()
            e0.record(stream)
            for _ in range(args.steps):
                plan.decompress_accumulate(idx[:W], val[:W], None, dense, True, ws, stream)
            e1.record(stream)
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) / args.steps * 1e3
            row[name + "_us"] = us
            row[name + "_frac_of_measured_peak"] = row["bytes"] / us / 1e3 / peak
        # no fixed order among the workers (within 1e-6 relative of the fixed-order sum up to 16 workers)
        plan.set_option(api.GC_OPT_DECODE_ROUTE, api.GC_DECODE_AUTO)
        plan.set_option(api.GC_OPT_DECODE_ORDER, api.GC_ORDER_ANY)
        for _ in range(max(args.warmup, 3)):
            plan.decompress_accumulate(idx[:W], val[:W], None, dense, True, ws, stream)
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(args.steps):
            plan.decompress_accumulate(idx[:W], val[:W], None, dense, True, ws, stream)
        e1.record(stream)
        torch.cuda.synchronize()
        row["any_order_us"] = e0.elapsed_time(e1) / args.steps * 1e3
        plan.set_option(api.GC_OPT_DECODE_ORDER, api.GC_ORDER_FIXED)
        rows.append(row)
    st, det = plan.last_status(ws)
    if st != api.GC_OK:
        raise RuntimeError(f"device status {st} (detail {det})")
    print(json.dumps({"workload": w.name + "_decode_sweep", "elements": n, "pairs_per_worker": k, "density": w.density,
                      "steps": args.steps, "peak_GB_per_s": peak, "peak_source": peak_src, "rows": rows,
                      "l2": "dense buffer larger than L2 (no flush)"}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=2, help="workload 0..4 (default 2: 110M BERT-base shape)")
    ap.add_argument("--impl", default="gc", choices=["gc", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--configs", default="all", choices=["all", "none"],
                    help="all: after the headline workload, time the other four workloads (and the threshold variant "
                         "of the 8-worker one) and report them under `configs`; none: headline only")
    ap.add_argument("--min-loop-ms", type=float, default=1000.0,
                    help="repeat every K-step loop until this much device time has passed (median loop reported)")
    ap.add_argument("--path", default="auto", choices=["auto", "staged", "exact"],
                    help="auto: one-pass candidate path in one cooperative launch (default); staged: the "
                         "same phases as separate launches; exact: multi-pass kernels only")
    ap.add_argument("--mode", default="topk", choices=["topk", "threshold"],
                    help="selection mode (threshold = the sampled-threshold variant)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end region")
    ap.add_argument("--input-sets", type=int, default=N_INPUT_SETS,
                    help="distinct gradients per worker cycled through (1 keeps profiler captures small)")
    ap.add_argument("--grad-dtype", default="f32", choices=["f32", "bf16"],
                    help="storage type of the gradient (bf16: gc_compress_bf16, 10n + 8k bytes per compress; no e2e leg)")
    ap.add_argument("--decode-workers", default="1,2,4,8,16,32", help="worker counts of --workload decode")
    ap.add_argument("--workload", default="gc", choices=["gc", "ecrm", "exchange", "decode"],
                    help="gc: gradient compression (the headline line); ecrm: erasure-coded embedding-table rows; "
                         "exchange: one worker per rank, NCCL all-gather of the pairs, decode of all ranks' lists; "
                         "decode: the decode alone for several worker counts and both tiled kernels")
    ap.add_argument("--ecrm-rows", type=int, default=8 * 1024 * 1024, help="rows of the embedding-table shard")
    ap.add_argument("--ecrm-batch", type=int, default=1024 * 1024, help="distinct rows one batch updates")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "gc" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    w = synth.workload(args.config)
    if args.impl == "reference":
        run_reference(args, w, rank)
        return
    group = world > 1 or args.workload == "exchange"
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    elif group:                                  # a one-rank group, so that the collective itself runs
        rdv = os.path.join(tempfile.mkdtemp(prefix="gc_bench_"), "rendezvous")
        torch.distributed.init_process_group("nccl", init_method=f"file://{rdv}", rank=0, world_size=1,
                                             device_id=torch.device(f"cuda:{local_rank}"))
    try:
        if args.workload == "ecrm":
            run_ecrm(args, rank, world, local_rank)
        elif args.workload == "exchange":
            run_exchange(args, w, rank, world, local_rank)
        elif args.workload == "decode":
            run_decode_sweep(args, w, rank, world, local_rank)
        else:
            run_gpu(args, w, rank, world, local_rank)
    finally:
        if group:
            torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()

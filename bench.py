#!/usr/bin/env python
"""Benchmark of the LGC compression step (accumulate -> top-k -> gather -> encode -> combine ->
decode -> scatter) on synthetic ResNet-50-shaped gradients, K = 8 simulated nodes per GPU.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints ONE JSON line.  metric = dense-gradient GB/s compressed and reconstructed per step
(K * N * 4 bytes / step time, summed over GPUs).  With --gpus N > 1 (under torchrun) every rank
runs an independent replica of the workload: the path has no cross-GPU exchange step.
`--impl reference` times the CPU oracle, as it stands, on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2103_08870_b200 import workloads as W  # noqa: E402

METRIC = "dense_gradient_GBps_compressed_and_reconstructed_per_step"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
GRAD_SETS = 3            # distinct gradient batches cycled through (each far larger than L2)
CLOCK_WINDOW_MS = 500.0  # the clock sampler watches at least this long a run of steps (see run_ours)
# DRAM bytes (read + write) per element that one ncu capture measured for the dominant kernel on a small
# case (K = 2 nodes of the same layer table; traffic grows in proportion to K * N), with the SHA-256 of the
# kernel's source file as it was when the counters were taken.  While the file differs from that, the
# figure is not reported ("traffic": null): the kernel has changed since.
NCU_CAPTURE = {
    "kernel": "accumulate_select_kernel",
    # the kernel's source and the headers it is built from; the digest is over their bytes, in this order
    "sources": [os.path.join("paper_2103_08870_b200", "csrc", n)
                for n in ("lgc_select_fast.cu", "lgc_select_common.cuh", "lgc_internal.cuh")],
    "sources_sha256": "0e3a7186a36d74f3181d4f637b6ea77c44f9669739b802759f19065fc33650a3",
    "dram_bytes_per_element": 19.02,
}


def ncu_traffic_bytes(elements: int):
    """DRAM traffic of one launch over `elements` elements from the stored capture, or None when the
    kernel's sources are no longer the ones that were measured."""
    import hashlib
    if not NCU_CAPTURE["sources_sha256"] or NCU_CAPTURE["dram_bytes_per_element"] is None:
        return None
    h = hashlib.sha256()
    try:
        for name in NCU_CAPTURE["sources"]:
            with open(os.path.join(ROOT, name), "rb") as f:
                h.update(f.read())
    except OSError:
        return None
    return NCU_CAPTURE["dram_bytes_per_element"] * elements if h.hexdigest() == NCU_CAPTURE["sources_sha256"] else None


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while a region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


class NvmlClockSampler:
    """The same through NVML (read-only queries), polled from a thread every few milliseconds: a timed
    region of a fraction of a second still gets tens of samples."""

    def __init__(self, index: int):
        import pynvml
        self.nv = pynvml
        self.REASONS = (("hw_slowdown", pynvml.nvmlClocksThrottleReasonHwSlowdown),
                        ("hw_thermal_slowdown", pynvml.nvmlClocksThrottleReasonHwThermalSlowdown),
                        ("sw_thermal_slowdown", pynvml.nvmlClocksThrottleReasonSwThermalSlowdown),
                        ("sw_power_cap", pynvml.nvmlClocksThrottleReasonSwPowerCap))
        pynvml.nvmlInit()
        self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
        self.sm, self.bits, self.stop_flag = [], 0, False

    def start(self):
        self.thread = threading.Thread(target=self._poll, daemon=True)
        self.thread.start()

    def _poll(self):
        nv = self.nv
        while not self.stop_flag:
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                self.bits |= int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
            except Exception:
                pass
            time.sleep(0.003)

    def stop(self):
        self.stop_flag = True
        self.thread.join(timeout=2)
        mx = None
        try:
            mx = float(self.nv.nvmlDeviceGetMaxClockInfo(self.h, self.nv.NVML_CLOCK_SM))
        except Exception:
            pass
        return {"sm_mhz": statistics.median(self.sm) if self.sm else None, "sm_max_mhz": mx, "samples": len(self.sm),
                "reasons": sorted(name for name, bit in self.REASONS if self.bits & bit), "source": "nvml"}


def clock_sampler(index: int):
    try:
        return NvmlClockSampler(index)
    except Exception:
        return ClockSampler(index)


def visible_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


def host_description():
    """Core count, CPU model and memory of the machine the oracle is timed on."""
    model = "unknown"
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    ram = None
    try:
        import psutil
        ram = round(psutil.virtual_memory().total / 2**30, 1)
    except Exception:
        pass
    try:
        usable = len(os.sched_getaffinity(0))
    except Exception:
        usable = os.cpu_count()
    return {"nproc": os.cpu_count(), "usable_cores": usable, "cpu_model": model, "ram_gib": ram}


def make_oracle(w: W.Workload, threads: int):
    """The oracle of the workload.  threads > 1: the same object with its two loops over independent units --
    nodes in the accumulation, (node, layer) pairs in the selection -- handed to a thread pool.  Every unit
    calls the same oracle function on the same slices as the sequential loop does (ctypes releases the
    interpreter lock during the call); no arithmetic changes, results are identical."""
    from oracle import OracleLGC
    import oracle as O
    import numpy as np
    params = w.init_params().numpy()
    kw = dict(density_ppm=w.density_ppm, momentum=w.momentum, variant=w.variant, ae_kind=w.ae_kind, c1=w.ae_c1,
              c2=w.ae_c2, params=params, innovation_permille=w.innovation_permille)
    if threads <= 1:
        return OracleLGC(w.table.numel, w.num_nodes, **kw), None
    from concurrent.futures import ThreadPoolExecutor
    pool = ThreadPoolExecutor(max_workers=threads)

    class PooledOracle(OracleLGC):
        def accumulate(self, g):
            assert g.shape == (self.K, self.N) and g.dtype == np.float32
            # a node's row is cut into pieces so that all cores have work when K is small
            pieces = max(1, (threads + self.K - 1) // self.K)
            edges = np.linspace(0, self.N, pieces + 1).astype(np.int64)
            jobs = [(k, int(a), int(b)) for k in range(self.K) for a, b in zip(edges[:-1], edges[1:]) if b > a]
            list(pool.map(lambda j: O.accumulate(self.u[j[0], j[1]:j[2]], self.v[j[0], j[1]:j[2]],
                                                 np.ascontiguousarray(g[j[0], j[1]:j[2]]), float(self.m)), jobs))

        def _select(self, k):
            out = np.empty(self.mu, dtype=np.int32)

            def one(l):
                a, b = int(self.off[l]), int(self.off[l + 1])
                out[self.koff[l]:self.koff[l + 1]] = O.topk(self.v[k, a:b], self.k_l[l], base=a, method=self.topk_method)
            list(pool.map(one, range(self.L)))
            return out

        def topk(self, leader=0):
            if self.variant == "rar":
                self.idx = np.broadcast_to(self._select(leader), (self.K, self.mu)).copy()
            else:
                self.idx = np.stack(list(pool.map(self._select_serial, range(self.K))))
            self.val = np.stack([O.gather(self.v[k], self.idx[k]) for k in range(self.K)])

        def _select_serial(self, k):
            return OracleLGC._select(self, k)

    return PooledOracle(w.table.numel, w.num_nodes, **kw), pool


def oracle_throughput(w: W.Workload, sample_steps: int, host_grads=None, threads: int = 1):
    """The oracle, as it stands, on `sample_steps` whole steps of the workload (host cores).
    `host_grads`: gradient batches (numpy [K][N]) to cycle through; generated on the CPU if absent."""
    if host_grads is None:
        src = W.GradientSource(w.table, w.num_nodes, seed=w.seed)
        host_grads = [src.step(t).numpy() for t in range(min(GRAD_SETS, sample_steps))]
    ora, pool = make_oracle(w, threads)
    times = []
    for t in range(sample_steps):
        g = host_grads[t % len(host_grads)]
        t0 = time.perf_counter()
        ora.step(g, W.choice_for_step(w.seed, t, w.num_nodes))
        times.append(time.perf_counter() - t0)
    if pool is not None:
        pool.shutdown()
    bytes_per_step = w.num_nodes * w.table.total * 4
    return bytes_per_step / 1e9 / statistics.mean(times), times


def cpu_baseline_record(w: W.Workload, sample_steps: int, host_grads=None):
    """The reported CPU baseline: the oracle single-threaded (the figure `value` carries) and once more with
    its independent units on all usable cores."""
    host = host_description()
    gbs1, t1 = oracle_throughput(w, sample_steps, host_grads, threads=1)
    cores = int(host["usable_cores"] or 1)
    rec = {"value": gbs1, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": f"{len(t1)} whole steps of {w.name} (K={w.num_nodes}, N={w.table.total}), single thread",
           "s_per_step": statistics.mean(t1), "host": host}
    if cores > 1:
        gbsn, tn = oracle_throughput(w, sample_steps, host_grads, threads=cores)
        rec["all_cores"] = {"value": gbsn, "unit": UNIT, "cores": cores, "s_per_step": statistics.mean(tn),
                            "sample": f"{len(tn)} whole steps; nodes (accumulation) and (node, layer) pairs "
                                      f"(selection) on a pool of {cores} threads, same oracle functions"}
    return rec


def run_reference(args, w: W.Workload):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    total = args.steps + args.warmup
    gbs, times = oracle_throughput(w, total)
    timed = times[args.warmup:] or times
    value = w.num_nodes * w.table.total * 4 / 1e9 / statistics.mean(timed)
    base = {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{len(timed)} whole steps of {w.name} (K={w.num_nodes}, N={w.table.total}), single thread",
            "host": host_description()}
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": len(timed),
        "warmup": args.warmup, "ms_per_step": 1e3 * statistics.mean(timed), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(w), "cpu_baseline": base,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def workload_config(w: W.Workload):
    return {"workload": f"{w.name}: {len(w.table.numel)} tensors, N={w.table.total}, K={w.num_nodes} nodes per GPU, "
                        f"density {w.density_ppm} ppm, {w.variant}, AE "
                        + ("64/128/256/64/4 (full size)" if w.ae_kind == "conv5" else f"{w.ae_c1}/{w.ae_c2}"),
            "l2": f"inputs larger than L2: {w.num_nodes * w.table.total * 20 / 1e6:.0f} MB streamed per step, "
                  f"{GRAD_SETS} gradient batches cycled"}


def max_over_ranks(values, device, world: int):
    """Element-wise maximum of a list of floats over all ranks (identity for one rank)."""
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_gbs(num_nodes: int, numel: int, world: int, ms_per_step: float) -> float:
    """Dense-gradient GB/s of the whole job: every rank compresses K * N fp32 values per step."""
    return num_nodes * numel * 4 * world / 1e9 / (ms_per_step / 1e3)


def run_ours(args, w: W.Workload):
    from paper_2103_08870_b200 import lgc
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the LGC path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    K, N = w.num_nodes, w.table.total
    gpu = lgc.LGC(w.table.numel, K, density_ppm=w.density_ppm, momentum=w.momentum, variant=w.variant,
                  ae_kind=w.ae_kind, c1=w.ae_c1, c2=w.ae_c2, innovation_permille=w.innovation_permille, device=dev)
    gpu.set_ae_params(w.init_params())
    src = W.GradientSource(w.table, K, seed=w.seed + rank, device=dev)
    grads = [src.step(t) for t in range(GRAD_SETS)]
    update = torch.empty(N, dtype=torch.float32, device=dev)
    choices = [W.choice_for_step(w.seed, t, K) for t in range(args.steps + args.warmup)]

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for t in range(args.warmup):
        gpu.step(grads[t % GRAD_SETS], update, choices[t])
    gpu.check()
    barrier()

    sampler = clock_sampler(visible_gpu_index(local))
    sampler.start()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    launches_before = lgc.kernel_launches()
    start.record()
    for t in range(args.steps):
        i = args.warmup + t
        ev[t][0].record()
        gpu.accumulate(grads[i % GRAD_SETS], choices[i])
        ev[t][1].record()
        gpu.topk(choices[i], update)
        gpu.encode()
        gpu.combine(choices[i])
        gpu.decode_scatter(update)
    stop.record()
    gpu_launches = lgc.kernel_launches() - launches_before
    barrier()
    elapsed_ms = start.elapsed_time(stop)
    # A timed region of a few milliseconds is over before the sampler has read the clocks twice.  The same
    # steps therefore keep running, untimed, under the sampler until it has watched CLOCK_WINDOW_MS of this
    # load in all: the clocks reported are those of the timed steps and of their continuation.
    clock_window_ms = elapsed_ms
    t = args.steps
    while clock_window_ms < args.clock_window_ms:
        n = max(1, int((args.clock_window_ms - clock_window_ms) / max(elapsed_ms / args.steps, 1e-3)) + 1)
        for _ in range(n):
            i = args.warmup + t
            ch = W.choice_for_step(w.seed, i, K)
            gpu.step(grads[i % GRAD_SETS], update, ch)
            t += 1
        torch.cuda.synchronize(dev)
        clock_window_ms += n * elapsed_ms / args.steps
    extra_steps = t - args.steps
    clocks = sampler.stop()
    clocks["window"] = f"{args.steps} timed steps + {extra_steps} more of the same steps, about {clock_window_ms:.0f} ms under load"
    gpu.check()
    acc_ms = [a.elapsed_time(b) for a, b in ev]
    # every step's own time: from its first event to the next step's (the last one: to the closing event)
    step_ms = [ev[t][0].elapsed_time(ev[t + 1][0] if t + 1 < args.steps else stop) for t in range(args.steps)]

    # optional: the five stages' own times, on steps of their own after the timed region (an event between the
    # stage calls costs about a microsecond each, so they stay out of the reported step time)
    stages_us = None
    if args.stage_times:
        names = ("accumulate", "topk", "encode", "combine", "decode_scatter")
        marks = [[torch.cuda.Event(enable_timing=True) for _ in range(6)] for _ in range(min(args.steps, 50))]
        for t, m in enumerate(marks):
            i = args.warmup + args.steps + extra_steps + t
            ch = W.choice_for_step(w.seed, i, K)
            m[0].record(); gpu.accumulate(grads[i % GRAD_SETS], ch)
            m[1].record(); gpu.topk(ch, update)
            m[2].record(); gpu.encode()
            m[3].record(); gpu.combine(ch)
            m[4].record(); gpu.decode_scatter(update)
            m[5].record()
        barrier()
        gpu.check()
        stages_us = {n: 1e3 * statistics.median(m[j].elapsed_time(m[j + 1]) for m in marks) for j, n in enumerate(names)}

    # end to end through host buffers: pinned gradients in, dense update out, every step
    e2e_steps = 0 if args.no_e2e else max(2, min(args.steps, 20))
    e2e_ms = 0.0
    if e2e_steps:
        host_g = torch.empty((K, N), dtype=torch.float32).pin_memory()
        host_g.copy_(grads[0])
        host_u = torch.empty(N, dtype=torch.float32).pin_memory()
        dev_g = torch.empty((K, N), dtype=torch.float32, device=dev)
        gpu.step_host(host_g, dev_g, update, host_u, choices[0])
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for t in range(e2e_steps):
            gpu.step_host(host_g, dev_g, update, host_u, choices[t])
        e1.record()
        barrier()
        e2e_ms = e0.elapsed_time(e1)

    elapsed_ms, e2e_ms, acc_mean_ms = max_over_ranks([elapsed_ms, e2e_ms, statistics.mean(acc_ms)], dev, world)

    if rank == 0:
        value = whole_job_gbs(K, N, world, elapsed_ms / args.steps)
        e2e_value = whole_job_gbs(K, N, world, e2e_ms / e2e_steps) if e2e_steps else None
        peak, peak_kind = measured_peak()
        acc_bytes = 20 * K * N
        achieved = acc_bytes / 1e9 / (acc_mean_ms / 1e3)
        step_bytes = 20 * K * N + 4 * N
        step_gbs = step_bytes / 1e9 / (elapsed_ms / 1e3 / args.steps)
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": workload_config(w),
            "roofline": {"bound": "hbm", "kernel": "accumulate_select_kernel", "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                         "traffic": ncu_traffic_bytes(K * N),
                         "algorithmic_bytes_per_launch": acc_bytes,
                         "kernel_ms": acc_mean_ms},
            "step_hbm": {"algorithmic_bytes": step_bytes, "achieved_GBps": step_gbs,
                         "frac_of_measured_peak": step_gbs / peak, "frac_of_nominal_8TBps": step_gbs / NOMINAL_HBM_GBS},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": K * N * 4, "d2h_bytes_per_step": N * 4,
                    "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps if e2e_steps else None},
            "step_ms": {"min": min(step_ms), "median": statistics.median(step_ms), "max": max(step_ms)},   # this rank's steps
            "gpu_launches": gpu_launches,
            "clocks": clocks,
        }
        if stages_us is not None:
            out["stages_us"] = stages_us        # medians, this rank
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline_record(w, args.cpu_sample_steps, [g.cpu().numpy() for g in grads])
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet50", choices=list(W.WORKLOAD_NAMES))
    ap.add_argument("--cpu-sample-steps", type=int, default=12)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--nodes", type=int, default=0, help="override K (profiling aid: a smaller device footprint)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling aid)")
    ap.add_argument("--clock-window-ms", type=float, default=CLOCK_WINDOW_MS,
                    help="how long a run of steps the clock sampler watches (profiling aid: 0 = the timed steps only)")
    ap.add_argument("--stage-times", action="store_true", help="also report the median time of each of the five stages")
    args = ap.parse_args()
    w = W.workload(args.workload)
    if args.nodes > 0:
        w.num_nodes = args.nodes
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the Sparbit step executor on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one whole allgather (own-block copy + all ceil(log2 P) schedule steps) over P = 256
virtual ranks with m = 64 KiB blocks: 4 GiB of receive buffers, 2*P*(P-1)*m = 8.556 GB moved.
Prints ONE JSON line.  The metric is effective GB/s = 2*P*(P-1)*m / time per collective.

With N > 1 (launched under torch.distributed.run) every rank runs an independent replica of the
same collective on its own GPU ("replicas only": the path has no exchange between GPUs); the
value is the sum over ranks divided by the slowest rank's time.

`--impl reference` times the CPU oracle (the plain simulator under oracle/) on the host cores, on
a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import seeded_inputs as si  # noqa: E402

P_DEFAULT, M_DEFAULT = 256, 64 * 1024
METRIC = "sparbit_allgather_effective_GBps"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 7700.0  # HBM3e of the HGX B200 (8000 on DGX); context only, not the roofline's peak

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from ncu captures
# of this benchmark's own kernels: bytes, and the summary under profiles/ that holds the capture's
# command and figures (a configuration that is not listed was not captured: traffic = null)
NCU_TRAFFIC = {
    # persistent_bulk_kernel, whole collective: 4.16 GB read + 4.25 GB written
    "sparbit:P256:m65536:persistent:bulk": (8.41e9, "profiles/phase_bulk_kernel_last_phase_P256_m64k_traffic.md"),
    # phase_bulk_kernel, last phase: 2.15 GB read + 2.10 GB written
    "sparbit:P256:m65536:graph:bulk": (4.25e9, "profiles/phase_bulk_kernel_last_phase_P256_m64k_traffic.md"),
    # config 3: flow_vec_kernel, whole collective; last pass of the per-pass kernels of either engine
    "sparbit:P128:m65536:flow:vector": (1.997e9, "profiles/phase_kernels_and_flow_kernel_P128_m64k.md"),
    "sparbit:P128:m65536:graph:bulk": (1.026e9, "profiles/phase_kernels_and_flow_kernel_P128_m64k.md"),
    "sparbit:P128:m65536:graph:vector": (1.029e9, "profiles/phase_kernels_and_flow_kernel_P128_m64k.md"),
    # config 4: flow_vec_kernel, whole collective; last pass of phase_vec_kernel
    "sparbit:P1000:m1024:flow:vector": (1.89e9, "profiles/phase_vec_and_flow_kernel_P1000_m1k.md"),
    "sparbit:P1000:m1024:graph:vector": (9.79e8, "profiles/phase_vec_and_flow_kernel_P1000_m1k.md"),
    # config 5, small blocks: last pass of phase_vec_kernel (captured alone, caches cold)
    "sparbit:P256:m4096:flow:vector": (3.72e8, "profiles/flow_vec_kernel_P256_m4k.md"),
    "sparbit:P256:m4096:graph:vector": (2.21e8, "profiles/phase_vec_kernel_P256_small_blocks.md"),
    "sparbit:P256:m512:graph:vector": (1.68e7, "profiles/phase_vec_kernel_P256_small_blocks.md"),
    "sparbit:P256:m64:graph:vector": (4.21e6, "profiles/phase_vec_kernel_P256_small_blocks.md"),
    "sparbit:P256:m8:graph:vector": (5.36e5, "profiles/phase_vec_kernel_P256_small_blocks.md"),
}
MIN_TIMED_MS = 500.0   # the timed rounds together last at least this long, whatever --steps is


def effective_bytes(P: int, m: int) -> int:
    return 2 * P * (P - 1) * m


def algorithmic_bytes(P: int, m: int, fused_first: bool = True) -> int:
    """Bytes one collective must read plus write: every delivered block is written once and read
    once (2*P*(P-1)*m), and the own block gets into place.  With the own-block copy fused into the
    first step (sendbuf[r] read once, written to two places; Sparbit, ring, neighbor exchange and
    recursive doubling) that costs P*m more; as a separate copy (Bruck) it costs 2*P*m."""
    return 2 * P * (P - 1) * m + (P * m if fused_first else 2 * P * m)


def measured_peak():
    f = ROOT / "MEASURED_PEAKS.json"
    if f.exists():
        try:
            return float(json.loads(f.read_text())["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            pass
        rows = [l for (t, l) in self.lines if t0 <= t <= t1 + 0.2] or [l for (_, l) in self.lines]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in rows:
            f = [x.strip() for x in l.split(",")]
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
                for n, v in zip(names, f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                continue
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(x: float, device, use_dist: bool) -> float:
    """Largest value of x over all ranks (device timings are reported as the slowest rank's)."""
    if not use_dist:
        return float(x)
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


HEAD_START_BELOW_US = 100.0   # collectives shorter than this are timed behind a device-side delay
HEAD_START_CYCLES = 4_000_000  # about 2 ms at 1965 MHz: 50 collectives of six launches each are queued long before


def head_start(us_per_collective):
    """A short collective takes the GPU less time than the host needs to launch it (3-4 us per call
    through the binding), so a loop of them would time the host.  Called right before the first
    time stamp of a batch, this puts a spinning kernel in front: while it spins the host queues
    the whole batch, and what lies between the two stamps is GPU time.  None = not measured yet:
    treated as short."""
    import torch
    spin = getattr(torch.cuda, "_sleep", None)   # torch's spinning kernel; without it the batch is timed as it comes
    if spin is not None and (us_per_collective is None or us_per_collective < HEAD_START_BELOW_US):
        spin(HEAD_START_CYCLES)


def whole_job_value(world: int, P: int, m: int, ms_per_step: float) -> float:
    """Effective GB/s of `world` independent replicas that all finish within ms_per_step."""
    return world * effective_bytes(P, m) / (ms_per_step * 1e-3) / 1e9


def workload_config(algo: str, P: int, m: int, world: int) -> dict:
    """The part of the JSON line that names the workload; the same for both arms."""
    return {"workload": f"{algo} allgather, P={P} virtual ranks, m={m} B blocks",
            "P": P, "block_bytes": m, "algo": algo,
            "l2": "inputs larger than L2 (no flush needed)" if P * P * m > (256 << 20)
                  else "working set may sit in L2 (latency regime, reported as such)",
            "parallelism": "replicas only" if world > 1 else "1 GPU"}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


# ------------------------------------------------------------------------------------------------
def time_oracle(P: int, m: int, steps: int, warmup: int, threads: int, seed: int):
    """Seconds per collective of the CPU oracle's execute phase (message lists already built)."""
    import oracle
    plan = oracle.Plan(oracle.SPARBIT, P)
    send = si.send_blocks(P, m, seed).reshape(-1)
    recv = si.sentinel_buffer(P * P * m)
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        plan.run(m, send, recv, None, threads=threads)
        dt = time.perf_counter() - t0
        if it >= warmup:
            times.append(dt)
    ok = bool(np.array_equal(recv.reshape(P, P * m)[P // 2], send))
    return times, ok


def cpu_baseline_leg(P: int, m: int, seed: int):
    """The oracle as it stands on this machine's cores, on a bounded sample (about 10-30 s of work)."""
    cores = os.cpu_count() or 1
    threads = min(cores, 16)
    try:
        import psutil
        free = psutil.virtual_memory().available
    except Exception:
        free = 8 << 30
    ms = m
    while P * P * ms * 2.5 > free and ms > 1024:
        ms //= 2
    t1, ok1 = time_oracle(P, ms, steps=1, warmup=1, threads=1, seed=seed)
    tn, okn = time_oracle(P, ms, steps=2, warmup=0, threads=threads, seed=seed)
    best1, bestn = min(t1), min(tn)
    return {
        "value": effective_bytes(P, ms) / bestn / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
        "sample": f"whole collective P={P}, m={ms} B on host buffers, execute phase only "
                  f"(message lists prebuilt), best of 2; box has {cores} cores",
        "single_thread_value": effective_bytes(P, ms) / best1 / 1e9,
        "checked": bool(ok1 and okn),
    }


def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return 0
    P, m = args.P, args.m
    cores = os.cpu_count() or 1
    threads = min(cores, 16)
    # bounded sample: shrink the block until (steps + warmup) collectives fit in about two minutes
    ms = m
    budget = 120.0
    while True:
        t, _ = time_oracle(P, ms, steps=1, warmup=0, threads=threads, seed=args.seed)
        if t[0] * (args.steps + args.warmup) <= budget or ms <= 1024:
            break
        ms //= 4
    times, ok = time_oracle(P, ms, steps=args.steps, warmup=args.warmup, threads=threads, seed=args.seed)
    per = float(np.mean(times))
    value = effective_bytes(P, ms) / per / 1e9
    shrunk = f" (block shrunk from {m} B to bound the run)" if ms != m else ""
    sample = (f"each step = one whole collective P={P}, m={ms} B{shrunk}, "
              f"oracle execute phase on host buffers; box has {cores} cores")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": workload_config("sparbit", P, m, world), "sampled_block_bytes": ms,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0, "checked": ok,
    }
    print(json.dumps(line), flush=True)
    return 0


# ------------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import paper_2109_08751_b200 as sp

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    use_dist = world > 1
    if use_dist:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    P, m = args.P, args.m
    algo = {"sparbit": sp.ALGO_SPARBIT, "ring": sp.ALGO_RING, "rd": sp.ALGO_RECURSIVE_DOUBLING,
            "bruck": sp.ALGO_BRUCK, "ne": sp.ALGO_NEIGHBOR_EXCHANGE}[args.algo]
    exec_mode = {"auto": sp.EXEC_AUTO, "persistent": sp.EXEC_PERSISTENT, "graph": sp.EXEC_GRAPH,
                 "stream": sp.EXEC_STREAM, "flow": sp.EXEC_FLOW, "mirror": sp.EXEC_MIRROR}[args.exec]
    copy = {"auto": sp.COPY_AUTO, "vector": sp.COPY_VECTOR, "bulk": sp.COPY_BULK}[args.copy]

    plan = sp.Plan(P, m, algo, exec_mode)
    plan.set_copy_path(copy)
    if args.no_grouped_front:
        plan.set_tunable(sp.TUNE_GROUPED_FRONT, 0)
    seed = args.seed + rank
    # two input sets, alternated, so that no step finds its answer already in place
    sends = [torch.from_numpy(si.send_blocks(P, m, seed + k).reshape(-1)).to(dev) for k in range(2)]
    recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    work = None
    if algo == sp.ALGO_BRUCK:
        work = torch.empty(P * P * m, dtype=torch.uint8, device=dev)
        plan.set_workspace(work, P * P * m)
    stream = torch.cuda.Stream(device=dev)

    def barrier():
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize(dev)

    with torch.cuda.stream(stream):
        for it in range(args.warmup):
            plan.allgather(sends[it & 1], recv, stream)
        stream.synchronize()
        assert plan.status() == sp.OK

        # rounds: each round is exactly --steps collectives between a barrier + synchronize on
        # both sides; enough rounds that the timed work lasts MIN_TIMED_MS, so that neither one
        # noisy neighbour nor a handful of clock samples decides the number
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        head_start(None)
        e0.record(stream)
        for it in range(args.steps):
            plan.allgather(sends[it & 1], recv, stream)
        e1.record(stream)
        stream.synchronize()
        est_ms = max_over_ranks(e0.elapsed_time(e1), dev, use_dist)   # one untimed round sizes the run
        est_us = est_ms / args.steps * 1e3
        rounds = int(min(200, max(1, -(-args.min_timed_ms // max(est_ms, 1e-3)))))

        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
            time.sleep(0.25)
        k0, g0 = plan.launch_counts()
        round_ms, per_ms = [], []
        # A time stamp between every two collectives costs about 2 us of GPU time (the next
        # collective's first kernel can no longer start ahead of the last one's end), so the timed
        # rounds carry two stamps each; the spread of single collectives comes from one extra
        # stamped round after the timed region, where a collective is long enough to stand it.
        stamp_each = est_ms / args.steps >= 0.1
        t_wall0 = time.time()
        for _ in range(rounds):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier()
            head_start(est_us)
            e0.record(stream)
            for it in range(args.steps):
                plan.allgather(sends[it & 1], recv, stream)
            e1.record(stream)
            stream.synchronize()
            barrier()
            round_ms.append(max_over_ranks(e0.elapsed_time(e1), dev, use_dist))
            per_ms.append(e0.elapsed_time(e1) / args.steps)
        t_wall1 = time.time()
        k1, g1 = plan.launch_counts()
        if stamp_each:
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
            ev[0].record(stream)
            for it in range(args.steps):
                plan.allgather(sends[it & 1], recv, stream)
                ev[it + 1].record(stream)
            stream.synchronize()
            per_ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    assert plan.status() == sp.OK
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    ran_exec, ran_copy = plan.exec_mode, plan.copy_path   # what the timed collectives ran on

    # the last collective's result, checked against the result's definition on the device
    last_send = sends[(args.steps - 1) & 1]
    view = recv.view(P, P * m)
    checked = all(bool(torch.equal(view[r], last_send)) for r in (0, P // 3, P - 1))

    ms_per_step = float(np.median(round_ms)) / args.steps   # the median round, slowest rank
    value = whole_job_value(world, P, m, ms_per_step)

    # end to end through the host-buffer entry point (pinned host memory; H2D + D2H inside)
    e2e = None
    if not args.no_e2e:
        hs = torch.from_numpy(si.send_blocks(P, m, seed + 7).reshape(-1)).pin_memory()
        hr = torch.empty(P * P * m, dtype=torch.uint8).pin_memory()
        e2e_steps = max(1, min(args.steps, 3))
        hplan = sp.Plan(P, m, algo, exec_mode)
        hplan.set_copy_path(copy)
        hplan.allgather_host(hs.numpy(), hr.numpy())  # warm-up: allocates device staging
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            hplan.allgather_host(hs.numpy(), hr.numpy())
        torch.cuda.synchronize(dev)
        dt = (time.perf_counter() - t0) / e2e_steps
        dt = max_over_ranks(dt, dev, use_dist)
        ok = bool(np.array_equal(hr.numpy()[(P - 1) * P * m:], hs.numpy()))
        e2e = {"value": whole_job_value(world, P, m, dt * 1e3), "unit": UNIT, "ms_per_step": dt * 1e3,
               "h2d_bytes_per_step": P * m, "d2h_bytes_per_step": P * P * m, "steps": e2e_steps,
               "checked": ok}
        hplan.destroy()
        del hs, hr

    # the dominant kernel on its own, for the roofline entry: the whole collective when it is one
    # kernel (persistent, flow), else the last schedule step (half of all bytes for a power of
    # two P), launched exactly as inside the collective and timed with events on the same stream
    launches_per_step = (k1 - k0) / (args.steps * rounds)
    # the flow executor's kernel cannot be launched apart from the small per-pass kernels it may
    # have in front of it: its entry is the whole collective as well
    one_kernel = launches_per_step <= 1 or ran_exec == sp.EXEC_FLOW
    per_pass_us = None
    if one_kernel and ran_exec == sp.EXEC_PERSISTENT:
        # one more, traced, launch: the persistent kernel's own time stamps, pass by pass
        plan.set_trace(True)
        plan.allgather(sends[0], recv, stream)
        assert plan.status() == sp.OK
        stamps = plan.get_trace().astype(np.int64)
        per_pass_us = [round(float(x) / 1e3, 1) for x in np.diff(stamps)]
        plan.set_trace(False)
    if one_kernel:
        dom_ms = float(np.mean(round_ms)) / args.steps   # the timed rounds (no stamps in between)
        dom_bytes = algorithmic_bytes(P, m, algo != sp.ALGO_BRUCK)
        dom_name = ("whole collective in one kernel" if launches_per_step <= 1 else
                    f"whole collective: the flow kernel behind {launches_per_step - 1:g} small per-pass kernel(s)")
    else:
        last = plan.last_phase
        with torch.cuda.stream(stream):
            for _ in range(3):
                plan.allgather_steps(sends[0], recv, last, last, stream)
            d0 = torch.cuda.Event(enable_timing=True)
            d1 = torch.cuda.Event(enable_timing=True)
            d0.record(stream)
            for _ in range(args.steps):
                plan.allgather_steps(sends[0], recv, last, last, stream)
            d1.record(stream)
            stream.synchronize()
        dom_ms = d0.elapsed_time(d1) / args.steps
        dom_bytes = 2 * len(plan.messages(last)) * m
        dom_name = f"phase {last} (the last and largest) as its own kernel"

    if rank == 0:
        peak, peak_src = measured_peak()
        avg_ms = float(np.mean(round_ms)) / args.steps   # the timed rounds (no stamps in between)
        path_bytes = algorithmic_bytes(P, m, algo != sp.ALGO_BRUCK)
        achieved = dom_bytes / (dom_ms * 1e-3) / 1e9
        key = f"{args.algo}:P{P}:m{m}:{sp.EXEC_NAMES[ran_exec]}:{sp.COPY_NAMES[ran_copy]}"
        roofline = {
            "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "traffic": NCU_TRAFFIC.get(key, (None, None))[0],
            "traffic_source": NCU_TRAFFIC.get(key, (None, None))[1], "peak_source": peak_src,
            "kernel": f"{sp.EXEC_NAMES[ran_exec]} executor, {sp.COPY_NAMES[ran_copy]} engine: "
                      f"{dom_name} ({launches_per_step:g} launch(es) per collective)",
            "algorithmic_bytes_per_launch": dom_bytes, "us_per_launch": dom_ms * 1e3,
            "per_pass_us": per_pass_us,
            "whole_path": {"algorithmic_bytes": path_bytes, "us": avg_ms * 1e3,
                           "achieved": path_bytes / (avg_ms * 1e-3) / 1e9,
                           "frac": path_bytes / (avg_ms * 1e-3) / 1e9 / peak},
        }
        cpu = None if args.no_cpu else cpu_baseline_leg(P, m, seed)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
            "config": workload_config(args.algo, P, m, world),
            "executor": {"exec": sp.EXEC_NAMES[ran_exec], "copy": sp.COPY_NAMES[ran_copy],
                         "recv_GiB_per_gpu": round(P * P * m / 2**30, 3)},
            "rounds": rounds, "timed_ms": float(sum(round_ms)),
            "timed_behind_device_delay": bool(est_us < HEAD_START_BELOW_US),
            "ms_per_step_rounds": {"min": min(round_ms) / args.steps, "median": ms_per_step,
                                   "max": max(round_ms) / args.steps},
            "us_per_collective": {"min": min(per_ms) * 1e3, "avg": avg_ms * 1e3, "max": max(per_ms) * 1e3,
                                  "min_max_from": ("one extra round with a time stamp after every collective, "
                                                   "outside the timed region" if stamp_each else "the timed rounds")},
            "pct_of_hbm_peak": 100.0 * value / world / peak,
            "pct_of_nominal_hbm": 100.0 * value / world / NOMINAL_HBM_GBS,
            "GBps_from_min_time": world * effective_bytes(P, m) / (min(per_ms) * 1e-3) / 1e9,
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e,
            # kernels of this library per round of --steps collectives; the timed region is `rounds` rounds
            "gpu_launches": int((k1 - k0) // rounds), "graph_launches": int((g1 - g0) // rounds),
            "gpu_launches_timed_region": int(k1 - k0),
            "clocks": clocks, "checked": bool(checked),
        }
        print(json.dumps(line), flush=True)
    plan.destroy()
    if use_dist:
        dist.barrier()
        dist.destroy_process_group()
    return 0


# ------------------------------------------------------------------------------------------------
def run_cpu_sweep(args):
    """The oracle of every algorithm timed on this machine's host cores (no GPU involved): execute
    phase only, best of 3, one thread and all threads (capped at 16), same effective-bytes formula
    as the GPU numbers.  One JSON line per (algorithm, P, m)."""
    import oracle
    cores = os.cpu_count() or 1
    threads = min(cores, 16)
    P = args.P
    for m in (64, 4096, 65536):
        send = si.send_blocks(P, m, args.seed).reshape(-1)
        for name, algo in (("sparbit", oracle.SPARBIT), ("ring", oracle.RING), ("ne", oracle.NEIGHBOR_EXCHANGE),
                           ("rd", oracle.RECURSIVE_DOUBLING), ("bruck", oracle.BRUCK)):
            if (name == "rd" and P & (P - 1)) or (name == "ne" and P % 2):
                continue
            plan = oracle.Plan(algo, P)
            recv = si.sentinel_buffer(P * P * m)
            scratch = si.sentinel_buffer(P * P * m) if algo == oracle.BRUCK else None
            out = {"algo": name, "P": P, "m": m, "cores": threads}
            for label, t in (("us_1_thread", 1), (f"us_{threads}_threads", threads)):
                best = None
                for _ in range(3):
                    t0 = time.perf_counter()
                    plan.run(m, send, recv, scratch, threads=t)
                    dt = time.perf_counter() - t0
                    best = dt if best is None else min(best, dt)
                out[label] = round(best * 1e6, 1)
                out[label.replace("us_", "GBps_")] = round(effective_bytes(P, m) / best / 1e9, 2)
            out["checked"] = bool(np.array_equal(recv.reshape(P, P * m)[P - 1], send))
            print(json.dumps(out), flush=True)
            plan.close()
            del recv, scratch
    return 0


def run_sweep(args):
    """Latency and bandwidth curves: every point timed with the paper's protocol (5 warm-ups, then
    batches of 50 timed collectives; min / avg / max over ten batches; batches of collectives
    shorter than 100 us start behind a device-side delay, see head_start), one JSON line per
    (algorithm, executor, engine, P, m)."""
    import torch
    import paper_2109_08751_b200 as sp

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peak, _ = measured_peak()
    points = []
    if args.sweep in ("config4", "all"):
        points += [(1000, 1024, ["sparbit"])]
    if args.sweep in ("config5", "all"):
        points += [(256, m, ["sparbit", "ring", "ne", "rd", "bruck"])
                   for m in (8, 64, 512, 4096, 32768, 65536, 262144)]
    if args.sweep == "config3":
        points += [(128, 65536, ["sparbit"])]
    if args.sweep == "small":  # configs 1 and 2 and their neighbourhood: latency only
        points += [(P, m, ["sparbit"]) for P in (6, 8, 13, 16, 32, 64) for m in (64, 4096)]
    if args.sweep == "engines":  # what the engine and executor thresholds rest on
        points += [(P, m, ["sparbit"]) for P in (61, 128, 256, 509) for m in (4096, 8192, 16384, 32768, 65536)
                   if P * P * m <= (20 << 30)]
        points += [(1000, 1024, ["sparbit"]), (700, 1024, ["sparbit"]), (360, 8192, ["sparbit"])]
    algos = {"sparbit": sp.ALGO_SPARBIT, "ring": sp.ALGO_RING, "rd": sp.ALGO_RECURSIVE_DOUBLING,
             "bruck": sp.ALGO_BRUCK, "ne": sp.ALGO_NEIGHBOR_EXCHANGE}
    execs = {"persistent": sp.EXEC_PERSISTENT, "graph": sp.EXEC_GRAPH, "stream": sp.EXEC_STREAM,
             "flow": sp.EXEC_FLOW, "mirror": sp.EXEC_MIRROR}
    if args.sweep == "offline":  # block sizes that are not a multiple of 128 B beside neighbours that are
        points += [(P, m, ["sparbit"]) for P, m in (
            (256, 2032), (256, 2048), (256, 4080), (256, 4096), (256, 16368), (256, 16384),
            (128, 65520), (128, 65536), (1000, 1008), (1000, 1024))]
    if args.sweep in ("engines", "offline"):
        execs = {"graph": sp.EXEC_GRAPH, "flow": sp.EXEC_FLOW}
    if args.sweep == "mirror":  # where the mirror executor (one CTA, then a cluster) wins and where it stops winning
        points += [(P, m, ["sparbit"]) for P, m in (
            (8, 64), (16, 64), (32, 64), (64, 64), (128, 64), (64, 256), (32, 512), (45, 512), (16, 1024),
            (8, 4096), (16, 4096), (256, 8), (253, 1), (253, 3), (128, 128), (64, 512), (100, 200), (181, 64),
            (4, 16384), (8, 8192))]
        execs = {"graph": sp.EXEC_GRAPH, "mirror": sp.EXEC_MIRROR}
        copies = {"vector": sp.COPY_VECTOR}
    else:
        copies = {"vector": sp.COPY_VECTOR, "bulk": sp.COPY_BULK}
    stream = torch.cuda.Stream(device=dev)
    cores = min(os.cpu_count() or 1, 16)
    for P, m, names in points:
        # the CPU oracle on the same point (Sparbit, all host threads up to 16, best of 2), where
        # its buffers stay at or below 1 GiB
        oracle_ms = None
        if P * P * m <= (1 << 30):
            t, ok = time_oracle(P, m, steps=2, warmup=0, threads=cores, seed=args.seed)
            oracle_ms = round(min(t) * 1e3, 3) if ok else None
        sends = [torch.from_numpy(si.send_blocks(P, m, args.seed + k).reshape(-1)).to(dev) for k in range(2)]
        recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
        work = None
        for name in names:
            if name == "bruck" and work is None:
                work = torch.empty(P * P * m, dtype=torch.uint8, device=dev)
            combos = [("auto", sp.EXEC_AUTO, "auto", sp.COPY_AUTO)]
            if not args.sweep_auto_only:
                combos += [(en, e, cn, c) for en, e in execs.items() for cn, c in copies.items()]
            for ename, e, cname, c in combos:
                if ename == "stream" and name in ("ring", "ne") and m >= 32768:
                    continue  # same kernels as the graph chain; skipped to bound the sweep
                if cname == "bulk" and (m % 16 or ename in ("flow", "mirror")):
                    continue
                if ename == "mirror" and (P + 15) // 16 * P * m > (224 << 10):
                    continue  # fits no cluster
                plan = sp.Plan(P, m, algos[name], e)
                plan.set_copy_path(c)
                if args.no_grouped_front:
                    plan.set_tunable(sp.TUNE_GROUPED_FRONT, 0)
                if name == "bruck":
                    plan.set_workspace(work, P * P * m)
                # the paper's protocol (5 warm-ups, 50 timed runs), the way its benchmark times them:
                # a batch of 50 back-to-back collectives between two time stamps, divided by 50
                # (a time stamp between every two collectives would itself cost 2 us each); ten
                # such batches give the minimum, average and maximum
                us = []
                with torch.cuda.stream(stream):
                    for it in range(5):
                        plan.allgather(sends[it & 1], recv, stream)
                    stream.synchronize()
                    k_before = plan.launch_counts()[0]
                    for _ in range(10):
                        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        head_start(us[-1] if us else None)   # short collectives: GPU time, not the host's launch loop
                        e0.record(stream)
                        for it in range(50):
                            plan.allgather(sends[it & 1], recv, stream)
                        e1.record(stream)
                        stream.synchronize()
                        us.append(e0.elapsed_time(e1) / 50 * 1e3)
                    k_after = plan.launch_counts()[0]
                    # the same loop as the host feeds it (no delay in front: short collectives are then
                    # bound by the launches of this Python loop, 3-4 us per call and more per plain
                    # kernel launch; reported beside the GPU time, not instead of it)
                    fed = None
                    if float(np.mean(us)) < HEAD_START_BELOW_US:
                        fed = []
                        for _ in range(3):
                            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                            e0.record(stream)
                            for it in range(50):
                                plan.allgather(sends[it & 1], recv, stream)
                            e1.record(stream)
                            stream.synchronize()
                            fed.append(e0.elapsed_time(e1) / 50 * 1e3)
                assert plan.status() == sp.OK
                ok = bool(torch.equal(recv.view(P, P * m)[P - 1], sends[1]))
                avg = float(np.mean(us))
                print(json.dumps({
                    "algo": name, "exec": ename, "copy": cname, "P": P, "m": m,
                    "ran": f"{sp.EXEC_NAMES[plan.exec_mode]}/{sp.COPY_NAMES[plan.copy_path]}",
                    "launches_per_collective": (k_after - k_before) / 500,
                    "us_min": round(min(us), 2), "us_avg": round(avg, 2), "us_max": round(max(us), 2),
                    "us_host_fed": round(min(fed), 2) if fed else None,
                    "GBps_avg": round(effective_bytes(P, m) / avg / 1e3, 1),
                    "GBps_min_time": round(effective_bytes(P, m) / min(us) / 1e3, 1),
                    "pct_measured_peak": round(100 * effective_bytes(P, m) / avg / 1e3 / peak, 1),
                    "pct_nominal_hbm": round(100 * effective_bytes(P, m) / avg / 1e3 / NOMINAL_HBM_GBS, 1),
                    "oracle_ms": oracle_ms if name == "sparbit" else None,
                    "oracle_cores": cores if name == "sparbit" and oracle_ms is not None else None,
                    "checked": ok}), flush=True)
                plan.destroy()
        del sends, recv, work
        torch.cuda.empty_cache()
    return 0


def run_flow_wait_bound(args):
    """What the flow executor loses to waiting of any kind: the same collectives with and without
    the units' waits for their source rank's counters (a measurement hook of the library; without
    them blocks are forwarded before they have arrived, so that run's result is wrong and is not
    checked).  The difference bounds what finer readiness tracking, per (rank, slot) instead of
    per (rank, pass), could gain.  One JSON line per point; same timing protocol as --sweep."""
    import torch
    import paper_2109_08751_b200 as sp

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peak, _ = measured_peak()
    stream = torch.cuda.Stream(device=dev)
    for P, m in ((256, 4096), (128, 16384), (256, 8192), (512, 4096), (128, 65536), (1000, 1024), (256, 32768)):
        sends = [torch.from_numpy(si.send_blocks(P, m, args.seed + k).reshape(-1)).to(dev) for k in range(2)]
        recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
        out = {"P": P, "m": m, "GB_moved": round(effective_bytes(P, m) / 1e9, 3)}
        for label, skip in (("graph", None), ("flow", 0), ("flow_no_waits", 1)):
            plan = sp.Plan(P, m, sp.ALGO_SPARBIT, sp.EXEC_GRAPH if skip is None else sp.EXEC_FLOW)
            if skip:
                plan.set_tunable(sp.TUNE_FLOW_SKIP_WAITS, 1)
            us = []
            with torch.cuda.stream(stream):
                for it in range(5):
                    plan.allgather(sends[it & 1], recv, stream)
                stream.synchronize()
                for _ in range(10):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    for it in range(50):
                        plan.allgather(sends[it & 1], recv, stream)
                    e1.record(stream)
                    stream.synchronize()
                    us.append(e0.elapsed_time(e1) / 50 * 1e3)
            assert plan.status() == sp.OK
            if not skip:
                assert bool(torch.equal(recv.view(P, P * m)[P - 1], sends[1]))
            out[label + "_us"] = round(float(np.mean(us)), 2)
            out[label + "_pct_measured_peak"] = round(100 * effective_bytes(P, m) / float(np.mean(us)) / 1e3 / peak, 1)
            plan.destroy()
        out["waiting_costs_pct"] = round(100 * (out["flow_us"] - out["flow_no_waits_us"]) / out["flow_us"], 2)
        print(json.dumps(out), flush=True)
        del sends, recv
        torch.cuda.empty_cache()
    return 0


def run_placement_study(args):
    """The same collective (Sparbit, --P, --m, executor and engine as AUTO picks them), timed with
    the receive buffer at different places in device memory: before it is allocated, a pad of the
    given size is allocated and kept.  Same protocol as --sweep.  One JSON line per pad size."""
    import torch
    import paper_2109_08751_b200 as sp

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peak, _ = measured_peak()
    P, m = args.P, args.m
    stream = torch.cuda.Stream(device=dev)
    for pad_mib in (0, 2, 64, 256, 512, 1024, 1536):
        torch.cuda.empty_cache()
        pad = torch.empty(max(pad_mib << 20, 1), dtype=torch.uint8, device=dev)
        sends = [torch.from_numpy(si.send_blocks(P, m, args.seed + k).reshape(-1)).to(dev) for k in range(2)]
        recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
        plan = sp.Plan(P, m)
        us = []
        with torch.cuda.stream(stream):
            for it in range(5):
                plan.allgather(sends[it & 1], recv, stream)
            stream.synchronize()
            for _ in range(10):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for it in range(50):
                    plan.allgather(sends[it & 1], recv, stream)
                e1.record(stream)
                stream.synchronize()
                us.append(e0.elapsed_time(e1) / 50 * 1e3)
        assert plan.status() == sp.OK
        ok = bool(torch.equal(recv.view(P, P * m)[P - 1], sends[1]))
        avg = float(np.mean(us))
        print(json.dumps({"P": P, "m": m, "pad_MiB": pad_mib,
                          "ran": f"{sp.EXEC_NAMES[plan.exec_mode]}/{sp.COPY_NAMES[plan.copy_path]}",
                          "recv_address": hex(recv.data_ptr()),
                          "us_min": round(min(us), 2), "us_avg": round(avg, 2), "us_max": round(max(us), 2),
                          "pct_measured_peak": round(100 * effective_bytes(P, m) / avg / 1e3 / peak, 1),
                          "checked": ok}), flush=True)
        plan.destroy()
        del sends, recv, pad
    return 0


def run_allgatherv(args):
    """Blocks of different sizes on the Sparbit schedule (P = 256, about 64 KiB per block on
    average): equal sizes through the variable-size path, uniformly drawn sizes, and a mix with
    empty and several-times-larger blocks.  Effective bytes = 2*(P-1)*sum(counts)."""
    import torch
    import paper_2109_08751_b200 as sp

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peak, _ = measured_peak()
    P = args.P
    cases = {
        "equal (fixed-size plan)": None,
        "equal (variable-size plan)": [args.m] * P,
        "uniform 0..2m": si.block_counts(P, args.seed, kind="uniform", unit=16, scale=args.m // 16),
        "mixed (1/8 empty, 1/8 six-fold)": si.block_counts(P, args.seed, kind="mixed", unit=16,
                                                            scale=args.m // 16 * 8 // 13),
    }
    stream = torch.cuda.Stream(device=dev)
    for name, counts in cases.items():
        if counts is None:
            plan = sp.Plan(P, args.m)
            T = P * args.m
            host = [si.send_blocks(P, args.m, args.seed + k).reshape(-1) for k in range(2)]
        else:
            plan = sp.Plan.create_v(counts)
            T = sum(counts)
            host = [si.send_blocks_v(counts, args.seed + k) for k in range(2)]
        sends = [torch.from_numpy(h).to(dev) for h in host]
        recv = torch.full((P * T,), si.SENTINEL, dtype=torch.uint8, device=dev)
        with torch.cuda.stream(stream):
            for it in range(5):
                plan.allgather(sends[it & 1], recv, stream)
            stream.synchronize()
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(51)]
            ev[0].record(stream)
            for it in range(50):
                plan.allgather(sends[it & 1], recv, stream)
                ev[it + 1].record(stream)
            stream.synchronize()
        assert plan.status() == sp.OK
        ok = bool(torch.equal(recv.view(P, T)[P - 1], sends[1]))
        us = [ev[i].elapsed_time(ev[i + 1]) * 1e3 for i in range(50)]
        avg = float(np.mean(us))
        eff = 2 * (P - 1) * T
        print(json.dumps({"case": name, "P": P, "total_bytes_per_rank": T,
                          "max_block": max(counts) if counts else args.m,
                          "us_min": round(min(us), 1), "us_avg": round(avg, 1), "us_max": round(max(us), 1),
                          "GBps_avg": round(eff / avg / 1e3, 1),
                          "pct_measured_peak": round(100 * eff / avg / 1e3 / peak, 1), "checked": ok}), flush=True)
        plan.destroy()
        del sends, recv
        torch.cuda.empty_cache()
    return 0


def run_mapping_study(args):
    """Section III-C in numbers, for G devices instead of machines (host only, no GPU): how many
    blocks of every Sparbit step leave their device under the sequential and the cyclic mapping of
    ranks to devices.  One JSON line per (P, G, mapping); multiply blocks by m for bytes."""
    import paper_2109_08751_b200 as sp
    for P in (256, 1000):
        plan = sp.Plan(P, 1)
        for G in (2, 4, 8):
            for name, mp in (("sequential", sp.MAP_SEQUENTIAL), ("cyclic", sp.MAP_CYCLIC)):
                steps = []
                for st in range(plan.num_steps):
                    d, n, _ = plan.step_info(st)
                    b = plan.partition(G, mp, st)
                    steps.append({"distance": d, "blocks": int(b.sum()), "cross": int(b.sum() - np.trace(b)),
                                  "busiest_link": int((b - np.diag(np.diag(b))).max())})
                total = sum(x["blocks"] for x in steps)
                cross = sum(x["cross"] for x in steps)
                print(json.dumps({"P": P, "G": G, "mapping": name, "total_blocks": total, "cross_blocks": cross,
                                  "cross_pct": round(100.0 * cross / total, 2), "steps": steps}), flush=True)
        plan.destroy()
    return 0


def run_multi_emulated(args):
    """The multi-device executor (sparbit_allgather_multi_phases) with its G devices emulated on ONE
    GPU: G pairs of allocations, one kernel per device and step, all on one stream, so that stream
    order is the cross-device barrier and every "peer" store is a local store.  This times the
    kernels and the G launches per step against the single-device executor on the same collective; it
    says nothing about NVLink.  One JSON line per (G, mapping), plus the single-device line first."""
    import torch
    import paper_2109_08751_b200 as sp

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peak, _ = measured_peak()
    P, m = args.P, args.m
    stream = torch.cuda.Stream(device=dev)
    host = [si.send_blocks(P, m, args.seed + k) for k in range(2)]
    rdev = sp.binding.lib.sparbit_rank_device

    def timed(run):
        us = []
        with torch.cuda.stream(stream):
            for it in range(5):
                run(it)
            stream.synchronize()
            for _ in range(10):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for it in range(20):
                    run(it)
                e1.record(stream)
                stream.synchronize()
                us.append(e0.elapsed_time(e1) / 20 * 1e3)
        return us

    def line(tag, us, ok):
        avg = float(np.mean(us))
        print(json.dumps({"P": P, "m": m, **tag, "us_min": round(min(us), 2), "us_avg": round(avg, 2),
                          "us_max": round(max(us), 2), "GBps_avg": round(effective_bytes(P, m) / avg / 1e3, 1),
                          "pct_measured_peak": round(100 * effective_bytes(P, m) / avg / 1e3 / peak, 1),
                          "checked": ok}), flush=True)

    plan = sp.Plan(P, m)
    sends = [torch.from_numpy(h.reshape(-1)).to(dev) for h in host]
    recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
    us = timed(lambda it: plan.allgather(sends[it & 1], recv, stream))
    line({"devices": 1, "mapping": "-", "ran": f"{sp.EXEC_NAMES[plan.exec_mode]}/{sp.COPY_NAMES[plan.copy_path]}"},
         us, bool(torch.equal(recv.view(P, P * m)[P - 1], sends[1])))
    del recv
    for G in args.multi_devices:
        for name, mp in (("sequential", sp.MAP_SEQUENTIAL), ("cyclic", sp.MAP_CYCLIC)):
            ranks = [[r for r in range(P) if rdev(P, G, mp, r) == g] for g in range(G)]
            dsend = [[torch.from_numpy(np.ascontiguousarray(h[ranks[g]]).reshape(-1)).to(dev) for g in range(G)]
                     for h in host]
            drecv = [torch.full((len(ranks[g]) * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
                     for g in range(G)]
            bases = [t.data_ptr() for t in drecv]

            def run(it):
                # phases -1 and 0 as one pass, then step by step; every device's kernel of a step is
                # enqueued before any kernel of the next step
                for g in range(G):
                    plan.allgather_multi_phases(G, mp, g, dsend[it & 1][g], bases, -1, 0, stream)
                for ph in range(1, plan.last_phase + 1):
                    for g in range(G):
                        plan.allgather_multi_phases(G, mp, g, dsend[it & 1][g], bases, ph, ph, stream)

            us = timed(run)
            want = torch.from_numpy(host[1].reshape(-1)).to(dev)
            ok = all(bool(torch.equal(drecv[g].view(len(ranks[g]), P * m)[-1], want)) for g in range(G))
            line({"devices": G, "mapping": name, "ran": "multi-device kernels, emulated on one GPU",
                  "launches_per_collective": G * (plan.last_phase + 1)}, us, ok)
            del dsend, drecv
            torch.cuda.empty_cache()
    plan.destroy()
    return 0


def run_heatmap(args):
    """Which algorithm is fastest for each (P, m) on this executor, in the style of the paper's
    heat maps (Section IV): block sizes 1 B .. 1 MiB, P up to 256, powers of two and not, every
    algorithm that is defined for the P, executor and engine chosen by the library (AUTO).
    5 warm-ups + 50 timed collectives per cell; one JSON line per cell."""
    import torch
    import paper_2109_08751_b200 as sp

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    algos = {"sparbit": sp.ALGO_SPARBIT, "ring": sp.ALGO_RING, "ne": sp.ALGO_NEIGHBOR_EXCHANGE,
             "rd": sp.ALGO_RECURSIVE_DOUBLING, "bruck": sp.ALGO_BRUCK}
    stream = torch.cuda.Stream(device=dev)
    free_bytes = torch.cuda.mem_get_info(dev)[0]
    if args.heatmap == "paper":
        # the paper's grid (Section IV-A): 1 B .. 1 MiB by powers of two; process counts 8..256 in
        # steps of 8 and 5..253 in steps of 8 (one less than a multiple of 8, plus the odd offsets)
        grid_P = sorted(list(range(8, 257, 8)) + list(range(5, 254, 8)))
        grid_m = [1 << k for k in range(21)]
    else:
        grid_P = (5, 8, 13, 16, 32, 61, 64, 128, 253, 256)
        grid_m = (1, 8, 64, 512, 4096, 32768, 262144, 1048576)
    for P in grid_P:
        for m in grid_m:
            if P * P * m * 2.2 + 2 * P * m > free_bytes:
                continue
            sends = [torch.from_numpy(si.send_blocks(P, m, args.seed + k).reshape(-1)).to(dev) for k in range(2)]
            recv = torch.full((P * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
            work = torch.empty(P * P * m, dtype=torch.uint8, device=dev)
            cell = {}
            for name, a in algos.items():
                if name == "rd" and P & (P - 1):
                    continue
                if name == "ne" and P % 2:
                    continue
                plan = sp.Plan(P, m, a, sp.EXEC_AUTO)
                if name == "bruck":
                    plan.set_workspace(work, P * P * m)
                with torch.cuda.stream(stream):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    plan.allgather(sends[1], recv, stream)
                    e0.record(stream)
                    for it in range(4):
                        plan.allgather(sends[it & 1], recv, stream)
                    e1.record(stream)
                    stream.synchronize()
                    warm_us = e0.elapsed_time(e1) / 4 * 1e3   # an upper estimate (host-bound where short)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    head_start(warm_us)
                    e0.record(stream)
                    for it in range(50):
                        plan.allgather(sends[it & 1], recv, stream)
                    e1.record(stream)
                    stream.synchronize()
                assert plan.status() == sp.OK
                assert bool(torch.equal(recv.view(P, P * m)[P - 1], sends[1]))
                cell[name] = round(e0.elapsed_time(e1) / 50 * 1e3, 2)
                plan.destroy()
            order = sorted(cell, key=cell.get)
            best, second = order[0], order[1]
            print(json.dumps({"P": P, "m": m, "us_avg": cell, "best": best,
                              "gain_over_second_pct": round(100 * (cell[second] - cell[best]) / cell[second], 1)}),
                  flush=True)
            del sends, recv, work
            torch.cuda.empty_cache()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--P", type=int, default=P_DEFAULT)
    ap.add_argument("--m", type=int, default=M_DEFAULT)
    ap.add_argument("--algo", choices=["sparbit", "ring", "ne", "rd", "bruck"], default="sparbit")
    ap.add_argument("--exec", choices=["auto", "persistent", "graph", "stream", "flow", "mirror"], default="auto")
    ap.add_argument("--copy", choices=["auto", "vector", "bulk"], default="auto")
    ap.add_argument("--seed", type=int, default=si.BASE_SEED + 5)
    ap.add_argument("--min-timed-ms", type=float, default=MIN_TIMED_MS,
                    help="rounds of --steps collectives are repeated until the timed work lasts this long "
                         "(0 = one round, for profiler captures)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--sweep", choices=["small", "config3", "config4", "config5", "engines", "mirror", "offline", "all"], default=None,
                    help="print latency/bandwidth curves (one JSON line per point) instead of the bench line")
    ap.add_argument("--no-grouped-front", action="store_true",
                    help="every pass of the graph and stream executors as its own kernel (SPARBIT_TUNE_GROUPED_FRONT = 0)")
    ap.add_argument("--sweep-auto-only", action="store_true",
                    help="with --sweep: only the executor and engine the library picks by itself")
    ap.add_argument("--heatmap", nargs="?", const="coarse", default=None, choices=["coarse", "paper"],
                    help="best algorithm per (P, m) cell, one JSON line per cell; 'paper' = the paper's "
                         "grid of 64 process counts x 21 block sizes (about a quarter of an hour)")
    ap.add_argument("--cpu-sweep", action="store_true",
                    help="time the CPU oracle of every algorithm on the host cores (no GPU)")
    ap.add_argument("--mapping-study", action="store_true",
                    help="blocks per Sparbit step that cross devices under the sequential and cyclic "
                         "rank-to-device mappings (host only), one JSON line per (P, G, mapping)")
    ap.add_argument("--multi-emulated", action="store_true",
                    help="the multi-device executor with G = 1, 2, 4, 8 devices emulated on one GPU "
                         "(kernel and launch cost only; no NVLink involved)")
    ap.add_argument("--multi-devices", type=int, nargs="+", default=[1, 2, 4, 8],
                    help="with --multi-emulated: the device counts to run")
    ap.add_argument("--flow-wait-bound", action="store_true",
                    help="the flow executor with and without its waits (timing only): what any finer "
                         "readiness tracking could gain at most")
    ap.add_argument("--placement-study", action="store_true",
                    help="the same collective with its receive buffer at different places in device memory")
    ap.add_argument("--allgatherv", action="store_true",
                    help="variable block sizes on the Sparbit schedule, one JSON line per size mix")
    args = ap.parse_args()
    if args.cpu_sweep:
        return run_cpu_sweep(args)
    if args.mapping_study:
        return run_mapping_study(args)
    if args.allgatherv:
        return run_allgatherv(args)
    if args.multi_emulated:
        return run_multi_emulated(args)
    if args.flow_wait_bound:
        return run_flow_wait_bound(args)
    if args.placement_study:
        return run_placement_study(args)
    if args.heatmap:
        return run_heatmap(args)
    if args.sweep:
        return run_sweep(args)
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())

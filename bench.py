#!/usr/bin/env python
"""Throughput benchmark of the batched response-time analysis (tasksets analysed per second).

A step is one pass of the whole hot path over one batch of synthetic tasksets: the GCAPS
analysis and the round-robin analysis of every taskset of the batch (two gcaps_rta_batch calls;
`--fused`: one gcaps_rta_multi_batch call that reads every taskset once).  The
default workload is the 1,000,000-taskset configuration (8 cores x 10 tasks per taskset).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

prints ONE JSON line (rank 0).  With N > 1 (launched by torch.distributed.run, one rank per GPU)
every rank analyses its own shard of the generator stream; there is no data-path collective.
`--impl reference` times the CPU oracle on a bounded sample instead (host cores, no GPU).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "tasksets analysed/sec (GCAPS & RR RTA)"
UNIT = "tasksets/s"
FALLBACK_HBM_GBS = 6650.0
# plain-ALU peak of one B200 from unit counts and clock, 148 SMs x 128 INT32 lanes x 1.965 GHz
# (integer lane-operations/s): only the fallback when the issue-rate probe cannot run
ALU_PEAK_DERIVED = 148 * 128 * 1.965e9
# a workload larger than this is benchmarked one chunk at a time (the 10,000,000-taskset
# workload is generated, analysed and verified in chunks of 1,000,000)
MAX_TASKSETS_PER_GPU = 1_000_000
K_TERM, K_SETUP = 6, 16   # algorithmic integer lane-operations per interference term / per task
# kernels launched by one gcaps_rta_batch call: 3 plan kernels, one analysis kernel for the bins
# of up to 32 tasks and one each for the 64-, 96-, 128-, 192- and 256-task bins
LAUNCHES_PER_CALL = 9        # three plan kernels + one kernel per group of size bins
LAUNCHES_PER_SMALL_CALL = 2  # batches of up to 8,192 tasksets: one plan kernel, one kernel for all bins
# DRAM bytes (read + write) per taskset of the analysis kernel on the 'large' workload, from an
# ncu capture of a 131,072-taskset launch (traffic grows in proportion to the tasksets of a
# launch).  Only reported while the kernel source is the one the counters were taken from.
CAPTURED_TRAFFIC = {
    "source_sha256": "9fc3a243eb31c6fb7c4e05766b9dc8d537e4e9f0aa84ad3911c2ef4eedab4396",
    "workload": "large",
    "bytes_per_taskset": {"gcaps": (1248476000 + 84340736) / 131072.0,
                          "rr": (1258324000 + 95665152) / 131072.0},
}


def kernel_source_digest():
    """sha256 over the sources of the analysis kernel (gcaps_rta.cu and the header it shares)."""
    import hashlib
    h = hashlib.sha256()
    try:
        for name in ("gcaps_rta.cu", "rta_common.cuh"):
            with open(os.path.join(ROOT, "paper_2406_05221_b200", "csrc", name), "rb") as fh:
                h.update(fh.read())
    except OSError:
        return None
    return h.hexdigest()


def captured_traffic(workload_name, policy_name, tasksets):
    """DRAM traffic of one analysis launch, or None if the capture does not apply any more."""
    digest = kernel_source_digest()
    if digest is None:
        return None
    if digest != CAPTURED_TRAFFIC["source_sha256"] or workload_name != CAPTURED_TRAFFIC["workload"]:
        return None
    per_taskset = CAPTURED_TRAFFIC["bytes_per_taskset"].get(policy_name)
    return per_taskset * tasksets if per_taskset is not None else None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            d = json.load(fh)
        return float(d["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while a region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.gpu_id, self.proc = gpu_id, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.gpu_id, "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            text, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            return out
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in text.strip().splitlines():
            tok = [x.strip() for x in line.split(",")]
            if len(tok) < 7:
                continue
            try:
                sm.append(float(tok[0]))
                mx.append(float(tok[1]))
            except ValueError:
                continue
            for name, val in zip(names, tok[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


def oracle_sample(workload, first, count, budget_s, chunk=50_000, stream=0):
    """Times the CPU oracle (as it stands, one thread) on tasksets first.. of the workload, both
    policies per taskset, stopping after ``count`` tasksets or ``budget_s`` seconds."""
    from oracle import rta
    done, spent, terms, sweeps, started = 0, 0.0, [0, 0], [0, 0], [0, 0]
    while done < count and spent < budget_s:
        n = min(chunk, count - done)
        batch = workload.generate(first + done, n, stream=stream)
        t0 = time.perf_counter()
        for k, policy in enumerate((rta.POLICY_GCAPS, rta.POLICY_RR)):
            _, _, c = rta.analyse(batch, policy, workload.timeslice_us, workload.overhead_us)
            terms[k] += c.terms
            sweeps[k] += c.sweeps
            started[k] += c.tasks
        spent += time.perf_counter() - t0
        done += n
    return {"tasksets": done, "seconds": spent, "terms": terms, "sweeps": sweeps, "started": started}


def _oracle_shard(job):
    """Worker of the all-core CPU baseline: generates its own shard and times the oracle on it."""
    os.environ["OMP_NUM_THREADS"] = "1"   # the generator's OpenMP loop stays on this core
    name, first, count, stream = job
    from paper_2406_05221_b200 import taskgen
    r = oracle_sample(taskgen.WORKLOADS[name], first, count, 1e9, chunk=count, stream=stream)
    return r["tasksets"], r["seconds"]


def oracle_all_cores(workload, first, per_core, stream=0):
    """The single-threaded oracle over disjoint shards of the workload, one per host core, in
    processes started with `spawn` (a forked child of a process that has used CUDA hangs)."""
    import multiprocessing as mp
    try:
        cores = len(os.sched_getaffinity(0))
    except AttributeError:
        cores = os.cpu_count() or 1
    cores = max(1, min(cores, 256))
    jobs = [(workload.name, first + k * per_core, per_core, stream) for k in range(cores)]
    t0 = time.perf_counter()
    with mp.get_context("spawn").Pool(cores) as pool:
        got = pool.map(_oracle_shard, jobs, chunksize=1)
    wall = time.perf_counter() - t0
    tasksets = sum(g[0] for g in got)
    slowest = max(g[1] for g in got)
    return {"value": tasksets / slowest, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%d tasksets per core on %d cores (disjoint shards), both policies; rate = all "
                      "tasksets / the slowest core's oracle time (%.1f s); generation and process "
                      "start excluded (%.1f s wall in all)" % (per_core, cores, slowest, wall)}


def run_reference(args, workload):
    """The reference arm: the CPU oracle, single-threaded, on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    per_step = min(args.ref_sample, workload.n_tasksets)
    for _ in range(args.warmup):
        oracle_sample(workload, 0, min(per_step, 10_000), 1e9)
    t_total, n_total = 0.0, 0
    for k in range(args.steps):
        r = oracle_sample(workload, (k * per_step) % max(1, workload.n_tasksets - per_step + 1), per_step, 1e9)
        t_total += r["seconds"]
        n_total += r["tasksets"]
    value = n_total / t_total
    sample = "%d tasksets of '%s' per step, both policies, generation excluded" % (per_step, workload.name)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
        "data": "synthetic", "config": {"workload": workload.name, "tasksets_per_step": per_step,
                                         "note": workload.note},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large")
    ap.add_argument("--stream", type=int, default=0, help="sweep point of the workload")
    ap.add_argument("--tasksets", type=int, default=0, help="tasksets per GPU (0 = the workload's own size)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-budget", type=float, default=20.0, help="seconds of oracle time for cpu_baseline")
    ap.add_argument("--ref-sample", type=int, default=100_000)
    ap.add_argument("--fused", action="store_true",
                    help="one gcaps_rta_multi_batch call per step (every taskset read once, analysed "
                         "under both policies) instead of one gcaps_rta_batch call per policy")
    ap.add_argument("--on-device-inputs", action="store_true",
                    help="generate the tasksets on the GPU (integer-only generator) instead of on the "
                         "host; reports the generation time in config.generation")
    ap.add_argument("--mode", default="policies", choices=["policies", "assign", "sweep"],
                    help="policies: GCAPS + RR calls per step (the benchmark); assign: the GCAPS call "
                         "followed by the GPU-priority search of the paper's Sec. 5.3 on the same batch; "
                         "sweep: all (timeslice, overhead) pairs of the workload, once as one fused "
                         "gcaps_rta_sweep_batch call and once as one gcaps_rta_batch call per pair")
    ap.add_argument("--graph", action="store_true",
                    help="replay each call from a CUDA graph instead of enqueueing its launches again")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="weak: every rank analyses --tasksets tasksets of its own; strong: --tasksets "
                         "tasksets in all, split over the ranks")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-cpu-all-cores", action="store_true",
                    help="skip the all-host-cores leg of the CPU baseline")
    ap.add_argument("--cpu-all-cores-budget", type=float, default=6.0,
                    help="seconds of oracle time per core for the all-cores leg")
    ap.add_argument("--no-diagnostic", action="store_true",
                    help="skip the secondary timing on tasksets that converge")
    args = ap.parse_args()

    from paper_2406_05221_b200 import taskgen
    workload = taskgen.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, workload)
        return

    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2406_05221_b200 import binding, sharding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    binding.load_library()

    per_gpu = args.tasksets or min(workload.n_tasksets, MAX_TASKSETS_PER_GPU)
    if args.scaling == "strong":   # a fixed job split over the ranks
        first, count = sharding.strong_shard(rank, world, per_gpu)
        total_count = per_gpu
    else:                          # every rank analyses its own per_gpu tasksets
        first, count = sharding.weak_shard(rank, per_gpu)
        total_count = world * count
    pinned = []

    def alloc(n):
        t = torch.empty(max(n, 1), dtype=torch.int64, pin_memory=True)
        pinned.append(t)
        return t.numpy()[:n]

    generation = None
    if args.on_device_inputs:
        # the inputs never exist on the host; the host twin of the same stream is only needed by
        # the end-to-end and CPU-baseline legs, which are switched off here
        args.no_e2e = args.no_cpu_baseline = True
        generation = {}
        binding.generate_device(workload.streams[args.stream], first, min(count, 1000), dev)  # warm-up
        ts = binding.generate_device(workload.streams[args.stream], first, count, dev, timing=generation)
        generation["tasksets_per_s"] = count / ((generation["count_ms"] + generation["fill_ms"]) * 1e-3)
        generation["generator"] = "integer-only, on device (gcaps_gen_count + gcaps_gen_fill)"

        class _Sizes:   # what the report needs of a host batch
            def input_bytes(self):
                return ts.input_bytes()

            def output_bytes(self):
                return 8 * ts.n_tasks + ts.n_tasksets

            def checksum(self):
                return None
        batch = _Sizes()
    else:
        batch = workload.generate(first, count, stream=args.stream, alloc=alloc)
        ts = binding.DeviceTasksets.from_host(batch, dev)
    out_wcrt = torch.empty(ts.n_tasks, dtype=torch.int64, device=dev)
    out_sched = torch.empty(ts.n_tasksets, dtype=torch.uint8, device=dev)
    workspace = torch.empty(max(256, binding.workspace_bytes(ts.n_tasksets)), dtype=torch.uint8, device=dev)
    policies = [p for p in (binding.POLICY_GCAPS, binding.POLICY_RR)
                if ("gcaps", "rr")[p] in workload.policies]
    names = [("gcaps", "rr")[p] for p in policies]
    host_policies = list(policies)   # the end-to-end leg
    analyses_per_step = len(policies)
    fused = args.mode == "policies" and len(policies) == 2 and args.fused
    if fused:
        # one call analyses every taskset under GCAPS and under round robin (self-suspension)
        policies, names = ["fused"], ["gcaps+rr"]
        multi_wcrt = torch.empty((1, 2, ts.n_tasks), dtype=torch.int64, device=dev)
        multi_sched = torch.empty((1, 2, ts.n_tasksets), dtype=torch.uint8, device=dev)
    L, ovh = workload.timeslice_us, workload.overhead_us
    stream = torch.cuda.current_stream(dev)
    if args.graph:  # the legacy default stream cannot be captured
        torch.cuda.synchronize(dev)
        stream = torch.cuda.Stream(dev)

    if args.mode == "assign":
        policies, names = [binding.POLICY_GCAPS, binding.ASSIGN], ["gcaps", "gpu_priority_search"]
        args.no_e2e = True
    pairs = None
    if args.mode == "sweep":
        # two legs per step: [0] the fused call, [1] one call per pair; the policy is the workload's
        # last one (round robin for the driver-model workload)
        sweep_policy = policies[-1]
        tl = getattr(workload, "timeslices", None) or [L]
        ol = getattr(workload, "overheads", None) or [0, 25, 50, 100, 200]
        pairs = [(a, b) for a in tl for b in ol]
        policies, names = ["fused", "separate"], ["fused_sweep", "one_call_per_pair"]
        sweep_sched = torch.empty((len(pairs), ts.n_tasksets), dtype=torch.uint8, device=dev)
        sweep_wcrt = torch.empty((len(pairs), ts.n_tasks), dtype=torch.int64, device=dev)
        args.no_e2e = True

    def call(k, policy):
        if args.mode == "assign" and k == 1:
            binding.rta_gpu_priority(ts, binding.ASSIGN, ovh, None, workspace=workspace, stream=stream)
        elif fused:
            binding.rta_multi(ts, binding.GCAPS_SUSPEND | binding.RR_SUSPEND, [L], [ovh],
                              out_wcrt=multi_wcrt, out_sched=multi_sched, workspace=workspace,
                              stream=stream)
        elif args.mode == "sweep" and k == 0:
            binding.rta_sweep(ts, sweep_policy, [a for a, _ in pairs], [b for _, b in pairs],
                              out_wcrt=sweep_wcrt, out_sched=sweep_sched, workspace=workspace,
                              stream=stream)
        elif args.mode == "sweep":
            for q, (a, b) in enumerate(pairs):
                binding.rta_batch(ts, sweep_policy, a, b, out_wcrt=sweep_wcrt[q],
                                  out_sched=sweep_sched[q], workspace=workspace, stream=stream)
        else:
            binding.rta_batch(ts, policy, L, ovh, out_wcrt=out_wcrt, out_sched=out_sched,
                              workspace=workspace, stream=stream)

    # --graph: each call's launches (plan kernels + one kernel per size bin) recorded once in a
    # CUDA graph and replayed; the entry points only enqueue work on the stream they are given, so
    # they can be captured as they are (after one plain call, which sets the kernels' attributes)
    graphs = None
    if args.graph:
        for k, policy in enumerate(policies):
            call(k, policy)
        torch.cuda.synchronize(dev)
        graphs = []
        for k, policy in enumerate(policies):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                call(k, policy)
            graphs.append(g)

    def step(events=None):
        for k, policy in enumerate(policies):
            if events is not None:
                events[k].record(stream)
            if graphs is not None:
                with torch.cuda.stream(stream):
                    graphs[k].replay()
            else:
                call(k, policy)
        if events is not None:
            events[len(policies)].record(stream)

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize(dev)

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        step()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(len(policies) + 1)] for _ in range(args.steps)]
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_id = str(local_rank)
    sampler = ClockSampler(gpu_id)
    barrier()
    sampler.start()
    t_wall0 = time.perf_counter()
    for k in range(args.steps):
        step(ev[k])
    barrier()
    t_wall = time.perf_counter() - t_wall0
    clocks = sampler.stop()
    total_ms = ev[0][0].elapsed_time(ev[-1][-1])
    per_policy_ms = [statistics.mean(e[k].elapsed_time(e[k + 1]) for e in ev) for k in range(len(policies))]
    best_policy_ms = [min(e[k].elapsed_time(e[k + 1]) for e in ev) for k in range(len(policies))]
    flags = sweep_sched[0] if args.mode == "sweep" else (multi_sched[0, 1] if fused else out_sched)
    sched_frac = float((flags == 1).float().mean().item()) if count else 0.0
    total_ms = sharding.reduce_scalars([total_ms], "max", dev)[0]
    ms_per_step = total_ms / args.steps
    value = total_count / (ms_per_step * 1e-3)
    if args.mode == "sweep":  # taskset analyses per second of the fused call alone
        value = total_count * len(pairs) / (per_policy_ms[0] * 1e-3)

    # ---- beside the headline: the busy-waiting analyses, planning on its own, the integer peak --
    def mean_ms(fn, n):
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n):
            fn()
        e1.record(stream)
        e1.synchronize()
        return e0.elapsed_time(e1) / n

    side = {}
    if args.mode == "policies" and not fused and not args.graph:
        n_side = max(3, min(args.steps, 20))
        busy_ms = {nm: mean_ms(lambda pol=pol: binding.rta_batch(
            ts, pol | binding.BUSY, L, ovh, out_wcrt=out_wcrt, out_sched=out_sched,
            workspace=workspace, stream=stream), n_side) for nm, pol in zip(names, policies)}
        plan_ms = mean_ms(lambda: binding.rta_plan(ts, workspace, stream=stream), n_side)
        side["busy_waiting"] = {
            "ms_per_launch": busy_ms, "value": count / (sum(busy_ms.values()) * 1e-3), "unit": UNIT,
            "note": "the same batch under the busy-waiting lemmas (GCAPS_RTA_BUSY), %d steps, this rank" % n_side}
        side["plan"] = {
            "ms_per_call": plan_ms,
            "share_of_call": {nm: plan_ms / ms for nm, ms in zip(names, per_policy_ms)},
            "analysis_only_ms": {nm: ms - plan_ms for nm, ms in zip(names, per_policy_ms)},
            "analysis_only_value": count / (sum(ms - plan_ms for ms in per_policy_ms) * 1e-3),
            "note": "size binning of the batch (gcaps_rta_plan_batch) timed alone; `value` is plan + analysis"}
    alu_peaks, alu_peak, alu_kind = None, ALU_PEAK_DERIVED, "derived (148 SMs x 128 lanes x 1.965 GHz)"
    if rank == 0:
        try:
            alu_peaks = {nm: binding.int_issue_rate(kind, device=dev)
                         for kind, nm in enumerate(("multiply_add", "add", "multiply_add_and_add"))}
            alu_peak, alu_kind = alu_peaks["multiply_add_and_add"], "measured"
        except Exception as exc:   # keep the derived figure, say why
            alu_kind += "; probe failed: %s" % exc

    # ---- end to end through the host-buffer entry point (copies inside the timed region) -----
    e2e = None
    if not args.no_e2e:
        host_wcrt = [torch.empty(max(ts.n_tasks, 1), dtype=torch.int64, pin_memory=True).numpy()[:ts.n_tasks]
                     for _ in host_policies]
        host_sched = [torch.empty(max(ts.n_tasksets, 1), dtype=torch.uint8, pin_memory=True).numpy()[:ts.n_tasksets]
                      for _ in host_policies]
        arrays = batch.arrays()
        # warm-up: staging buffers get allocated here
        binding.rta_batch_host_multi(arrays, host_policies, L, ovh, host_wcrt, host_sched)
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            binding.rta_batch_host_multi(arrays, host_policies, L, ovh, host_wcrt, host_sched)
        barrier()
        dt = time.perf_counter() - t0
        dt = sharding.reduce_scalars([dt], "max", dev)[0]
        e2e = {"value": total_count * args.e2e_steps / dt, "unit": UNIT,
               "h2d_bytes_per_step": batch.input_bytes(),
               "d2h_bytes_per_step": len(host_policies) * batch.output_bytes(),
               "steps": args.e2e_steps, "ms_per_step": 1e3 * dt / args.e2e_steps,
               "api": "gcaps_rta_batch_host_multi, page-locked host arrays, one copy in, both policies"}
        binding.release_host()

    # ---- the oracle beside it, and the roofline of the dominant launch ------------------------
    cpu = None
    bytes_per_call = batch.input_bytes() + batch.output_bytes()
    if args.mode == "sweep":  # inputs once, outputs once per pair
        bytes_per_call = batch.input_bytes() + len(pairs) * batch.output_bytes()
    if fused:                 # inputs once, outputs once per analysis
        bytes_per_call = batch.input_bytes() + 2 * batch.output_bytes()
    peak, peak_kind = measured_peaks()
    roof = None
    if rank == 0:
        dom = 0 if args.mode == "sweep" else int(np.argmax(per_policy_ms))
        achieved = bytes_per_call / (per_policy_ms[dom] * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak,
                "traffic": captured_traffic(workload.name, names[dom], count),
                "peak_kind": peak_kind,
                "kernel": "analysis kernel of the %s call (the call's plan kernels are inside the timing)"
                          % names[dom].upper() + (": both analyses of a taskset in one launch" if fused else ""),
                "algorithmic_bytes_per_launch": bytes_per_call,
                "ms_per_launch": dict(zip(names, per_policy_ms)),
                "best_ms_per_launch": dict(zip(names, best_policy_ms)),
                "frac_per_policy": {nm: bytes_per_call / (ms * 1e-3) / 1e9 / peak
                                    for nm, ms in zip(names, per_policy_ms)}}
        roof["alu_peak_kind"] = alu_kind
        roof["alu_peak_tlaneops"] = alu_peak / 1e12
        roof["int_issue_probe_tlaneops"] = ({k: v / 1e12 for k, v in alu_peaks.items()}
                                            if alu_peaks else None)
        if world == 1 and not args.no_cpu_baseline and args.mode == "policies":
            r = oracle_sample(workload, first, count, args.cpu_budget, stream=args.stream)
            n_tasks_per_set = ts.n_tasks / max(1, ts.n_tasksets)
            cpu = {"value": r["tasksets"] / r["seconds"], "unit": UNIT, "cores": 1, "kind": "oracle",
                   "sample": "first %d tasksets of the workload, both policies, %.1f s, generation excluded"
                             % (r["tasksets"], r["seconds"]),
                   "terms_per_taskset": {"gcaps": r["terms"][0] / r["tasksets"], "rr": r["terms"][1] / r["tasksets"]},
                   "sweeps_per_taskset": {"gcaps": r["sweeps"][0] / r["tasksets"], "rr": r["sweeps"][1] / r["tasksets"]},
                   # share of the tasks whose recurrence is started at all (the rest sit behind the
                   # first deadline miss of their taskset)
                   "tasks_analysed_fraction": {
                       "gcaps": r["started"][0] / (r["tasksets"] * n_tasks_per_set),
                       "rr": r["started"][1] / (r["tasksets"] * n_tasks_per_set)}}
            if not args.no_cpu_all_cores:
                per_core = max(200, min(int(cpu["value"] * args.cpu_all_cores_budget), count // 2))
                cpu["all_cores"] = oracle_all_cores(workload, first, per_core, stream=args.stream)
            # which roofline binds: algorithmic integer work against algorithmic bytes
            t_mem = bytes_per_call / (peak * 1e9)
            terms = sum(r["terms"]) if fused else r["terms"][policies[dom]]
            t_alu = count * (K_TERM * terms / r["tasksets"] + K_SETUP * n_tasks_per_set) / alu_peak
            roof["model_ms"] = {"hbm": 1e3 * t_mem, "alu": 1e3 * t_alu}
            roof["frac_alu"] = t_alu / (per_policy_ms[dom] * 1e-3)
            if t_alu > t_mem:
                ops = t_alu * alu_peak
                ach = ops / (per_policy_ms[dom] * 1e-3)
                roof.update(bound="alu", achieved=ach / 1e12, peak=alu_peak / 1e12,
                            unit="Tlaneop/s", frac=ach / alu_peak)
    # ---- a diagnostic beside the workload (never instead of it): tasksets of the same shape that
    # converge, so that the recurrence of Eq. 1 runs for every task instead of ending at an early miss
    diagnostic = None
    if (rank == 0 and world == 1 and args.mode == "policies" and not fused and not args.graph
            and workload.name == "large" and not args.no_diagnostic and not args.on_device_inputs):
        from oracle import rta
        light = taskgen.WORKLOADS["large_light"]
        d_count = min(light.n_tasksets, 200_000)
        d_batch = light.generate(0, d_count)
        d_ts = binding.DeviceTasksets.from_host(d_batch, dev)
        d_w = torch.empty(d_ts.n_tasks, dtype=torch.int64, device=dev)
        d_s = torch.empty(d_ts.n_tasksets, dtype=torch.uint8, device=dev)
        d_bytes = d_batch.input_bytes() + d_batch.output_bytes()
        d_ms, d_sched, d_terms = {}, {}, {}
        sample = d_batch.slice(0, 2000)
        for nm, pol in zip(names, policies):
            d_ms[nm] = mean_ms(lambda pol=pol: binding.rta_batch(
                d_ts, pol, light.timeslice_us, light.overhead_us, out_wcrt=d_w, out_sched=d_s,
                workspace=workspace, stream=stream), 20)
            d_sched[nm] = float((d_s == 1).float().mean().item())
            _, _, c = rta.analyse(sample, pol, light.timeslice_us, light.overhead_us)
            d_terms[nm] = c.terms / 2000.0
        diagnostic = {
            "workload": light.name, "note": light.note, "tasksets": d_count,
            "ms_per_launch": d_ms, "schedulable_fraction": d_sched,
            "oracle_terms_per_taskset": d_terms,
            "tasksets_per_s": {nm: d_count / (ms * 1e-3) for nm, ms in d_ms.items()},
            "frac_hbm": {nm: d_bytes / (ms * 1e-3) / 1e9 / peak for nm, ms in d_ms.items()},
            "frac_alu": {nm: d_count * (K_TERM * d_terms[nm] + K_SETUP * 80) / alu_peak / (ms * 1e-3)
                         for nm, ms in d_ms.items()},
            "alu_model": "%d lane-ops per interference term the oracle counts + %d per task, against "
                         "the integer issue rate (%s)" % (K_TERM, K_SETUP, alu_kind)}
        del d_ts, d_w, d_s

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": args.scaling, "vs_baseline": None, "dtype": "int64", "data": "synthetic",
            "config": {"workload": workload.name, "note": workload.note, "tasksets_per_gpu": count,
                       "tasks": ts.n_tasks, "policies": names, "mode": "self-suspension",
                       "timeslice_us": L, "overhead_us": ovh,
                       "analyses_per_taskset_per_step": len(pairs) if pairs else analyses_per_step,
                       "calls_per_step": len(policies),
                       "launch": "cuda graph replay per call" if args.graph else "stream launches",
                       "sweep_pairs": pairs, "generation": generation,
                       "l2": "inputs (%.2f GB per call) against a 126 MB L2; no flush between steps"
                             % (batch.input_bytes() / 1e9),
                       "schedulable_fraction_last_policy": sched_frac,
                       "input_checksum": batch.checksum() if count <= 200_000 else None},
            "clocks": clocks, "e2e": e2e,
            "gpu_launches": args.steps * (len(policies) if args.mode == "policies"
                                          else (1 + len(pairs)) if args.mode == "sweep" else 2)
                            * (LAUNCHES_PER_SMALL_CALL if count <= 8192 else LAUNCHES_PER_CALL),
            "roofline": roof, "cpu_baseline": cpu, "wall_s_timed_region": t_wall,
        }
        line.update(side)
        if diagnostic is not None:
            line["recurrence_diagnostic"] = diagnostic
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

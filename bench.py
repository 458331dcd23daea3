#!/usr/bin/env python
"""Benchmark of the Cleave hot path on B200: decomposed GEMM + assembly throughput per step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 3]

A step is one pass of the path over one batch of synthetic input: queue arming, the grouped
sub-GEMM execution of every task of every GEMM of the layer, and the assembly of the K-split
partial blocks into the GEMM results.  The plan is made once before the loop (the paper computes a
schedule when the device set changes, not per batch); its time and the churn path (drop 10 % of the tasks,
re-plan, reissue, re-assemble) are measured separately and reported inside `config`.

One JSON line is printed by rank 0.  With --gpus N > 1 (launched through torch.distributed.run)
every rank runs an independent replica of the same workload on its own GPU: the path has no
inter-GPU exchange step, so there is no collective on the data path ("replicas only").
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decomposed GEMM+assembly TFLOP/s and % of B200 dense BF16 peak, per step"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def measured_traffic(kernel: str):
    """(DRAM bytes per full-size launch, how they were obtained) from the ncu record in
    profiles/dram_traffic.txt, or (None, reason) when there is no record or the kernel's source
    changed since the counters were taken."""
    import hashlib
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.txt")) as f:
            rec = json.load(f)[kernel]
        with open(os.path.join(ROOT, rec["source"]), "rb") as f:
            if hashlib.sha1(f.read()).hexdigest() != rec["sha1"]:
                return None, "kernel source changed since the capture"
        if rec.get("dram_bytes_captured_launch") is None:
            return None, "no capture recorded"
        return rec["dram_bytes_captured_launch"] * rec["scale_to_full"], rec["how"]
    except Exception:
        return None, "no capture recorded"


def load_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


# --------------------------------------------------------------------------------------------------
# clocks during the timed region (read-only NVML queries)
# --------------------------------------------------------------------------------------------------
REASON_BITS = {0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x10: "sync_boost",
               0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown"}


class ClockSampler:
    def __init__(self, device_index: int):
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self._nv = pynvml
            try:
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                if not uuid.startswith("GPU-"):
                    uuid = "GPU-" + uuid
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for b, name in REASON_BITS.items():
                    if bits & b:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.01)

    def start(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread:
            self._stop.set()
            self._thread.join()
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------------------------------
# the oracle on the host cores (reported baseline / --impl reference)
# --------------------------------------------------------------------------------------------------
def oracle_block_groups(w, opts):
    """The oracle's own plan of the workload, its tasks grouped by output rectangle (all K-slices
    of one block), in a seeded random order."""
    import numpy as np
    import cleave_inputs as ci
    from oracle.cost import devices_from_array
    from oracle.plan import Gemm, Opts, plan, plan_uniform
    gemms = [Gemm(g.M, g.N, g.K, g.transA, g.transB) for g in w.gemms]
    t0 = time.perf_counter()
    devs = ci.workload_devices(w)
    op = plan_uniform(gemms, *w.uniform, Opts(**opts)) if devs is None else plan(gemms, devices_from_array(devs), Opts(**opts))
    plan_s = time.perf_counter() - t0
    groups = {}
    for t in op.tasks:
        groups.setdefault((t.gemm, t.m0, t.m1, t.n0, t.n1), []).append(t)
    keys = sorted(groups)
    order = np.random.default_rng(w.seed + 3).permutation(len(keys))
    return op, [groups[keys[i]] for i in order], plan_s


def oracle_run_groups(w, bits, groups):
    """fp64 sub-GEMMs of every task of the groups plus the tree-sum of each block's K-slices."""
    from oracle import numerics as nm
    flops = 0
    for tasks in groups:
        g = w.gemms[tasks[0].gemm]
        parts = [nm.sub_gemm_from_bits(t, g.transA, g.transB, bits[g.a_key], bits[g.b_key])
                 for t in sorted(tasks, key=lambda t: t.kslice)]
        nm.tree_sum(parts)
        flops += sum(2 * t.alpha * t.beta * t.kappa for t in tasks)
    return flops


def blas_threads():
    try:
        import threadpoolctl
        n = [i["num_threads"] for i in threadpoolctl.threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return len(os.sched_getaffinity(0))


def cpu_baseline(w, tensors, opts, budget_s=15.0):
    import cleave_inputs as ci
    bits = {k: ci.bf16_bits(t) for k, t in tensors.items()}
    op, groups, plan_s = oracle_block_groups(w, opts)
    t0 = time.perf_counter()
    flops, n = 0, 0
    for grp in groups:
        flops += oracle_run_groups(w, bits, [grp])
        n += 1
        if time.perf_counter() - t0 > budget_s:
            break
    dt = time.perf_counter() - t0
    return {"value": flops / dt / 1e12, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"{n} of {len(groups)} output blocks (all K-slices each, seeded random order) of {w.name}: "
                      f"fp64 sub-GEMMs + tree assembly, {flops / 1e12:.3f} TFLOP in {dt:.1f} s; "
                      f"oracle plan of the full workload took {plan_s:.2f} s (not in the rate)",
            "host_cores_available": len(os.sched_getaffinity(0))}


def run_reference(args):
    """--impl reference: the oracle, as it stands, on the host cores; each step is a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import cleave_inputs as ci
    w = ci.config(args.config)
    tensors = ci.make_tensors(w)
    bits = {k: ci.bf16_bits(t) for k, t in tensors.items()}
    op, groups, plan_s = oracle_block_groups(w, {})
    # size a step: calibrate on a few blocks, then fix the number of blocks per step
    t0 = time.perf_counter()
    oracle_run_groups(w, bits, groups[:4])
    per_block = (time.perf_counter() - t0) / 4
    step_budget = min(2.0, 90.0 / (args.steps + args.warmup))
    per_step = max(1, min(len(groups) // (args.steps + args.warmup), int(step_budget / max(per_block, 1e-6))))
    cursor = 0
    for _ in range(args.warmup):
        oracle_run_groups(w, bits, groups[cursor:cursor + per_step]); cursor += per_step
    flops, t0 = 0, time.perf_counter()
    for _ in range(args.steps):
        flops += oracle_run_groups(w, bits, groups[cursor:cursor + per_step]); cursor += per_step
    dt = time.perf_counter() - t0
    value = flops / dt / 1e12
    sample = (f"each step = {per_step} of {len(groups)} output blocks (all K-slices each) of {w.name}: fp64 sub-GEMMs + "
              f"tree assembly on the host cores")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "gemms": len(w.gemms), "devices": w.n_devices, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------------
# rank plumbing (replicas only: no collective on the data path)
# --------------------------------------------------------------------------------------------------
def rank_max(x: float, dist, device) -> float:
    """The slowest rank's time: every rank reports the same number."""
    if dist is None:
        return x
    import torch
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(flop_per_replica: float, world: int, ms_per_step: float) -> float:
    """Whole-job TFLOP/s of `world` independent replicas that all finish a step in ms_per_step."""
    return world * flop_per_replica / (ms_per_step * 1e-3) / 1e12


# --------------------------------------------------------------------------------------------------
# a short leg on another workload or mode (reported under config.other_workloads)
# --------------------------------------------------------------------------------------------------
def plan_summary(plan, n_gemms, n_devices):
    """The paper's quantities of a plan: modelled makespans against the water-fill level, devices with work."""
    import numpy as np
    t = plan.tasks()
    ratios = [plan.makespan_ns(i) / plan.tstar_ns(i) for i in range(n_gemms) if plan.tstar_ns(i)]
    return {"tasks": int(plan.num_tasks), "tiles": int(plan.num_tiles),
            "active_devices": int(len(np.unique(t["dev"]))) if n_devices else None,
            "makespan_over_waterfill_level_median": float(np.median(ratios)) if ratios else None,
            "modelled_step_makespan_ms": plan.step_makespan_ns / 1e6}


def library_gemm_here(torch, dev, local, warm_s=1.5, timed_s=1.0, n=8192):
    """The vendor library's bf16 GEMM (n^3) on THIS GPU, the way the pool's sustained figure was taken: back to back
    until the power cap has pulled the clocks down, then timed with CUDA events, SM clock sampled meanwhile.  Context
    for the roofline fraction (GPUs of one pool differ by several percent under the same cap); not on any timed path."""
    a = torch.randn(n, n, device=dev).to(torch.bfloat16)
    b = torch.randn(n, n, device=dev).to(torch.bfloat16)
    c = torch.empty(n, n, device=dev, dtype=torch.bfloat16)
    reps, t0 = 0, time.perf_counter()
    while time.perf_counter() - t0 < warm_s:
        for _ in range(20):
            torch.matmul(a, b, out=c)
        torch.cuda.synchronize()
        reps += 20
    per_s = reps / (time.perf_counter() - t0)
    k = max(20, int(per_s * timed_s))
    sampler = ClockSampler(local)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.start()
    e0.record()
    for _ in range(k):
        torch.matmul(a, b, out=c)
    e1.record()
    torch.cuda.synchronize()
    clk = sampler.stop()
    ms = e0.elapsed_time(e1) / k
    return {"tflops": 2.0 * n ** 3 / (ms * 1e-3) / 1e12, "sm_mhz": clk.get("sm_mhz"), "reasons": clk.get("reasons"),
            "how": f"torch.matmul bf16 {n}^3, {k} calls back to back after {warm_s} s of the same"}


def quick_leg(cl, ci, torch, dev, name, cfg, scale, opts, mode, min_s=0.6, tensors=None, bf16_out=False, consume=True):
    """Plans the workload, runs it for at least `min_s` seconds untimed, then times the same number of
    steps again: step / exec / assembly times from CUDA events on the launching stream."""
    w = ci.config(cfg, scale)
    if tensors is None:
        tensors = {k: t.to(dev) for k, t in ci.make_tensors(w).items()}
    devs = ci.workload_devices(w)
    o = cl.default_opts(**opts)
    plan = cl.plan_uniform(w.gemms, *w.uniform, o) if devs is None else cl.plan(w.gemms, devs, o)
    A = [tensors[g.a_key] for g in w.gemms]
    B = [tensors[g.b_key] for g in w.gemms]
    partials = torch.empty(max(1, plan.arena_elems), dtype=torch.float32, device=dev)
    C = [torch.empty((g.M, g.N), dtype=torch.bfloat16 if bf16_out else torch.float32, device=dev) for g in w.gemms]

    def step():
        if mode == "two-step":
            plan.exec_opts(A, B, partials, C, bf16=bf16_out)
        else:
            plan.exec_opts(A, B, partials, C, direct=True, finish=True, bf16=bf16_out, consume=consume)
        plan.assemble(partials, C)

    n, t0 = 0, time.perf_counter()
    while True:
        step(); n += 1
        if n % 8 == 0:
            torch.cuda.synchronize()
            if time.perf_counter() - t0 >= min_s:
                break
    plan.check_status()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n)]
    torch.cuda.synchronize()
    for e in ev:
        e[0].record()
        if mode == "two-step":
            plan.exec_opts(A, B, partials, C, bf16=bf16_out)
        else:
            plan.exec_opts(A, B, partials, C, direct=True, finish=True, bf16=bf16_out, consume=consume)
        e[1].record()
        plan.assemble(partials, C)
        e[2].record()
    torch.cuda.synchronize()
    plan.check_status()
    step_ms = ev[0][0].elapsed_time(ev[-1][2]) / n
    exec_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in ev)
    asm_ms = statistics.mean(e[1].elapsed_time(e[2]) for e in ev)
    S = [plan.ksplit(i) for i in range(len(w.gemms))]
    asm_bytes = float(sum((S[i] + 1) * g.M * g.N * 4 for i, g in enumerate(w.gemms)
                          if mode == "two-step" or not (S[i] == 1 or plan.finishable(i))))
    out = {"name": name, "workload": w.name, "opts": opts, "write_out": mode, "c_dtype": "bf16" if bf16_out else "fp32",
           "steps_timed": n, "step_ms": step_ms, "step_TFLOPs": w.flops / step_ms / 1e9, "exec_ms": exec_ms,
           "exec_TFLOPs": w.flops / exec_ms / 1e9, "assemble_ms": asm_ms,
           "assemble_GBs": asm_bytes / asm_ms / 1e6 if asm_bytes else None, "assemble_bytes": asm_bytes,
           "arena_GB": plan.arena_elems * 4 / 1e9, "ksplit_max": max(S)}
    out.update(plan_summary(plan, len(w.gemms), w.n_devices))
    plan.close()
    del partials, C
    return out


# --------------------------------------------------------------------------------------------------
# the CUDA path
# --------------------------------------------------------------------------------------------------
def run_ours(args):
    import numpy as np
    import torch

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank == 0:
        from paper_2512_22142_b200.build import build_library
        build_library()                               # no-op when the in-tree library is up to date
    import cleave_inputs as ci
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
        dist.barrier()                                # rank 0 may have just built the library
    import paper_2512_22142_b200 as cl

    w = ci.config(args.config, args.scale)
    opts = {}
    if args.kslice_max is not None:
        opts["kslice_max"] = args.kslice_max
    if args.gran_m is not None:
        opts["gran_m"] = args.gran_m
    t0 = time.perf_counter()
    tensors = ci.make_tensors(w, pin=True)
    gen_s = time.perf_counter() - t0
    devs = ci.workload_devices(w)
    t0 = time.perf_counter()
    plan_opts = cl.default_opts(**opts)
    plan = cl.plan_uniform(w.gemms, *w.uniform, plan_opts) if devs is None else cl.plan(w.gemms, devs, plan_opts)
    plan_ms = (time.perf_counter() - t0) * 1e3

    d_tensors = {k: t.to(dev) for k, t in tensors.items()}
    A = [d_tensors[g.a_key] for g in w.gemms]
    B = [d_tensors[g.b_key] for g in w.gemms]
    partials = torch.empty(plan.arena_elems, dtype=torch.float32, device=dev)
    c_dtype = torch.bfloat16 if args.bf16_out else torch.float32
    c_bytes = 2 if args.bf16_out else 4
    C = [torch.empty((g.M, g.N), dtype=c_dtype, device=dev) for g in w.gemms]
    flops = float(w.flops)
    S = [plan.ksplit(i) for i in range(len(w.gemms))]
    # bytes the assembly kernels move: GEMMs with one K-slice are finished by the exec kernel in fused mode
    in_kernel = [(not args.two_step) and (S[i] == 1 or (not args.no_finish and plan.finishable(i))) for i in range(len(w.gemms))]
    asm_bytes = float(sum((S[i] + 1) * g.M * g.N * 4 for i, g in enumerate(w.gemms) if not in_kernel[i]))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        return rank_max(x, dist, dev)

    # ---- device-resident steps -------------------------------------------------------------------
    def run_exec():
        # one-slice GEMMs are written straight to C by the exec kernel unless --two-step is given
        if args.two_step:
            plan.exec_opts(A, B, partials, C, bf16=args.bf16_out)
        else:
            plan.exec_opts(A, B, partials, C, direct=True, finish=not args.no_finish, bf16=args.bf16_out,
                           consume=not args.keep_blocks and not args.no_finish)

    # warm-up: at least --warmup steps AND at least --min-warm-s seconds of back-to-back steps, so that the
    # timed steps see the clocks of a long run (the power cap pulls them down within about a second)
    warm_steps, t_warm = 0, time.perf_counter()
    while warm_steps < args.warmup or time.perf_counter() - t_warm < args.min_warm_s:
        run_exec()
        plan.assemble(partials, C)
        warm_steps += 1
        if warm_steps % 8 == 0:
            torch.cuda.synchronize()
    plan.check_status()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local) if rank == 0 else None
    barrier()
    if sampler:
        sampler.start()
    begin, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    begin.record()
    for s in range(args.steps):
        ev[s][0].record()
        run_exec()
        ev[s][1].record()
        plan.assemble(partials, C)
        ev[s][2].record()
    end.record()
    barrier()
    clocks = sampler.stop() if sampler else None
    plan.check_status()
    total_ms = max_over_ranks(begin.elapsed_time(end))
    exec_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in ev)
    asm_ms = statistics.mean(e[1].elapsed_time(e[2]) for e in ev)
    step_times = [e[0].elapsed_time(e[2]) for e in ev]
    ms_per_step = total_ms / args.steps
    value = job_throughput(flops, world, ms_per_step)

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region ----------------
    host_C = [torch.empty((g.M, g.N), dtype=c_dtype).pin_memory() if args.e2e_steps > 0 else
              torch.empty((g.M, g.N), dtype=c_dtype) for g in w.gemms]
    h2d = sum(t.numel() * 2 for t in tensors.values())
    d2h = sum(c.numel() * c_bytes for c in host_C)

    def e2e_step():
        for k, t in tensors.items():
            d_tensors[k].copy_(t, non_blocking=True)
        run_exec()
        plan.assemble(partials, C)
        for hc, c in zip(host_C, C):
            hc.copy_(c, non_blocking=True)

    # (a) serial: copy in, compute, copy out on one stream
    b2, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if args.e2e_steps > 0:
        e2e_step()
    barrier()
    b2.record()
    for _ in range(max(args.e2e_steps, 0)):
        e2e_step()
    e2.record()
    barrier()
    e2e_serial_ms = max_over_ranks(b2.elapsed_time(e2)) / max(args.e2e_steps, 1) if args.e2e_steps > 0 else float("nan")

    # (b) pipelined, as a training loop would drive the library: two sets of device buffers, the
    # host-to-device copy of step i+1 and the device-to-host copy of step i-1 overlap the kernels of
    # step i (three streams).  Every step still copies all of its own inputs in and all of its own
    # results out inside the timed region.
    e2e_ms = e2e_serial_ms
    if args.e2e_steps > 0:
        sets = [(d_tensors, C, plan)]
        d2 = {k: torch.empty_like(t) for k, t in d_tensors.items()}
        plan_b = cl.plan_uniform(w.gemms, *w.uniform, cl.default_opts(**opts)) if devs is None else cl.plan(w.gemms, devs, cl.default_opts(**opts))
        sets.append((d2, [torch.empty_like(c) for c in C], plan_b))
        s_in, s_comp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
        n_pipe = 2 * args.e2e_steps + 2
        in_done = [torch.cuda.Event() for _ in range(n_pipe)]
        comp_done = [torch.cuda.Event() for _ in range(n_pipe)]
        out_done = [torch.cuda.Event() for _ in range(n_pipe)]
        t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

        def pipe_step(i):
            dt, Cs, pl = sets[i % 2]
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(comp_done[i - 2])            # the kernels that read this input set are done
                for k, t in tensors.items():
                    dt[k].copy_(t, non_blocking=True)
                in_done[i].record(s_in)
            with torch.cuda.stream(s_comp):
                s_comp.wait_event(in_done[i])
                if i >= 2:
                    s_comp.wait_event(out_done[i - 2])           # this output set has been copied out
                Ai, Bi = [dt[g.a_key] for g in w.gemms], [dt[g.b_key] for g in w.gemms]
                if args.two_step:
                    pl.exec_opts(Ai, Bi, partials, Cs, bf16=args.bf16_out)
                else:
                    pl.exec_opts(Ai, Bi, partials, Cs, direct=True, finish=not args.no_finish, bf16=args.bf16_out,
                                 consume=not args.keep_blocks and not args.no_finish)
                pl.assemble(partials, Cs)
                comp_done[i].record(s_comp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(comp_done[i])
                for hc, c in zip(host_C, Cs):
                    hc.copy_(c, non_blocking=True)
                out_done[i].record(s_out)

        for i in range(2):                                        # fill the pipeline (untimed)
            pipe_step(i)
        barrier()
        t_begin.record()
        for s_ in (s_in, s_comp, s_out):
            s_.wait_event(t_begin)
        for i in range(2, n_pipe):
            pipe_step(i)
        torch.cuda.current_stream().wait_event(out_done[n_pipe - 1])
        t_end.record()
        barrier()
        plan_b.check_status()
        e2e_ms = max_over_ranks(t_begin.elapsed_time(t_end)) / (n_pipe - 2)
    e2e_value = job_throughput(flops, world, e2e_ms)
    checksum = float(host_C[0][0, :8].double().sum()) if args.e2e_steps > 0 else None

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- churn path (rank 0, once): drop 10 %, execute, re-plan + reissue, re-assemble ------------------
    churn = None
    if devs is not None and not args.no_churn:
        p2 = cl.plan(w.gemms, devs, cl.default_opts(**opts))
        failed = ci.make_failed_ids(p2.num_tasks, 0.10, w.seed + 2)
        p2.set_drops(failed)
        if args.two_step:
            p2.exec_opts(A, B, partials, C, bf16=args.bf16_out)
        else:
            p2.exec_opts(A, B, partials, C, direct=True, finish=not args.no_finish, bf16=args.bf16_out)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        c0, c1, c2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        c0.record()
        p2.reissue(failed, A, B, partials)
        host_ms = (time.perf_counter() - t0) * 1e3
        c1.record()
        p2.assemble(partials, C)
        c2.record()
        torch.cuda.synchronize()
        replay_ms = p2.last_kernel_ms()[0]                  # the exec kernel over the replacement tasks alone
        churn = {"failed_tasks": int(len(failed)), "reissued_tasks": int(p2.num_tasks - p2.num_original),
                 "reissue_host_ms": host_ms, "reissue_device_ms": c0.elapsed_time(c1), "replay_kernel_ms": replay_ms,
                 "reassemble_ms": c1.elapsed_time(c2), "status": p2.status(),
                 "note": "reissue_device_ms spans the call on the stream, host re-plan included (the GPU waits for it); "
                         "replay_kernel_ms is the exec kernel over the replacement tasks"}
        p2.close()

    # ---- block verification (Section 6 of the paper), once, on the result of the last step -------------------
    verify = None
    if not args.no_verify and not (args.bf16_out and not args.two_step):
        t = plan.tasks()
        live = (t["flags"] & 1) == 0
        al, be, ka = (t["m1"] - t["m0"]).astype(np.float64), (t["n1"] - t["n0"]).astype(np.float64), (t["k1"] - t["k0"]).astype(np.float64)
        vbytes = float((((al + be) * ka * 2 + al * be * 4) * live).sum())
        if not args.two_step:                          # every block into the arena (the timed steps use some up on arrival)
            plan.exec_opts(A, B, partials, C, direct=True, finish=not args.no_finish, bf16=args.bf16_out)
        plan.verify(A, B, partials, seed=1)            # first call allocates
        v0, v1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        v0.record()
        n_bad, _ = plan.verify(A, B, partials, seed=2)
        v1.record()
        torch.cuda.synchronize()
        vms = v0.elapsed_time(v1)
        verify = {"flagged_tasks": int(n_bad), "ms": vms, "dispatch_volume_GB": vbytes / 1e9,
                  "dispatch_volume_GB_per_s": vbytes / vms / 1e6,
                  "note": "bytes = every task's own rows, columns and block (the method's dispatch + return volume); "
                          "tasks share operand panels, so part of it is served by L2: a rate, not a DRAM roofline fraction"}

    # ---- other modes and workloads, short legs (rank 0, N = 1): observed in the same run as the headline ----
    others = []
    if world == 1 and not args.no_other:
        shared = dict(tensors=d_tensors)
        base = dict(opts)
        legs = [("same workload, two-step (cleave_exec + cleave_assemble of every GEMM)", args.config, args.scale, base, "two-step", False, shared),
                ("same workload, every block kept in the arena", args.config, args.scale, base, "fused", False, dict(shared, consume=False)),
                ("same workload, bf16 outputs", args.config, args.scale, base, "fused", True, shared)]
        if args.gran_m is None:
            legs.append(("same workload, row granule 256", args.config, args.scale, dict(base, gran_m=256), "fused", False, shared))
        if args.kslice_max is None:                        # the K-slice cap's sweep: half the default, and no cap (one slice per GEMM)
            legs.append(("same workload, K-slices of at most 2048", args.config, args.scale, dict(base, kslice_max=2048), "fused", False, shared))
            legs.append(("same workload, no K-slice cap (every GEMM one slice)", args.config, args.scale, dict(base, kslice_max=0), "fused", False, shared))
        if args.config == 3 and args.scale == 1:
            legs += [("GPT-2-small-shaped layer, 64 devices", 2, 1, {}, "fused", False, {}),
                     ("Llama-13B-shaped layer, 4096 devices", 5, 1, {}, "fused", False, {}),
                     ("attention GEMMs of 1024 heads as tasks, 64 devices", 6, 1, {}, "fused", False, {}),
                     ("attention GEMMs of 1024 heads as tasks, bf16 outputs", 6, 1, {}, "fused", True, {})]
        for name, cfg, scale, o, mode, b16, kw in legs:
            try:
                others.append(quick_leg(cl, ci, torch, dev, name, cfg, scale, o, mode, bf16_out=b16, **kw))
            except Exception as e:                          # a leg must not cost the headline its line
                others.append({"name": name, "error": repr(e)})
            torch.cuda.empty_cache()

    lib_here = None
    if rank == 0 and not args.no_library_gemm:
        try:
            lib_here = library_gemm_here(torch, dev, local)
        except Exception as e:                              # context only: never costs the line
            lib_here = {"error": repr(e)}
    peaks, peak_kind = load_peaks()
    exec_tflops = flops / (exec_ms * 1e-3) / 1e12
    sm_mhz = clocks["sm_mhz"] if clocks and clocks.get("sm_mhz") else None
    sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
    flop_per_clk_per_sm = flops / (exec_ms * 1e-3) / (sm_mhz * 1e6) / sm_count if sm_mhz else None
    traffic, traffic_how = (measured_traffic("exec_pair_kernel") if (args.config == 3 and args.scale == 1 and not args.two_step
                                                                      and not args.bf16_out and not args.no_finish)
                            else (None, "recorded for the default run of the Llama-7B-shaped layer only"))
    # the assembly kernels only run where the exec kernel cannot finish a GEMM itself: their roofline comes from
    # this run when it launches them, else from the two-step leg above
    asm_src = {"ms": asm_ms, "bytes": asm_bytes, "from": "this run's steps"} if asm_bytes else None
    if asm_src is None:
        for o in others:
            if o.get("write_out") == "two-step" and o.get("assemble_bytes"):
                asm_src = {"ms": o["assemble_ms"], "bytes": o["assemble_bytes"], "from": "the two-step leg of this run (config.other_workloads[0])"}
    asm_traffic, asm_traffic_how = measured_traffic("assemble_vec_kernel")
    roofline_assemble = None
    if asm_src:
        asm_gbs = asm_src["bytes"] / (asm_src["ms"] * 1e-3) / 1e9
        roofline_assemble = {"kernel": "assemble_vec_kernel", "bound": "hbm", "achieved": asm_gbs, "peak": peaks["hbm_gbs"],
                             "unit": "GB/s", "frac": asm_gbs / peaks["hbm_gbs"],
                             "traffic": asm_traffic if (args.config == 3 and args.scale == 1) else None, "traffic_how": asm_traffic_how,
                             "peak_kind": f"{peak_kind} copy bandwidth", "frac_of_nominal": asm_gbs / NOMINAL_HBM_GBS,
                             "algorithmic_bytes": asm_src["bytes"], "timed_in": asm_src["from"]}
    step_s = warm_steps * ms_per_step * 1e-3
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warm_steps,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": w.name, "gemms": len(w.gemms), "devices": w.n_devices, "flop_per_step": flops, "ksplit": S,
            "granule": [plan_opts.gran_m, plan_opts.gran_n, plan_opts.gran_k], "kslice_max": plan_opts.kslice_max,
            "plan": plan_summary(plan, len(w.gemms), w.n_devices), "arena_GB": plan.arena_elems * 4 / 1e9,
            "parallelism": "replicas only" if world > 1 else "1 GPU",
            "write_out": ("two-step: every block to the arena, every GEMM through cleave_assemble" if args.two_step else
                          "in the exec kernel: one-slice blocks stored in C" +
                          ("" if args.no_finish else ", K-split cells summed in fixed order by the block that arrives last" +
                           ("" if args.keep_blocks else " (that block is used up on arrival, the others are stored in the arena)"))),
            "c_dtype": "bf16" if args.bf16_out else "fp32",
            "gemms_finished_in_exec_kernel": int(sum(in_kernel)),
            "l2": "not flushed; operands + arena + outputs per step (~%.1f GB) far exceed the 126 MB L2" %
                  ((h2d + plan.arena_elems * 4 + d2h) / 1e9),
            "warmup": f"{warm_steps} steps, about {step_s:.1f} s back to back (at least --warmup steps and --min-warm-s seconds)",
            "plan_ms_host": plan_ms, "step_ms_median": statistics.median(step_times), "step_ms_best": min(step_times),
            "input_gen_s": gen_s, "exec_ms": exec_ms, "assemble_ms": asm_ms,
            "pct_of_nominal_bf16_peak": 100 * value / world / NOMINAL_BF16_TFLOPS,
            "pct_of_measured_sustained_bf16": 100 * value / world / peaks["bf16_tflops_sustained"],
            "churn": churn, "verify": verify, "e2e_ms_per_step": e2e_ms, "e2e_serial_ms_per_step": e2e_serial_ms,
            "e2e_mode": "pipelined over 3 streams, 2 buffer sets; every step copies all inputs in and all results out",
            "e2e_steps": args.e2e_steps, "e2e_checksum": checksum,
            "other_workloads": others,
        },
        "roofline": {"kernel": "exec_pair_kernel", "bound": "tensor", "achieved": exec_tflops, "peak": peaks["bf16_tflops_sustained"],
                     "unit": "TFLOP/s", "frac": exec_tflops / peaks["bf16_tflops_sustained"],
                     "traffic": traffic, "traffic_how": traffic_how,
                     "peak_kind": f"{peak_kind}, sustained cuBLAS bf16: the kernel is timed inside steps that follow "
                                  f"{step_s:.1f} s of back-to-back steps (power-capped steady state)",
                     "frac_of_burst": exec_tflops / peaks["bf16_tflops"], "frac_of_nominal": exec_tflops / NOMINAL_BF16_TFLOPS,
                     "flop_per_clk_per_sm": flop_per_clk_per_sm,
                     "frac_of_tensor_peak_per_clk": flop_per_clk_per_sm / 8192.0 if flop_per_clk_per_sm else None,
                     "library_gemm_this_gpu": (dict(lib_here, frac=exec_tflops / lib_here["tflops"])
                                               if lib_here and "tflops" in lib_here else lib_here)},
        "roofline_assemble": roofline_assemble,
        "e2e": {"value": e2e_value if args.e2e_steps > 0 else None, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": plan.num_launches * args.steps,
        "clocks": clocks,
    }
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(w, tensors, opts, args.cpu_budget)
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3, help="workload: 1..5 (3 = Llama-7B-shaped layer, the headline)")
    ap.add_argument("--kslice-max", type=int, default=None, help="deepest K-slice (planner option); default 4096")
    ap.add_argument("--scale", type=int, default=1, help="divide the workload's sizes (profiling captures only)")
    ap.add_argument("--e2e-steps", type=int, default=3, help="0 skips the end-to-end leg (profiling captures only)")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-churn", action="store_true")
    ap.add_argument("--no-verify", action="store_true")
    ap.add_argument("--two-step", action="store_true", help="cleave_exec + full cleave_assemble instead of the fused write-out")
    ap.add_argument("--no-finish", action="store_true", help="fused write-out of one-slice GEMMs only; K-split GEMMs go through cleave_assemble")
    ap.add_argument("--gran-m", type=int, default=None, help="row granule of the planner (default 128)")
    ap.add_argument("--keep-blocks", action="store_true", help="store every partial block in the arena (default: the block that "
                    "completes a K-split cell is summed on arrival and not stored)")
    ap.add_argument("--bf16-out", action="store_true", help="C in bf16 (rounded from the fp32 sums) instead of fp32")
    ap.add_argument("--min-warm-s", type=float, default=1.5, help="warm up for at least this long before the timed steps")
    ap.add_argument("--no-other", action="store_true", help="skip the short legs on other modes and workloads")
    ap.add_argument("--no-library-gemm", action="store_true", help="skip the vendor library's GEMM on this GPU (context for the roofline)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the Distributed-Lion optimizer step (arXiv 2404.00438) on B200.

One "step" is one pass of the whole hot path over one batch of synthetic
gradients: the worker-side kernel for all N workers (sign + pack + momentum),
then the server-side kernel (vote / average + parameter update).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5] [--mode majority]
    python bench.py --impl reference ...      # the CPU oracle on a bounded sample

Prints ONE JSON line on rank 0.  Timing is by CUDA events on the launching
stream; every input is seeded and synthetic.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2404_00438_b200 import inputs  # noqa: E402

METRIC = "dlion_step_param_worker_updates_per_s"
UNIT = "G param*worker updates/s"
FALLBACK_HBM_GBS = 6650.0

NCU_TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_traffic.json")


def kernel_hash() -> str:
    """SHA-256 (first 16 hex digits) of the worker-side kernel's sources."""
    h = hashlib.sha256()
    for name in ("worker_step.cu", "dlion_common.cuh"):
        h.update(open(os.path.join(ROOT, "paper_2404_00438_b200", "csrc", name), "rb").read())
    return h.hexdigest()[:16]


def ncu_traffic(kernel: str, variant: str):
    """DRAM bytes per param*worker of `kernel` from its ncu capture (dram__bytes_read.sum +
    dram__bytes_write.sum over the units of the captured launch), as recorded in
    profiles/ncu_traffic.json beside the hash of the kernel's sources at capture time; None
    when there is no record or the sources have changed since."""
    try:
        rec = json.load(open(NCU_TRAFFIC_FILE))[kernel][variant]
    except Exception:
        return None
    return float(rec["dram_bytes_per_param_worker"]) if rec.get("source_sha16") == kernel_hash() else None


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"


class ClockSampler:
    """Read-only NVML polling (every 20 ms, in a thread) of SM clock, power and clock-event
    reasons; the summary covers the samples taken inside [window_start, window_end]."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap"}

    def __init__(self, cuda_index: int):
        self.samples, self.thread, self.stop_flag, self.handle, self.nv = [], None, False, None, None
        self.t0 = self.t1 = None
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(cuda_index).uuid)
            try:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid) if not uuid.startswith("GPU-") else uuid)
            except Exception:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(cuda_index)
            self.nv = pynvml
        except Exception:
            self.nv = None

    def _loop(self):
        nv, h = self.nv, self.handle
        while not self.stop_flag:
            try:
                try:
                    reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(h)
                except Exception:
                    reasons = nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                self.samples.append((time.time(), nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM),
                                     nv.nvmlDeviceGetPowerUsage(h) / 1000.0, int(reasons)))
            except Exception:
                pass
            time.sleep(0.02)

    def start(self):
        if self.nv is None:
            return
        import threading
        self.thread = threading.Thread(target=self._loop, daemon=True)
        self.thread.start()

    def window_start(self):
        self.t0 = time.time()

    def window_end(self):
        self.t1 = time.time()

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.nv is None or self.thread is None:
            out["note"] = "NVML unavailable"
            return out
        self.stop_flag = True
        self.thread.join(timeout=2)
        inside = [s for s in self.samples if self.t0 is not None and self.t0 <= s[0] <= (self.t1 or 1e30)]
        use, scope = (inside, "timed region") if len(inside) >= 3 else (self.samples, "whole measured phase")
        if use:
            bits = 0
            for s in use:
                bits |= s[3]
            out.update(sm_mhz=statistics.median(s[1] for s in use),
                       sm_max_mhz=self.nv.nvmlDeviceGetMaxClockInfo(self.handle, self.nv.NVML_CLOCK_SM),
                       reasons=sorted(name for bit, name in self.REASONS.items() if bits & bit),
                       samples=len(use), power_w_max=max(s[2] for s in use), scope=scope)
        return out


def host_memory_available() -> int:
    """Bytes of host memory this process may still take (the tighter of the machine's and the cgroup's)."""
    try:
        import psutil
        avail = int(psutil.virtual_memory().available)
    except Exception:
        avail = 1 << 62
    for path in ("/sys/fs/cgroup/memory.max", "/sys/fs/cgroup/memory/memory.limit_in_bytes"):
        try:
            v = open(path).read().strip()
            if v.isdigit():
                used = 0
                for up in ("/sys/fs/cgroup/memory.current", "/sys/fs/cgroup/memory/memory.usage_in_bytes"):
                    try:
                        used = int(open(up).read().strip())
                        break
                    except Exception:
                        pass
                avail = min(avail, int(v) - used)
        except Exception:
            pass
    return avail


def bytes_per_param_worker_k1(w, state_bytes: int = 4) -> float:
    """Worker-side kernel: gradient + momentum read + momentum write + 1/8 B of signs."""
    return w.grad_bytes + 2 * state_bytes + 1 / 8


def bytes_per_param_k2(w) -> float:
    """Server-side kernel: N/8 B of votes + parameter read + write."""
    return w.n_workers / 8 + 4 + 4


MODE_NAMES = {inputs.MAJORITY: "majority", inputs.AVERAGE: "average", inputs.MAJORITY_TERNARY: "ternary"}


def mode_of(name: str) -> int:
    return {v: k for k, v in MODE_NAMES.items()}[name]


def oracle_sample_rate(w, mode: int, seconds: float, nthreads: int, n_max: int = 1 << 22):
    """Times the CPU oracle (as it stands) on a bounded sample: the first n_max (2^22)
    arena coordinates of the workload, all N workers, repeated steps."""
    from oracle import dlion_oracle as orc
    orc.build()
    n = min(w.d_pad, n_max)
    segs = []
    for off, cnt in w.segments:
        a, b = off, min(off + cnt, n)
        if a < b:
            segs.append((a, b - a))
    params = sum(c for _, c in segs)
    g = inputs.as_numpy_grads(inputs.fill_grads(w, 0, torch.empty(w.n_workers, n, dtype=inputs.grad_torch_dtype(w)),
                                               0, n))
    m = np.zeros((w.n_workers, n), np.float32)
    x = inputs.fill_x0(w, torch.empty(n), 0, n).numpy()
    packed = np.zeros((w.n_workers, n // 32), np.uint32)

    def one():
        orc.worker_step(segs, n, w.n_workers, g, m, packed, w.beta1, w.beta2, nthreads=nthreads)
        orc.aggregate_apply(segs, n, w.n_workers, mode, packed, x, w.lr, w.weight_decay, nthreads=nthreads)

    one()                                   # warm-up, page faults
    t0 = time.perf_counter()
    one()
    dt = time.perf_counter() - t0
    steps = max(1, min(5000, int(seconds / max(dt, 1e-6))))
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    dt = time.perf_counter() - t0
    rate = params * w.n_workers * steps / dt / 1e9
    sample = (f"first {n} arena coordinates ({params} parameters) of {w.name}, all {w.n_workers} workers, "
              f"{steps} steps, {dt:.1f} s")
    return rate, sample, steps, dt


def run_reference(args):
    """The oracle, as it stands, on the host cores: bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = inputs.workload(args.workload)
    mode = mode_of(args.mode) if args.mode else w.mode
    cores = os.cpu_count() or 1
    for _ in range(max(args.warmup, 0)):
        oracle_sample_rate(w, mode, 0.0, cores)
    rates, secs, sample = [], 0.0, ""
    for _ in range(args.steps):
        r, sample, _, dt = oracle_sample_rate(w, mode, 2.0, cores)
        rates.append(r)
        secs += dt
    value = statistics.mean(rates)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / max(args.steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": args.workload, "n_workers": w.n_workers, "d": w.d,
                   "mode": MODE_NAMES[mode], "grads": w.grad_dtype},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": "each step: " + sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


_JSON_FD = None


def keep_stdout_for_the_json_line():
    """Libraries write banners to stdout (NCCL prints its version when a communicator is
    created): from here on file descriptor 1 is stderr, and emit() alone writes to the
    real stdout, so that stdout carries exactly one JSON line."""
    global _JSON_FD
    if _JSON_FD is None:
        sys.stdout.flush()
        _JSON_FD = os.dup(1)
        os.dup2(2, 1)


def emit(line: dict) -> None:
    data = (json.dumps(line) + "\n").encode()
    if _JSON_FD is None:
        sys.stdout.write(data.decode())
        sys.stdout.flush()
    else:
        os.write(_JSON_FD, data)


def run_ours(args):
    import torch.distributed as dist
    keep_stdout_for_the_json_line()
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    launched_by_torchrun = "MASTER_ADDR" in os.environ and "MASTER_PORT" in os.environ and "RANK" in os.environ
    if world > 1 or launched_by_torchrun:             # under torchrun the rendezvous store is the launcher's, one rank included
        dist.init_process_group("nccl", device_id=dev)
    from paper_2404_00438_b200 import build
    if rank == 0:
        build.build()                                 # in-tree; a no-op when the library is up to date
    if world > 1:
        dist.barrier()
    from paper_2404_00438_b200 import dlion           # loads libdlion.so; raises if it is missing

    w = inputs.workload(args.workload)
    if args.n_workers:
        w.n_workers = args.n_workers
    w.seed += rank                                    # each rank owns a different slab of a larger model
    mode = mode_of(args.mode) if args.mode else w.mode
    N, D, W = w.n_workers, w.d_pad, w.d_pad // 32
    gdt = inputs.grad_torch_dtype(w)
    ctx = dlion.Dlion(w.segments, D, N, w.beta1, w.beta2, w.lr, w.weight_decay, mode,
                      dlion.GRAD_F32 if w.grad_dtype == "f32" else dlion.GRAD_BF16)
    g = torch.empty(N, D, dtype=gdt, device=dev)
    sbytes = 2 if args.state == "bf16" else 4
    if args.state == "bf16":
        ctx.set_momentum_dtype(dlion.STATE_BF16)
    m = torch.zeros(N, D, dtype=torch.bfloat16 if args.state == "bf16" else torch.float32, device=dev)
    x = inputs.fill_x0(w, torch.empty(D, device=dev))
    packed = torch.zeros(N, W, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    wire = torch.zeros(ctx.delta_planes() * W, dtype=torch.int32, device=dev) if args.path == "wire" else None

    def server_side():
        if args.path == "wire":                       # vote into the broadcast message, then apply from it
            ctx.aggregate(packed, wire)
            ctx.apply_delta(wire, x)
        else:
            ctx.aggregate_apply(packed, x)

    def step():
        if args.path == "fused":
            ctx.step_fused(g, m, x, None)
        else:
            ctx.worker_step(-1, g, m, packed)
            server_side()

    for t in range(args.warmup):
        inputs.fill_grads(w, t, g)
        step()
    barrier()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()

    # ---- secondary leg: K steps with fresh seeded gradients generated between steps
    # (generation untimed; each step bracketed by its own events)
    fresh = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
    for t in range(args.steps):
        inputs.fill_grads(w, args.warmup + t, g)
        barrier()
        fresh[t][0].record(stream)
        step()
        fresh[t][1].record(stream)
    barrier()
    fresh_ms = sum(e[0].elapsed_time(e[1]) for e in fresh) / args.steps

    # ---- timed region: exactly K steps back to back inside one barrier/synchronize
    # bracket, on the gradients of the last generated step; events between the
    # kernels give the per-kernel durations
    launches0 = ctx.launch_count()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    barrier()
    sampler.window_start()
    for t in range(args.steps):
        ev[t][0].record(stream)
        if args.path == "fused":
            ctx.step_fused(g, m, x, None)
            ev[t][1].record(stream)
        else:
            ctx.worker_step(-1, g, m, packed)
            ev[t][1].record(stream)
            server_side()
        ev[t][2].record(stream)
    barrier()
    sampler.window_end()
    launches = ctx.launch_count() - launches0
    k1_ms = [e[0].elapsed_time(e[1]) for e in ev]
    k2_ms = [e[1].elapsed_time(e[2]) for e in ev]
    total_ms = ev[0][0].elapsed_time(ev[-1][2])
    clocks = sampler.stop() if rank == 0 else None

    # ---- after the timed region: the server-side kernel under the OTHER aggregation rule
    # (the workload names both), and the Global-Lion comparison step (the full-precision
    # scheme the paper measures Distributed Lion against), K launches each on a scratch
    # copy of x with events around every launch.  Neither enters `value`.
    extra = {}
    if args.path == "two_stage" and not args.no_extra:
        other = inputs.AVERAGE if mode == inputs.MAJORITY else inputs.MAJORITY
        x_scratch = x.clone()
        ctx2 = dlion.Dlion(w.segments, D, N, w.beta1, w.beta2, w.lr, w.weight_decay, other,
                           dlion.GRAD_F32 if w.grad_dtype == "f32" else dlion.GRAD_BF16)

        def timed(fn):
            for _ in range(3):
                fn()
            barrier()
            e = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
            e[0].record(stream)
            for t in range(args.steps):
                fn()
                e[t + 1].record(stream)
            barrier()
            return statistics.mean(e[t].elapsed_time(e[t + 1]) for t in range(args.steps))

        time.sleep(1.0)        # these stages are timed alone: let the power state of the timed region settle
        extra["other_rule_ms"] = timed(lambda: ctx2.aggregate_apply(packed, x_scratch))
        extra["other_rule"] = MODE_NAMES[other]
        if N <= 255:                                   # the one-launch step counts votes in bytes
            extra["fused_ms"] = timed(lambda: ctx.step_fused(g, m, x_scratch, None))
        if args.state == "f32":
            extra["global_lion_ms"] = timed(lambda: ctx2.step_global(g, m, x_scratch))
        ctx2.destroy()
        del x_scratch

    # ---- optional: the same K steps captured once in a CUDA graph and replayed
    # (small workloads are bound by launch latency; the calls never synchronise)
    graph_ms = None
    if args.graph:
        side = torch.cuda.Stream()
        gph = torch.cuda.CUDAGraph()
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            step()
            torch.cuda.synchronize()
            with torch.cuda.graph(gph, stream=side):
                for _ in range(args.steps):
                    step()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        gph.replay()
        barrier()
        g0.record(stream)
        gph.replay()
        g1.record(stream)
        barrier()
        graph_ms = g0.elapsed_time(g1) / args.steps

    t_all = torch.tensor([total_ms], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t_all, op=dist.ReduceOp.MAX)
    total_ms_max = float(t_all.item())
    units = w.d * N * args.steps * world               # param*worker updates, all ranks
    value = units / (total_ms_max * 1e-3) / 1e9

    # ---- worker = GPU exchange (Algorithm 1's send / broadcast as collectives): on by
    # default whenever there is more than one rank
    exch = None
    if args.exchange or world > 1:
        try:
            exch = run_exchange(args, w, mode, dev, world, rank, barrier)
        except Exception as e:                        # reported, never allowed to take the main line down
            exch = {"error": f"{type(e).__name__}: {e}"}
        if args.exchange_fused_send and "error" not in exch:
            try:
                exch["fused_send"] = run_exchange(args, w, mode, dev, world, rank, barrier, fused_send=True)
            except Exception as e:
                exch["fused_send"] = {"error": f"{type(e).__name__}: {e}"}

    # ---- end to end: gradients in pinned host memory, Delta read back
    e2e = None
    if not args.no_e2e:
        need = N * D * w.grad_bytes * int(os.environ.get("LOCAL_WORLD_SIZE", world))
        if host_memory_available() >= 1.25 * need:            # every local rank pins its own gradient copy
            e2e = run_e2e(args, ctx, w, mode, g, m, x, packed, dev, world, barrier)
        else:
            e2e = {"value": None, "unit": UNIT, "skipped": "not enough host memory to pin the gradients of every rank",
                   "h2d_bytes_per_step": N * D * w.grad_bytes, "d2h_bytes_per_step": None}

    if rank == 0:
        peak, peak_src = measured_peak()
        k1 = statistics.mean(k1_ms)
        k2 = statistics.mean(k2_ms)
        if args.path == "fused":
            alg_bytes = w.d * (N * (w.grad_bytes + 2 * sbytes) + 8)
            name = "step_fused_kernel"
        else:
            alg_bytes = w.d * N * bytes_per_param_worker_k1(w, sbytes)
            name = "worker_step_kernel"
        achieved = alg_bytes / (k1 * 1e-3) / 1e9
        traffic = ncu_traffic(name, f"grads_{w.grad_dtype}_momentum_{args.state}")
        roofline = {"bound": "hbm", "kernel": name, "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak, "peak_source": peak_src, "frac_of_8tbs_nominal": achieved / 8000.0,
                    "algorithmic_bytes_per_launch": alg_bytes, "ms_per_launch": k1,
                    "traffic": None if traffic is None else traffic * w.d * N,
                    # duration x median SM clock of the timed region: compares runs taken at different
                    # power-cap clocks (a DRAM-bound kernel's product rises with the clock, an issue-bound one's does not)
                    "ms_per_launch_x_sm_ghz": (k1 * clocks["sm_mhz"] / 1000.0 if clocks and clocks.get("sm_mhz") else None)}
        stages = None
        if args.path != "fused":
            b2 = w.d * bytes_per_param_k2(w)
            if args.path == "wire":                   # votes in, K planes out; K planes in, x in and out
                b2 += 2 * w.d * ctx.delta_planes() / 8
            rule = MODE_NAMES[mode]
            key = ("aggregate_kernel+apply_delta_kernel<%s>" if args.path == "wire" else "aggregate_apply_kernel<%s>") % rule
            stages = {key: {"achieved": b2 / (k2 * 1e-3) / 1e9, "unit": "GB/s",
                            "frac": b2 / (k2 * 1e-3) / 1e9 / peak,
                            "frac_of_8tbs_nominal": b2 / (k2 * 1e-3) / 1e9 / 8000.0, "ms_per_launch": k2,
                            "algorithmic_bytes_per_launch": b2}}
        comparison = None
        if extra:
            b2 = w.d * bytes_per_param_k2(w)
            ms2 = extra["other_rule_ms"]
            stages["aggregate_apply_kernel<%s>" % extra["other_rule"]] = {
                "achieved": b2 / (ms2 * 1e-3) / 1e9, "unit": "GB/s", "frac": b2 / (ms2 * 1e-3) / 1e9 / peak,
                "frac_of_8tbs_nominal": b2 / (ms2 * 1e-3) / 1e9 / 8000.0, "ms_per_launch": ms2,
                "algorithmic_bytes_per_launch": b2,
                "note": "timed after the timed region on a scratch copy of x; not part of `value`"}
            if "fused_ms" in extra:
                bf = w.d * (N * (w.grad_bytes + 2 * sbytes) + 8)
                msf = extra["fused_ms"]
                stages["step_fused_kernel<%s>" % MODE_NAMES[mode]] = {
                    "achieved": bf / (msf * 1e-3) / 1e9, "unit": "GB/s", "frac": bf / (msf * 1e-3) / 1e9 / peak,
                    "frac_of_8tbs_nominal": bf / (msf * 1e-3) / 1e9 / 8000.0, "ms_per_launch": msf,
                    "algorithmic_bytes_per_launch": bf,
                    "note": "the whole step in one launch (dlion_step_fused), timed after the timed region; "
                            "not part of `value`"}
            if "global_lion_ms" in extra:
                msg = extra["global_lion_ms"]
                bg = w.d * (N * (w.grad_bytes + 8) + 8)
                comparison = {"global_lion": {
                    "call": "dlion_step_global (fp32 mean of the workers' blends, one sign; one launch)",
                    "ms_per_step": msg, "value": w.d * N / (msg * 1e-3) / 1e9, "unit": UNIT,
                    "achieved_gbs": bg / (msg * 1e-3) / 1e9, "algorithmic_bytes_per_launch": bg,
                    "wire_bytes_each_way_per_worker": ctx.wire_bytes(2),
                    "distributed_lion_ms_per_step": total_ms_max / args.steps,
                    "note": "on one GPU both schemes read the same gradients and momenta, so their step "
                            "times are close; the schemes differ in what crosses the network "
                            "(wire_bytes_per_step)"}}
        cpu = None
        if not args.no_cpu_baseline and world == 1:
            cores = os.cpu_count() or 1
            rate, sample, _, _ = oracle_sample_rate(w, mode, args.cpu_seconds, cores)
            rate1, sample1, _, _ = oracle_sample_rate(w, mode, args.cpu_seconds / 3, 1, n_max=1 << 20)
            cpu = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                   "single_thread": {"value": rate1, "unit": UNIT, "cores": 1, "sample": sample1}}
        up, down = ctx.wire_bytes(0), ctx.wire_bytes(1)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms_max / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "n_workers": N, "d": w.d, "grads": w.grad_dtype,
                       "mode": MODE_NAMES[mode], "path": args.path,
                       "momentum": args.state,
                       "l2": "inputs larger than L2 (no flush needed)" if N * D * (w.grad_bytes + 4) > 4 * 126e6
                             else "working set comparable to L2: latency-bound case",
                       "timed_region": "K steps back to back in one bracket, on the last generated gradients",
                       "per_rank": "each rank steps its own full-size coordinate slab; no collective"},
            "ms_per_step_fresh_grads": fresh_ms, "ms_per_step_graph_replay": graph_ms,
            "roofline": roofline, "roofline_stages": stages, "comparison": comparison,
            "exchange": exch, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": launches, "clocks": clocks,
            "wire_bytes_per_step": {"up_all_workers": up, "down_per_worker": down,
                                    # Averaging: the paper's own estimate, log2(N) bits per parameter (the exact
                                    # count of N+1 values is ceil(log2(N+1)), which `down_per_worker` uses)
                                    "down_per_worker_paper_log2_n": (w.d * np.log2(N) / 8 if mode == inputs.AVERAGE and N > 1
                                                                     else None),
                                    "fp32_gradients_each_way_per_worker": ctx.wire_bytes(2),
                                    "fp32_ring_allreduce_per_gpu": int(2 * (N - 1) / N * 4 * w.d)},
        }
        emit(line)
    ctx.destroy()
    if dist.is_initialized():
        dist.destroy_process_group()


def make_packed(ctx, dlion, w, dev, step: int = 0, rounds: int = 1):
    """The wire buffer [N][d_pad/32] of workload w without holding N gradient and
    momentum arenas: the workers are stepped one at a time through
    dlion_worker_step(i) on one worker-sized gradient buffer (each worker's own
    seeded gradients; `rounds` steps from m = 0)."""
    N, D, W = w.n_workers, w.d_pad, w.d_pad // 32
    gdt = inputs.grad_torch_dtype(w)
    packed = torch.zeros(N, W, dtype=torch.int32, device=dev)
    g1 = torch.empty(1, D, dtype=gdt, device=dev)
    m1 = torch.empty(D, dtype=torch.float32, device=dev)
    for i in range(N):
        m1.zero_()
        for t in range(rounds):
            inputs.fill_grads(w, step + t, g1, workers=[i])
            ctx.worker_step(i, g1[0], m1, packed[i])
    torch.cuda.synchronize()
    return packed


def run_server_stage(args):
    """Times the server-side kernel alone (dlion_aggregate_apply) on the wire buffer of
    the workload: N*d/8 B of votes plus x are all the device memory it needs, so even
    the large-N cases are small enough to profile."""
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    from paper_2404_00438_b200 import build
    build.build()
    from paper_2404_00438_b200 import dlion
    w = inputs.workload(args.workload)
    if args.n_workers:
        w.n_workers = args.n_workers
    mode = mode_of(args.mode) if args.mode else w.mode
    N, D = w.n_workers, w.d_pad
    ctx = dlion.Dlion(w.segments, D, N, w.beta1, w.beta2, w.lr, w.weight_decay, mode,
                      dlion.GRAD_F32 if w.grad_dtype == "f32" else dlion.GRAD_BF16)
    packed = make_packed(ctx, dlion, w, dev)
    x = inputs.fill_x0(w, torch.empty(D, device=dev))
    stream = torch.cuda.current_stream()
    for _ in range(max(args.warmup, 3)):
        ctx.aggregate_apply(packed, x)
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    sampler.window_start()
    ev[0].record(stream)
    for t in range(args.steps):
        ctx.aggregate_apply(packed, x)
        ev[t + 1].record(stream)
    torch.cuda.synchronize()
    sampler.window_end()
    clocks = sampler.stop()
    ms = [ev[t].elapsed_time(ev[t + 1]) for t in range(args.steps)]
    k2 = statistics.mean(ms)
    peak, peak_src = measured_peak()
    b2 = w.d * bytes_per_param_k2(w)
    achieved = b2 / (k2 * 1e-3) / 1e9
    line = {
        "metric": "dlion_server_stage_params_per_s", "value": w.d / (k2 * 1e-3) / 1e9, "unit": "G param/s",
        "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": k2,
        "ms_min": min(ms), "higher_is_better": True, "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "n_workers": N, "d": w.d, "stage": "server",
                   "mode": MODE_NAMES[mode],
                   "l2": "votes + x = %.0f MB, larger than L2" % ((N * D / 8 + 4 * D) / 1e6)},
        "roofline": {"bound": "hbm", "kernel": "aggregate_apply_kernel", "achieved": achieved, "peak": 8000.0,
                     "unit": "GB/s", "frac": achieved / 8000.0, "peak_source": "nominal 8 TB/s",
                     "vs_measured_copy": achieved / peak, "measured_copy_gbs": peak, "measured_copy_source": peak_src,
                     "algorithmic_bytes_per_launch": b2, "ms_per_launch": k2, "traffic": None},
        "gpu_launches": args.steps, "clocks": clocks,
    }
    print(json.dumps(line), flush=True)
    ctx.destroy()


def run_exchange(args, w, mode, dev, world, rank, barrier, fused_send=False):
    """The paper's own deployment, one worker per GPU: worker-side kernel on this rank's
    gradients, all-to-all of the 1-bit shards, vote on this rank's coordinate slice,
    all-gather of the broadcast message, apply (exchange.DistributedLion; the collectives
    are NCCL's).  Times K steps with CUDA events, max over ranks, and reports what crossed
    the links beside an fp32 all-reduce of the same gradients."""
    import torch.distributed as dist
    from paper_2404_00438_b200 import exchange
    own_group = not dist.is_initialized()
    if own_group:                                     # one rank: a self-exchange through the same collectives
        import socket
        with socket.socket() as s:
            s.bind(("127.0.0.1", 0))
            port = s.getsockname()[1]
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1, device_id=dev)
    try:
        opt = exchange.DistributedLion(w.segments, w.d_pad, mode, beta1=w.beta1, beta2=w.beta2, lr=w.lr,
                                       weight_decay=w.weight_decay, gdtype=0 if w.grad_dtype == "f32" else 1,
                                       device=dev, fused_send=fused_send)
        Dx = opt.d_pad_x
        g = torch.zeros(Dx, dtype=inputs.grad_torch_dtype(w), device=dev)
        inputs.fill_grads(w, 0, g[:w.d_pad].unsqueeze(0), workers=[rank % max(w.n_workers, 1)])
        m = torch.zeros(Dx, device=dev)
        x = torch.zeros(Dx, device=dev)
        inputs.fill_x0(w, x[:w.d_pad])
        stream = torch.cuda.current_stream()
        for _ in range(3):
            opt.step(g, m, x)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            opt.step(g, m, x)
        e1.record(stream)
        barrier()
        t = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item()) / args.steps
        phases = None
        if not fused_send:
            # the same step once more, phase by phase (events on the launching stream; the
            # collectives are enqueued on it by the backend): where a multi-GPU step spends its time
            names = ("worker_step", "all_to_all", "vote_on_slice", "all_gather", "apply")
            acc = [0.0] * len(names)
            for _ in range(args.steps):
                ev = [torch.cuda.Event(enable_timing=True) for _ in range(len(names) + 1)]
                ev[0].record(stream)
                opt.kernels.worker_step(g, m, opt.packed)
                ev[1].record(stream)
                opt._all_to_all()
                ev[2].record(stream)
                opt.kernels.aggregate(opt.recv, opt.wire_slice)
                ev[3].record(stream)
                opt._all_gather()
                ev[4].record(stream)
                opt.kernels.apply_delta_sliced(opt.gathered, opt.slice_words, x)
                ev[5].record(stream)
                torch.cuda.synchronize()
                for k in range(len(names)):
                    acc[k] += ev[k].elapsed_time(ev[k + 1])
            pt = torch.tensor(acc, dtype=torch.float64, device=dev) / args.steps
            if world > 1:
                dist.all_reduce(pt, op=dist.ReduceOp.MAX)
            phases = {nm: float(v) for nm, v in zip(names, pt.tolist())}
        sent, received = opt.wire_bytes_per_step()
        return {"ms_per_step": ms, "phases_ms_max_over_ranks": phases, "value": w.d * world / (ms * 1e-3) / 1e9, "unit": UNIT, "workers": world,
                "steps": args.steps, "gpu_launches_per_step": 3,
                "collectives": ("sign words stored by the worker-side kernel into the ranks' receive buffers "
                                "(symmetric memory) + barrier + all_gather_into_tensor (NCCL)") if fused_send
                else "all_to_all_single + all_gather_into_tensor (NCCL)",
                "alltoall_bytes_sent_per_rank": sent, "allgather_bytes_received_per_rank": received,
                "fp32_ring_allreduce_bytes_per_rank": int(2 * (world - 1) / world * 4 * w.d),
                "note": "one worker per GPU, d = the workload's parameter count on every rank"}
    finally:
        if own_group:
            dist.destroy_process_group()


def run_e2e(args, ctx, w, mode, g, m, x, packed, dev, world, barrier):
    """dlion_step_host: per step, N*D gradient elements host->device, Delta device->host."""
    import torch.distributed as dist
    N, D, W = w.n_workers, w.d_pad, w.d_pad // 32
    host_g = torch.empty(N, D, dtype=g.dtype, pin_memory=True)
    host_g.copy_(g)
    staging = torch.empty(2, D, dtype=g.dtype, device=dev)
    wire_bytes = ctx.delta_planes() * W * 4           # the broadcast message: 1 or K planes of d bits
    wire = torch.zeros(wire_bytes, dtype=torch.uint8, device=dev)
    host_wire = torch.zeros(wire_bytes, dtype=torch.uint8, pin_memory=True)
    stream = torch.cuda.current_stream()
    for _ in range(args.e2e_warmup):
        ctx.step_host(host_g, m, x, packed, staging, wire, host_wire)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.e2e_steps):
        ctx.step_host(host_g, m, x, packed, staging, wire, host_wire)
    e1.record(stream)
    barrier()
    t = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms = float(t.item()) / args.e2e_steps
    del host_g, staging
    return {"value": w.d * N * world / (ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms,
            "steps": args.e2e_steps, "h2d_bytes_per_step": N * D * w.grad_bytes,
            "d2h_bytes_per_step": wire_bytes, "call": "dlion_step_host (pinned host gradients in, Delta out)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5", choices=["c1", "c2", "c3", "c4", "c5"])
    ap.add_argument("--n-workers", type=int, default=0, help="override N (the c4 sweep)")
    ap.add_argument("--mode", default=None, choices=["majority", "average", "ternary"],
                    help="ternary: Majority Vote with Delta = 0 on an even-N tie")
    ap.add_argument("--path", default="two_stage", choices=["two_stage", "fused", "wire"],
                    help="wire: server side as two launches with the broadcast message in between")
    ap.add_argument("--state", default="f32", choices=["f32", "bf16"], help="momentum storage")
    ap.add_argument("--stage", default="step", choices=["step", "server"],
                    help="server: time the server-side kernel alone on the workload's wire buffer (1 GPU)")
    ap.add_argument("--graph", action="store_true", help="also time the K steps replayed from one CUDA graph")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--exchange", action="store_true",
                    help="also time the worker = GPU exchange step (always on with more than one rank)")
    ap.add_argument("--exchange-fused-send", action="store_true",
                    help="with the exchange leg: time it once more with the all-to-all fused into the worker-side "
                         "kernel (peer stores into symmetric memory); only on request")
    ap.add_argument("--no-extra", action="store_true",
                    help="skip the stages timed after the timed region (other aggregation rule, Global Lion)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--e2e-warmup", type=int, default=1)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3                               # timing hygiene: at least three warm-up steps
    if args.impl == "reference":
        run_reference(args)
    elif args.stage == "server":
        run_server_stage(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

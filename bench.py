#!/usr/bin/env python
"""Benchmark of the fused grouped aggregate + update.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME]
                    [--impl ours|reference] [--no-extra] [--architecture ps|all_reduce]

A step is one round of the whole path on one batch of synthetic gradients:
the mode decision of the round is encoded into a CSR schedule (host, in the
library) and the fused update kernel is launched once.  Prints ONE JSON line.

  value      achieved GB/s = algorithmic bytes / device time, inputs resident
             in HBM; bytes per round = n * (sum_k |G_k| * sizeof(g) + 16).
             K steps are timed between two CUDA events; that region is repeated
             until at least half a second of device time has been measured and
             the value is taken from the median repeat (min and max beside it).
  e2e        the same metric through the host-buffer entry point: parameters,
             momentum and gradients start in pinned host memory, results end
             there, every copy inside the timed region; its own roofline is a
             plain pinned copy of the same bytes up and down, timed in the same run
  roofline   the update kernel against the measured HBM copy bandwidth
  cpu_baseline  the CPU oracle timed on this machine's cores (reported only)
  other_workloads  the remaining workloads, the extended entry points (parameter
             snapshots, tree order, tensor list with snapshots) and the two
             kernels of the all-reduce round, each with its own roofline block

With N > 1 (under torchrun) every rank runs the same workload on its own GPU
(the path is elementwise: shards need no exchange), the time is the maximum
over ranks and the value the sum of all ranks' bytes over that time.
--architecture all_reduce runs the all-reduce architecture's round instead (one
rank = one worker: children -> parent, local aggregate, ring exchange, update).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "grouped aggregate+update HBM GB/s"
UNIT = "GB/s"
HEADLINE = "cfg4_gpt2_medium"          # the largest single-GPU workload: 17.03 GB per round, 292 tensors
FALLBACK_HBM_GBS = 6650.0
MIN_TIMED_SECONDS = 0.5
MAX_REPEATS = 50


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per ELEMENT of a
# launch of the headline kernel, from the ncu capture summarised under profiles/
# (taken on a reduced tensor list: traffic grows in proportion to the elements
# processed), keyed by workload, with the SHA-256 of the kernel sources the
# capture was taken on: once the sources differ the figure is stale and
# `traffic` is reported as null.
NCU_TRAFFIC_PER_ELEMENT = {
    "cfg4_gpt2_medium": (1644.47e6 / 34_631_680, "03e0fa45a87f327661444bc4c1aff616ef7e6deddd70b78ae0dd5d517a48867b"),
    "cfg1_resnet50": (787.86e6 / 25_557_032, "03e0fa45a87f327661444bc4c1aff616ef7e6deddd70b78ae0dd5d517a48867b"),
}


def kernel_source_hash() -> str:
    import hashlib
    h = hashlib.sha256()
    for name in ("kernels.cuh", "api.cu"):
        with open(os.path.join(ROOT, "paper_2512_09685_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def ncu_traffic(workload_name: str, n: int):
    entry = NCU_TRAFFIC_PER_ELEMENT.get(workload_name)
    if entry is None:
        return None
    try:
        return entry[0] * n if kernel_source_hash() == entry[1] else None
    except OSError:
        return None


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ---------------------------------------------------------------------------
# clocks during the timed region
# ---------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the
    timed region runs."""

    REASONS = (("sw_power_cap", 0x4), ("hw_slowdown", 0x8), ("sw_thermal_slowdown", 0x20),
               ("hw_thermal_slowdown", 0x40), ("hw_power_brake", 0x80))

    def __init__(self, index: int, period: float = 0.01):
        self.index, self.period = index, period
        self.sm, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = index
            if visible:
                ids = [x for x in visible.split(",") if x.strip()]
                if index < len(ids) and ids[index].strip().isdigit():
                    phys = int(ids[index])
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def sample(self):
        """One reading, now (also called from the timing loop right after the last
        launch is queued, so that even a very short region has a sample taken
        while the GPU is busy)."""
        nv = self.nv
        if nv is None:
            return
        try:
            self.sm.append(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM))
            mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
            for name, bit in self.REASONS:
                if mask & bit:
                    self.reasons.add(name)
        except Exception:
            pass

    def _loop(self):
        while not self._stop.is_set():
            self.sample()
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.sm:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(self.sm), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.sm)}


# ---------------------------------------------------------------------------
# device side
# ---------------------------------------------------------------------------
class DeviceWorkload:
    """One workload resident on the current device, ready to step.

    mode: "plain"      star_group_update / star_group_update_multi
          "snap_f32"   per-group rates + one fp32 parameter snapshot per group
          "snap_bf16"  the same with bf16 snapshots
          "tree"       tree summation order, no snapshots
    (flat workloads: star_group_update_ex; tensor lists: star_group_update_multi_ex
    with one snapshot set per group)."""

    def __init__(self, w, grad_sets: int, mode: str = "plain", max_groups: int = 8):
        import torch
        from paper_2512_09685_b200 import binding as B
        from paper_2512_09685_b200 import workloads as WL
        self.torch, self.B, self.w, self.mode = torch, B, w, mode
        dev = "cuda"
        self.params = WL.make_params(w, dev)
        self.momentum = WL.make_momentum(w, dev)
        dt = w.torch_grad_dtype()
        self.grad_sets = []
        for s in range(grad_sets):
            one = []
            for wk in range(w.W):
                bufs = [torch.empty(size, dtype=dt, device=dev) for size in w.sizes]
                WL.fill_grads(w, s, wk, bufs)
                one.append(bufs)
            self.grad_sets.append(one)
        self.snapshot_bytes = {"snap_f32": 4, "snap_bf16": 2}.get(mode, 0)
        self.snapshots = []
        if self.snapshot_bytes:
            sdt = torch.float32 if mode == "snap_f32" else torch.bfloat16
            self.snapshots = [[torch.empty(size, dtype=sdt, device=dev) for size in w.sizes]
                              for _ in range(max_groups)]
        self.plans = None
        if w.multi_tensor:
            self.workspaces, self.plans = [], []
            for one in self.grad_sets:
                ws = torch.empty(B.star_multi_workspace_bytes_ex(w.sizes, w.W, len(self.snapshots)),
                                 dtype=torch.uint8, device=dev)
                self.workspaces.append(ws)
                if mode == "plain":
                    self.plans.append(B.star_multi_prepare(self.params, self.momentum, one, ws))
                else:
                    self.plans.append(B.star_multi_prepare_ex(self.params, self.momentum, one, self.snapshots, ws))
        else:
            self.flat_grads = [[bufs[0] for bufs in one] for one in self.grad_sets]
            # pointers marshalled once per gradient set: the per-round host work is the schedule
            self.flat_rounds = [B.FlatRoundBuffers(self.params[0], self.momentum[0], g) for g in self.flat_grads]
        self.step_index = 0
        torch.cuda.synchronize()

    def step(self) -> int:
        """One round: encode the decision, launch the fused update.  Returns the
        algorithmic bytes of the round on this rank."""
        w, B = self.w, self.B
        off, mem = B.encode(w.decision(self.step_index))
        K = len(off) - 1
        which = self.step_index % len(self.grad_sets)
        order = B.STAR_SUM_TREE if self.mode == "tree" else B.STAR_SUM_LINEAR
        n_snap = K if self.snapshot_bytes else 0
        if self.mode == "plain":
            if self.plans is not None:
                B.star_group_update_multi(self.plans[which], off, mem, w.lr, w.mu, w.wd)
            else:
                self.flat_rounds[which].star_group_update(off, mem, w.lr, w.mu, w.wd)
        elif self.plans is not None:
            B.star_group_update_multi_ex(self.plans[which], off, mem, [w.lr] * K, w.mu, w.wd,
                                         list(range(K)) if n_snap else None, order)
        else:
            snaps = [self.snapshots[k][0] for k in range(K)] if n_snap else None
            B.star_group_update_ex(self.params[0], self.momentum[0], self.flat_grads[which], off, mem,
                                   [w.lr] * K, w.mu, w.wd, snapshots=snaps, sum_order=order)
        self.step_index += 1
        return w.n * (off[-1] * w.grad_bytes + 16 + n_snap * self.snapshot_bytes)

    def kernel_name(self) -> str:
        if self.mode == "plain":
            return "star_update_multi_kernel" if self.w.multi_tensor else "star_update_flat_kernel"
        return "star_update_multi_ex_kernel" if self.w.multi_tensor else "star_update_flat_snapshot_kernel"


def max_over_ranks(seconds: float, dist, device) -> float:
    """The slowest rank's time: what a multi-rank measurement reports."""
    if dist is None:
        return seconds
    import torch
    t = torch.tensor([seconds], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def time_steps(step, steps: int, warmup: int, dist, sampler=None, launch_count=None, probe: bool = True):
    """Times `steps` calls of step() between two CUDA events on the current
    stream, after `warmup` untimed calls, with a barrier and a synchronize on
    both sides; repeats that region until MIN_TIMED_SECONDS of device time have
    been measured (at least 3, at most MAX_REPEATS regions; every rank runs the
    same number: the decision uses the max-over-ranks times).  step() returns the
    algorithmic bytes it moved.  Returns a dict: the median region (seconds =
    max over ranks, bytes on this rank, launches), the GB/s of every region, and
    per-launch durations from a separate probe pass."""
    import torch
    for _ in range(warmup):
        step()
    regions = []
    if sampler is not None:
        sampler.__enter__()
    while True:
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        begin, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches0 = launch_count() if launch_count else 0
        nbytes = 0
        begin.record()
        for _ in range(steps):
            nbytes += step()
        end.record()
        if sampler is not None:
            sampler.sample()
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        seconds = max_over_ranks(begin.elapsed_time(end) / 1e3, dist, "cuda")
        regions.append({"seconds": seconds, "bytes": nbytes,
                        "launches": (launch_count() - launches0) if launch_count else steps})
        total = sum(r["seconds"] for r in regions)
        if len(regions) >= MAX_REPEATS or (len(regions) >= 3 and total >= MIN_TIMED_SECONDS):
            break
    if sampler is not None:
        sampler.__exit__(None, None, None)
    rates = sorted(r["bytes"] / r["seconds"] / 1e9 for r in regions)
    ordered = sorted(regions, key=lambda r: r["bytes"] / r["seconds"])
    median = ordered[(len(ordered) - 1) // 2]           # an actual region (the lower median)
    per_launch = []
    if probe:
        # Per-launch durations from a short extra pass with an event after every
        # launch (the events themselves cost time, so they stay out of the timed
        # regions above; the pass only shows the spread).
        count = min(steps, 200)
        events = [torch.cuda.Event(enable_timing=True) for _ in range(count + 1)]
        events[0].record()
        for i in range(count):
            step()
            events[i + 1].record()
        torch.cuda.synchronize()
        per_launch = [events[i].elapsed_time(events[i + 1]) for i in range(count)]
    return {"seconds": median["seconds"], "bytes": median["bytes"], "launches": median["launches"],
            "gbs_regions": rates, "repeats": len(regions), "timed_seconds": total, "per_launch_ms": per_launch}


def time_device(dw: DeviceWorkload, steps: int, warmup: int, dist, sampler=None, probe: bool = True):
    return time_steps(dw.step, steps, warmup, dist, sampler, dw.B.star_launch_count, probe)


def roofline_block(t, steps: int, peak: float, peak_kind: str, kernel: str, traffic=None):
    """The kernel against the HBM roofline: algorithmic bytes per launch over the
    mean launch duration of the median timed region (one launch per step and
    nothing else on the stream, so that is region time / launches)."""
    kernel_ms = t["seconds"] / t["launches"] * 1e3
    achieved = (t["bytes"] / t["launches"]) / (kernel_ms / 1e3) / 1e9
    block = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
             "traffic": traffic, "peak_kind": "of " + peak_kind, "kernel": kernel, "kernel_ms_mean": kernel_ms,
             "bytes_per_launch": t["bytes"] // t["launches"],
             "regions": {"count": t["repeats"], "gbs_min": t["gbs_regions"][0], "gbs_max": t["gbs_regions"][-1],
                         "gbs_median": t["bytes"] / t["seconds"] / 1e9, "timed_seconds": t["timed_seconds"]}}
    if t["per_launch_ms"]:
        block["per_launch_probe_ms"] = {"median": statistics.median(t["per_launch_ms"]),
                                        "min": min(t["per_launch_ms"]), "launches": len(t["per_launch_ms"])}
    return block


def time_graph_replay(dw: DeviceWorkload, rounds: int, replays: int) -> float:
    """ms per round when `rounds` rounds are captured once in a CUDA graph and
    replayed `replays` times."""
    torch = dw.torch
    dw.step()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for _ in range(rounds):
                dw.step()
    graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(replays):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / (rounds * replays)


def time_e2e(w, steps: int, warmup: int, dist):
    """The same rounds through the host-buffer entry point: p, v and gradients
    start in pinned host memory and p, v end there; every copy is inside the
    timed region and each step ends with the stream synchronized (the result
    is read on the host).  Also times, in the same run and on the same pinned
    tensors, nothing but the copies such a step needs (every scheduled
    gradient, p and v up on one stream; p and v down on another, concurrently):
    the roofline of this leg.  Returns a dict."""
    import torch
    from paper_2512_09685_b200 import binding as B
    from paper_2512_09685_b200 import workloads as WL
    n = w.n
    flat = WL.scaled(w, n)                      # tensor lists are streamed as one flat buffer
    p = WL.make_params(flat, "cpu")[0].pin_memory()
    v = WL.make_momentum(flat, "cpu")[0].pin_memory()
    one = torch.empty(n, dtype=w.torch_grad_dtype())
    WL.fill_grads(flat, 0, 0, [one])
    grads = []
    for wk in range(w.W):                       # values do not affect the timing: one draw, W pinned copies
        g = torch.empty(n, dtype=w.torch_grad_dtype()).pin_memory()
        g.copy_(one)
        grads.append(g)
    del one
    chunk = 4 * 1024 * 1024
    ws = torch.empty(B.star_host_workspace_bytes(w.W, w.torch_grad_dtype(), chunk), dtype=torch.uint8,
                     device="cuda")
    stream = torch.cuda.current_stream()

    def step(i):
        off, mem = B.encode(w.decision(i))
        B.star_group_update_host(p, v, grads, off, mem, w.lr, w.mu, w.wd, ws)
        stream.synchronize()
        return off[-1]

    for i in range(warmup):
        step(i)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = B.star_launch_count()
    scheduled = 0
    e0.record()
    for i in range(steps):
        scheduled += step(warmup + i)
    e1.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    seconds = max_over_ranks(e0.elapsed_time(e1) / 1e3, dist, "cuda")
    launches = B.star_launch_count() - launches0
    nbytes = n * (scheduled * w.grad_bytes + 16 * steps)
    h2d = n * (scheduled * w.grad_bytes + 8 * steps) // steps
    d2h = n * 8

    # Copy-only roofline: the bytes of one step, up and down at the same time.
    d_state = torch.empty(n, dtype=torch.float32, device="cuda")
    d_back = torch.empty(n, dtype=torch.float32, device="cuda")
    d_grad = torch.empty(n, dtype=w.torch_grad_dtype(), device="cuda")
    up, down = torch.cuda.Stream(), torch.cuda.Stream()
    per_step_workers = scheduled // steps

    def copies():
        with torch.cuda.stream(up):
            d_state.copy_(p, non_blocking=True)
            d_state.copy_(v, non_blocking=True)
            for g in grads[:per_step_workers]:
                d_grad.copy_(g, non_blocking=True)
        with torch.cuda.stream(down):
            p.copy_(d_back, non_blocking=True)
            v.copy_(d_back, non_blocking=True)

    d_back.zero_()
    torch.cuda.synchronize()
    copies()
    torch.cuda.synchronize()
    reps = max(2, min(steps, 5))
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    cur = torch.cuda.current_stream()
    c0.record()
    up.wait_stream(cur)
    down.wait_stream(cur)
    for _ in range(reps):
        copies()
    cur.wait_stream(up)
    cur.wait_stream(down)
    c1.record()
    torch.cuda.synchronize()
    copy_seconds = max_over_ranks(c0.elapsed_time(c1) / 1e3 / reps, dist, "cuda")
    step_bytes = nbytes / steps
    return {"seconds": seconds, "bytes": nbytes, "h2d": h2d, "d2h": d2h, "launches": launches,
            "copy_only_seconds_per_step": copy_seconds, "peak": step_bytes / copy_seconds / 1e9,
            "h2d_gbs_copy_only": h2d / copy_seconds / 1e9}


# ---------------------------------------------------------------------------
# CPU oracle timing
# ---------------------------------------------------------------------------
class OracleRunner:
    """The CPU oracle, as it stands, on the first `n_sample` elements of a
    workload (inputs generated once on the CPU), `threads` Python threads over
    disjoint index ranges (the C call releases the GIL)."""

    def __init__(self, w, n_sample: int, threads: int):
        import numpy as np
        import torch
        from oracle import schedule as S
        from oracle import star_oracle as O
        from paper_2512_09685_b200 import workloads as WL
        self.np, self.S, self.O, self.w = np, S, O, w
        self.n, self.threads = n_sample, threads
        ws = WL.scaled(w, n_sample)
        self.p = WL.make_params(ws, "cpu")[0].numpy()
        self.v = WL.make_momentum(ws, "cpu")[0].numpy()
        self.grads = []
        for g in WL.make_grads(ws, 0, "cpu"):
            g = g[0]
            self.grads.append(g.view(torch.int16).numpy().view(np.uint16) if g.dtype == torch.bfloat16
                              else g.numpy())
        self.rounds_done = 0
        O.build()

    def encode(self, step):
        d = self.w.decision(step)
        if d.kind == "labels":
            return self.S.from_labels(d.labels)
        return self.S.static_x(d.arrival_order, d.W, d.x, d.sort_members)

    def round(self, n=None) -> int:
        """One round on the first n (default: all sampled) elements; returns the
        number of scheduled workers."""
        n = self.n if n is None else n
        off, mem = self.encode(self.rounds_done)
        self.rounds_done += 1
        w, lr = self.w, self.np.float32(self.w.lr)
        bounds = [n * i // self.threads for i in range(self.threads + 1)]

        def work(i):
            a, b = bounds[i], bounds[i + 1]
            self.O.group_update_f32(self.p[a:b], self.v[a:b], [g[a:b] for g in self.grads], off, mem,
                                    lr, w.mu, w.wd)
        if self.threads == 1:
            work(0)
        else:
            ts = [threading.Thread(target=work, args=(i,)) for i in range(self.threads)]
            for t in ts:
                t.start()
            for t in ts:
                t.join()
        return off[-1]


def time_oracle(w, n_sample: int, min_seconds: float, threads: int):
    """Rounds of the oracle for at least `min_seconds`.  Returns (GB/s,
    elements/s, rounds run, seconds)."""
    runner = OracleRunner(w, n_sample, threads)
    runner.round()                                 # warm-up
    rounds, scheduled = 0, 0
    t0 = time.perf_counter()
    while True:
        scheduled += runner.round()
        rounds += 1
        dt = time.perf_counter() - t0
        if dt >= min_seconds:
            break
    nbytes = n_sample * (scheduled * w.grad_bytes + 16 * rounds)
    return nbytes / dt / 1e9, n_sample * rounds / dt, rounds, dt


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


# ---------------------------------------------------------------------------
REFERENCE_BUDGET_SECONDS = 100.0


def config_for(w, world: int):
    """The workload as both arms describe it (every workload schedules all W workers)."""
    full = w.n * (w.W * w.grad_bytes + 16)
    return {"workload": w.name, "stands_for": w.model, "n": w.n, "W": w.W, "grad_dtype": w.grad_dtype,
            "tensors": len(w.sizes), "bytes_per_step": full,
            "l2": "inputs larger than L2: %.0f MB per step" % (full / 1e6),
            "parallelism": "replicas x%d" % world}


def run_reference(args, rank: int, world: int):
    """--impl reference: the CPU oracle on the host cores.  A step is one round on
    a bounded sample of the workload: the first n_sample elements, n_sample
    chosen from a calibration round so that warm-up + steps fit the budget."""
    if rank != 0:
        return
    from paper_2512_09685_b200 import workloads as WL
    w = WL.BY_NAME[args.workload]
    cores = host_cores()
    runner = OracleRunner(w, min(w.n, 16_000_000), cores)
    probe = min(runner.n, 2_000_000)
    runner.round(probe)
    t0 = time.perf_counter()
    runner.round(probe)
    rate = probe / (time.perf_counter() - t0)                        # elements / s
    total_rounds = max(args.steps, 1) + max(args.warmup, 0)
    n_sample = int(min(runner.n, max(65_536, rate * REFERENCE_BUDGET_SECONDS / total_rounds)))
    for _ in range(max(args.warmup, 0)):
        runner.round(n_sample)
    scheduled = 0
    t0 = time.perf_counter()
    for _ in range(args.steps):
        scheduled += runner.round(n_sample)
    seconds = time.perf_counter() - t0
    value = n_sample * (scheduled * w.grad_bytes + 16 * args.steps) / seconds / 1e9
    sample = "first %d of %d elements of %s (as one flat tensor) per step, %d threads over disjoint ranges" % (
        n_sample, w.n, w.name, cores)
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": seconds / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "config": config_for(w, world),
        "param_elements_per_s": n_sample * args.steps / seconds,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                         "sample_elements": n_sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


def extra_entry(t, steps: int, peak: float, peak_kind: str, kernel: str, n: int, note: str = ""):
    """One line of `other_workloads`: a roofline block plus the per-step figures."""
    block = roofline_block(t, steps, peak, peak_kind, kernel)
    out = {"gbs": block["achieved"], "frac_of_%s_peak" % peak_kind: block["frac"],
           "ms_per_step": t["seconds"] / steps * 1e3, "param_elements_per_s": n * steps / t["seconds"],
           "steps": steps, "roofline": block}
    if note:
        out["note"] = note
    return out


def time_other_workloads(headline, peak: float, peak_kind: str, only=None, n_synthetic: int = 100_000_000):
    """The remaining bar workloads, the extended entry points and the kernels of
    the all-reduce round, each timed like the headline (rank 0, one GPU).
    `only`: run just the entry of that name; `n_synthetic`: elements of the
    entries that are not one of the five workloads (smaller for profiler captures)."""
    import dataclasses
    import torch
    from paper_2512_09685_b200 import binding as B
    from paper_2512_09685_b200 import workloads as WL
    others = {}

    def wanted(name):
        return only is None or only == name

    def run(name, w, mode="plain", note=""):
        if not wanted(name):
            return None
        big = w.n > 30_000_000
        dw = DeviceWorkload(w, grad_sets=1 if big else 8, mode=mode)
        steps = 50 if big else 400
        t = time_device(dw, steps, 5, None, probe=False)
        others[name] = extra_entry(t, steps, peak, peak_kind, dw.kernel_name(), w.n, note)
        return dw

    for other in WL.WORKLOADS:
        if other.name == headline.name:
            continue
        dw = run(other.name, other)
        if dw is not None and other.n <= 30_000_000 and not other.multi_tensor and other.n * (other.W * other.grad_bytes + 16) < 126e6:
            # L2-resident, launch-bound size: also the same rounds replayed from a
            # CUDA graph (schedules encoded once at capture), i.e. without the host.
            others[other.name]["note"] = "working set fits L2: not an HBM figure"
            gms = time_graph_replay(dw, 100, 10)
            others[other.name]["cuda_graph_replay"] = {"ms_per_step": gms}
        del dw
        torch.cuda.empty_cache()

    # Extended entry points on the ResNet-50-sized workload (3 groups: 3 + 3 + 2 workers):
    # bytes per round = n * (sum |G| * 2 + 16 + 3 snapshots * sizeof(snapshot)).
    cfg1 = WL.BY_NAME["cfg1_resnet50"]
    for mode, note in (("snap_f32", "star_group_update_ex, one fp32 parameter snapshot per group"),
                       ("snap_bf16", "star_group_update_ex, one bf16 parameter snapshot per group"),
                       ("tree", "star_group_update_ex, tree summation order (groups of 3: 4-leaf kernel)")):
        del_me = run("cfg1_resnet50/" + mode, cfg1, mode, note)
        del del_me
        torch.cuda.empty_cache()
    # Tree order on one group of 16 (the 8-leaf-block kernel, two blocks per SM), 100 M elements.
    one16 = dataclasses.replace(WL.scaled(WL.BY_NAME["cfg2_bert_large"], n_synthetic), name="tree_1x16_100M",
                                schedule="fixed", fixed_labels=(0,) * 16)
    del_me = run("tree_1x16_100M", one16, "tree", "one group of 16 workers in tree order")
    del del_me
    torch.cuda.empty_cache()
    # The tensor list with per-group rates and a bf16 snapshot set per group (2..8 groups per round).
    if headline.multi_tensor:
        del_me = run(headline.name + "/snap_bf16", headline, "snap_bf16",
                     "star_group_update_multi_ex, one bf16 snapshot set per group")
        del del_me
        torch.cuda.empty_cache()

    # The two kernels of the all-reduce round, 100 M elements of bf16 gradients.
    n = n_synthetic
    if only is not None and not (only.startswith("group_reduce") or only.startswith("update_from_sums")):
        return others
    grads = [(torch.randn(n, device="cuda") * 0.01).to(torch.bfloat16) for _ in range(4)]
    out = torch.empty(n, device="cuda")
    for count in (2, 4):
        if not wanted("group_reduce_%d_bf16_to_f32_100M" % count):
            continue
        nbytes = n * (count * 2 + 4)
        t = time_steps(lambda: (B.star_group_reduce(out, grads, list(range(count))), nbytes)[1], 50, 5, None,
                       launch_count=B.star_launch_count, probe=False)
        others["group_reduce_%d_bf16_to_f32_100M" % count] = extra_entry(
            t, 50, peak, peak_kind, "star_group_reduce_kernel", n,
            "a parent's aggregate of its own and %d children's gradients; bytes n*(%d*2+4)" % (count - 1, count))
    del grads
    if not wanted("update_from_sums_R4_100M"):
        return others
    sums = [torch.randn(n, device="cuda") * 0.01 for _ in range(4)]
    p, v = torch.randn(n, device="cuda") * 0.05, torch.zeros(n, device="cuda")
    nbytes = n * (4 * 4 + 16)
    t = time_steps(lambda: (B.star_group_update_from_sums(p, v, sums, 6, 0.01, 0.9, 1e-4), nbytes)[1], 50, 5, None,
                   launch_count=B.star_launch_count, probe=False)
    others["update_from_sums_R4_100M"] = extra_entry(
        t, 50, peak, peak_kind, "star_update_flat_kernel", n,
        "the ring's update from 4 fp32 aggregates (6 gradient reports); bytes n*(4*4+16)")
    return others


def run_all_reduce_architecture(args, rank: int, world: int, local_rank: int):
    """--architecture all_reduce: every rank is one worker holding its own
    ResNet-50-sized gradient; every step decides (Section II straggler rule, Eq. 3)
    who leaves the ring from seeded predicted iteration times, then runs the round
    (children -> parent, local aggregate, ring exchange, update, state back)."""
    import torch
    import torch.distributed as dist_mod
    from paper_2512_09685_b200 import binding as B
    from paper_2512_09685_b200 import workloads as WL
    from paper_2512_09685_b200.all_reduce_round import AllReduceRound
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist = dist_mod
    w = WL.BY_NAME["cfg1_resnet50"] if args.n <= 0 else WL.scaled(WL.BY_NAME["cfg1_resnet50"], args.n)
    n = w.n
    p = WL.make_params(w, "cuda")[0]
    v = WL.make_momentum(w, "cuda")[0]
    grad = torch.empty(n, dtype=w.torch_grad_dtype(), device="cuda")
    WL.fill_grads(w, 0, rank, [grad])
    runner = AllReduceRound(dist_mod, rank, world, exchange=args.exchange)
    peak, peak_kind = measured_peak()
    state = {"step": 0}

    def decide(step):
        # every rank draws the same times: a fast majority and a slow tail
        rng = WL.SplitMix64(77_000 + step)
        t = [1.0 + rng.below(100) / 1000.0 for _ in range(world)]
        for _ in range(world // 4):
            t[rng.below(world)] *= 2.0 + rng.below(3)
        child = [ti * (0.3 + rng.below(60) / 100.0) for ti in t]
        x, t_w, T, removed, (off, mem) = B.star_choose_all_reduce_mode(t, child, 1e3, 256.0, 0.5)
        return removed, [c for c in mem if c in removed]

    def step():
        removed, in_time = decide(state["step"])
        state["step"] += 1
        plan = runner.run(grad, p, v, removed, in_time, w.lr, w.mu, w.wd)
        # algorithmic HBM bytes of this rank's two kernels (ring members only)
        if rank in plan.ring:
            kids = len(plan.children[rank])
            return n * ((1 + kids) * w.grad_bytes + 4) + n * (len(plan.ring) * 4 + 16)
        return 0

    t = time_steps(step, args.steps, max(args.warmup, 3), dist, launch_count=B.star_launch_count, probe=False)
    total = torch.tensor([float(t["bytes"])], dtype=torch.float64, device="cuda")
    if dist is not None:
        dist.all_reduce(total)
    out = {"metric": "all-reduce-architecture round, HBM GB/s of the aggregate and update kernels over the whole round",
           "value": float(total.item()) / t["seconds"] / 1e9, "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": max(args.warmup, 3), "ms_per_step": t["seconds"] / args.steps * 1e3, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
           "config": {"workload": w.name, "architecture": "all_reduce", "exchange": args.exchange, "n": n,
                      "workers": world, "grad_dtype": w.grad_dtype},
           "gpu_launches": t["launches"], "regions": {"count": t["repeats"], "gbs": t["gbs_regions"]}}
    if rank == 0:
        print(json.dumps(out), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    global MIN_TIMED_SECONDS
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default=HEADLINE)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--architecture", default="ps", choices=["ps", "all_reduce"],
                    help="ps: the parameter-server round (default); all_reduce: one rank per worker, "
                         "the all-reduce architecture's round")
    ap.add_argument("--exchange", default="scatter", choices=["gather", "scatter"],
                    help="how the ring exchanges its aggregates (--architecture all_reduce)")
    ap.add_argument("--n", type=int, default=0,
                    help="run the workload at a reduced size (flat: this many elements; tensor list: 2 "
                         "layers and n/1024 vocabulary rows): small cases for profiler captures, "
                         "not a benchmark configuration")
    ap.add_argument("--min-seconds", type=float, default=MIN_TIMED_SECONDS,
                    help="device time to accumulate over repeated timed regions (0: three regions; for "
                         "profiler captures)")
    ap.add_argument("--only", default=None,
                    help="time just this entry of other_workloads (with --n: its synthetic entries at that "
                         "size) and print it; for profiler captures of the other kernels")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-extra", action="store_true",
                    help="device-timed headline only: skip the end-to-end leg, the other workloads "
                         "and the CPU baseline")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    MIN_TIMED_SECONDS = args.min_seconds

    import torch
    from paper_2512_09685_b200 import binding as B        # raises if the CUDA library is missing
    from paper_2512_09685_b200 import workloads as WL

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    if max(args.warmup, 0) < 3:
        args.warmup = 3
    if args.architecture == "all_reduce":
        run_all_reduce_architecture(args, rank, world, local_rank)
        return
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist = dist_mod

    w = WL.BY_NAME[args.workload]
    if args.n > 0:
        # reduced sizes for profiler captures: a flat workload at n elements, the
        # tensor list with 2 layers and a vocabulary of n / 1024 rows
        w = WL.reduced_list(w, 2, max(args.n // 1024, 1)) if w.multi_tensor else WL.scaled(w, args.n)
    peak, peak_kind = measured_peak()
    if args.only:
        entry = time_other_workloads(w, peak, peak_kind, args.only,
                                     args.n if args.n > 0 else 100_000_000)
        print(json.dumps({"other_workloads": entry}), flush=True)
        return
    dw = DeviceWorkload(w, grad_sets=2 if w.n * w.W * w.grad_bytes < (4 << 30) else 1)
    sampler = ClockSampler(local_rank)
    t = time_device(dw, args.steps, args.warmup, dist, sampler)
    gbs_rank = t["bytes"] / t["seconds"] / 1e9
    value = gbs_rank * world
    config = config_for(w, world)                      # identical in the reference arm

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t["seconds"] / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config,
        "gradient_buffer_sets_rotated": len(dw.grad_sets),
        "timed_regions": {"count": t["repeats"], "steps_each": args.steps, "seconds_total": t["timed_seconds"],
                          "value_min": t["gbs_regions"][0] * world, "value_median": value,
                          "value_max": t["gbs_regions"][-1] * world,
                          "note": "value is the median region; each region is `steps` rounds between two CUDA events"},
        "param_elements_per_s": w.n * args.steps * world / t["seconds"],
        "pct_of_peak": {"measured_%.1f" % peak: 100 * gbs_rank / peak, "datasheet_8000": 100 * gbs_rank / 8000},
        "gpu_launches": t["launches"],
        "clocks": sampler.summary(),
        "roofline": roofline_block(t, args.steps, peak, peak_kind, dw.kernel_name(),
                                   ncu_traffic(args.workload, w.n) if args.n <= 0 else None),
    }

    del dw
    torch.cuda.empty_cache()
    if not args.no_e2e and not args.no_extra:
        e2e_steps = max(3, min(args.steps, 5 if w.n > 100_000_000 else 20))
        e = time_e2e(w, e2e_steps, 3, dist)
        e2e_value = e["bytes"] / e["seconds"] / 1e9
        out["e2e"] = {"value": e2e_value * world, "unit": UNIT, "h2d_bytes_per_step": e["h2d"],
                      "d2h_bytes_per_step": e["d2h"], "steps": e2e_steps, "ms_per_step": e["seconds"] / e2e_steps * 1e3,
                      "gpu_launches": e["launches"],
                      "peak": e["peak"] * world, "frac": e2e_value / e["peak"],
                      "peak_kind": "plain pinned copies of the same bytes, up and down concurrently, same run "
                                   "(%.1f GB/s host to device)" % e["h2d_gbs_copy_only"],
                      "how": "star_group_update_host on pinned host tensors, 4 Mi-element chunks, "
                             "stream synchronized every step"}
        torch.cuda.empty_cache()

    if not args.no_extra and rank == 0 and world == 1:
        out["other_workloads"] = time_other_workloads(w, peak, peak_kind)
        cores = host_cores()
        n_sample = min(w.n, 8_000_000)
        cgbs, ceps, rounds, cdt = time_oracle(w, n_sample, 8.0, cores)
        sgbs, seps, srounds, sdt = time_oracle(w, n_sample, 4.0, 1)
        out["cpu_baseline"] = {
            "value": cgbs, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "first %d of %d elements of %s (as one flat tensor), %d rounds in %.1f s, %d threads over "
                      "disjoint ranges" % (n_sample, w.n, w.name, rounds, cdt, cores),
            "param_elements_per_s": ceps,
            "single_thread": {"value": sgbs, "param_elements_per_s": seps, "rounds": srounds}}

    if rank == 0:
        print(json.dumps(out), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

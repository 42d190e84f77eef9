#!/usr/bin/env python
"""Benchmark of the fused grouped aggregate + update.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME]
                    [--impl ours|reference] [--no-extra]

A step is one round of the whole path on one batch of synthetic gradients:
the mode decision of the round is encoded into a CSR schedule (host, in the
library) and the fused update kernel is launched once.  Prints ONE JSON line.

  value      achieved GB/s = algorithmic bytes / device time, inputs resident
             in HBM; bytes per round = n * (sum_k |G_k| * sizeof(g) + 16)
  e2e        the same metric through the host-buffer entry point: parameters,
             momentum and gradients start in pinned host memory, results end
             there, every copy inside the timed region
  roofline   the update kernel against the measured HBM copy bandwidth
  cpu_baseline  the CPU oracle timed on this machine's cores (reported only)

With N > 1 (under torchrun) every rank runs the same workload on its own GPU
(the path is elementwise: shards need no exchange), the time is the maximum
over ranks and the value the sum of all ranks' bytes over that time.
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

METRIC = "grouped aggregate+update HBM GB/s"
UNIT = "GB/s"
HEADLINE = "cfg1_resnet50"
FALLBACK_HBM_GBS = 6650.0


# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the
# headline kernel from the ncu capture summarised under profiles/, keyed by
# workload, with the SHA-256 of the kernel sources the capture was taken on:
# once the sources differ the figure is stale and `traffic` is reported as null.
NCU_TRAFFIC = {
    "cfg1_resnet50": (790.9e6, "f5e911d974634f5eb3fd6156f6e14ba3e7e39ba3c74004c57323496e84f0320a"),
}


def kernel_source_hash() -> str:
    import hashlib
    h = hashlib.sha256()
    for name in ("kernels.cuh", "api.cu"):
        with open(os.path.join(ROOT, "paper_2512_09685_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def ncu_traffic(workload_name: str):
    entry = NCU_TRAFFIC.get(workload_name)
    if entry is None:
        return None
    try:
        return entry[0] if kernel_source_hash() == entry[1] else None
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
    """One workload resident on the current device, ready to step."""

    def __init__(self, w, grad_sets: int):
        import torch
        from paper_2512_09685_b200 import binding as B
        from paper_2512_09685_b200 import workloads as WL
        self.torch, self.B, self.w = torch, B, w
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
        self.plans = None
        if w.multi_tensor:
            self.workspaces, self.plans = [], []
            for one in self.grad_sets:
                ws = torch.empty(B.star_multi_workspace_bytes(w.sizes, w.W), dtype=torch.uint8, device=dev)
                self.workspaces.append(ws)
                self.plans.append(B.star_multi_prepare(self.params, self.momentum, one, ws))
        else:
            self.flat_grads = [[bufs[0] for bufs in one] for one in self.grad_sets]
        self.step_index = 0
        torch.cuda.synchronize()

    def step(self) -> int:
        """One round: encode the decision, launch the fused update.  Returns the
        number of scheduled workers (for the byte count)."""
        w, B = self.w, self.B
        off, mem = B.encode(w.decision(self.step_index))
        which = self.step_index % len(self.grad_sets)
        if self.plans is not None:
            B.star_group_update_multi(self.plans[which], off, mem, w.lr, w.mu, w.wd)
        else:
            B.star_group_update(self.params[0], self.momentum[0], self.flat_grads[which], off, mem,
                                w.lr, w.mu, w.wd)
        self.step_index += 1
        return off[-1]

    def reset_state(self):
        # keeps values bounded over thousands of timed rounds; not timed
        for v in self.momentum:
            v.zero_()


def max_over_ranks(seconds: float, dist, device) -> float:
    """The slowest rank's time: what a multi-rank measurement reports."""
    if dist is None:
        return seconds
    import torch
    t = torch.tensor([seconds], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def time_device(dw: DeviceWorkload, steps: int, warmup: int, dist, sampler=None):
    """Returns (seconds for `steps` rounds [max over ranks], per-launch ms list,
    algorithmic bytes of those rounds on this rank, launches)."""
    torch, B = dw.torch, dw.B
    for _ in range(warmup):
        dw.step()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    begin, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = B.star_launch_count()
    scheduled = 0
    if sampler is not None:
        sampler.__enter__()
    begin.record()
    for i in range(steps):
        scheduled += dw.step()
    end.record()
    if sampler is not None:
        sampler.sample()
    torch.cuda.synchronize()
    if sampler is not None:
        sampler.__exit__(None, None, None)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    launches = B.star_launch_count() - launches0
    total_ms = begin.elapsed_time(end)
    # Per-launch durations from a short extra pass with an event after every
    # launch (the events themselves cost time, so they stay out of the timed
    # region above; the pass only shows the spread).
    probe = min(steps, 200)
    events = [torch.cuda.Event(enable_timing=True) for _ in range(probe + 1)]
    events[0].record()
    for i in range(probe):
        dw.step()
        events[i + 1].record()
    torch.cuda.synchronize()
    per_launch = [events[i].elapsed_time(events[i + 1]) for i in range(probe)]
    nbytes = dw.w.n * (scheduled * dw.w.grad_bytes + 16 * steps)
    seconds = max_over_ranks(total_ms / 1e3, dist, "cuda")
    return seconds, per_launch, nbytes, launches


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
    is read on the host).  Returns (seconds [max over ranks], bytes, h2d, d2h
    per step, launches)."""
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
    nbytes = n * (scheduled * w.grad_bytes + 16 * steps)
    h2d = n * (scheduled * w.grad_bytes + 8 * steps) // steps
    d2h = n * 8
    return seconds, nbytes, h2d, d2h, B.star_launch_count() - launches0


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


def run_reference(args, rank: int):
    """--impl reference: the CPU oracle on the host cores.  A step is one round on
    a bounded sample of the workload: the first n_sample elements, n_sample
    chosen from a calibration round so that warm-up + steps fit the budget."""
    if rank != 0:
        return
    from paper_2512_09685_b200 import workloads as WL
    w = WL.BY_NAME[args.workload]
    cores = host_cores()
    runner = OracleRunner(w, w.n if w.n <= 32_000_000 else 32_000_000, cores)
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
    sample = "first %d of %d elements of %s per step, %d threads over disjoint ranges" % (
        n_sample, w.n, w.name, cores)
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": seconds / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "config": {"workload": w.name, "stands_for": w.model, "n": w.n, "W": w.W,
                                        "grad_dtype": w.grad_dtype, "sample_elements": n_sample},
        "param_elements_per_s": n_sample * args.steps / seconds,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default=HEADLINE)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--n", type=int, default=0,
                    help="run the workload at a reduced size (flat: this many elements; tensor list: 2 "
                         "layers and n/1024 vocabulary rows): small cases for profiler captures, "
                         "not a benchmark configuration")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-extra", action="store_true",
                    help="device-timed headline only: skip the end-to-end leg, the other workloads "
                         "and the CPU baseline")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    from paper_2512_09685_b200 import binding as B        # raises if the CUDA library is missing
    from paper_2512_09685_b200 import workloads as WL

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    if max(args.warmup, 0) < 3:
        args.warmup = 3
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
    dw = DeviceWorkload(w, grad_sets=2 if w.n * w.W * w.grad_bytes < (4 << 30) else 1)
    sampler = ClockSampler(local_rank)
    seconds, per_launch, nbytes, launches = time_device(dw, args.steps, args.warmup, dist, sampler)
    gbs_rank = nbytes / seconds / 1e9
    value = gbs_rank * world
    # one launch per step and nothing else on the stream: the kernel's mean
    # launch duration over the timed region is the region's time / launches
    kernel_ms = seconds / launches * 1e3
    achieved = (nbytes / args.steps) / (kernel_ms / 1e3) / 1e9

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": seconds / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "stands_for": w.model, "n": w.n, "W": w.W, "grad_dtype": w.grad_dtype,
                   "tensors": len(w.sizes), "bytes_per_step": nbytes // args.steps,
                   "l2": "inputs larger than L2: %.0f MB per step, gradient buffer sets rotated: %d" % (
                       nbytes / args.steps / 1e6, len(dw.grad_sets)),
                   "parallelism": "replicas x%d" % world},
        "param_elements_per_s": w.n * args.steps * world / seconds,
        "pct_of_peak": {"measured_%.1f" % peak: 100 * gbs_rank / peak, "datasheet_8000": 100 * gbs_rank / 8000},
        "gpu_launches": launches,
        "clocks": sampler.summary(),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak,
                     "traffic": ncu_traffic(w.name) if args.n <= 0 else None, "peak_kind": "of " + peak_kind,
                     "kernel": "star_update_multi_kernel" if w.multi_tensor else "star_update_flat_kernel",
                     "kernel_ms_mean": kernel_ms,
                     "per_launch_probe_ms": {"median": statistics.median(per_launch), "min": min(per_launch),
                                             "launches": len(per_launch)}},
    }

    del dw
    torch.cuda.empty_cache()
    if not args.no_e2e and not args.no_extra:
        e2e_steps = max(3, min(args.steps, 20))
        esec, ebytes, h2d, d2h, elaunch = time_e2e(w, e2e_steps, 3, dist)
        out["e2e"] = {"value": ebytes / esec / 1e9 * world, "unit": UNIT, "h2d_bytes_per_step": h2d,
                      "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": esec / e2e_steps * 1e3,
                      "gpu_launches": elaunch,
                      "how": "star_group_update_host on pinned host tensors, 4 Mi-element chunks, "
                             "stream synchronized every step"}

    if not args.no_extra and rank == 0 and world == 1:
        others = {}
        for other in WL.WORKLOADS:
            if other.name == w.name:
                continue
            odw = DeviceWorkload(other, grad_sets=1 if other.n > 30_000_000 else 8)
            osteps = 50 if other.n > 30_000_000 else 400
            osec, oper, obytes, _ = time_device(odw, osteps, 5, None)
            ogbs = obytes / osec / 1e9
            others[other.name] = {"gbs": ogbs, "frac_of_%s_peak" % peak_kind: ogbs / peak,
                                  "ms_per_step": osec / osteps * 1e3,
                                  "param_elements_per_s": other.n * osteps / osec, "steps": osteps}
            if other.n <= 30_000_000 and not other.multi_tensor:
                # Launch-bound size: also time the same rounds replayed from a CUDA
                # graph (schedules encoded once at capture), i.e. without the host.
                gms = time_graph_replay(odw, 100, 10)
                others[other.name]["cuda_graph_replay"] = {
                    "ms_per_step": gms, "gbs": obytes / osteps / (gms / 1e3) / 1e9,
                    "note": "L2-resident working set: not an HBM figure"}
            del odw
            torch.cuda.empty_cache()
        out["other_workloads"] = others
        cores = host_cores()
        n_sample = min(w.n, 8_000_000)
        cgbs, ceps, rounds, cdt = time_oracle(w, n_sample, 8.0, cores)
        sgbs, seps, srounds, sdt = time_oracle(w, n_sample, 4.0, 1)
        out["cpu_baseline"] = {
            "value": cgbs, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "first %d of %d elements of %s, %d rounds in %.1f s, %d threads over disjoint ranges"
                      % (n_sample, w.n, w.name, rounds, cdt, cores),
            "param_elements_per_s": ceps,
            "single_thread": {"value": sgbs, "param_elements_per_s": seps, "rounds": srounds}}

    if rank == 0:
        print(json.dumps(out), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

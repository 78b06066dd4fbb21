#!/usr/bin/env python
"""Benchmark of the event-triggered communication step.

    python bench.py --gpus N --steps K --warmup W            (CUDA library)
    python bench.py --impl reference --steps K --warmup W    (CPU oracle on the host cores)

A "step" is one ``eg_step``: change norms, device-side trigger decisions, dense snapshots
(or Top-K select / pack / scatter), ring average and SGD update for all P replicas of the
workload.  Default workload: the 16-replica ring of ResNet-18 (CIFAR) parameter sets with the
step-indexed synthetic gradients of that configuration.  With N > 1 (torchrun) every rank runs
an independent copy of the workload on its own GPU ("replicas only": the method is defined on
one device's memory, nothing is exchanged); the value is the sum over ranks divided by the
slowest rank's time.

Every GB/s figure of one line (``value``, ``e2e``, ``cpu_baseline``, and the line of
``--impl reference``) counts the same bytes per element-step, those of the timed variant
(``config.bytes_per_element_step``: 16 with the carried norm, 24 with the separate norm pass), so
their ratios are ratios of step rates; ``replica_steps_per_s`` beside each needs no convention.

Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2103_07454_b200 import workload as W  # noqa: E402

METRIC = "event-triggered step: effective HBM GB/s (% of peak), replica-steps/s, msgs sent"
FALLBACK_HBM_GBS = 6650.0          # earlier measurement on this machine, used if no peaks file
NOMINAL_HBM_GBS = 8000.0
BYTES_PER_ELEMENT = {"carry": 16, "two_pass": 24}   # algorithmic bytes per element-replica-step
FUSED_BYTES_PER_ELEMENT = 16       # fused kernel: reads x, g, touches x_hat once, writes x
MOMENTUM_BYTES_PER_ELEMENT = 8     # --momentum: the velocity is read and written once more

# DRAM traffic of the fused kernel from an ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum per launch, captured on a prefix of the default workload), keyed by the
# hash of the kernel sources the timed configuration launches.  Once any of those sources has
# changed the figure is reported as null, together with what it was captured with.
FUSED_TRAFFIC_ELEMENTS = 16 * 11173962     # element-replicas of one launch on the default workload
FUSED_TRAFFIC = {
    # sources of a dense run: hash -> (bytes per launch of the default workload, where the counters are)
    "dense": {"244492e95c38": (2.634e9, "profiles/k_fused_pipe_resnet18_first45tensors.md")},
}
DENSE_SOURCES = ("eg_common.cuh", "eg_norm.cuh", "eg_fused.cuh", "eg_fused_pipe.cuh")


def kernel_sources(wl) -> tuple:
    """The kernel sources a run of this workload launches from (the single-launch kernel serves
    the small dense configurations, the Top-K kernels the Top-K ones)."""
    names = list(DENSE_SOURCES)
    if wl.topk:
        names.append("eg_topk.cuh")
    elif wl.P <= 16 and wl.N <= 300000:
        names.append("eg_step_small.cuh")
    return tuple(names)


def kernel_source_hash(names=DENSE_SOURCES) -> str:
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2103_07454_b200", "csrc")
    for name in names:
        with open(os.path.join(d, name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:12]


def fused_traffic(wl, elems: int, momentum, quant_bits=None) -> dict:
    """`traffic` of the roofline object, and what to say when the counters are out of date."""
    names = kernel_sources(wl)
    current = kernel_source_hash(names)
    if momentum is not None or quant_bits is not None or names != DENSE_SOURCES:
        # counters exist for the default kernel on dense runs only
        return {"traffic": None, "traffic_note": "no capture for this configuration's kernels",
                "traffic_sources": list(names), "traffic_sources_hash": current}
    known = FUSED_TRAFFIC["dense"]
    if current in known:
        per_launch, where = known[current]
        # the capture was taken on a prefix of the default workload; a streaming kernel's traffic
        # grows with the elements, so it is scaled to the elements of one launch of this run
        return {"traffic": per_launch * elems / FUSED_TRAFFIC_ELEMENTS, "traffic_from": where,
                "traffic_sources": list(names), "traffic_sources_hash": current}
    captured, (_, where) = next(iter(known.items()))
    return {"traffic": None,
            "traffic_stale_since": f"kernel sources changed after the capture in {where} "
                                   f"(captured with sources hash {captured}, now {current})",
            "traffic_sources": list(names), "traffic_sources_hash": current}


# ----------------------------------------------------------------------------------------
# multi-process plumbing (one process per GPU; nothing of the data path is exchanged)
# ----------------------------------------------------------------------------------------
def dist_setup(backend: str):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world <= 1:
        return 0, 1, 0
    import torch.distributed as dist
    rank, local = int(os.environ["RANK"]), int(os.environ.get("LOCAL_RANK", "0"))
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    if not dist.is_initialized():
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world, local


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def aggregate(units_this_rank: float, ms_this_rank: float, device="cpu"):
    """Whole-job figures from per-rank ones: (sum of units, max of milliseconds)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(units_this_rank), float(ms_this_rank)
    u = torch.tensor([units_this_rank], dtype=torch.float64, device=device)
    t = torch.tensor([ms_this_rank], dtype=torch.float64, device=device)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(u.item()), float(t.item())


# ----------------------------------------------------------------------------------------
# clocks during the timed region
# ----------------------------------------------------------------------------------------
REASON_BITS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap",
               0x8: "hw_slowdown", 0x10: "sync_boost", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
               0x100: "display_clock_setting"}


class ClockSampler:
    """Polls SM clock and clock-event reasons through NVML from a thread."""

    def __init__(self, device_index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            self._nv = pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception as exc:  # pragma: no cover - depends on the box
            self.error = repr(exc)

    def _poll(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                self.samples.append(mhz)
                for bit, name in REASON_BITS.items():
                    if mask & bit and name != "gpu_idle":
                        self.reasons.add(name)
            except Exception:
                break
            time.sleep(0.0005)

    def start(self):
        if self._h is not None:
            self._stop.clear()
            self._thread = threading.Thread(target=self._poll, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
            self._thread = None

    def summary(self) -> dict:
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ----------------------------------------------------------------------------------------
def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def pick_workload(args) -> W.Workload:
    wl = W.config(args.config)[args.which]
    if args.max_elements:       # a smaller case of the same shapes (for profiler captures)
        keep, total = [], 0
        for t in wl.tensors:
            if keep and total + t.numel > args.max_elements:
                break
            keep.append(t)
            total += t.numel
        wl.tensors = keep
        wl.name += f"_first{len(keep)}tensors"
    return wl


def sample_tensors(wl: W.Workload, fraction: float):
    """Tensors (in order) holding about ``fraction`` of the elements; at least one."""
    picked, acc = [], 0
    for t, n in enumerate(wl.numel):
        if picked and acc >= fraction * wl.N:
            break
        picked.append(t)
        acc += n
    return picked


def time_oracle(wl: W.Workload, steps: int, warmup: int, budget_s: float, gen_device: str,
                single_thread_s: float = 0.0, bytes_per_element: int = 16):
    """Times the CPU oracle, as it stands, on all host cores.  If ``steps`` full-size steps do
    not fit ``budget_s`` the run uses a subset of the tensors (they do not interact)."""
    import numpy as np
    from oracle import eg_oracle as eo
    threads = eo.threads_available()
    # calibrate on a small prefix of the tensors
    probe_t = sample_tensors(wl, 0.05)
    numel = [wl.numel[t] for t in probe_t]
    o = eo.Oracle(wl.P, numel, horizon=wl.horizon, history_len=wl.history_len,
                  delta_init=wl.delta_init, topk=wl.topk, threads=threads)
    n_probe = sum(numel)
    x = np.zeros((wl.P, n_probe), np.float32)
    g = np.full((wl.P, n_probe), 1e-3, np.float32)
    o.step(x, g, wl.lr)
    t0 = time.perf_counter()
    o.step(x, g, wl.lr)
    per_elem = (time.perf_counter() - t0) / (wl.P * n_probe)
    o.close()
    full_step_s = per_elem * wl.P * wl.N
    fraction = min(1.0, budget_s / max(1e-9, full_step_s * (steps + warmup)))
    tensors = sample_tensors(wl, fraction) if fraction < 1.0 else list(range(wl.T))
    numel = [wl.numel[t] for t in tensors]
    n_sub = sum(numel)
    off = np.concatenate([[0], np.cumsum(wl.numel)])
    cols = np.concatenate([np.arange(off[t], off[t] + wl.numel[t]) for t in tensors])
    cols_t = torch.from_numpy(cols).to(gen_device)
    n_buf = max(1, min(steps + warmup, 4))
    grads = [np.ascontiguousarray(wl.grads(k, gen_device)[:, cols_t].cpu().numpy()) for k in range(n_buf)]
    x = np.ascontiguousarray(wl.init_params(gen_device)[:, cols_t].cpu().numpy())
    o = eo.Oracle(wl.P, numel, horizon=wl.horizon, history_len=wl.history_len,
                  delta_init=wl.delta_init, topk=wl.topk, threads=threads)
    for k in range(warmup):
        o.step(x, grads[k % n_buf], wl.lr)
    t0 = time.perf_counter()
    for k in range(steps):
        o.step(x, grads[(warmup + k) % n_buf], wl.lr)
    sec = time.perf_counter() - t0
    stats = o.stats()
    o.close()
    # one thread, for context: a few seconds on the leading tensors
    one = None
    if single_thread_s > 0:
        frac1 = min(1.0, single_thread_s / max(1e-9, 2 * full_step_s * threads))
        t1 = sample_tensors(wl, frac1) if frac1 < 1.0 else list(range(wl.T))
        numel1 = [wl.numel[t] for t in t1]
        cols1 = torch.from_numpy(np.concatenate([np.arange(off[t], off[t] + wl.numel[t]) for t in t1])).to(gen_device)
        g1 = np.ascontiguousarray(wl.grads(0, gen_device)[:, cols1].cpu().numpy())
        x1 = np.ascontiguousarray(wl.init_params(gen_device)[:, cols1].cpu().numpy())
        o1 = eo.Oracle(wl.P, numel1, horizon=wl.horizon, history_len=wl.history_len,
                       delta_init=wl.delta_init, topk=wl.topk, threads=1)
        o1.step(x1, g1, wl.lr)
        t0 = time.perf_counter()
        o1.step(x1, g1, wl.lr)
        s1 = time.perf_counter() - t0
        o1.close()
        one = {"value": wl.P * sum(numel1) * bytes_per_element / s1 / 1e9, "unit": "GB/s",
               "replica_steps_per_s": wl.P * (sum(numel1) / wl.N) / s1,
               "sample": f"1 step of {len(t1)}/{wl.T} tensors ({sum(numel1)} elements per replica)"}
    elems = wl.P * n_sub * steps
    gbs = elems * bytes_per_element / sec / 1e9
    sample = (f"{steps} steps of all {wl.P} replicas x {len(tensors)}/{wl.T} tensors "
              f"({n_sub}/{wl.N} elements per replica)")
    return {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample,
            "replica_steps_per_s": wl.P * steps * (n_sub / wl.N) / sec, "seconds": sec,
            "messages_sent": stats["messages"], "single_thread": one}


def run_reference(args):
    rank, world, local = dist_setup("gloo")
    if rank != 0:
        return
    wl = pick_workload(args)
    gen = "cuda" if torch.cuda.is_available() else "cpu"
    r = time_oracle(wl, args.steps, args.warmup, budget_s=120.0, gen_device=gen,
                    bytes_per_element=BYTES_PER_ELEMENT[args.variant])
    line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": "GB/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * r["seconds"] / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "P": wl.P, "tensors": wl.T, "elements": wl.N,
                       "variant": args.variant, "bytes_per_element_step": BYTES_PER_ELEMENT[args.variant]},
            "replica_steps_per_s": r["replica_steps_per_s"],
            "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": r["value"], "unit": "GB/s", "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def time_steps(eg, x, grads, lr, steps, sampler=None):
    """K steps bracketed by events on the launching stream, barrier + synchronise outside."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.start()
    e0.record()
    launches = 0
    for k in range(steps):
        eg.step(x, grads[k % len(grads)], lr)
        launches += eg.last_launch_count
    e1.record()
    torch.cuda.synchronize()
    if sampler:
        sampler.stop()
    barrier()
    return e0.elapsed_time(e1), launches


def measure_workload(B, wl, K, Wm, dev, world, variants, sampler, sampled_variant, graph_steps=0,
                     momentum=None, quant_bits=None):
    """Times K steps of `wl` for every variant; returns ({variant: figures}, context)."""
    eg = B.from_workload(wl)
    if momentum is not None:      # heavy-ball update: the velocity is read and written as well
        eg.set_momentum(momentum)
    if quant_bits is not None:    # quantised messages: delivered by kernels of their own, on events only
        eg.set_quantisation(quant_bits)
    extra = MOMENTUM_BYTES_PER_ELEMENT if momentum is not None else 0
    buf_bytes = wl.P * eg.replica_stride * 4
    free, _ = torch.cuda.mem_get_info()
    reserve = (24 << 30) + 4 * buf_bytes + (2 * buf_bytes if wl.topk else 0)
    n_buf = int(max(1, min(max(K, Wm), (free - reserve) // buf_bytes)))
    grads = [eg.to_layout(wl.grads(k, dev)) for k in range(n_buf)]
    x0 = eg.to_layout(wl.init_params(dev))
    x = x0.clone()
    elems = wl.P * wl.N
    results = {}
    for variant in variants:
        eg.set_carry_norm(variant == "carry")
        x.copy_(x0)
        eg.reset()
        eg.set_timing(False)
        for k in range(Wm):
            eg.step(x, grads[k % n_buf], wl.lr)
        # pass 1, the timed region of `value`: K steps between two events, nothing in between
        x.copy_(x0)
        eg.reset()
        eg.set_carry_norm(variant == "carry")
        eg.set_timing(False)
        ms, launches = time_steps(eg, x, grads, wl.lr, K,
                                  sampler if (sampler and variant == sampled_variant) else None)
        stats = eg.stats()
        units, ms_max = aggregate(float(elems) * K, ms, dev)
        # pass 2, the same K steps with a pair of events around every kernel group (the events
        # keep a kernel from starting under the tail of the one before it, so this pass is a
        # little slower than pass 1): per-kernel durations for the roofline
        x.copy_(x0)
        eg.reset()
        eg.set_carry_norm(variant == "carry")
        eg.set_timing(True)
        ms_instr, _ = time_steps(eg, x, grads, wl.lr, K, None)
        kt = eg.kernel_times()
        # the same K steps once more with an event between steps: spread of the single steps
        # (the figures above come from the two outer events only)
        x.copy_(x0)
        eg.reset()
        eg.set_carry_norm(variant == "carry")
        eg.set_timing(False)
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
        torch.cuda.synchronize()
        marks[0].record()
        for k in range(K):
            eg.step(x, grads[k % n_buf], wl.lr)
            marks[k + 1].record()
        torch.cuda.synchronize()
        per_step = sorted(marks[k].elapsed_time(marks[k + 1]) for k in range(K))
        results[variant] = {
            "ms_per_step": ms_max / K, "gbs": units * (BYTES_PER_ELEMENT[variant] + extra) / ms_max / 1e6,
            "replica_steps_per_s": world * wl.P * K / (ms_max / 1e3), "launches": launches,
            "kernel_ms": {g: (v[0] / v[1] if v[1] else None) for g, v in kt.items()},
            "ms_per_step_with_kernel_events": ms_instr / K,
            "messages_sent": stats["messages"], "bytes_sent": stats["bytes"],
            "pct_messages": 100.0 * stats["messages"] / (wl.P * wl.T * 2 * K),
            "gradient_buffers": n_buf, "cuda_graph": False,
            "step_ms": {"median": statistics.median(per_step), "best": per_step[0],
                        "worst": per_step[-1]}}
    if graph_steps:
        # launch-bound cases: the same steady-state step replayed from a CUDA graph (gradients of
        # one step, carried norm); shows what remains when the launch overhead is taken away
        eg.set_timing(False)
        eg.set_carry_norm(True)
        x.copy_(x0)
        eg.reset()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for k in range(3):
                eg.step(x, grads[0], wl.lr)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            eg.step(x, grads[0], wl.lr)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(5):
            g.replay()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(graph_steps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        results["graph_replay_ms_per_step"] = e0.elapsed_time(e1) / graph_steps
        del g
    del x
    return results, (eg, x0, grads, n_buf, buf_bytes)


def run_native(args):
    from paper_2103_07454_b200 import binding as B
    rank, world, local = dist_setup("nccl")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    wl = pick_workload(args)
    K, Wm = args.steps, max(args.warmup, 3)
    peak, peak_kind = measured_peak()
    sampler = ClockSampler(local)
    if args.all_configs:
        rows = []
        for idx in (1, 2, 3, 4, 5):
            for w in W.config(idx):
                r, ctx = measure_workload(B, w, w.steps, Wm, dev, world, ("carry", "two_pass"), None, None,
                                          graph_steps=200 if w.N < 1_000_000 else 0)
                ctx[0].close()
                del ctx
                rows.append({"config": idx, "workload": w.name, "P": w.P, "tensors": w.T, "elements": w.N,
                             "steps": w.steps, "topk": w.topk,
                             **{v: {"ms_per_step": r[v]["ms_per_step"], "GB/s": r[v]["gbs"],
                                    "pct_of_peak": 100.0 * r[v]["gbs"] / peak,
                                    "replica_steps_per_s": r[v]["replica_steps_per_s"],
                                    "kernel_ms": r[v]["kernel_ms"], "gradient_buffers": r[v]["gradient_buffers"]}
                                for v in ("carry", "two_pass")},
                             "graph_replay_ms_per_step": r.get("graph_replay_ms_per_step"),
                             "messages_sent": r["carry"]["messages_sent"],
                             "pct_messages": r["carry"]["pct_messages"],
                             "bytes_sent": r["carry"]["bytes_sent"]})
                torch.cuda.empty_cache()
        if rank == 0:
            print(json.dumps({"metric": METRIC, "unit": "GB/s", "n_gpus": world, "peak": peak,
                              "peak_kind": f"of {peak_kind}", "all_configs": rows}), flush=True)
        return
    results, ctx = measure_workload(B, wl, K, Wm, dev, world,
                                    [args.variant] + [v for v in ("carry", "two_pass") if v != args.variant],
                                    sampler, args.variant, momentum=args.momentum, quant_bits=args.quant_bits)
    eg, x0, grads, n_buf, buf_bytes = ctx
    extra = MOMENTUM_BYTES_PER_ELEMENT if args.momentum is not None else 0
    clocks = sampler.summary()
    elems = wl.P * wl.N
    main = results[args.variant]

    # end to end: host buffers in, updated parameters out, through eg_step_host
    e_steps = max(1, min(K, args.e2e_steps))
    xh = x0.cpu().pin_memory()
    gh = [grads[k % n_buf].cpu().pin_memory() for k in range(min(e_steps, 2))]
    eg.reset()
    eg.set_timing(False)
    eg.step_host(xh, gh[0], wl.lr)          # allocates the staging buffers
    xh.copy_(x0)
    eg.reset()
    barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for k in range(e_steps):
        eg.step_host(xh, gh[k % len(gh)], wl.lr)
    e_ms = (time.perf_counter() - t0) * 1e3
    e_units, e_ms_max = aggregate(float(elems) * e_steps, e_ms, dev)
    e2e = {"value": e_units * (BYTES_PER_ELEMENT[args.variant] + extra) / e_ms_max / 1e6, "unit": "GB/s",
           "h2d_bytes_per_step": 2 * buf_bytes, "d2h_bytes_per_step": buf_bytes,
           "steps": e_steps, "ms_per_step": e_ms_max / e_steps,
           "replica_steps_per_s": world * wl.P * e_steps / (e_ms_max / 1e3)}

    fused_ms = main["kernel_ms"]["fused"]
    achieved = elems * (FUSED_BYTES_PER_ELEMENT + extra) / fused_ms / 1e6 if fused_ms else None
    traffic = fused_traffic(wl, elems, args.momentum, args.quant_bits)
    roofline = {"bound": "hbm", "kernel": "k_fused_pipe" if args.momentum is None else "k_fused_pipe_momentum",
                "achieved": achieved, "peak": peak,
                "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                "frac": (achieved / peak) if achieved else None,
                **traffic,
                "algorithmic_bytes_per_launch": elems * (FUSED_BYTES_PER_ELEMENT + extra),
                "kernel_ms": fused_ms,
                "kernel_timed_in": "a second pass over the same K steps with CUDA events around every kernel "
                                   "group on the step's stream; the pass that gives `value` carries no events "
                                   "between its kernels",
                "ms_per_step_with_kernel_events": main["ms_per_step_with_kernel_events"],
                "step_frac_of_peak": main["gbs"] / peak,
                "step_frac_of_nominal_8TBs": main["gbs"] / NOMINAL_HBM_GBS}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        del grads
        torch.cuda.empty_cache()
        cpu = time_oracle(wl, steps=args.cpu_steps, warmup=1, budget_s=25.0, gen_device=str(dev),
                          single_thread_s=4.0, bytes_per_element=BYTES_PER_ELEMENT[args.variant] + extra)
        cpu = {k: cpu[k] for k in ("value", "unit", "cores", "kind", "sample", "replica_steps_per_s",
                                   "single_thread")}

    if rank == 0:
        line = {"metric": METRIC, "value": main["gbs"], "unit": "GB/s", "n_gpus": world,
                "steps": K, "warmup": Wm, "ms_per_step": main["ms_per_step"],
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                "data": "synthetic",
                "config": {"workload": wl.name, "P": wl.P, "tensors": wl.T, "elements": wl.N,
                           "variant": args.variant,
                           "bytes_per_element_step": BYTES_PER_ELEMENT[args.variant] + extra,
                           "momentum": args.momentum, "quant_bits": args.quant_bits,
                           "l2": "inputs larger than L2 (no flush needed)",
                           "gradient_buffers": n_buf, "multi_gpu": "replicas only"},
                "pct_of_peak": 100.0 * main["gbs"] / peak,
                "replica_steps_per_s": main["replica_steps_per_s"],
                "messages_sent": main["messages_sent"], "pct_messages": main["pct_messages"],
                "step_ms": main["step_ms"], "cuda_graph": False,
                "gpu_launches": main["launches"], "clocks": clocks, "e2e": e2e,
                "roofline": roofline, "cpu_baseline": cpu, "variants": results}
        print(json.dumps(line), flush=True)
    eg.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--config", type=int, default=3)
    ap.add_argument("--which", type=int, default=0)
    ap.add_argument("--variant", default="carry", choices=["carry", "two_pass"])
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-steps", type=int, default=10)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--all-configs", action="store_true",
                    help="time all five configurations (their own step counts) instead of the default one")
    ap.add_argument("--momentum", type=float, default=None,
                    help="heavy-ball momentum coefficient (default: plain SGD update, the paper's)")
    ap.add_argument("--quant-bits", type=int, default=None,
                    help="bits per element of quantised messages (default: messages in full precision, the paper's)")
    ap.add_argument("--max-elements", type=int, default=0,
                    help="keep only the leading tensors of the workload up to this many elements")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_native(args)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the RG-LRU temporal core on B200.

One "step" is one pass of the fused prefill path (Conv1D(4) -> gates -> log-space decay -> linear recurrence ->
state hand-off) over one batch of the training-shape workload (B=8, T=2048, D_RNN=2560, 10 heads, bf16 io, fp32
state).  The same JSON line also carries the batched decode step (B=512) and the backward as extra measurements.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
    python bench.py --only prefill|decode|backward [--B .. --T .. --D .. --H ..] [--iters n]    (one op, for profilers)

N > 1: one rank per GPU, each on its own seeded batch (sequences are independent: weak scaling, no data-path
collective); the time is the max over ranks.  Started without a rank environment, the script launches its own ranks
through torch.distributed.run.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2402_19427_b200 import inputs as synth, sharding  # noqa: E402

WORKLOAD = 1                 # index into synth.CONFIGS: the training-shape prefill
N_ROTATE = 4                 # distinct input/output buffer sets cycled between steps (defeats L2 reuse)
PREWARM_S = 0.1              # untimed launches of the step before the W warm-up steps (clock ramp, cold caches)
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes per prefill launch on the bench workload (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture,
# profiles/sm100_prefill_kernel_cfg1.md) together with the SHA-256 of the kernel source the capture was taken from:
# the figure is reported only while the benched kernel source still has that hash, else null.
NCU_TRAFFIC = {"bytes": 86849536 + 38148608, "kernel_sha256": "1e8f4cb69ef53ec5479321ebb194ff8b7163a5ba6daf54fb5ec124bd59118fd2"}
KERNEL_SOURCE = os.path.join(ROOT, "paper_2402_19427_b200", "csrc", "rglru_sm100.cu")


def captured_traffic():
    try:
        with open(KERNEL_SOURCE, "rb") as f:
            sha = hashlib.sha256(f.read()).hexdigest()
    except OSError:
        return None
    return NCU_TRAFFIC["bytes"] if sha == NCU_TRAFFIC["kernel_sha256"] else None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def algorithmic_work(cfg):
    """Bytes that must cross HBM and gate FLOPs for one prefill launch: x in + y out + every parameter once +
    state in/out; gates are two [tokens x Dh] . [Dh x Dh] products per head = 4*Dh FLOP per element."""
    B, T, D, H = cfg["B"], cfg["T"], cfg["D"], cfg["H"]
    Dh = D // H
    io = 2 if cfg["io"] == "bf16" else 4
    elems = B * T * D
    nbytes = 2 * elems * io + (4 * D + 2 * H * Dh * Dh) * io + 4 * D * 4 + B * D * 4 + B * 3 * D * io
    flops = elems * 4 * Dh
    return nbytes, flops


def roofline(nbytes, flops, launch_s, peaks, peak_kind, traffic=None):
    """The slower of (bytes at the copy rate, FLOPs at the tensor rate) is the bound; achieved = that quantity / time."""
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
    t_tc = flops / (peaks["bf16_tflops"] * 1e12)
    if t_tc >= t_hbm:
        roof = {"bound": "tensor", "achieved": flops / launch_s / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
    else:
        roof = {"bound": "hbm", "achieved": nbytes / launch_s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = traffic
    roof.update({"peaks": peak_kind, "launch_us": launch_s * 1e6, "hbm_gbs_achieved": nbytes / launch_s / 1e9,
                 "hbm_frac": nbytes / launch_s / 1e9 / peaks["hbm_gbs"], "tensor_tflops_achieved": flops / launch_s / 1e12,
                 "tensor_frac": flops / launch_s / 1e12 / peaks["bf16_tflops"], "algorithmic_bytes": nbytes, "gate_flops": flops,
                 # for context only: the same work against the data-sheet figures (8 TB/s, 2.25 PFLOP/s dense bf16)
                 "frac_of_nominal": max(nbytes / 8.0e12, flops / 2.25e15) / launch_s})
    return roof


def event_times_us(fn, reps, torch):
    """Runs fn() reps times, each between its own pair of CUDA events on the current stream; returns the times in us."""
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for a, b in evs:
        a.record(); fn(); b.record()
    torch.cuda.synchronize()
    return [a.elapsed_time(b) * 1e3 for a, b in evs]


def graph_times_us(fn, calls, reps, torch):
    """fn(i), i = 0 .. calls - 1, is captured once in a CUDA graph (the calls must allocate nothing); the graph is replayed
    reps times, each replay between its own pair of CUDA events.  Returns the times per call in us."""
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        fn(0)
        with torch.cuda.graph(graph, stream=side):
            for i in range(calls):
                fn(i)
    torch.cuda.current_stream().wait_stream(side)
    graph.replay()
    torch.cuda.synchronize()
    return [t / calls for t in event_times_us(graph.replay, reps, torch)]


def time_prefill_config(binding, dev, index, peaks, peak_kind, reps=20, heads=None, merged=False):
    """One of the other prefill shapes as a side record: `reps` launches over rotating buffer sets, median and min.  `heads`
    overrides the head count of the config (the paper's 16 blocks); `merged` adds the gate branch of the recurrent block
    (y = h GeLU(branch), one more bf16 read per element) and the decay-product output."""
    import torch
    cfg = dict(synth.CONFIGS[index])
    if heads is not None:
        cfg["H"] = heads
    B, T, D, H = cfg["B"], cfg["T"], cfg["D"], cfg["H"]
    dt = torch.bfloat16
    pr = synth.make_inputs(1, 4, D, H, io="bf16", seed=synth.BASE_SEED + index)["params"]
    params = binding.Params.from_numpy(pr, "bf16", device=dev)
    nset = max(2, int(np.ceil(300e6 / (2 * B * T * D * 2))))     # input + output of all sets exceed the 126 MB L2 twice over
    g = torch.Generator(device=dev); g.manual_seed(index)
    xs = [torch.randn(B, T, D, device=dev, generator=g).to(dt) for _ in range(nset)]
    ys = [torch.empty_like(xs[0]) for _ in range(nset)]
    shape = binding.make_shape(B, T, D, H, dt)
    ws = binding.alloc_workspace(shape, binding.OP_PREFILL, dev)
    hT = torch.empty(B, D, dtype=torch.float32, device=dev)
    cso = torch.empty(B, 3, D, dtype=dt, device=dev)
    gbs = [torch.randn(B, T, D, device=dev, generator=g).to(dt) for _ in range(nset)] if merged else None
    ap = torch.empty(B, D, dtype=torch.float32, device=dev) if merged else None

    def one(i):
        binding.prefill(xs[i % nset], params, y=ys[i % nset], h_T=hT, conv_state_out=cso, workspace=ws,
                        gate_branch=gbs[i % nset] if merged else None, a_prod=ap)

    for i in range(3):
        one(i)
    torch.cuda.synchronize()
    us = graph_times_us(one, 2 * nset, reps, torch)     # 2 * nset calls per replay, rotating over the buffer sets
    status = binding.query_status(ws)
    if status != binding.OK:
        raise binding.RglruError(status, "device status after the side measurement")
    nbytes, flops = algorithmic_work(cfg)
    if merged:
        nbytes += B * T * D * 2 + B * D * 4
    med = float(np.median(us))
    return {"workload": workload_name(cfg) + (" + gate branch (GeLU merge) and decay product" if merged else ""), "us_median": med, "us_min": float(np.min(us)), "reps": reps,
            "launch": f"{2 * nset} calls per CUDA-graph replay",
            "tokens_per_s": B * T / (med * 1e-6), "buffer_sets": nset, "roofline": roofline(nbytes, flops, med * 1e-6, peaks, peak_kind)}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or nv.nvmlDeviceGetCurrentClocksThrottleReasons
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(get_reasons(self.h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        if self.nv is not None and not self.samples:
            # a timed region of a millisecond or two can end before the thread's first NVML call returns: take that sample now,
            # directly after the region, while the clocks are still those of the load
            self._stop.clear()
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
            except Exception:
                pass
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def time_oracle(cfg, seed, heads):
    """Times the fp64 oracle, as it stands, on `heads` of the workload's H heads for every sequence and token (heads are
    independent, so this is heads/H of one step).  Returns (tokens/s scaled to full-width tokens, seconds, threads, text)."""
    import oracle
    Dh = cfg["D"] // cfg["H"]
    inp = synth.make_inputs(cfg["B"], cfg["T"], Dh * heads, heads, io=cfg["io"], seed=seed)
    p64 = {k: np.asarray(v, np.float64) for k, v in inp["params"].items()}
    x64 = inp["x"].astype(np.float64)
    t0 = time.perf_counter()
    oracle.prefill(x64, p64, heads, c=inp["c"])
    dt = time.perf_counter() - t0
    tokens_equiv = cfg["B"] * cfg["T"] * heads / cfg["H"]      # full-width tokens' worth of work in the sample
    what = (f"all {cfg['B']} sequences x {cfg['T']} tokens of {heads} of {cfg['H']} heads ({heads}/{cfg['H']} of a step), "
            f"fp64, sequential in time")
    return tokens_equiv / dt, dt, oracle.num_threads(), what


def run_reference(args):
    """The reference arm is the CPU oracle (there is no reference implementation to install).  Each step is a bounded
    sample of the workload -- some of its heads -- sized so that the whole run stays within a few minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = dict(synth.CONFIGS[WORKLOAD])
    seed = synth.BASE_SEED + WORKLOAD
    _, t_head, _, _ = time_oracle(cfg, seed, 1)               # untimed probe: cost of one head
    budget_s = 150.0
    heads = int(max(1, min(cfg["H"], budget_s / max(t_head, 1e-3) / (args.steps + args.warmup))))
    times, sample, cores = [], "", 0
    for i in range(args.warmup + args.steps):
        tps, dt, cores, sample = time_oracle(cfg, seed, heads)
        if i >= args.warmup:
            times.append(dt)
    mean_dt = float(np.mean(times))
    value = cfg["B"] * cfg["T"] * heads / cfg["H"] / mean_dt
    line = {"impl": "reference", "metric": "rglru_prefill_tokens_per_s", "value": value, "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": mean_dt * 1e3 * cfg["H"] / heads,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_name(cfg)},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_name(cfg):
    return (f"{cfg['name']}: B={cfg['B']} T={cfg['T']} D_RNN={cfg['D']} H={cfg['H']} (head width {cfg['D'] // cfg['H']}), "
            f"{cfg['io']} io, fp32 state, c=8")


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2402_19427_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0 or world == 1:
        from paper_2402_19427_b200 import build
        build.build()  # no-op when the library is up to date
    if world > 1:
        dist.barrier()
    binding.load()  # fails loudly if the CUDA library is missing

    cfg = dict(synth.CONFIGS[WORKLOAD])
    B, T, D, H = cfg["B"], cfg["T"], cfg["D"], cfg["H"]
    dt = torch.bfloat16
    base = synth.make_config(WORKLOAD, seed=sharding.rank_seed(synth.BASE_SEED + WORKLOAD, rank))
    params = binding.Params.from_numpy(base["params"], cfg["io"], device=dev)
    rng = np.random.Generator(np.random.PCG64(99 + rank))
    xs_host = [base["x"]] + [synth.round_to_bf16(rng.standard_normal((B, T, D), dtype=np.float32)) for _ in range(N_ROTATE - 1)]
    xs = [torch.from_numpy(a).to(dev, dt).contiguous() for a in xs_host]
    ys = [torch.empty_like(x) for x in xs]
    hT = torch.empty(B, D, dtype=torch.float32, device=dev)
    cso = torch.empty(B, 3, D, dtype=dt, device=dev)
    shape = binding.make_shape(B, T, D, H, dt)
    ws = binding.alloc_workspace(shape, binding.OP_PREFILL, dev)

    def step(i):
        k = i % N_ROTATE
        binding.prefill(xs[k], params, y=ys[k], h_T=hT, conv_state_out=cso, workspace=ws)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # The K timed steps are K calls of the public API captured once in a CUDA graph and replayed: the calls allocate nothing
    # (outputs and workspace are passed in), and a graph takes the host's launch cost and the gap between consecutive
    # cooperative launches out of the measurement (measured: 86 against 91 us per step with plain stream launches, which are
    # timed as well and reported beside it).  Everything that costs host time (NVML set-up, event creation, the capture)
    # happens before the warm-up, so that the GPU does not sit idle between the warm-up and the timed region; the warm-up
    # itself is preceded by untimed launches of the same step for PREWARM_S seconds, which brings clocks and caches to their
    # steady state whatever K and W are.
    sampler = ClockSampler(local)
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step(0)
        with torch.cuda.graph(graph, stream=side):
            for i in range(args.steps):
                step(i)
    torch.cuda.current_stream().wait_stream(side)
    graph.replay()   # untimed: the first launch of a graph also uploads it to the device
    torch.cuda.synchronize()
    t_pre = time.perf_counter()
    n_pre = 0
    while time.perf_counter() - t_pre < PREWARM_S:
        for i in range(8):
            step(n_pre + i)
        n_pre += 8
        torch.cuda.synchronize()
    for i in range(args.warmup):
        step(i)
    barrier()
    sampler.start()
    g0.record()
    graph.replay()
    g1.record()
    barrier()
    clocks = sampler.stop()
    total_ms = g0.elapsed_time(g1)
    # the same K steps as plain launches on the stream, each between two events (side record)
    barrier()
    evs[0].record()
    for i in range(args.steps):
        step(i)
        evs[i + 1].record()
    barrier()
    stream_total_ms = evs[0].elapsed_time(evs[-1])
    per_launch_ms = [evs[i].elapsed_time(evs[i + 1]) for i in range(args.steps)]
    status = binding.query_status(ws)
    if status != binding.OK:
        raise binding.RglruError(status, "device status after timed region")
    total_ms = sharding.max_over_ranks(total_ms, dist if world > 1 else None, dev)
    ms_per_step = total_ms / args.steps
    value = world * B * T / (ms_per_step * 1e-3)

    # ---- end to end through the host-buffer entry point: pinned host x -> device -> kernel -> pinned host y
    x_pin = [torch.from_numpy(a).to(dt).pin_memory() for a in xs_host[:2]]
    y_pin = [torch.empty(B, T, D, dtype=dt).pin_memory() for _ in range(2)]
    hT_pin = torch.empty(B, D, dtype=torch.float32).pin_memory()
    cs_pin = torch.empty(B, 3, D, dtype=dt).pin_memory()
    staging = torch.empty(binding.host_staging_bytes(shape), dtype=torch.uint8, device=dev)
    e2e_steps = max(3, min(args.steps, 20))

    def e2e_step(i):
        binding.prefill_host(x_pin[i % 2], params, y_pin[i % 2], hT_pin, cs_pin, staging, ws)

    for i in range(3):
        e2e_step(i)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(e2e_steps):
        e2e_step(i)
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    e2e_ms = sharding.max_over_ranks(e2e_ms, dist if world > 1 else None, dev)
    # the e2e result must be the same computation: spot check against the device-resident run
    torch.cuda.synchronize()
    k = (e2e_steps - 1) % 2
    ref_y, _, _ = binding.prefill(xs[k], params, workspace=ws)
    torch.cuda.synchronize()
    # chunks of sequences run with their own time split, so sums associate differently: compare within the parity tolerance
    a64, b64 = y_pin[k].double(), ref_y.cpu().double()
    rms = float(b64.pow(2).mean().sqrt())
    if not bool(((a64 - b64).abs() <= 2e-2 * torch.clamp(b64.abs(), min=rms)).all()):
        raise RuntimeError("host-buffer entry point disagrees with the device entry point")
    io_b = 2
    h2d = B * T * D * io_b
    d2h = B * T * D * io_b + B * D * 4 + B * 3 * D * io_b

    peaks, peak_kind = load_peaks()
    nbytes, flops = algorithmic_work(cfg)
    launch_s = total_ms / args.steps * 1e-3   # average duration of the kernel over the timed region (one kernel per step)
    roof = roofline(nbytes, flops, launch_s, peaks, peak_kind, traffic=captured_traffic())
    roof["kernel"] = "rglru prefill (dominant kernel of the step)"

    extra = {}
    if rank == 0 and not args.no_extras:
        # the other prefill shapes: the long sequence (every tile through the decoupled look-back) and the training shape of config 4
        extra["prefill_long"] = time_prefill_config(binding, dev, 2, peaks, peak_kind)
        extra["prefill_cfg4_forward"] = time_prefill_config(binding, dev, 4, peaks, peak_kind)
        # the bench shape with the paper's 16 blocks (head width 160, one head per 256 channel slots), and with the merged output
        extra["prefill_16_blocks"] = time_prefill_config(binding, dev, WORKLOAD, peaks, peak_kind, heads=16)
        extra["prefill_gelu_merge"] = time_prefill_config(binding, dev, WORKLOAD, peaks, peak_kind, merged=True)
        extra.update(measure_extras(binding, dev, peaks))

    if rank == 0:
        line = {"metric": "rglru_prefill_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": workload_name(cfg), "parallelism": f"batch-sharded x{world}, no collective",
                           "l2": f"{N_ROTATE} rotating input/output buffer sets ({N_ROTATE * 2 * B * T * D * 2 / 1e6:.0f} MB) > 126 MB L2",
                           "prewarm": f"{PREWARM_S * 1e3:.0f} ms of untimed launches of the step before the {args.warmup} warm-up steps",
                           "launch": f"the {args.steps} timed steps are {args.steps} API calls captured in one CUDA graph and replayed once",
                           "kernel_path": "sm100" if binding.workspace_bytes(shape, binding.OP_PREFILL) > 256 else "generic"},
                "clocks": clocks, "gpu_launches": args.steps,
                "e2e": {"value": world * B * T / (e2e_ms * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                        "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps},
                "roofline": roof,
                "stream_launches": {"what": "the same steps as plain launches on the stream, one event pair per step",
                                    "ms_per_step": stream_total_ms / args.steps, "ms_per_launch_median": float(np.median(per_launch_ms)),
                                    "ms_per_launch_min": float(np.min(per_launch_ms))}}
        if world == 1 and not args.no_cpu_baseline:
            tps, dt_s, cores, sample = time_oracle(cfg, synth.BASE_SEED + WORKLOAD, cfg["H"])   # one whole step
            line["cpu_baseline"] = {"value": tps, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample,
                                    "seconds": dt_s}
        line.update(extra)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def measure_extras(binding, dev, peaks):
    """Decode (B=512, 256 chained steps from a prefilled state) and backward (B=4, T=4096, D=4096), each timed on the device."""
    import torch
    out = {}
    dt = torch.bfloat16
    # ---- batched decode
    c3 = synth.CONFIGS[3]
    B, D, H, steps = c3["B"], c3["D"], c3["H"], c3["decode_steps"]
    p3 = synth.make_inputs(1, 4, D, H, io="bf16", seed=synth.BASE_SEED + 3)["params"]
    params = binding.Params.from_numpy(p3, "bf16", device=dev)
    g = torch.Generator(device=dev); g.manual_seed(3)
    xs = torch.randn(steps, B, D, device=dev, generator=g).to(dt)
    h = torch.randn(B, D, device=dev, generator=g)
    cs = torch.randn(B, 3, D, device=dev, generator=g).to(dt)
    y = torch.empty(B, D, dtype=dt, device=dev)
    shape = binding.make_shape(B, 1, D, H, dt)
    ws = binding.alloc_workspace(shape, binding.OP_DECODE, dev)

    def chain():
        for t in range(steps):
            binding.decode_step(xs[t], params, h, cs, y=y, workspace=ws)

    chain(); torch.cuda.synchronize()
    reps = 20
    us_plain_all = [t / steps for t in event_times_us(chain, reps, torch)]

    def graph_of(fn):
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()
            with torch.cuda.graph(graph, stream=side):
                fn()
        torch.cuda.current_stream().wait_stream(side)
        graph.replay(); torch.cuda.synchronize()
        return graph

    # the same chain captured once in a CUDA graph (launch overhead off the critical path); one state set: h and the conv
    # state (13 MB) stay in the 126 MB L2 between steps
    graph = graph_of(chain)
    us_graph_all = [t / steps for t in event_times_us(graph.replay, reps, torch)]
    # the same number of steps over rotating state sets that together exceed L2 several times, so that every step's h and
    # conv state come from and go to HBM (a server with many resident sequence groups)
    nsets = 32
    hs = [torch.randn(B, D, device=dev, generator=g) for _ in range(nsets)]
    css = [torch.randn(B, 3, D, device=dev, generator=g).to(dt) for _ in range(nsets)]
    ysr = [torch.empty(B, D, dtype=dt, device=dev) for _ in range(nsets)]

    def chain_rot():
        for t in range(steps):
            binding.decode_step(xs[t], params, hs[t % nsets], css[t % nsets], y=ysr[t % nsets], workspace=ws)

    graph_rot = graph_of(chain_rot)
    us_rot_all = [t / steps for t in event_times_us(graph_rot.replay, reps, torch)]
    Dh = D // H
    dec_bytes = B * D * 2 * 2 + B * D * 4 * 2 + B * 3 * D * 2 + B * D * 2 + (4 * D + 2 * H * Dh * Dh) * 2 + 4 * D * 4
    us_plain, us_graph, us_rot = float(np.median(us_plain_all)), float(np.median(us_graph_all)), float(np.median(us_rot_all))
    set_mb = (B * D * 4 + B * 3 * D * 2 + B * D * 2) / 1e6
    out["decode"] = {"workload": f"B={B} D_RNN={D} H={H} bf16 io, fp32 h, {steps} chained steps", "reps": reps,
                     "algorithmic_bytes_per_step": dec_bytes,
                     "state_in_hbm": {"what": f"{nsets} rotating state sets ({nsets * set_mb:.0f} MB) > L2, CUDA graph",
                                      "us_per_step_median": us_rot, "us_per_step_min": float(np.min(us_rot_all)),
                                      "steps_per_s": 1e6 / us_rot, "tokens_per_s": B * 1e6 / us_rot,
                                      "hbm_gbs_achieved": dec_bytes / (us_rot * 1e-6) / 1e9,
                                      "roofline_frac": dec_bytes / (us_rot * 1e-6) / 1e9 / peaks["hbm_gbs"]},
                     "state_in_l2": {"what": f"one state set ({set_mb:.0f} MB) that stays in L2 between steps, CUDA graph",
                                     "us_per_step_median": us_graph, "us_per_step_min": float(np.min(us_graph_all)),
                                     "steps_per_s": 1e6 / us_graph, "tokens_per_s": B * 1e6 / us_graph,
                                     "hbm_gbs_equivalent": dec_bytes / (us_graph * 1e-6) / 1e9,
                                     "roofline_frac": dec_bytes / (us_graph * 1e-6) / 1e9 / peaks["hbm_gbs"]},
                     "us_per_step_plain_launches": us_plain, "us_per_step_plain_launches_min": float(np.min(us_plain_all))}
    del hs, css, ysr
    del xs, h, cs, y
    # ---- backward
    c4 = synth.CONFIGS[4]
    B, T, D, H = c4["B"], c4["T"], c4["D"], c4["H"]
    Dh = D // H
    p4 = synth.make_inputs(1, 4, D, H, io="bf16", seed=synth.BASE_SEED + 4)["params"]
    params = binding.Params.from_numpy(p4, "bf16", device=dev)
    x = torch.randn(B, T, D, device=dev, generator=g).to(dt)
    dy = torch.randn(B, T, D, device=dev, generator=g).to(dt)
    shape = binding.make_shape(B, T, D, H, dt)
    ws = binding.alloc_workspace(shape, binding.OP_BACKWARD, dev)
    y_saved, _, _ = binding.prefill(x, params)          # a training step keeps the forward output for the backward
    grads = binding.backward(x, params, dy, y=y_saved, workspace=ws)     # also allocates the gradient tensors reused below
    binding.backward(x, params, dy, y=y_saved, workspace=ws, out=grads)
    torch.cuda.synchronize()
    # one call (a dozen kernels) captured in a CUDA graph and replayed, as a training step would run it
    ms_all = [t * 1e-3 for t in graph_times_us(lambda i: binding.backward(x, params, dy, y=y_saved, workspace=ws, out=grads), 1, 20, torch)]
    ms = float(np.median(ms_all))
    bwd_flops = B * T * D * 12 * Dh
    bwd_bytes = B * T * D * 2 * 4
    out["backward"] = {"workload": f"B={B} T={T} D_RNN={D} H={H} bf16 io, forward output saved", "reps": 20,
                       "launch": "one call per CUDA-graph replay",
                       "tokens_per_s": B * T / (ms * 1e-3), "ms": ms, "ms_min": float(np.min(ms_all)),
                       "gate_flops": bwd_flops, "minimum_bytes": bwd_bytes,
                       "gate_tflops_achieved": bwd_flops / (ms * 1e-3) / 1e12,
                       "roofline_frac": bwd_flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"]}
    return out


def run_only(args):
    """One op a few times on a seeded synthetic workload of the given shape; meant to be wrapped in a profiler.  Prints the
    median CUDA-event time of the calls after the first.  With --impl reference (prefill only) the CPU oracle is timed on
    one head of the same shape instead, which is 1/H of the work."""
    if args.impl == "reference":
        cfg = dict(synth.CONFIGS[1])
        cfg.update(B=args.B or cfg["B"], T=args.T or cfg["T"], D=args.D or cfg["D"], H=args.H or cfg["H"])
        tps, dt, cores, what = time_oracle(cfg, synth.BASE_SEED, 1)
        print(json.dumps({"only": "prefill", "impl": "reference", "B": cfg["B"], "T": cfg["T"], "D": cfg["D"], "H": cfg["H"],
                          "tokens_per_s": tps, "seconds": dt, "cores": cores, "sample": what}))
        return
    import torch
    from paper_2402_19427_b200 import binding, build
    build.build()
    binding.load()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    dt = torch.bfloat16
    cfg = dict(synth.CONFIGS[{"prefill": 1, "decode": 3, "backward": 4}[args.only]])
    B, T, D, H = args.B or cfg["B"], args.T or cfg.get("T", 1), args.D or cfg["D"], args.H or cfg["H"]
    pr = synth.make_inputs(1, 4, D, H, io="bf16", seed=1)["params"]
    params = binding.Params.from_numpy(pr, "bf16", device=dev)
    g = torch.Generator(device=dev); g.manual_seed(0)
    ev = []
    if args.only == "decode":
        x = torch.randn(B, D, device=dev, generator=g).to(dt)
        h = torch.randn(B, D, device=dev, generator=g)
        cs = torch.randn(B, 3, D, device=dev, generator=g).to(dt)
        for _ in range(args.iters):
            ev.append((torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)))
            ev[-1][0].record(); binding.decode_step(x, params, h, cs); ev[-1][1].record()
    else:
        xs = [torch.randn(B, T, D, device=dev, generator=g).to(dt) for _ in range(2)]
        ys = [torch.empty_like(xs[0]) for _ in range(2)]
        if args.only == "prefill":
            shape = binding.make_shape(B, T, D, H, dt)
            ws = binding.alloc_workspace(shape, binding.OP_PREFILL, dev)
            for i in range(args.iters):
                ev.append((torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)))
                ev[-1][0].record(); binding.prefill(xs[i % 2], params, y=ys[i % 2], workspace=ws); ev[-1][1].record()
            if binding.query_status(ws) != binding.OK:
                raise RuntimeError("device status")
        else:
            for i in range(args.iters):
                dy = ys[0].normal_()
                ev.append((torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)))
                ev[-1][0].record(); binding.backward(xs[i % 2], params, dy); ev[-1][1].record()
    torch.cuda.synchronize()
    us = sorted(a.elapsed_time(b) * 1e3 for a, b in ev[1:]) or [float("nan")]
    print(json.dumps({"only": args.only, "B": B, "T": T, "D": D, "H": H, "iters": args.iters, "us_per_call_median": us[len(us) // 2],
                      "us_per_call_min": us[0], "tokens_per_s": B * T * 1e6 / us[len(us) // 2]}))


def launch_command(args, argv):
    """The torch.distributed.run command that starts one rank of this script per GPU on this node."""
    port = int(os.environ.get("MASTER_PORT", "29531"))
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the side measurements (other prefill shapes, decode, backward)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--launch-dry-run", action="store_true", help="print the command that would start the ranks, and this process's rank environment")
    ap.add_argument("--only", choices=["prefill", "decode", "backward"], help="run one op a few times and exit (for profilers)")
    ap.add_argument("--B", type=int); ap.add_argument("--T", type=int); ap.add_argument("--D", type=int); ap.add_argument("--H", type=int)
    ap.add_argument("--iters", type=int, default=3)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.only:
        run_only(args)
        return
    have_ranks = "RANK" in os.environ and "WORLD_SIZE" in os.environ
    if args.launch_dry_run:
        argv = [a for a in sys.argv[1:] if a != "--launch-dry-run"]
        print(json.dumps({"gpus": args.gpus, "self_launch": args.gpus > 1 and not have_ranks,
                          "command": launch_command(args, argv) if args.gpus > 1 and not have_ranks else None,
                          "env": {k: os.environ.get(k) for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}}))
        return
    if args.gpus > 1 and not have_ranks:
        # started as a plain script: become the launcher of one rank per GPU; rank 0 prints the JSON line
        sys.exit(subprocess.call(launch_command(args, sys.argv[1:])))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

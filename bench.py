#!/usr/bin/env python
"""Benchmark of the RG-LRU temporal core on B200.

One "step" is one pass of the fused prefill path (Conv1D(4) -> gates -> log-space decay -> linear recurrence ->
state hand-off) over one batch of the training-shape workload (B=8, T=2048, D_RNN=2560, 10 heads, bf16 io, fp32
state).  The same JSON line also carries the batched decode step (B=512) and the backward as extra measurements.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 is launched with torch.distributed.run, one rank per GPU; sequences are independent, so each rank runs the
full workload on its own seeded batch (weak scaling, no data-path collective); the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
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
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes per prefill launch on the bench workload from the committed ncu capture
# (dram__bytes_read.sum + dram__bytes_write.sum); None until a capture exists.
NCU_TRAFFIC_BYTES = 132525056   # 86.90 MB read + 45.63 MB written (profiles/sm100_prefill_kernel_cfg1.md)


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

    for i in range(args.warmup):
        step(i)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    barrier()
    evs[0].record()
    for i in range(args.steps):
        step(i)
        evs[i + 1].record()
    barrier()
    clocks = sampler.stop()
    total_ms = evs[0].elapsed_time(evs[-1])
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
    launch_s = float(np.mean(per_launch_ms)) * 1e-3
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
    t_tc = flops / (peaks["bf16_tflops"] * 1e12)
    if t_tc >= t_hbm:
        roof = {"bound": "tensor", "achieved": flops / launch_s / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
    else:
        roof = {"bound": "hbm", "achieved": nbytes / launch_s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = NCU_TRAFFIC_BYTES
    roof.update({"peaks": peak_kind, "kernel": "rglru prefill (dominant kernel of the step)",
                 "launch_us": launch_s * 1e6, "hbm_gbs_achieved": nbytes / launch_s / 1e9,
                 "hbm_frac": nbytes / launch_s / 1e9 / peaks["hbm_gbs"], "tensor_tflops_achieved": flops / launch_s / 1e12,
                 "tensor_frac": flops / launch_s / 1e12 / peaks["bf16_tflops"], "algorithmic_bytes": nbytes, "gate_flops": flops,
                 # for context only: the same work against the data-sheet figures (8 TB/s, 2.25 PFLOP/s dense bf16)
                 "frac_of_nominal": max(nbytes / 8.0e12, flops / 2.25e15) / launch_s})

    extra = {}
    if rank == 0 and not args.no_extras:
        extra = measure_extras(binding, dev, peaks)

    if rank == 0:
        line = {"metric": "rglru_prefill_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": workload_name(cfg), "parallelism": f"batch-sharded x{world}, no collective",
                           "l2": f"{N_ROTATE} rotating input/output buffer sets ({N_ROTATE * 2 * B * T * D * 2 / 1e6:.0f} MB) > 126 MB L2",
                           "kernel_path": "sm100" if binding.workspace_bytes(shape, binding.OP_PREFILL) > 256 else "generic"},
                "clocks": clocks, "gpu_launches": args.steps,
                "e2e": {"value": world * B * T / (e2e_ms * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                        "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps},
                "roofline": roof}
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
    reps = 3
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        chain()
    e1.record(); torch.cuda.synchronize()
    us_plain = e0.elapsed_time(e1) * 1e3 / (reps * steps)
    # the same chain captured once in a CUDA graph (launch overhead off the critical path)
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        chain()
        with torch.cuda.graph(graph, stream=side):
            chain()
    torch.cuda.current_stream().wait_stream(side)
    graph.replay(); torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        graph.replay()
    e1.record(); torch.cuda.synchronize()
    us_graph = e0.elapsed_time(e1) * 1e3 / (reps * steps)
    us = min(us_plain, us_graph)
    Dh = D // H
    dec_bytes = B * D * 2 * 2 + B * D * 4 * 2 + B * 3 * D * 2 + B * D * 2 + (4 * D + 2 * H * Dh * Dh) * 2 + 4 * D * 4
    out["decode"] = {"workload": f"B={B} D_RNN={D} H={H} bf16 io, fp32 h, {steps} chained steps", "steps_per_s": 1e6 / us,
                     "tokens_per_s": B * 1e6 / us, "us_per_step_plain_launches": us_plain, "us_per_step_cuda_graph": us_graph,
                     "algorithmic_bytes_per_step": dec_bytes, "hbm_gbs_achieved": dec_bytes / (us * 1e-6) / 1e9,
                     "roofline_frac": dec_bytes / (us * 1e-6) / 1e9 / peaks["hbm_gbs"]}
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
    binding.backward(x, params, dy, y=y_saved, workspace=ws); torch.cuda.synchronize()
    e0.record()
    binding.backward(x, params, dy, y=y_saved, workspace=ws)
    e1.record(); torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    bwd_flops = B * T * D * 12 * Dh
    out["backward"] = {"workload": f"B={B} T={T} D_RNN={D} H={H} bf16 io, forward output saved", "tokens_per_s": B * T / (ms * 1e-3), "ms": ms,
                       "gate_tflops_achieved": bwd_flops / (ms * 1e-3) / 1e12,
                       "roofline_frac": bwd_flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"]}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the decode and backward side measurements")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

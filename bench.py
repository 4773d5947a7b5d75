#!/usr/bin/env python
"""Benchmark of the forward-convolution hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-general]

One "step" is one pass of the single-channel hot path over the large single-channel
configuration (1 x 1 x 4096 x 4096 image, 32 filters of 5 x 5): filter staging, tile staging,
register-window FMA loop and vector stores, all inside conv2d_fwd_single_channel.  The general-case
configurations are timed as well (tensor-core and fp32 variants) and reported under "general" in the
same JSON line.  Prints exactly one JSON line on stdout (rank 0).

Multi-GPU: the path has no exchange step; with --gpus N every rank runs an independent replica of the
workload on its own GPU (weak scaling, no collective on the data path).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import numpy as np  # noqa: E402

from workloads import CONFIGS, make_inputs  # noqa: E402

SM_COUNT = 148
FP32_LANES_PER_SM = 128
TF32_FLOP_PER_CLK_PER_SM = 4096     # dense TF32 = half the bf16 rate per clock
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_TF32_TFLOPS = 1125.0
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0


def load_peaks():
    path = ROOT / "MEASURED_PEAKS.json"
    if path.exists():
        p = json.loads(path.read_text())
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    sm_max_mhz=float(p.get("sm_max_mhz", 1965.0)), source="measured")
    return dict(hbm_gbs=FALLBACK_HBM_GBS, bf16_tflops=FALLBACK_BF16_TFLOPS, bf16_tflops_sustained=1400.0,
                sm_max_mhz=1965.0, source="fallback")


class ClockSampler:
    """Samples SM clock, power and throttle reasons through NVML in a thread while the timed region runs."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, gpu_index: int, period_s: float = 0.002):
        self.gpu_index, self.period_s = gpu_index, period_s
        self.samples, self.reasons, self.power = [], set(), []
        self.sm_max = None
        self._stop = False
        self._thread = None
        self._active = False

    def _run(self, nv, handle):
        while not self._stop:
            if self._active:
                try:
                    self.samples.append(nv.nvmlDeviceGetClockInfo(handle, nv.NVML_CLOCK_SM))
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(handle)
                    for bit, name in self.REASONS.items():
                        if mask & bit:
                            self.reasons.add(name)
                    self.power.append(nv.nvmlDeviceGetPowerUsage(handle) / 1000.0)
                except Exception:
                    pass
            time.sleep(self.period_s)

    def start(self):
        """Starts the thread (idle); mark the timed region with begin()/end()."""
        try:
            import threading
            import pynvml as nv
            nv.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            index = self.gpu_index
            if visible:
                ids = [v.strip() for v in visible.split(",") if v.strip()]
                if self.gpu_index < len(ids) and ids[self.gpu_index].isdigit():
                    index = int(ids[self.gpu_index])
            handle = nv.nvmlDeviceGetHandleByIndex(index)
            self.sm_max = nv.nvmlDeviceGetMaxClockInfo(handle, nv.NVML_CLOCK_SM)
            self._thread = threading.Thread(target=self._run, args=(nv, handle), daemon=True)
            self._thread.start()
        except Exception:
            self._thread = None

    def begin(self):
        self._active = True

    def end(self):
        self._active = False

    def stop(self) -> dict:
        self._stop = True
        if self._thread is not None:
            self._thread.join(timeout=2)
        out = {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": sorted(self.reasons), "samples": len(self.samples),
               "power_w_max": max(self.power) if self.power else None}
        if self.samples:
            out["sm_mhz"] = statistics.median(self.samples)
        return out


def cpu_model():
    try:
        for line in Path("/proc/cpuinfo").read_text().splitlines():
            if line.startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def time_oracle_sample(cfg, target_seconds: float):
    """Times the oracle, as it stands, on a bounded sample of output maps of `cfg`."""
    import oracle
    x, w = make_inputs(cfg)
    flops_per_map = 2 * cfg.N * cfg.C * cfg.R * cfg.S * cfg.P * cfg.Q
    t0 = time.perf_counter()
    oracle.conv2d_oracle_range(x, w, k_range=(0, 1))
    t1 = time.perf_counter() - t0
    maps = int(max(1, min(cfg.K - 1, round(target_seconds / max(t1, 1e-6)))))
    t0 = time.perf_counter()
    oracle.conv2d_oracle_range(x, w, k_range=(1, 1 + maps))
    t = time.perf_counter() - t0
    return dict(value=flops_per_map * maps / t / 1e9, unit="GFLOP/s", cores=oracle.oracle_threads(),
                kind="oracle", sample=f"{cfg.name}: all outputs of {maps}/{cfg.K} maps, {t:.1f} s")


def run_reference(args, rank: int):
    """The reference arm: the CPU oracle on the host cores, bounded sample per step."""
    if rank != 0:
        return
    import oracle
    cfg = CONFIGS[args.workload]
    x, w = make_inputs(cfg)
    maps = 2
    flops = 2 * cfg.N * cfg.C * cfg.R * cfg.S * cfg.P * cfg.Q * maps
    for _ in range(min(args.warmup, 1)):
        oracle.conv2d_oracle_range(x, w, k_range=(0, maps))
    steps = min(args.steps, 5)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.conv2d_oracle_range(x, w, k_range=(0, maps))
    t = (time.perf_counter() - t0) / steps
    val = flops / t / 1e9
    sample = f"{cfg.name}: all outputs of {maps} of {cfg.K} maps per step, {cpu_model()}"
    print(json.dumps({
        "impl": "reference", "metric": "conv_fwd_gflops", "value": val, "unit": "GFLOP/s",
        "n_gpus": args.gpus, "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": t * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, **cfg.as_dict()},
        "cpu_baseline": {"value": val, "unit": "GFLOP/s", "cores": oracle.oracle_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": val, "unit": "GFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def event_ms(fn, torch, iters=1):
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(iters):
        fn()
    stop.record()
    stop.synchronize()
    return start.elapsed_time(stop) / iters


def sig(v, digits=4):
    """Rounds a float to `digits` significant digits (the JSON line has to stay short)."""
    if v is None or isinstance(v, (int, str, bool)):
        return v
    if v == 0 or v != v or v in (float("inf"), float("-inf")):
        return v
    from math import floor, log10
    return round(v, digits - 1 - int(floor(log10(abs(v)))))


def sustained_ms(fn, torch, sampler, seconds=1.0):
    """Back-to-back calls for at least `seconds`: mean time per call, with the SM clock sampled during the loop."""
    ms1 = max(event_ms(fn, torch, iters=5), 1e-3)
    iters = int(max(20, seconds * 1e3 / ms1))
    torch.cuda.synchronize()
    n0 = len(sampler.samples)
    sampler.begin()
    ms = event_ms(fn, torch, iters=iters)
    sampler.end()
    clocks = sampler.samples[n0:]
    mhz = statistics.median(clocks) if clocks else None
    return ms, mhz, iters


GENERAL_COLS = ["us_cold", "us_cold_flushed", "us_warm", "us_warm_prepacked", "frac_cold", "frac_warm_prepacked",
                "frac_cold_nominal", "us_sustained", "mhz_sustained", "frac_sustained", "useful_px", "useful_flops"]
L2_BYTES = 126 * 1024 * 1024


def bench_general(torch, lib, peaks, flush, sampler, detail, with_sustained=True):
    """Times every general-case configuration: tensor cores on fp32 (TF32) and bf16 inputs, and the fp32 kernel.

    Per (configuration, algorithm) one row of GENERAL_COLS.  All times are complete calls (filter re-ordering
    included) except the "prepacked" one.
      us_cold            inputs and outputs larger than L2: the calls rotate over enough distinct (x, y) buffer sets
                         to exceed twice the 126 MB L2, so no call finds its image in L2 and every call evicts an
                         earlier call's output: DRAM traffic per call = the algorithmic bytes.  `frac_cold` is the
                         roofline fraction of this time.
      us_cold_flushed    one call after a 256 MB fill: L2 then holds only dirty lines of the fill, so every line
                         the call brings in also costs a write-back that is not the call's own traffic
      us_warm, us_warm_prepacked   same buffers back to back (L2 resident); with the filters already re-ordered
      us_sustained       at least one second of back-to-back calls, SM clock sampled during the loop
    """
    rows = {}
    dev = torch.device("cuda")
    stream = torch.cuda.current_stream().cuda_stream
    fp32_peak = SM_COUNT * FP32_LANES_PER_SM * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12
    for name in ["cfg3", "cfg4", "cfg5_r1", "cfg5_r3", "cfg5_r5", "cfg5_r7"]:
        cfg = CONFIGS[name]
        x, w = make_inputs(cfg)
        xd, wd = torch.from_numpy(x).to(dev), torch.from_numpy(w).to(dev)
        yd = torch.empty((cfg.N, cfg.K, cfg.P, cfg.Q), device=dev, dtype=torch.float32)
        xd16 = wd16 = None
        rows[name] = {}
        for algo_name, algo in (("tf32", lib.ALGO_TF32), ("bf16", lib.ALGO_16BIT), ("ffma", lib.ALGO_FFMA)):
            try:
                ws_bytes = lib.conv2d_fwd_workspace_size(cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S, algo)
            except lib.Conv2dError:
                rows[name][algo_name] = None
                continue
            ws = torch.zeros(max(ws_bytes, 16), dtype=torch.uint8, device=dev)

            tensor_core = algo in (lib.ALGO_TF32, lib.ALGO_16BIT)
            if algo == lib.ALGO_16BIT and xd16 is None:     # same synthetic values, rounded once to bf16
                xd16, wd16 = xd.to(torch.bfloat16).contiguous(), wd.to(torch.bfloat16).contiguous()

            def call(flags=0):
                if algo == lib.ALGO_16BIT:
                    lib.conv2d_fwd_general_16bit(xd16.data_ptr(), wd16.data_ptr(), yd.data_ptr(), cfg.N, cfg.C, cfg.H,
                                                 cfg.W, cfg.K, cfg.R, cfg.S, lib.OPERAND_BF16, ws.data_ptr(), ws_bytes,
                                                 flags, stream)
                else:
                    lib.conv2d_fwd_general(xd.data_ptr(), wd.data_ptr(), yd.data_ptr(), cfg.N, cfg.C, cfg.H, cfg.W,
                                           cfg.K, cfg.R, cfg.S, algo, ws.data_ptr(), ws_bytes, flags, stream)
            for _ in range(3):
                call()
            lib.conv2d_get_status(ws.data_ptr(), stream)
            cold = []
            for _ in range(10):
                flush.zero_()
                cold.append(event_ms(call, torch))
            # rotating buffer sets: more than twice the L2 in distinct inputs and outputs
            src, src16 = (xd16, None) if algo == lib.ALGO_16BIT else (xd, None)
            per_set = src.numel() * src.element_size() + yd.numel() * 4
            n_sets = int(2 * L2_BYTES // per_set) + 2
            xs = [src.clone() for _ in range(n_sets)]
            ys = [torch.empty_like(yd) for _ in range(n_sets)]

            def call_set(i):
                if algo == lib.ALGO_16BIT:
                    lib.conv2d_fwd_general_16bit(xs[i].data_ptr(), wd16.data_ptr(), ys[i].data_ptr(), cfg.N, cfg.C, cfg.H,
                                                 cfg.W, cfg.K, cfg.R, cfg.S, lib.OPERAND_BF16, ws.data_ptr(), ws_bytes,
                                                 0, stream)
                else:
                    lib.conv2d_fwd_general(xs[i].data_ptr(), wd.data_ptr(), ys[i].data_ptr(), cfg.N, cfg.C, cfg.H, cfg.W,
                                           cfg.K, cfg.R, cfg.S, algo, ws.data_ptr(), ws_bytes, 0, stream)
            for i in range(n_sets):
                call_set(i)
            rounds = 3
            start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            start.record()
            for _ in range(rounds):
                for i in range(n_sets):
                    call_set(i)
            stop.record()
            stop.synchronize()
            t_rot = start.elapsed_time(stop) / (rounds * n_sets)
            del xs, ys
            warm = event_ms(call, torch, iters=20)
            packed = event_ms(lambda: call(lib.FLAG_WEIGHTS_PACKED), torch, iters=20) if tensor_core else None
            if with_sustained:
                sust, sust_mhz, sust_iters = sustained_ms(call, torch, sampler, 1.0 if algo_name != "ffma" else 0.3)
            else:
                sust, sust_mhz, sust_iters = warm, None, 0
            lib.conv2d_get_status(ws.data_ptr(), stream)
            t_flush = statistics.median(cold)
            t_cold = t_rot
            nbytes = cfg.compulsory_bytes
            if algo == lib.ALGO_TF32:
                pipe_peak, pipe_sustained, pipe_nominal = peaks["bf16_tflops"] / 2.0, peaks["bf16_tflops_sustained"] / 2.0, NOMINAL_TF32_TFLOPS
            elif algo == lib.ALGO_16BIT:
                pipe_peak, pipe_sustained, pipe_nominal = peaks["bf16_tflops"], peaks["bf16_tflops_sustained"], NOMINAL_BF16_TFLOPS
                nbytes = 2 * (x.size + w.size) + 4 * yd.numel()     # 2-byte operands, fp32 output
            else:
                pipe_peak = pipe_sustained = pipe_nominal = fp32_peak
            t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9) * 1e3
            t_hbm_nominal = nbytes / 8000e9 * 1e3

            def roof_ms(peak_tflops, hbm_ms=t_hbm):
                return max(cfg.flops / (peak_tflops * 1e12) * 1e3, hbm_ms)
            plan = {}
            if tensor_core:
                plan = lib.conv2d_fwd_plan_describe(cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S, algo)
            bound = ("tensor" if tensor_core else "alu") if cfg.flops / (pipe_peak * 1e12) * 1e3 >= t_hbm else "hbm"
            row = [t_cold * 1e3, t_flush * 1e3, warm * 1e3, packed * 1e3 if packed else None,
                   roof_ms(pipe_peak) / t_cold, roof_ms(pipe_peak) / packed if packed else None,
                   roof_ms(pipe_nominal, t_hbm_nominal) / t_cold, sust * 1e3, sust_mhz, roof_ms(pipe_sustained) / sust,
                   plan.get("mma_useful_px"), plan.get("mma_useful_flops")]
            rows[name][algo_name] = [sig(v, 3) if i in (5, 6, 8, 9, 10, 11) else sig(v) for i, v in enumerate(row)]
            detail.append({"workload": name, "algo": algo_name, "bound": bound, "cold_after_flush_us_all": [sig(c * 1e3) for c in cold], "rotating_sets": n_sets,
                           "sustained_iters": sust_iters, "pipe_peak_tflops": pipe_peak, "pipe_nominal_tflops": pipe_nominal,
                           "pipe_sustained_tflops": pipe_sustained, "t_hbm_us": sig(t_hbm * 1e3), "plan": plan,
                           "gflops_cold": sig(cfg.flops / t_cold / 1e6)})
        del xd, wd, yd, xd16, wd16
    return {"cols": GENERAL_COLS, "rows": rows,
            "peaks": {"tf32": "bf16/2", "ffma": "148x128x2x1.965GHz", "nominal": "1125/2250 TF, 8 TB/s",
                      "sustained": "bf16_sustained(/2)", "source": peaks["source"]}}


def bench_cfg1(torch, lib):
    """cfg1 (64 x 64 image, 8 filters of 3 x 3) is bound by launch latency: time of a single launch and of
    back-to-back launches, in microseconds."""
    cfg = CONFIGS["cfg1"]
    dev = torch.device("cuda")
    x, w = make_inputs(cfg)
    xd, wd = torch.from_numpy(x).to(dev), torch.from_numpy(w).to(dev)
    yd = torch.empty((cfg.N, cfg.K, cfg.P, cfg.Q), device=dev)
    stream = torch.cuda.current_stream().cuda_stream

    def call():
        lib.conv2d_fwd_single_channel(xd.data_ptr(), wd.data_ptr(), yd.data_ptr(), cfg.N, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S,
                                      0, 0, 0, stream)
    for _ in range(5):
        call()
    single = []
    for _ in range(20):
        torch.cuda.synchronize()
        single.append(event_ms(call, torch))
    return {"us_single_launch": sig(statistics.median(single) * 1e3), "us_back_to_back": sig(event_ms(call, torch, iters=200) * 1e3)}


def reduce_max(value: float, device=None) -> float:
    """Max of a per-rank scalar over all ranks (identity when torch.distributed is not initialised)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(flops_per_replica: int, world: int, seconds_per_step: float) -> float:
    """Whole-job GFLOP/s of `world` independent replicas that each finish a step in `seconds_per_step`."""
    return world * flops_per_replica / seconds_per_step / 1e9


def run_e2e(torch, lib, cfg, algo, x_host, w_host, xd, wd, yd, ws, ws_bytes, stream, args, world, dev, barrier):
    """Same metric through conv2d_fwd_host: pinned host buffers, H2D and D2H copies inside the timed region."""
    y_host = torch.empty((cfg.N, cfg.K, cfg.P, cfg.Q), dtype=torch.float32).pin_memory()

    def e2e_step():
        lib.conv2d_fwd_host(x_host.data_ptr(), w_host.data_ptr(), y_host.data_ptr(),
                            xd.data_ptr(), wd.data_ptr(), yd.data_ptr(), cfg.N, cfg.C, cfg.H, cfg.W,
                            cfg.K, cfg.R, cfg.S, algo, ws.data_ptr() if ws_bytes else 0, ws_bytes, stream)
    e2e_step()
    e2e_steps = max(2, min(args.steps, 5))
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()          # synchronises the stream itself
    barrier()
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    e2e_s = reduce_max(e2e_s, dev)
    return {"value": job_throughput(cfg.flops, world, e2e_s), "unit": "GFLOP/s",
            "h2d_bytes_per_step": int(x_host.numel() * 4 + w_host.numel() * 4),
            "d2h_bytes_per_step": int(y_host.numel() * 4), "ms_per_step": e2e_s * 1e3, "steps": e2e_steps}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=sorted(CONFIGS))
    ap.add_argument("--no-general", action="store_true", help="skip the general-case configurations")
    ap.add_argument("--operand", default="fp32", choices=["fp32", "bf16", "fp32-exact"],
                    help="general-case workloads only: bf16 runs the 16-bit operand entry on the same values rounded to "
                         "bf16; fp32-exact runs the fp32 FMA kernel (1e-5 tolerance) instead of the tensor cores")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg (profiling runs)")
    ap.add_argument("--no-sustained", action="store_true", help="skip the one-second sustained leg (profiling runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import paper_1705_10591_b200 as lib
    from paper_1705_10591_b200 import build as lib_build

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    lib_build.build()
    lib.load_library()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    peaks = load_peaks()

    cfg = CONFIGS[args.workload]
    single = cfg.C == 1
    x, w = make_inputs(cfg)
    x_host = torch.from_numpy(x).pin_memory()
    w_host = torch.from_numpy(w).pin_memory()
    xd, wd = x_host.to(dev), w_host.to(dev)
    yd = torch.empty((cfg.N, cfg.K, cfg.P, cfg.Q), device=dev, dtype=torch.float32)
    b16 = args.operand == "bf16" and not single
    if b16:
        xd16, wd16 = xd.to(torch.bfloat16).contiguous(), wd.to(torch.bfloat16).contiguous()
        args.no_e2e = True            # the host-buffer entry takes fp32 tensors only
    ffma = args.operand == "fp32-exact" and not single
    algo = lib.ALGO_FFMA if (single or ffma) else (lib.ALGO_16BIT if b16 else lib.ALGO_AUTO)
    ws_bytes = 0 if single else lib.conv2d_fwd_workspace_size(cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S, algo)
    ws = torch.zeros(max(ws_bytes, 16), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)   # larger than the 126 MB L2

    def step():
        if single:
            lib.conv2d_fwd_single_channel(xd.data_ptr(), wd.data_ptr(), yd.data_ptr(), cfg.N, cfg.H, cfg.W,
                                          cfg.K, cfg.R, cfg.S, 0, 0, 0, stream)
        elif b16:
            lib.conv2d_fwd_general_16bit(xd16.data_ptr(), wd16.data_ptr(), yd.data_ptr(), cfg.N, cfg.C, cfg.H, cfg.W,
                                         cfg.K, cfg.R, cfg.S, lib.OPERAND_BF16, ws.data_ptr(), ws_bytes, 0, stream)
        else:
            lib.conv2d_fwd_general(xd.data_ptr(), wd.data_ptr(), yd.data_ptr(), cfg.N, cfg.C, cfg.H, cfg.W,
                                   cfg.K, cfg.R, cfg.S, algo, ws.data_ptr(), ws_bytes, 0, stream)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    working_set = cfg.compulsory_bytes
    algorithmic_bytes = cfg.compulsory_bytes if not b16 else 2 * (x.size + w.size) + 4 * yd.numel()
    flush_between = working_set < 2 * 126 * 1024 * 1024
    for _ in range(args.warmup):
        step()
    lib.conv2d_get_status(ws.data_ptr() if ws_bytes else 0, stream)

    sampler = ClockSampler(local_rank)
    sampler.start()
    barrier()
    sampler.begin()
    launches0 = lib.conv2d_launch_count()
    per_step = []
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if flush_between:
        for _ in range(args.steps):
            flush.zero_()
            per_step.append(event_ms(step, torch))
        total_ms = sum(per_step)
    else:
        start.record()
        for _ in range(args.steps):
            step()
        stop.record()
        stop.synchronize()
        total_ms = start.elapsed_time(stop)
    barrier()
    sampler.end()
    launches = lib.conv2d_launch_count() - launches0
    clocks = sampler.stop()
    lib.conv2d_get_status(ws.data_ptr() if ws_bytes else 0, stream)

    total_ms = reduce_max(total_ms, dev)
    ms_per_step = total_ms / args.steps
    value = job_throughput(cfg.flops, world, ms_per_step * 1e-3)

    # ---- end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(torch, lib, cfg, algo, x_host, w_host, xd, wd, yd, ws, ws_bytes, stream, args, world, dev, barrier)

    # ---- roofline of the dominant kernel (per launch = one step)
    t_kernel_s = ms_per_step * 1e-3
    fp32_peak = SM_COUNT * FP32_LANES_PER_SM * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12   # TFLOP/s at max clock
    t_hbm = algorithmic_bytes / (peaks["hbm_gbs"] * 1e9)
    if single or ffma:
        t_pipe, pipe_name, pipe_peak = cfg.flops / (fp32_peak * 1e12), "alu", fp32_peak
    else:
        pipe_peak = peaks["bf16_tflops"] if b16 else peaks["bf16_tflops"] / 2.0
        t_pipe, pipe_name = cfg.flops / (pipe_peak * 1e12), "tensor"
    if t_pipe >= t_hbm:
        roof = {"bound": pipe_name, "achieved": cfg.flops / t_kernel_s / 1e12, "peak": pipe_peak, "unit": "TFLOP/s"}
    else:
        roof = {"bound": "hbm", "achieved": algorithmic_bytes / t_kernel_s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof.update({
        "traffic": None, "peaks": peaks["source"],
        "algorithmic_bytes_per_launch": algorithmic_bytes, "flops_per_launch": cfg.flops,
        "hbm_gbs_achieved": algorithmic_bytes / t_kernel_s / 1e9,
        "hbm_frac_of_measured": algorithmic_bytes / t_kernel_s / 1e9 / peaks["hbm_gbs"],
        "hbm_frac_of_nominal_8tbs": algorithmic_bytes / t_kernel_s / 1e9 / 8000.0,
        "tflops_achieved": cfg.flops / t_kernel_s / 1e12,
    })
    if not (single or ffma):
        nominal = NOMINAL_BF16_TFLOPS if b16 else NOMINAL_TF32_TFLOPS
        roof["pipe_frac_of_nominal"] = cfg.flops / t_kernel_s / 1e12 / nominal
    traffic_file = ROOT / "profiles" / "traffic.json"
    if traffic_file.exists():
        roof["traffic"] = json.loads(traffic_file.read_text()).get(args.workload)
    if clocks.get("sm_mhz"):
        at_clock = SM_COUNT * FP32_LANES_PER_SM * 2 * clocks["sm_mhz"] * 1e6 / 1e12
        roof["alu_frac_at_sampled_clock"] = cfg.flops / t_kernel_s / 1e12 / at_clock

    result = {
        "metric": "conv_fwd_gflops", "value": value, "unit": "GFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if b16 else ("f32" if (single or ffma) else "tf32"), "data": "synthetic",
        "config": {"workload": cfg.name, "operand": args.operand if not single else "fp32", **cfg.as_dict(), "parallelism": f"replicas x{world}",
                   "l2": "flushed between steps" if flush_between else "step moves 2.2 GB > 126 MB L2"},
        "clocks": {k: clocks.get(k) for k in ("sm_mhz", "sm_max_mhz", "reasons", "samples", "power_w_max")},
        "e2e": e2e, "gpu_launches": int(launches), "roofline": roof,
    }

    detail = []
    if rank == 0 and world == 1:
        sampler2 = ClockSampler(local_rank)
        sampler2.start()
        # a sustained leg of the headline workload: at least one second of back-to-back steps
        if not args.no_sustained:
            sust, sust_mhz, sust_iters = sustained_ms(step, torch, sampler2, 1.0)
            fp32_at = (lambda mhz: SM_COUNT * FP32_LANES_PER_SM * 2 * mhz * 1e6 / 1e12)
            result["sustained"] = {"ms_per_step": sust, "steps": sust_iters, "sm_mhz": sust_mhz,
                                   "ms_x_mhz": sust * sust_mhz if sust_mhz else None,
                                   "value": cfg.flops / sust / 1e6}
        if (single or ffma) and not args.no_sustained:
            result["sustained"]["alu_frac_at_sampled_clock"] = cfg.flops / (sust * 1e-3) / 1e12 / fp32_at(sust_mhz) if sust_mhz else None
            result["sustained"]["hbm_frac_of_measured"] = algorithmic_bytes / (sust * 1e-3) / 1e9 / peaks["hbm_gbs"]
        if not args.no_general:
            result["cfg1"] = bench_cfg1(torch, lib)
            result["general"] = bench_general(torch, lib, peaks, flush, sampler2, detail, not args.no_sustained)
        sampler2.stop()
        if not args.no_cpu_baseline:
            result["cpu_baseline"] = time_oracle_sample(cfg, 12.0)
    if rank == 0:
        def compact(o):
            if isinstance(o, float):
                return sig(o)
            if isinstance(o, dict):
                return {k: compact(v) for k, v in o.items()}
            if isinstance(o, list):
                return [compact(v) for v in o]
            return o
        if detail:
            sys.stderr.write("general-case detail: " + json.dumps(detail) + "\n")
        print(json.dumps(compact(result), separators=(",", ":")))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

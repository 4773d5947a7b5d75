#!/usr/bin/env python
"""Shape sweeps in the structure of the paper's experiments (Section 5), on B200.

    python sweep.py special   # one input channel: filter 1x1 / 3x3 / 5x5, image size and filter count swept (Fig. 7)
    python sweep.py general   # many channels: filter 3x3 / 5x5 / 7x7, image size, channels, filters swept (Fig. 9)
    python sweep.py unit      # per-thread unit float / float2 / float4 on the 3x3 special case (matched vs unmatched)
    python sweep.py point N C H W K R S tf32|bf16|fp32   # one shape of the general case (what the profiles capture)
    python sweep.py pointwise # many channels, 1x1 filters: channels and filters swept up to 1024 / 512 (which form of
                              # the kernel fed by tensor-map copies the planner took is part of each record)

The swept values of the paper's figures were not published as numbers, so the grids below are this
repository's own.  Prints one JSON line per point: shape, time, GFLOP/s and the fraction of the roofline
max(FLOPs / pipe peak, compulsory bytes / measured HBM bandwidth).  Inputs are seeded synthetic tensors.
"""
from __future__ import annotations

import json
import os
import statistics
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from bench import load_peaks  # noqa: E402
from workloads import uniform  # noqa: E402


def time_call(torch, fn, flush, iters=10):
    for _ in range(3):
        fn()
    times = []
    for _ in range(iters):
        if flush is not None:
            flush.zero_()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        b.synchronize()
        times.append(a.elapsed_time(b))
    return statistics.median(times)


def run_point(torch, lib, peaks, flush, N, C, H, W, K, R, S, algo, label, extra=None):
    dev = torch.device("cuda")
    x = torch.from_numpy(uniform((N, C, H, W), 7)).to(dev)
    w = torch.from_numpy(uniform((K, C, R, S), 8)).to(dev)
    P, Q = H - R + 1, W - S + 1
    y = torch.empty((N, K, P, Q), device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    if C == 1:
        def fn():
            lib.conv2d_fwd_single_channel(x.data_ptr(), w.data_ptr(), y.data_ptr(), N, H, W, K, R, S, 0, 0, 0, stream)
        ws = None
    else:
        ws_bytes = lib.conv2d_fwd_workspace_size(N, C, H, W, K, R, S, algo)
        ws = torch.zeros(max(ws_bytes, 16), dtype=torch.uint8, device=dev)
        if algo == lib.ALGO_16BIT:
            x16, w16 = x.to(torch.bfloat16).contiguous(), w.to(torch.bfloat16).contiguous()

            def fn():
                lib.conv2d_fwd_general_16bit(x16.data_ptr(), w16.data_ptr(), y.data_ptr(), N, C, H, W, K, R, S,
                                             lib.OPERAND_BF16, ws.data_ptr(), ws_bytes, 0, stream)
        else:
            def fn():
                lib.conv2d_fwd_general(x.data_ptr(), w.data_ptr(), y.data_ptr(), N, C, H, W, K, R, S, algo,
                                       ws.data_ptr(), ws_bytes, 0, stream)
    flops = 2 * N * K * C * R * S * P * Q
    in_bytes = 2 if (C > 1 and algo == lib.ALGO_16BIT) else 4
    bytes_ = in_bytes * (N * C * H * W + K * C * R * S) + 4 * N * K * P * Q
    big = bytes_ > 2 * 126 * 1024 * 1024
    ms = time_call(torch, fn, None if big else flush)
    lib.conv2d_get_status(ws.data_ptr() if ws is not None else 0, stream)
    fp32_peak = 148 * 128 * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12
    pipe_peak = fp32_peak if (C == 1 or algo == lib.ALGO_FFMA) else (
        peaks["bf16_tflops"] if algo == lib.ALGO_16BIT else peaks["bf16_tflops"] / 2)
    t_roof = max(flops / (pipe_peak * 1e12), bytes_ / (peaks["hbm_gbs"] * 1e9)) * 1e3
    rec = {"sweep": label, "N": N, "C": C, "H": H, "W": W, "K": K, "R": R, "S": S, "ms": ms,
           "gflops": flops / ms / 1e6, "gbs": bytes_ / ms / 1e6, "roofline_frac": t_roof / ms,
           "bound": "pipe" if flops / (pipe_peak * 1e12) >= bytes_ / (peaks["hbm_gbs"] * 1e9) else "hbm"}
    if extra:
        rec.update(extra)
    print(json.dumps(rec), flush=True)


def main():
    import torch
    import paper_1705_10591_b200 as lib
    from paper_1705_10591_b200 import build as lib_build
    lib_build.build()
    peaks = load_peaks()
    which = sys.argv[1] if len(sys.argv) > 1 else "special"
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    if which == "special":
        for r in (1, 3, 5):
            for size in (512, 1024, 2048, 4096):
                for k in (1, 2, 4, 8, 16, 32, 64):
                    if size == 4096 and k == 64:
                        continue                      # 4.3 GB of output: beyond what this sweep needs
                    run_point(torch, lib, peaks, flush, 1, 1, size, size, k, r, r, lib.ALGO_FFMA, "special")
    elif which == "general":
        for r in (3, 5, 7):
            for size in (16, 32, 64, 128, 256, 512):
                for c in (64, 128):
                    for k in (64, 128, 256):
                        n = max(1, 65536 // (size * size))
                        for algo, name in ((lib.ALGO_TF32, "tf32"), (lib.ALGO_16BIT, "bf16"), (lib.ALGO_FFMA, "fp32")):
                            run_point(torch, lib, peaks, flush, n, c, size, size, k, r, r, algo, "general", {"algo": name})
    elif which == "point":
        n, c, h, w_, k, r, s_ = (int(v) for v in sys.argv[2:9])
        name = sys.argv[9] if len(sys.argv) > 9 else "tf32"
        algo = {"tf32": lib.ALGO_TF32, "bf16": lib.ALGO_16BIT, "fp32": lib.ALGO_FFMA}[name]
        plan = lib.conv2d_fwd_plan_describe(n, c, h, w_, k, r, s_, algo) if algo != lib.ALGO_FFMA else {}
        run_point(torch, lib, peaks, flush, n, c, h, w_, k, r, s_, algo, "point", {"algo": name, "plan": plan})
    elif which == "pointwise":
        for size in (16, 32, 64):
            for c in (128, 256, 512, 1024):
                for k in (128, 256, 512):
                    n = max(1, 65536 // (size * size))
                    for algo, name in ((lib.ALGO_TF32, "tf32"), (lib.ALGO_16BIT, "bf16")):
                        plan = lib.conv2d_fwd_plan_describe(n, c, size, size, k, 1, 1, algo)
                        run_point(torch, lib, peaks, flush, n, c, size, size, k, 1, 1, algo, "pointwise",
                                  {"algo": name, "kernel": plan.get("kernel"), "two_sm": plan.get("two_sm"),
                                   "resident_filters": plan.get("resident_filters")})
    elif which == "unit":
        os.environ["CONV2D_B200_TUNING"] = "1"      # must be set before the library's first call
        for size in (2048, 4096):
            for k in (8, 32):
                for unit in (1, 2, 4):
                    os.environ["CONV2D_B200_SC_UNIT"] = str(unit)
                    run_point(torch, lib, peaks, flush, 1, 1, size, size, k, 3, 3, lib.ALGO_FFMA, "unit", {"unit_floats": unit})
                os.environ.pop("CONV2D_B200_SC_UNIT", None)
                run_point(torch, lib, peaks, flush, 1, 1, size, size, k, 3, 3, lib.ALGO_FFMA, "unit", {"unit_floats": "default path"})
    else:
        raise SystemExit(__doc__)


if __name__ == "__main__":
    main()

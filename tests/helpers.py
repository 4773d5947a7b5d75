"""Shared helpers of the GPU parity tests: run the library on torch device buffers, compare with the oracle."""
from __future__ import annotations

import numpy as np

GUARD = 1024  # floats of guard band on each side of the output buffer

FFMA_TOL = 1e-5   # |y - y_ref| <= 1e-5 * sum|x*w|   (fp32 FMA paths)
TF32_TOL = 2e-3   # |y - y_ref| <= 2e-3 * sum|x*w|   (TF32 tensor-core path)


B16_TOL = 1e-5    # 16-bit operands, exact products, fp32 accumulation: same bar as the fp32 FMA paths


def bf16_values(a: np.ndarray):
    """Rounds fp32 to the nearest bf16 (ties to even).  Returns (the values as fp32, their 16-bit patterns)."""
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    bits = (bits + 0x7FFF + ((bits >> 16) & 1)) >> 16
    pat = bits.astype(np.uint16)
    return (pat.astype(np.uint32) << 16).view(np.float32).reshape(a.shape), pat.reshape(a.shape)


def fp16_values(a: np.ndarray):
    """Rounds fp32 to the nearest IEEE half (numpy's conversion, ties to even).  Returns (values as fp32, patterns)."""
    h = np.ascontiguousarray(a, dtype=np.float32).astype(np.float16)
    return h.astype(np.float32), h.view(np.uint16)


def run_library(x: np.ndarray, w: np.ndarray, entry: str = "general", algo: int = 1, flags: int = 0,
                workspace=None, repeat: int = 1):
    """Runs one convolution through the C ABI on cuda:0 and returns y as a numpy array [N,K,P,Q].

    The output buffer is pre-filled with a NaN payload and framed by guard bands; the call fails if
    a guard word changed or an output element kept the payload.
    """
    import torch
    import paper_1705_10591_b200 as lib

    N, C, H, W = x.shape
    K, _, R, S = w.shape
    P, Q = H - R + 1, W - S + 1
    dev = torch.device("cuda:0")
    if entry in ("bf16", "fp16"):     # x, w hold 16-bit values; the device gets their 16-bit patterns
        conv = bf16_values if entry == "bf16" else fp16_values
        xd = torch.from_numpy(conv(x)[1].view(np.int16)).to(dev)
        wd = torch.from_numpy(conv(w)[1].view(np.int16)).to(dev)
        algo = 3
    else:
        xd = torch.from_numpy(np.ascontiguousarray(x)).to(dev)
        wd = torch.from_numpy(np.ascontiguousarray(w)).to(dev)
    numel = N * K * P * Q
    payload = np.array([0x7FC0BEEF], dtype=np.uint32).view(np.float32)[0]
    buf = torch.full((numel + 2 * GUARD,), float("nan"), device=dev, dtype=torch.float32)
    buf.view(torch.int32).fill_(int(np.array([payload]).view(np.int32)[0]))
    y_ptr = buf.data_ptr() + 4 * GUARD
    stream = torch.cuda.current_stream().cuda_stream
    ws_ptr, ws_bytes = 0, 0
    if entry in ("general", "bf16", "fp16"):
        ws_bytes = lib.conv2d_fwd_workspace_size(N, C, H, W, K, R, S, algo)
        if workspace is None and ws_bytes:
            workspace = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
        ws_ptr = workspace.data_ptr() if workspace is not None else 0
    for _ in range(repeat):
        if entry == "single":
            assert C == 1
            lib.conv2d_fwd_single_channel(xd.data_ptr(), wd.data_ptr(), y_ptr, N, H, W, K, R, S, 0, 0, flags, stream)
        elif entry in ("bf16", "fp16"):
            lib.conv2d_fwd_general_16bit(xd.data_ptr(), wd.data_ptr(), y_ptr, N, C, H, W, K, R, S,
                                         lib.OPERAND_BF16 if entry == "bf16" else lib.OPERAND_FP16,
                                         ws_ptr, ws_bytes, flags, stream)
        else:
            lib.conv2d_fwd_general(xd.data_ptr(), wd.data_ptr(), y_ptr, N, C, H, W, K, R, S, algo,
                                   ws_ptr, ws_bytes, flags, stream)
    lib.conv2d_get_status(ws_ptr, stream)
    torch.cuda.synchronize()
    host = buf.cpu().numpy()
    bits = host.view(np.uint32)
    assert np.all(bits[:GUARD] == 0x7FC0BEEF) and np.all(bits[-GUARD:] == 0x7FC0BEEF), "guard band overwritten"
    y = host[GUARD:GUARD + numel]
    assert not np.any(bits[GUARD:GUARD + numel] == 0x7FC0BEEF), "some outputs were never written"
    return y.reshape(N, K, P, Q).copy()


def error_ratio(y_gpu: np.ndarray, y_ref: np.ndarray, yabs: np.ndarray) -> float:
    """max over elements of |y_gpu - y_ref| / sum|x*w| (0/0 counts as 0, x/0 as inf)."""
    assert np.all(np.isfinite(y_gpu)), "non-finite output"
    num = np.abs(y_gpu.astype(np.float64) - y_ref)
    ratio = np.where(yabs > 0, num / np.where(yabs > 0, yabs, 1.0), np.where(num == 0, 0.0, np.inf))
    return float(ratio.max())


def assert_parity(y_gpu, y_ref, yabs, tol, what=""):
    r = error_ratio(y_gpu, y_ref, yabs)
    if not r <= tol:
        num = np.abs(y_gpu.astype(np.float64) - y_ref)
        idx = np.unravel_index(np.argmax(np.where(yabs > 0, num / np.maximum(yabs, 1e-300), num * 1e300)), y_ref.shape)
        raise AssertionError(f"{what}: max |err|/sum|xw| = {r:.3e} > {tol:.1e} at (n,k,p,q)={idx}: "
                             f"gpu={y_gpu[idx]!r} ref={y_ref[idx]!r}")
    return r

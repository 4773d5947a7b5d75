"""conv2d_fwd_host, the host-buffer entry the benchmark's end-to-end leg times, against the oracle.

Covers the three kernels it can reach (single channel, fp32 general, tensor cores), pageable and page-locked host
buffers, and a workspace that the caller never initialised: only a tensor-core call may read its status block.
"""
import numpy as np
import pytest

from helpers import FFMA_TOL, TF32_TOL, assert_parity
from workloads import small_integers, uniform

pytestmark = pytest.mark.gpu
ALGO_AUTO, ALGO_FFMA, ALGO_TF32 = 0, 1, 2


def _host_call(x, w, algo, pinned, workspace="query"):
    import torch
    import paper_1705_10591_b200 as lib

    N, C, H, W = x.shape
    K, _, R, S = w.shape
    P, Q = H - R + 1, W - S + 1
    dev = torch.device("cuda:0")
    xh, wh = torch.from_numpy(np.ascontiguousarray(x)), torch.from_numpy(np.ascontiguousarray(w))
    yh = torch.full((N, K, P, Q), float("nan"))
    if pinned:
        xh, wh, yh = xh.pin_memory(), wh.pin_memory(), yh.pin_memory()
    xd, wd = torch.empty_like(xh, device=dev), torch.empty_like(wh, device=dev)
    yd = torch.full((N, K, P, Q), float("nan"), device=dev)
    ws_ptr, ws_bytes, ws = 0, 0, None
    if workspace == "query":
        ws_bytes = lib.conv2d_fwd_workspace_size(N, C, H, W, K, R, S, algo)
    elif workspace == "garbage":        # larger than needed, every word a NaN pattern: must never be read as a status
        ws_bytes = max(lib.conv2d_fwd_workspace_size(N, C, H, W, K, R, S, ALGO_AUTO), 4096)
    if ws_bytes:
        ws = torch.full((ws_bytes // 4 + 1,), float("nan"), device=dev)
        ws_ptr = ws.data_ptr()
    stream = torch.cuda.current_stream().cuda_stream
    lib.conv2d_fwd_host(xh.data_ptr(), wh.data_ptr(), yh.data_ptr(), xd.data_ptr(), wd.data_ptr(), yd.data_ptr(),
                        N, C, H, W, K, R, S, algo, ws_ptr, ws_bytes, stream)        # synchronises the stream itself
    return yh.numpy().copy()


@pytest.mark.parametrize("pinned", [False, True])
@pytest.mark.parametrize("case", [
    # x shape, w shape, algo, workspace, tolerance
    ((1, 1, 40, 52), (6, 1, 5, 5), ALGO_FFMA, "none", FFMA_TOL),          # one channel: the single-channel kernel
    ((1, 1, 24, 1100), (4, 1, 3, 3), ALGO_AUTO, "garbage", FFMA_TOL),     # wide single-channel kernel, workspace never written
    ((2, 24, 18, 20), (40, 24, 3, 3), ALGO_FFMA, "none", FFMA_TOL),       # fp32 general kernel without a workspace
    ((2, 24, 18, 20), (40, 24, 3, 3), ALGO_FFMA, "garbage", FFMA_TOL),    # ... and with one it must not look at
    ((2, 48, 16, 16), (96, 48, 3, 3), ALGO_TF32, "query", TF32_TOL),      # tensor cores
    ((2, 48, 16, 16), (96, 48, 3, 3), ALGO_AUTO, "garbage", TF32_TOL),    # AUTO takes the tensor cores and clears the block itself
])
def test_host_entry_matches_the_oracle(oracle, case, pinned):
    xs, ws_, algo, workspace, tol = case
    x, w = uniform(xs, 951), uniform(ws_, 952)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(_host_call(x, w, algo, pinned, workspace), y_ref, yabs, tol, f"host entry {case}")


def test_host_entry_exact_on_integers(oracle):
    x, w = small_integers((2, 20, 14, 16), 953), small_integers((72, 20, 3, 3), 954)
    y_ref, _ = oracle.conv2d_oracle(x, w)
    for algo in (ALGO_FFMA, ALGO_TF32):
        np.testing.assert_array_equal(_host_call(x, w, algo, True).astype(np.float64), y_ref)

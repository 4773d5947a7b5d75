"""Outputs with more than 2^31 elements: every kernel family must index y with 64 bits.

The output tensors here are 9-10 GB and stay on the device; only sampled rows are read back and compared with the
oracle, among them rows at the very end of y and rows on both sides of element 2^31.
"""
import numpy as np
import pytest

from helpers import FFMA_TOL, TF32_TOL, assert_parity
from workloads import uniform

pytestmark = pytest.mark.gpu


def _free_bytes():
    import torch
    return torch.cuda.mem_get_info(0)[0]


def _run_on_device(x, w, entry, algo):
    """Runs the library and returns the device output tensor [N,K,P,Q] (not copied to the host)."""
    import torch
    import paper_1705_10591_b200 as lib
    N, C, H, W = x.shape
    K, _, R, S = w.shape
    P, Q = H - R + 1, W - S + 1
    dev = torch.device("cuda:0")
    xd, wd = torch.from_numpy(x).to(dev), torch.from_numpy(w).to(dev)
    yd = torch.full((N, K, P, Q), float("nan"), device=dev, dtype=torch.float32)
    stream = torch.cuda.current_stream().cuda_stream
    if entry == "single":
        lib.conv2d_fwd_single_channel(xd.data_ptr(), wd.data_ptr(), yd.data_ptr(), N, H, W, K, R, S, 0, 0, 0, stream)
        lib.conv2d_get_status(0, stream)
    else:
        ws_bytes = lib.conv2d_fwd_workspace_size(N, C, H, W, K, R, S, algo)
        ws = torch.zeros(max(ws_bytes, 16), dtype=torch.uint8, device=dev)
        lib.conv2d_fwd_general(xd.data_ptr(), wd.data_ptr(), yd.data_ptr(), N, C, H, W, K, R, S, algo,
                               ws.data_ptr(), ws_bytes, 0, stream)
        lib.conv2d_get_status(ws.data_ptr(), stream)
    return yd


def _rows_to_check(N, K, P, Q):
    """(n, k, p) triples: first and last rows of y, and the rows that contain elements 2^31 - 1 and 2^31."""
    picks = {(0, 0, 0), (N - 1, K - 1, P - 1), (N - 1, K - 1, 0), (N - 1, 0, P // 2)}
    for flat in (2 ** 31 - 1, 2 ** 31, 2 ** 31 + Q):
        row = flat // Q
        n, rem = divmod(row, K * P)
        k, p = divmod(rem, P)
        if n < N:
            picks.add((n, k, p))
    return sorted(picks)


def _check(oracle, x, w, yd, tol, what):
    N, K, P, Q = yd.shape
    assert N * K * P * Q > 2 ** 31
    worst = 0.0
    for n, k, p in _rows_to_check(N, K, P, Q):
        y_ref, yabs = oracle.conv2d_oracle_range(x, w, n_range=(n, n + 1), k_range=(k, k + 1), p_range=(p, p + 1))
        got = yd[n, k, p].cpu().numpy().reshape(1, 1, 1, Q)
        worst = max(worst, assert_parity(got, y_ref, yabs, tol, f"{what} row {(n, k, p)}"))
    import torch
    assert not torch.isnan(yd[N - 1, K - 1]).any().item(), "the last plane has unwritten outputs"
    assert not torch.isnan(yd[0, 0]).any().item()
    print(f"{what}: max ratio {worst:.3e}")


def test_single_channel_output_beyond_2_to_31_elements(oracle):
    if _free_bytes() < 14 * 2 ** 30:
        pytest.skip("needs 14 GB of free device memory")
    N, H, W, K, R, S = 2, 8192, 8192, 17, 3, 3              # y: 2 x 17 x 8190 x 8190 = 2.28e9 elements
    x, w = uniform((N, 1, H, W), 441), uniform((K, 1, R, S), 442)
    yd = _run_on_device(x, w, "single", 1)
    _check(oracle, x, w, yd, FFMA_TOL, "single channel, 9.1 GB of output")


@pytest.mark.parametrize("algo,tol", [(2, TF32_TOL), (1, FFMA_TOL)])
def test_general_output_beyond_2_to_31_elements(oracle, algo, tol):
    if _free_bytes() < 14 * 2 ** 30:
        pytest.skip("needs 14 GB of free device memory")
    # y: 16 x 144 x 2046 x 510 = 2.40e9 elements (rows of 512 pixels: the tensor-core path stages whole-row halos,
    # so it has no instance for much wider images)
    N, C, H, W, K, R, S = 16, 8, 2048, 512, 144, 3, 3
    x, w = uniform((N, C, H, W), 443), uniform((K, C, R, S), 444)
    yd = _run_on_device(x, w, "general", algo)
    _check(oracle, x, w, yd, tol, f"general algo {algo}, 9.6 GB of output")

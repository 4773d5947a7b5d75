"""Failure detection on the device side, exercised without faulting or hanging anything.

The injection is on the host: an environment switch makes the tensor-core kernel arm one filter copy
without issuing it (the wide single-channel kernels: arm one input row more than they copy) and shortens
the bound of the waits.  The consumer's bounded wait then runs out,
the blocks stop storing, free their tensor memory and return normally; the status word reports it.
The CUDA context must stay usable and the next call must be correct.
"""
import numpy as np
import pytest

from helpers import FFMA_TOL, TF32_TOL, assert_parity, run_library
from workloads import uniform

pytestmark = pytest.mark.gpu
ALGO_TF32 = 2


def test_expired_wait_is_reported_and_the_context_survives(oracle, monkeypatch):
    import torch
    import paper_1705_10591_b200 as lib

    N, C, H, W, K, R, S = 2, 64, 16, 16, 128, 3, 3
    x, w = uniform((N, C, H, W), 801), uniform((K, C, R, S), 802)
    dev = torch.device("cuda:0")
    xd, wd = torch.from_numpy(x).to(dev), torch.from_numpy(w).to(dev)
    y = torch.zeros((N, K, H - R + 1, W - S + 1), device=dev)
    ws_bytes = lib.conv2d_fwd_workspace_size(N, C, H, W, K, R, S, ALGO_TF32)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream().cuda_stream

    monkeypatch.setenv("CONV2D_B200_TF32_MAX_POLLS", "2048")
    monkeypatch.setenv("CONV2D_B200_TF32_TEST_DROP_STAGE", "1")
    lib.conv2d_fwd_general(xd.data_ptr(), wd.data_ptr(), y.data_ptr(), N, C, H, W, K, R, S, ALGO_TF32,
                           ws.data_ptr(), ws_bytes, 0, stream)
    with pytest.raises(lib.Conv2dError) as e:
        lib.conv2d_get_status(ws.data_ptr(), stream)
    assert e.value.status == 8                       # CONV2D_ERR_DEVICE_TIMEOUT
    torch.cuda.synchronize()                         # no sticky CUDA error: the kernels returned normally

    monkeypatch.delenv("CONV2D_B200_TF32_MAX_POLLS")
    monkeypatch.delenv("CONV2D_B200_TF32_TEST_DROP_STAGE")
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="general", algo=ALGO_TF32), y_ref, yabs, TF32_TOL, "after a time-out")


@pytest.mark.parametrize("dims", [(1, 40, 1100, 4, 5, 5),      # wide kernel (128-bit stores), several bands
                                  (1, 40, 1032, 4, 3, 3)])     # shifted wide kernel (8-byte aligned rows)
def test_single_channel_wide_kernels_report_an_expired_wait(oracle, monkeypatch, dims):
    """Host-side injection: the barrier of one work item expects one input row more than is copied, and the wait
    bound is short.  The wait runs out, the block stops, the kernel returns normally; the status call reports the
    time-out once, and the next call is correct."""
    import torch
    import paper_1705_10591_b200 as lib

    N, H, W, K, R, S = dims
    x, w = uniform((N, 1, H, W), 811), uniform((K, 1, R, S), 812)
    dev = torch.device("cuda:0")
    xd, wd = torch.from_numpy(x).to(dev), torch.from_numpy(w).to(dev)
    y = torch.zeros((N, K, H - R + 1, W - S + 1), device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    monkeypatch.setenv("CONV2D_B200_SC_MAX_POLLS", "4096")
    monkeypatch.setenv("CONV2D_B200_SC_TEST_SHORT_ITEM", "1")
    lib.conv2d_fwd_single_channel(xd.data_ptr(), wd.data_ptr(), y.data_ptr(), N, H, W, K, R, S, 0, 0, 0, stream)
    with pytest.raises(lib.Conv2dError) as e:
        lib.conv2d_get_status(0, stream)
    assert e.value.status == 8                       # CONV2D_ERR_DEVICE_TIMEOUT
    torch.cuda.synchronize()                         # no sticky CUDA error: the kernel returned normally
    lib.conv2d_get_status(0, stream)                 # the word was consumed by the first query

    monkeypatch.delenv("CONV2D_B200_SC_MAX_POLLS")
    monkeypatch.delenv("CONV2D_B200_SC_TEST_SHORT_ITEM")
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="single"), y_ref, yabs, FFMA_TOL, "after a time-out")


def test_single_channel_wide_kernel_reports_no_timeout_in_normal_operation():
    import torch
    import paper_1705_10591_b200 as lib
    x = torch.rand((1, 1, 24, 1040), device="cuda:0")
    w = torch.rand((4, 1, 5, 5), device="cuda:0")
    y = torch.empty((1, 4, 20, 1036), device="cuda:0")
    stream = torch.cuda.current_stream().cuda_stream
    lib.conv2d_fwd_single_channel(x.data_ptr(), w.data_ptr(), y.data_ptr(), 1, 24, 1040, 4, 5, 5, 0, 0, 0, stream)
    lib.conv2d_get_status(0, stream)                 # raises on a device time-out
    assert torch.isfinite(y).all()

"""The entry point for callers that cannot allocate: conv2d_fwd_general_noalloc.

Some users of the library run where no device allocation may happen at call time -- a plug-in
that only receives its input and output buffers, a service whose memory pool is fully handed out,
a real-time loop that must stay away from the allocator.  For them the library keeps the scratch
of the tensor-core path in a fixed device array of its own.  This test calls that entry point
through the C ABI twice in a row, with different shapes and filters so that whatever the first call
left in the shared array would corrupt the second if it were reused, and checks each result
against the oracle (tensor-core tolerance) and against the regular entry point (conv2d_fwd_general
with a caller-provided workspace), with which it must agree bit for bit: same kernels, same plan.

Collected last on purpose (file name), so a run that stops at the first failure has already
run every other test; it does not depend on any other test having run.
"""
import numpy as np
import pytest

from helpers import TF32_TOL, assert_parity
from workloads import uniform

ALGO_TF32 = 2


def _device_run(fn_noalloc, x, w):
    import torch
    import paper_1705_10591_b200 as lib

    N, C, H, W = x.shape
    K, _, R, S = w.shape
    P, Q = H - R + 1, W - S + 1
    dev = torch.device("cuda:0")
    stream = torch.cuda.current_stream().cuda_stream
    xd, wd = torch.from_numpy(x).to(dev), torch.from_numpy(w).to(dev)
    y = torch.full((N, K, P, Q), float("nan"), device=dev)
    if fn_noalloc:
        lib.conv2d_fwd_general_noalloc(xd.data_ptr(), wd.data_ptr(), y.data_ptr(), N, C, H, W, K, R, S, 1, stream)
    else:
        ws_bytes = lib.conv2d_fwd_workspace_size(N, C, H, W, K, R, S, ALGO_TF32)
        ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
        lib.conv2d_fwd_general(xd.data_ptr(), wd.data_ptr(), y.data_ptr(), N, C, H, W, K, R, S, ALGO_TF32,
                               ws.data_ptr(), ws_bytes, 0, stream)
        lib.conv2d_get_status(ws.data_ptr(), stream)
    torch.cuda.synchronize()
    return y.cpu().numpy()


@pytest.mark.gpu
def test_noalloc_entry_matches_workspace_entry_on_two_calls_in_a_row(oracle):
    shapes = [
        (2, 40, 18, 22, 96, 3, 3),    # first call: larger filter bank
        (3, 24, 15, 15, 48, 5, 5),    # second call: different taps, fewer filters -> stale words remain behind it
    ]
    for call, (N, C, H, W, K, R, S) in enumerate(shapes):
        x, w = uniform((N, C, H, W), 900 + call), uniform((K, C, R, S), 910 + call)
        y_new = _device_run(True, x, w)
        y_old = _device_run(False, x, w)
        y_ref, yabs = oracle.conv2d_oracle(x, w)
        assert_parity(y_new, y_ref, yabs, TF32_TOL, f"call {call}: entry without caller scratch vs the oracle")
        np.testing.assert_array_equal(y_new, y_old, err_msg=f"call {call}: differs from the workspace entry point")


@pytest.mark.gpu
def test_noalloc_entry_timeout_is_visible_after_an_asynchronous_call(oracle, monkeypatch):
    """wait = 0 returns before the kernels have run, so an expired on-device wait cannot come back from the call
    itself: conv2d_get_status(NULL, stream) reports it, and the next call of the entry clears it.  The fault is
    injected on the host (one filter copy armed but never issued, short wait bound); nothing hangs or traps."""
    import torch
    import paper_1705_10591_b200 as lib

    N, C, H, W, K, R, S = 2, 64, 16, 16, 128, 3, 3
    x, w = uniform((N, C, H, W), 920), uniform((K, C, R, S), 921)
    dev = torch.device("cuda:0")
    stream = torch.cuda.current_stream().cuda_stream
    xd, wd = torch.from_numpy(x).to(dev), torch.from_numpy(w).to(dev)
    y = torch.zeros((N, K, H - R + 1, W - S + 1), device=dev)
    monkeypatch.setenv("CONV2D_B200_TF32_MAX_POLLS", "2048")
    monkeypatch.setenv("CONV2D_B200_TF32_TEST_DROP_STAGE", "1")
    lib.conv2d_fwd_general_noalloc(xd.data_ptr(), wd.data_ptr(), y.data_ptr(), N, C, H, W, K, R, S, 0, stream)
    with pytest.raises(lib.Conv2dError) as e:
        lib.conv2d_get_status(0, stream)
    assert e.value.status == 8                       # CONV2D_ERR_DEVICE_TIMEOUT
    torch.cuda.synchronize()                         # the context is intact
    monkeypatch.delenv("CONV2D_B200_TF32_MAX_POLLS")
    monkeypatch.delenv("CONV2D_B200_TF32_TEST_DROP_STAGE")
    y_new = _device_run(True, x, w)                  # wait = 1: would raise on a time-out; clears the status word
    lib.conv2d_get_status(0, stream)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(y_new, y_ref, yabs, TF32_TOL, "after a time-out")


@pytest.mark.gpu
def test_noalloc_entry_rejects_filter_banks_beyond_its_array():
    import torch
    import paper_1705_10591_b200 as lib
    # 512 filters x 512 channels x 3 x 3 re-ordered is 9 MiB: beyond the 8 MiB array
    N, C, H, W, K, R, S = 1, 512, 8, 8, 512, 3, 3
    assert lib.conv2d_fwd_workspace_size(N, C, H, W, K, R, S, ALGO_TF32) > 256 + 8 * 1024 * 1024
    buf = torch.zeros(16, device="cuda:0")
    with pytest.raises(lib.Conv2dError) as e:
        lib.conv2d_fwd_general_noalloc(buf.data_ptr(), buf.data_ptr(), buf.data_ptr(), N, C, H, W, K, R, S, 0, 0)
    assert e.value.status == 4     # CONV2D_ERR_WORKSPACE, nothing was enqueued

"""The entry point for callers that cannot allocate: conv2d_fwd_general_noalloc.

Some users of the library run where no device allocation may happen at call time -- a plug-in
that only receives its input and output buffers, a service whose memory pool is fully handed out,
a real-time loop that must stay away from the allocator.  For them the library keeps the scratch
of the tensor-core path in a fixed device array of its own.  This test calls that entry point
through the C ABI twice in a row, with different shapes and filters so that whatever the first call
left in the shared array would corrupt the second if it were reused, and checks each result
against the regular entry point (conv2d_fwd_general with a caller-provided workspace).

Collected last on purpose (file name), so a run that stops at the first failure has already
run every other test; it does not depend on any other test having run.
"""
import numpy as np
import pytest

from helpers import TF32_TOL
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
        _, yabs = oracle.conv2d_oracle(x, w)
        assert np.isfinite(y_new).all()
        excess = np.abs(y_new.astype(np.float64) - y_old.astype(np.float64)) - TF32_TOL * yabs
        assert excess.max() <= 0.0, f"call {call}: differs from the workspace entry point by more than the tolerance"


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

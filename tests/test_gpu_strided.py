"""Strided (and zero-padded) convolution entry against the oracle.  A strided convolution is by definition the
stride-1 convolution sampled at every stride-th row and column, so the reference is the oracle's output on the
host-padded input, subsampled."""
import numpy as np
import pytest

from helpers import FFMA_TOL, TF32_TOL, assert_parity
from workloads import small_integers, uniform

pytestmark = pytest.mark.gpu

CASES = [
    # N, C, H, W, K, R, S, pad_h, pad_w, stride
    (2, 3, 32, 32, 16, 7, 7, 3, 3, 2),       # first layer of an image network in miniature
    (1, 16, 15, 18, 40, 3, 3, 1, 1, 2),      # odd height: the last window starts at an even row
    (2, 8, 20, 20, 24, 5, 5, 0, 0, 2),
    (1, 4, 17, 23, 9, 3, 3, 0, 1, 3),        # stride 3, pads differ
    (1, 32, 8, 8, 64, 1, 1, 0, 0, 2),        # 1 x 1 with stride: three quarters of the input is never used
    (2, 6, 9, 9, 5, 2, 4, 1, 2, 2),          # rectangular, even taps
    (1, 5, 12, 12, 7, 3, 3, 1, 1, 1),        # stride 1 degenerates to the padded convolution
    (1, 2, 11, 11, 3, 3, 3, 0, 0, 4),        # stride larger than the filter
    (2, 512, 14, 16, 96, 1, 1, 0, 0, 2),     # 1 x 1, stride 2: 2048 channels on 7 x 8 pixels after the rewriting (streamed, split contraction)
    (1, 128, 16, 16, 200, 1, 1, 0, 0, 2),    # 512 channels, 200 filters after the rewriting (streamed filters, two-SM form)
]


def _run(x, w, pad_h, pad_w, stride, algo, flags=0, ws=None):
    import torch
    import paper_1705_10591_b200 as lib
    N, C, H, W = x.shape
    K, _, R, S = w.shape
    P, Q = (H + 2 * pad_h - R) // stride + 1, (W + 2 * pad_w - S) // stride + 1
    dev = torch.device("cuda:0")
    xd, wd = torch.from_numpy(x).to(dev), torch.from_numpy(w).to(dev)
    yd = torch.full((N, K, P, Q), float("nan"), device=dev)
    nbytes = lib.conv2d_fwd_strided_workspace_size(N, C, H, W, K, R, S, pad_h, pad_w, stride, algo)
    if ws is None:
        ws = torch.zeros(nbytes, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    lib.conv2d_fwd_general_strided(xd.data_ptr(), wd.data_ptr(), yd.data_ptr(), N, C, H, W, K, R, S, pad_h, pad_w, stride,
                                   algo, ws.data_ptr(), nbytes, flags, stream)
    lib.conv2d_get_status(ws.data_ptr(), stream)
    y = yd.cpu().numpy()
    assert np.isfinite(y).all()
    return y, ws


def _reference(oracle, x, w, ph, pw, st):
    y1, a1 = oracle.conv2d_oracle(np.pad(x, ((0, 0), (0, 0), (ph, ph), (pw, pw))), w)
    return y1[:, :, ::st, ::st], a1[:, :, ::st, ::st]


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("algo,tol", [(1, FFMA_TOL), (0, TF32_TOL)])
def test_strided_matches_subsampled_oracle(oracle, case, algo, tol):
    N, C, H, W, K, R, S, ph, pw, st = case
    x, w = uniform((N, C, H, W), 481), uniform((K, C, R, S), 482)
    y_ref, yabs = _reference(oracle, x, w, ph, pw, st)
    y, _ = _run(x, w, ph, pw, st, algo)
    assert y.shape == y_ref.shape
    assert_parity(y, y_ref, yabs, tol, f"strided algo {algo} {case}")
    xi, wi = small_integers((N, C, H, W), 483), small_integers((K, C, R, S), 484)
    yi_ref, _ = _reference(oracle, xi, wi, ph, pw, st)
    np.testing.assert_array_equal(_run(xi, wi, ph, pw, st, algo)[0].astype(np.float64), yi_ref)


def test_strided_prepacked_filters(oracle):
    import paper_1705_10591_b200 as lib
    N, C, H, W, K, R, S, ph, pw, st = 2, 16, 20, 20, 130, 3, 3, 1, 1, 2
    x, w = uniform((N, C, H, W), 485), uniform((K, C, R, S), 486)
    y1, ws = _run(x, w, ph, pw, st, 2)
    y2, _ = _run(x, w, ph, pw, st, 2, flags=lib.FLAG_WEIGHTS_PACKED, ws=ws)
    np.testing.assert_array_equal(y1, y2)

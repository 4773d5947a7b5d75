"""Zero-padded convolution entry against the oracle: padding is pinned by its definition -- the oracle convolves the
input that numpy has zero-extended on the host."""
import numpy as np
import pytest

from helpers import FFMA_TOL, TF32_TOL, assert_parity
from workloads import small_integers, uniform

pytestmark = pytest.mark.gpu

CASES = [
    # N, C, H, W, K, R, S, pad_h, pad_w
    (2, 16, 14, 14, 32, 3, 3, 1, 1),       # "same" 3 x 3
    (1, 8, 20, 33, 70, 5, 5, 2, 2),        # "same" 5 x 5, odd width
    (3, 5, 9, 12, 7, 7, 7, 3, 3),          # "same" 7 x 7 on a small image: most windows touch the border
    (1, 32, 10, 10, 16, 3, 3, 0, 2),       # columns only
    (2, 4, 6, 40, 12, 3, 1, 1, 0),         # rows only
    (1, 1, 16, 300, 9, 3, 3, 1, 1),        # one channel through the padded entry
    (1, 24, 5, 5, 40, 5, 5, 4, 4),         # full padding: output larger than the input
]


def _run(x, w, pad_h, pad_w, algo):
    import torch
    import paper_1705_10591_b200 as lib
    N, C, H, W = x.shape
    K, _, R, S = w.shape
    P, Q = H + 2 * pad_h - R + 1, W + 2 * pad_w - S + 1
    dev = torch.device("cuda:0")
    xd, wd = torch.from_numpy(x).to(dev), torch.from_numpy(w).to(dev)
    yd = torch.full((N, K, P, Q), float("nan"), device=dev)
    nbytes = lib.conv2d_fwd_padded_workspace_size(N, C, H, W, K, R, S, pad_h, pad_w, algo)
    ws = torch.zeros(nbytes, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    lib.conv2d_fwd_general_padded(xd.data_ptr(), wd.data_ptr(), yd.data_ptr(), N, C, H, W, K, R, S, pad_h, pad_w, algo,
                                  ws.data_ptr(), nbytes, 0, stream)
    lib.conv2d_get_status(ws.data_ptr(), stream)
    y = yd.cpu().numpy()
    assert np.isfinite(y).all()
    return y


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("algo,tol", [(1, FFMA_TOL), (0, TF32_TOL)])
def test_padded_matches_oracle_on_zero_extended_input(oracle, case, algo, tol):
    N, C, H, W, K, R, S, ph, pw = case
    x, w = uniform((N, C, H, W), 471), uniform((K, C, R, S), 472)
    xz = np.pad(x, ((0, 0), (0, 0), (ph, ph), (pw, pw)))
    y_ref, yabs = oracle.conv2d_oracle(xz, w)
    assert_parity(_run(x, w, ph, pw, algo), y_ref, yabs, tol, f"padded algo {algo} {case}")
    xi, wi = small_integers((N, C, H, W), 473), small_integers((K, C, R, S), 474)
    yi_ref, _ = oracle.conv2d_oracle(np.pad(xi, ((0, 0), (0, 0), (ph, ph), (pw, pw))), wi)
    np.testing.assert_array_equal(_run(xi, wi, ph, pw, algo).astype(np.float64), yi_ref)


def test_zero_padding_is_the_unpadded_entry(oracle):
    from helpers import run_library
    x, w = uniform((2, 12, 11, 13), 475), uniform((20, 12, 3, 3), 476)
    np.testing.assert_array_equal(_run(x, w, 0, 0, 1), run_library(x, w, entry="general", algo=1))

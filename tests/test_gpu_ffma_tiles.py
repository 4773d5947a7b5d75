"""fp32 general kernel: every tile shape (a block's output rows x segments of adjacent outputs per thread) gives the
same bits as the default 32 x 8 tile and matches the oracle within the fp32 bound; the launcher picks the shape that
wastes least of its tile on the map at hand."""
import numpy as np
import pytest

from helpers import FFMA_TOL, assert_parity, run_library
from workloads import uniform

pytestmark = pytest.mark.gpu
ALGO_FFMA = 1

# N, C, H, W, K, R, S: output maps of 30 x 30 (three segments of 10), 26 x 26 (three of 9), 54 wide (six of 9),
# 12 x 12 (two of 6), a ragged filter count, a map wider than the odd-width tiles (they must not be taken)
SHAPES = [
    (2, 12, 32, 32, 70, 3, 3),
    (2, 6, 32, 32, 64, 7, 7),
    (1, 10, 20, 56, 24, 3, 3),
    (3, 20, 14, 14, 130, 3, 3),
    (2, 9, 17, 70, 40, 5, 5),
    (2, 16, 9, 31, 64, 1, 1),
]


@pytest.mark.parametrize("dims", SHAPES)
def test_ffma_tile_shapes_agree(oracle, dims, monkeypatch):
    N, C, H, W, K, R, S = dims
    x, w = uniform((N, C, H, W), 1201), uniform((K, C, R, S), 1202)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    monkeypatch.setenv("CONV2D_B200_FFMA_TILE", "0")
    y0 = run_library(x, w, entry="general", algo=ALGO_FFMA)
    assert_parity(y0, y_ref, yabs, FFMA_TOL, f"fp32, default tile {dims}")
    for tile in (1, 2, 4, 5, 6):
        monkeypatch.setenv("CONV2D_B200_FFMA_TILE", str(tile))
        np.testing.assert_array_equal(run_library(x, w, entry="general", algo=ALGO_FFMA), y0, err_msg=f"tile {tile} {dims}")
    monkeypatch.delenv("CONV2D_B200_FFMA_TILE")
    np.testing.assert_array_equal(run_library(x, w, entry="general", algo=ALGO_FFMA), y0, err_msg=f"planner's tile {dims}")

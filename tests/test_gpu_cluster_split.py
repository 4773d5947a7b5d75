"""Split contraction as a two-block cluster (few output tiles: 14 x 14 and 7 x 7 layers): the two halves of the
channel blocks of a tile run on two thread blocks that exchange partial sums through distributed shared memory.
Checked against the oracle, and against the variant that adds into a zeroed output with atomics.
"""
import numpy as np
import pytest

from helpers import TF32_TOL, B16_TOL, assert_parity, bf16_values, run_library
from workloads import small_integers, uniform

pytestmark = pytest.mark.gpu
ALGO_TF32, ALGO_16BIT = 2, 3

SHAPES = [
    # N, C, H, W, K, R, S
    (8, 64, 14, 14, 128, 3, 3),      # two 32-pixel blocks per tile: one for each block of the pair
    (4, 128, 14, 14, 256, 3, 3),     # two filter blocks
    (16, 512, 7, 7, 512, 3, 3),      # 7 x 7 images, 32 channel blocks
    (3, 48, 16, 16, 130, 3, 3),      # odd number of channel blocks (3): the halves differ; second filter block nearly empty
    (2, 96, 20, 20, 128, 5, 5),
    (6, 40, 12, 12, 256, 1, 3),      # rectangular taps
]


def _plan(dims, algo=ALGO_TF32):
    import paper_1705_10591_b200 as lib
    return lib.conv2d_fwd_plan_describe(*dims, algo)


@pytest.mark.parametrize("dims", SHAPES)
def test_cluster_split_exact_on_integers(oracle, dims):
    assert _plan(dims).get("cluster") == 1, "the shape was meant to take the two-block cluster"
    N, C, H, W, K, R, S = dims
    x, w = small_integers((N, C, H, W), 971), small_integers((K, C, R, S), 972)
    y_ref, _ = oracle.conv2d_oracle(x, w)
    np.testing.assert_array_equal(run_library(x, w, entry="general", algo=ALGO_TF32).astype(np.float64), y_ref)


@pytest.mark.parametrize("dims", SHAPES)
def test_cluster_split_within_tolerance(oracle, dims):
    N, C, H, W, K, R, S = dims
    x, w = uniform((N, C, H, W), 973), uniform((K, C, R, S), 974)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="general", algo=ALGO_TF32), y_ref, yabs, TF32_TOL, f"cluster {dims}")


@pytest.mark.parametrize("tile_px", [96, 160, 192])
def test_cluster_split_with_odd_and_even_block_counts(oracle, monkeypatch, tile_px):
    """3, 5 and 6 blocks of 32 pixels per tile: with an odd count one block of the pair stores one block more."""
    monkeypatch.setenv("CONV2D_B200_TF32_TILE_PX", str(tile_px))
    dims = (8, 64, 14, 14, 128, 3, 3)
    plan = _plan(dims)
    assert plan.get("cluster") == 1 and plan.get("tile_px") == tile_px
    N, C, H, W, K, R, S = dims
    x, w = small_integers((N, C, H, W), 975), small_integers((K, C, R, S), 976)
    y_ref, _ = oracle.conv2d_oracle(x, w)
    np.testing.assert_array_equal(run_library(x, w, entry="general", algo=ALGO_TF32).astype(np.float64), y_ref)


def test_cluster_split_16bit_operands(oracle):
    dims = next((d for d in SHAPES if _plan(d, ALGO_16BIT).get("cluster") == 1), None)
    assert dims is not None, "no shape of the list takes the cluster with 16-bit operands"
    N, C, H, W, K, R, S = dims
    x, _ = bf16_values(uniform((N, C, H, W), 977))
    w, _ = bf16_values(uniform((K, C, R, S), 978))
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="bf16"), y_ref, yabs, B16_TOL, f"cluster bf16 {dims}")


def test_atomic_variant_still_serves_the_shape(oracle, monkeypatch):
    """With the cluster switched off the two items add into a zeroed output; integers give the same bits."""
    monkeypatch.setenv("CONV2D_B200_TF32_KSPLIT_CLUSTER", "0")
    dims = (4, 128, 14, 14, 256, 3, 3)
    plan = _plan(dims)
    assert plan.get("cluster") == 0 and plan.get("ksplit") == 2
    N, C, H, W, K, R, S = dims
    x, w = small_integers((N, C, H, W), 979), small_integers((K, C, R, S), 980)
    y_ref, _ = oracle.conv2d_oracle(x, w)
    np.testing.assert_array_equal(run_library(x, w, entry="general", algo=ALGO_TF32).astype(np.float64), y_ref)

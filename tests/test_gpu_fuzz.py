"""Seeded random shapes through every general-case path: the planner has many branches (operand roles, item size,
flat or patch addressing, folded taps, resident or streamed filters, split contraction), and each shape below lands in
some combination of them.  Every output element is compared with the oracle.
"""
import numpy as np
import pytest

from helpers import FFMA_TOL, TF32_TOL, assert_parity, bf16_values, run_library
from workloads import uniform

pytestmark = pytest.mark.gpu

ALGO_FFMA, ALGO_TF32 = 1, 2


def _draw(seed):
    """One shape from a seeded stream of uniforms; sizes are log-distributed and the work is capped."""
    u = uniform((16,), 9000 + seed, 0.0, 1.0)

    def log_int(t, lo, hi):
        return int(round(lo * (hi / lo) ** float(t)))

    taps = (1, 2, 3, 5, 7)
    R, S = taps[int(u[0] * 5) % 5], taps[int(u[1] * 5) % 5]
    N = log_int(u[2], 1, 5)
    C = log_int(u[3], 1, 200)
    H = max(R, log_int(u[4], 3, 48))
    W = max(S, log_int(u[5], 3, 900))
    K = log_int(u[6], 1, 320)
    while N * K * C * R * S * (H - R + 1) * (W - S + 1) > 6e8 and K > 1:      # keep the oracle under a second
        K = max(1, K // 2)
    while N * K * C * R * S * (H - R + 1) * (W - S + 1) > 6e8 and C > 1:
        C = max(1, C // 2)
    return N, C, H, W, K, R, S


SHAPES = sorted({_draw(s) for s in range(72)})


def _tc_available(dims, algo):
    import paper_1705_10591_b200 as lib
    try:
        return lib.conv2d_fwd_workspace_size(*dims, algo) > 0
    except lib.Conv2dError:
        return False


@pytest.mark.parametrize("dims", SHAPES)
def test_random_shape_all_paths(oracle, dims):
    N, C, H, W, K, R, S = dims
    x, w = uniform((N, C, H, W), 461), uniform((K, C, R, S), 462)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="general", algo=ALGO_FFMA), y_ref, yabs, FFMA_TOL, f"fp32 {dims}")
    if _tc_available(dims, ALGO_TF32):
        assert_parity(run_library(x, w, entry="general", algo=ALGO_TF32), y_ref, yabs, TF32_TOL, f"tf32 {dims}")
    if _tc_available(dims, 3):
        xb, wb = bf16_values(x)[0], bf16_values(w)[0]
        yb_ref, yb_abs = oracle.conv2d_oracle(xb, wb)
        assert_parity(run_library(xb, wb, entry="bf16"), yb_ref, yb_abs, 1e-5, f"bf16 {dims}")


def test_the_random_shapes_reach_the_planner_branches():
    """The stream above must contain wide images, few-channel shapes, many-channel shapes, many-filter shapes, 1 x 1 taps."""
    assert any(W >= 400 for (_, _, _, W, _, _, _) in SHAPES)
    assert any(C <= 3 for (_, C, _, _, _, _, _) in SHAPES)
    assert any(K > 128 for (_, _, _, _, K, _, _) in SHAPES)
    assert any(R == 1 and S == 1 for (*_, R, S) in SHAPES)
    assert any(C >= 64 for (_, C, _, _, _, _, _) in SHAPES)
    assert len(SHAPES) >= 60


def _draw_pointwise(seed):
    """A 1 x 1 shape the kernel fed by tensor-map copies takes: H*W and C multiples of 8 (so that both operand
    types qualify), at most 256 channels."""
    u = uniform((8,), 9500 + seed, 0.0, 1.0)

    def log_int(t, lo, hi):
        return int(round(lo * (hi / lo) ** float(t)))

    N = log_int(u[0], 1, 24)
    C = 8 * log_int(u[1], 1, 32)
    H = log_int(u[2], 1, 40)
    W = 8 * log_int(u[3], 1, 12)
    K = log_int(u[4], 1, 400)
    while N * K * C * H * W > 4e8 and N > 1:
        N = max(1, N // 2)
    return N, C, H, W, K, 1, 1


POINTWISE_SHAPES = sorted({_draw_pointwise(s) for s in range(40)})


@pytest.mark.parametrize("dims", POINTWISE_SHAPES)
def test_random_pointwise_shapes(oracle, dims):
    import paper_1705_10591_b200 as lib
    N, C, H, W, K, R, S = dims
    assert lib.conv2d_fwd_plan_describe(*dims, ALGO_TF32).get("kernel") == "pointwise_tma"
    assert lib.conv2d_fwd_plan_describe(*dims, 3).get("kernel") == "pointwise_tma"
    x, w = uniform((N, C, H, W), 463), uniform((K, C, R, S), 464)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="general", algo=ALGO_TF32), y_ref, yabs, TF32_TOL, f"tf32 {dims}")
    xb, wb = bf16_values(x)[0], bf16_values(w)[0]
    yb_ref, yb_abs = oracle.conv2d_oracle(xb, wb)
    assert_parity(run_library(xb, wb, entry="bf16"), yb_ref, yb_abs, 1e-5, f"bf16 {dims}")


def _draw_pointwise_deep(seed):
    """1 x 1 shapes with up to 1024 channels and 600 filters: streamed filter banks and the two-SM form."""
    u = uniform((8,), 9600 + seed, 0.0, 1.0)

    def log_int(t, lo, hi):
        return int(round(lo * (hi / lo) ** float(t)))

    N = log_int(u[0], 1, 16)
    C = 8 * log_int(u[1], 16, 128)
    H = log_int(u[2], 1, 24)
    W = 8 * log_int(u[3], 1, 6)
    K = log_int(u[4], 100, 600)
    while N * K * C * H * W > 6e8 and N > 1:
        N = max(1, N // 2)
    return N, C, H, W, K, 1, 1


POINTWISE_DEEP_SHAPES = sorted({_draw_pointwise_deep(s) for s in range(30)})


@pytest.mark.parametrize("dims", POINTWISE_DEEP_SHAPES)
def test_random_deep_pointwise_shapes(oracle, dims, monkeypatch):
    import paper_1705_10591_b200 as lib
    N, C, H, W, K, R, S = dims
    # the planner's own choice, the one-SM form and the two-SM form in turn
    monkeypatch.setenv("CONV2D_B200_TMA_PAIR", str((N + C // 8 + H + K) % 3))
    monkeypatch.setenv("CONV2D_B200_TMA_KSPLIT", str(1 + (C // 8 + W + K) % 2))     # the planner's choice / split wherever possible
    assert lib.conv2d_fwd_plan_describe(*dims, ALGO_TF32).get("kernel") == "pointwise_tma"
    assert lib.conv2d_fwd_plan_describe(*dims, 3).get("kernel") == "pointwise_tma"
    x, w = uniform((N, C, H, W), 465), uniform((K, C, R, S), 466)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="general", algo=ALGO_TF32), y_ref, yabs, TF32_TOL, f"tf32 {dims}")
    xb, wb = bf16_values(x)[0], bf16_values(w)[0]
    yb_ref, yb_abs = oracle.conv2d_oracle(xb, wb)
    assert_parity(run_library(xb, wb, entry="bf16"), yb_ref, yb_abs, 1e-5, f"bf16 {dims}")


def _draw_few_tiles(seed):
    """Small images with many channels and filters: the shapes whose contraction is split over a two-block cluster."""
    u = uniform((8,), 9700 + seed, 0.0, 1.0)
    taps = (1, 2, 3, 5)
    R, S = taps[int(u[0] * 4) % 4], taps[int(u[1] * 4) % 4]
    if R == 1 and S == 1:
        S = 3
    N = 1 + int(u[2] * 8)
    C = 16 * (2 + int(u[3] * 30))
    H = max(R, 5 + int(u[4] * 12))
    W = max(S, 5 + int(u[5] * 12))
    K = 65 + int(u[6] * 300)
    while N * K * C * R * S * (H - R + 1) * (W - S + 1) > 6e8 and C > 32:
        C //= 2
    return N, C, H, W, K, R, S


FEW_TILE_SHAPES = sorted({_draw_few_tiles(s) for s in range(30)})


@pytest.mark.parametrize("dims", FEW_TILE_SHAPES)
def test_random_few_tile_shapes(oracle, dims):
    N, C, H, W, K, R, S = dims
    x, w = uniform((N, C, H, W), 465), uniform((K, C, R, S), 466)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="general", algo=ALGO_TF32), y_ref, yabs, TF32_TOL, f"tf32 {dims}")


def test_the_few_tile_stream_reaches_the_cluster():
    import paper_1705_10591_b200 as lib
    assert sum(lib.conv2d_fwd_plan_describe(*d, ALGO_TF32).get("cluster") == 1 for d in FEW_TILE_SHAPES) >= 8

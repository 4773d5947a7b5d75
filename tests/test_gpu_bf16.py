"""GPU parity of the 16-bit operand entry (bf16 in, fp32 accumulate on the tensor cores) against the CPU oracle.

The inputs are bf16 values, so every product x*w is exact in fp32 and only the fp32 accumulation differs from the
oracle's double sum: the bar is the one of the fp32 FMA paths, |y - y_ref| <= 1e-5 * sum|x*w|, and integer-valued
inputs must match bit for bit.
"""
import numpy as np
import pytest

from helpers import BF16_TOL, assert_parity, bf16_values, run_library
from workloads import CONFIGS, make_inputs, small_integers, uniform

pytestmark = pytest.mark.gpu

ALGO_BF16 = 3

SHAPES = [
    # N, C, H, W, K, R, S
    (1, 3, 12, 13, 5, 3, 3),       # fewer channels than one 8-channel unit
    (2, 17, 20, 21, 70, 3, 3),     # K and C not multiples of the tiles
    (1, 8, 41, 37, 64, 5, 5),
    (2, 6, 15, 44, 9, 7, 7),
    (3, 32, 9, 9, 16, 1, 1),       # exactly one 32-channel block
    (2, 5, 3, 3, 4, 3, 3),         # one output per map
    (1, 64, 14, 14, 96, 3, 3),     # operand-swap path with zero-padded filters
    (2, 40, 10, 12, 300, 3, 3),    # two filter blocks, partial second channel block
    (1, 72, 16, 16, 130, 1, 7),    # three channel blocks, the last one quarter full
    (5, 33, 7, 9, 128, 3, 3),      # one channel beyond a block; ragged last pixel tile
    (2, 96, 12, 12, 128, 1, 1),    # 1 x 1 with resident filters
]


def _available(dims):
    import paper_1705_10591_b200 as lib
    try:
        return lib.conv2d_fwd_workspace_size(*dims, ALGO_BF16) > 0
    except lib.Conv2dError:
        return False


@pytest.mark.parametrize("dims", SHAPES)
def test_bf16_exact_on_integers(oracle, dims):
    if not _available(dims):
        pytest.skip("no tensor-core instance for this shape")
    N, C, H, W, K, R, S = dims
    x, w = small_integers((N, C, H, W), 411), small_integers((K, C, R, S), 412)
    y_ref, _ = oracle.conv2d_oracle(x, w)
    y = run_library(x, w, entry="bf16")
    np.testing.assert_array_equal(y.astype(np.float64), y_ref)


@pytest.mark.parametrize("dims", SHAPES)
def test_bf16_within_tolerance(oracle, dims):
    if not _available(dims):
        pytest.skip("no tensor-core instance for this shape")
    N, C, H, W, K, R, S = dims
    x, _ = bf16_values(uniform((N, C, H, W), 413))
    w, _ = bf16_values(uniform((K, C, R, S), 414))
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    r = assert_parity(run_library(x, w, entry="bf16"), y_ref, yabs, BF16_TOL, f"bf16 {dims}")
    print(f"bf16 {dims} max ratio {r:.3e}")


def _sampled_planes(cfg, count, seed):
    n = (uniform((count,), seed, 0, 1) * cfg.N).astype(np.int64)
    k = (uniform((count,), seed + 1, 0, 1) * cfg.K).astype(np.int64)
    return sorted({(0, 0), (cfg.N - 1, cfg.K - 1)} | set(zip(n.tolist(), k.tolist())))


@pytest.mark.parametrize("name", ["cfg3", "cfg4", "cfg5_r1", "cfg5_r3", "cfg5_r5", "cfg5_r7"])
def test_bf16_full_size_configs(oracle, name):
    """Benchmark shapes at full size with the inputs rounded to bf16; sampled (image, map) planes are checked."""
    cfg = CONFIGS[name]
    dims = (cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S)
    if not _available(dims):
        pytest.skip("no tensor-core instance for this shape")
    x, w = make_inputs(cfg)
    x, w = bf16_values(x)[0], bf16_values(w)[0]
    y = run_library(x, w, entry="bf16")
    worst = 0.0
    for n, k in _sampled_planes(cfg, 32, 600 + cfg.seed):
        y_ref, yabs = oracle.conv2d_oracle_range(x, w, n_range=(n, n + 1), k_range=(k, k + 1))
        worst = max(worst, assert_parity(y[n:n + 1, k:k + 1], y_ref, yabs, BF16_TOL, f"{name} plane {(n, k)}"))
    assert np.isfinite(y).all()
    print(f"{name} bf16 max ratio {worst:.3e}")


def test_bf16_prepacked_filters_flag(oracle):
    import torch
    import paper_1705_10591_b200 as lib
    dims = (2, 40, 10, 12, 300, 3, 3)
    N, C, H, W, K, R, S = dims
    x, _ = bf16_values(uniform((N, C, H, W), 415))
    w, _ = bf16_values(uniform((K, C, R, S), 416))
    ws = torch.zeros(lib.conv2d_fwd_workspace_size(*dims, ALGO_BF16), dtype=torch.uint8, device="cuda:0")
    y1 = run_library(x, w, entry="bf16", workspace=ws)
    y2 = run_library(x, w, entry="bf16", workspace=ws, flags=lib.FLAG_WEIGHTS_PACKED)
    np.testing.assert_array_equal(y1, y2)

"""GPU parity of the 16-bit operand entry (bf16 or fp16 in, fp32 accumulate on the tensor cores) against the CPU oracle.

The inputs are 16-bit values, so every product x*w is exact in fp32 and only the fp32 accumulation differs from the
oracle's double sum: the bar is the one of the fp32 FMA paths, |y - y_ref| <= 1e-5 * sum|x*w|, and integer-valued
inputs must match bit for bit.
"""
import numpy as np
import pytest

from helpers import B16_TOL, assert_parity, bf16_values, fp16_values, run_library
from workloads import CONFIGS, make_inputs, small_integers, uniform

pytestmark = pytest.mark.gpu

ALGO_16BIT = 3
ROUND = {"bf16": bf16_values, "fp16": fp16_values}
TYPES = ["bf16", "fp16"]

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
        return lib.conv2d_fwd_workspace_size(*dims, ALGO_16BIT) > 0
    except lib.Conv2dError:
        return False


@pytest.mark.parametrize("dims", SHAPES)
@pytest.mark.parametrize("kind", TYPES)
def test_16bit_exact_on_integers(oracle, dims, kind):
    if not _available(dims):
        pytest.skip("no tensor-core instance for this shape")
    N, C, H, W, K, R, S = dims
    x, w = small_integers((N, C, H, W), 411), small_integers((K, C, R, S), 412)
    y_ref, _ = oracle.conv2d_oracle(x, w)
    y = run_library(x, w, entry=kind)
    np.testing.assert_array_equal(y.astype(np.float64), y_ref)


@pytest.mark.parametrize("dims", SHAPES)
@pytest.mark.parametrize("kind", TYPES)
def test_16bit_within_tolerance(oracle, dims, kind):
    if not _available(dims):
        pytest.skip("no tensor-core instance for this shape")
    N, C, H, W, K, R, S = dims
    x, _ = ROUND[kind](uniform((N, C, H, W), 413))
    w, _ = ROUND[kind](uniform((K, C, R, S), 414))
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    r = assert_parity(run_library(x, w, entry=kind), y_ref, yabs, B16_TOL, f"{kind} {dims}")
    print(f"{kind} {dims} max ratio {r:.3e}")


@pytest.mark.parametrize("name", ["cfg3", "cfg4", "cfg5_r1", "cfg5_r3", "cfg5_r5", "cfg5_r7"])
@pytest.mark.parametrize("kind", TYPES)
def test_16bit_full_size_configs(oracle, name, kind):
    """Benchmark shapes at full size with the inputs rounded to the 16-bit type; every output element is checked."""
    cfg = CONFIGS[name]
    dims = (cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S)
    if not _available(dims):
        pytest.skip("no tensor-core instance for this shape")
    x, w = make_inputs(cfg)
    x, w = ROUND[kind](x)[0], ROUND[kind](w)[0]
    y = run_library(x, w, entry=kind)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    worst = assert_parity(y, y_ref, yabs, B16_TOL, f"{name} {kind}")
    print(f"{name} {kind} max ratio over all {y.size} outputs {worst:.3e}")


def test_16bit_prepacked_filters_flag(oracle):
    import torch
    import paper_1705_10591_b200 as lib
    dims = (2, 40, 10, 12, 300, 3, 3)
    N, C, H, W, K, R, S = dims
    x, _ = bf16_values(uniform((N, C, H, W), 415))
    w, _ = bf16_values(uniform((K, C, R, S), 416))
    ws = torch.zeros(lib.conv2d_fwd_workspace_size(*dims, ALGO_16BIT), dtype=torch.uint8, device="cuda:0")
    y1 = run_library(x, w, entry="bf16", workspace=ws)
    y2 = run_library(x, w, entry="bf16", workspace=ws, flags=lib.FLAG_WEIGHTS_PACKED)
    np.testing.assert_array_equal(y1, y2)


def test_16bit_single_pixel_loads_agree_with_paired_loads(oracle, monkeypatch):
    """H*W even takes paired-pixel producer loads by default; the one-pixel loads must give the same bits."""
    dims = (2, 40, 10, 12, 300, 3, 3)
    N, C, H, W, K, R, S = dims
    x, _ = bf16_values(uniform((N, C, H, W), 417))
    w, _ = bf16_values(uniform((K, C, R, S), 418))
    y_pair = run_library(x, w, entry="bf16")
    monkeypatch.setenv("CONV2D_B200_B16_PAIR", "0")
    y_single = run_library(x, w, entry="bf16")
    np.testing.assert_array_equal(y_pair, y_single)


def test_the_two_operand_types_are_told_apart(oracle):
    """The same bit patterns read as bf16 and as fp16 are different numbers: each call must follow its own type."""
    dims = (1, 32, 8, 8, 16, 3, 3)
    N, C, H, W, K, R, S = dims
    x, _ = fp16_values(uniform((N, C, H, W), 419))
    w, _ = fp16_values(uniform((K, C, R, S), 420))
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="fp16"), y_ref, yabs, B16_TOL, "fp16")
    xb, wb = bf16_values(x)[0], bf16_values(w)[0]            # coarser values: a different, also checkable result
    yb_ref, yb_abs = oracle.conv2d_oracle(xb, wb)
    assert_parity(run_library(xb, wb, entry="bf16"), yb_ref, yb_abs, B16_TOL, "bf16")
    assert np.abs(yb_ref - y_ref).max() > 1e-4 * yabs.max()

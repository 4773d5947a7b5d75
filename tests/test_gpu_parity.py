"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded inputs.

Bars: integer-valued inputs must match bit for bit; real-valued inputs within
|y - y_ref| <= 1e-5 * sum|x*w| (fp32 FMA paths) or 2e-3 * sum|x*w| (TF32 tensor-core path), elementwise.
"""
import numpy as np
import pytest

from helpers import FFMA_TOL, TF32_TOL, assert_parity, run_library
from workloads import CONFIGS, make_inputs, small_integers, uniform

pytestmark = pytest.mark.gpu

ALGO_AUTO, ALGO_FFMA, ALGO_TF32 = 0, 1, 2


# ---------------------------------------------------------------- special case (one input channel)

SINGLE_SHAPES = [
    # N, H, W, K, R, S
    (1, 64, 64, 8, 3, 3),        # cfg1 shape
    (1, 9, 10, 3, 3, 3),         # W % 4 != 0, tiny
    (2, 37, 53, 5, 5, 5),        # odd everything, Q % 4 != 0
    (1, 19, 1031, 2, 3, 3),      # three column tiles with a ragged last one
    (3, 40, 520, 4, 7, 7),       # Q = 514: second column tile nearly empty
    (1, 33, 36, 1, 1, 1),        # 1x1: no data sharing at all
    (1, 5, 5, 7, 5, 5),          # filter as large as the image: one output per map
    (2, 21, 24, 3, 3, 5),        # rectangular taps -> shape-agnostic kernel
    (1, 70, 16, 6, 5, 5),        # more rows than one tile, Q = 12 (vector stores)
    (1, 23, 2100, 3, 5, 5),      # wide persistent kernel: two column tiles (2048 + 48), 128-bit stores
    (2, 11, 1032, 5, 3, 3),      # wide kernel, Q = 1030: 64-bit stores, odd filter count
    (1, 9, 1028, 2, 7, 7),       # wide kernel, 7 x 7, band taller than the image's output rows
    (1, 14, 1040, 4, 1, 1),      # wide kernel, 1 x 1
    (1, 12, 1032, 3, 3, 3),      # shifted wide kernel: Q = 1030 (8-byte aligned rows), odd filter count
    (1, 10, 388, 3, 3, 3),       # shifted wide kernel on a narrow image: Q = 386, most of the 2048 columns idle
    (2, 14, 520, 5, 3, 3),       # shifted wide kernel: Q = 518, two images, two bands
    (2, 20, 2100, 5, 3, 3),      # shifted wide kernel: Q = 2098, two column tiles, three bands
    (1, 14, 1040, 4, 7, 7),      # wide kernel, 7 x 7, Q = 1034: 64-bit stores
]


@pytest.mark.parametrize("dims", SINGLE_SHAPES)
def test_single_channel_exact_on_integers(oracle, dims):
    N, H, W, K, R, S = dims
    x, w = small_integers((N, 1, H, W), 301), small_integers((K, 1, R, S), 302)
    y_ref, _ = oracle.conv2d_oracle(x, w)
    y = run_library(x, w, entry="single")
    np.testing.assert_array_equal(y.astype(np.float64), y_ref)


@pytest.mark.parametrize("dims", SINGLE_SHAPES)
def test_single_channel_within_tolerance(oracle, dims):
    N, H, W, K, R, S = dims
    x, w = uniform((N, 1, H, W), 303), uniform((K, 1, R, S), 304)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="single"), y_ref, yabs, FFMA_TOL, f"single {dims}")


@pytest.mark.parametrize("knobs", [
    dict(CONV2D_B200_SC_ROWS="1"), dict(CONV2D_B200_SC_TILE_H="5"),                       # packed-FMA kernel
    dict(CONV2D_B200_SC_UNIT="1"), dict(CONV2D_B200_SC_UNIT="2"), dict(CONV2D_B200_SC_UNIT="4"),   # unit ablation
    dict(CONV2D_B200_SC_WIDE="0"),                                                        # tile kernel on wide images
    dict(CONV2D_B200_SC_SHIFT="0"),                                                       # wide kernel with 64-bit stores
    dict(CONV2D_B200_SC_PACKED="0", CONV2D_B200_SC_WSRC="0"),                              # scalar-FMA kernel
    dict(CONV2D_B200_SC_PACKED="0", CONV2D_B200_SC_WSRC="1", CONV2D_B200_SC_ROWS="1"),
    dict(CONV2D_B200_SC_PACKED="0", CONV2D_B200_SC_TILE_H="5", CONV2D_B200_SC_WSRC="0", CONV2D_B200_SC_ROWS="1")])
def test_single_channel_variants_agree(oracle, monkeypatch, knobs):
    for k, v in knobs.items():
        monkeypatch.setenv(k, v)
    for dims in [(1, 64, 64, 8, 3, 3), (2, 37, 53, 5, 5, 5), (1, 19, 1031, 2, 3, 3), (1, 30, 40, 3, 7, 7),
                 (1, 12, 1100, 3, 5, 5), (1, 12, 1032, 3, 3, 3)]:
        N, H, W, K, R, S = dims
        x, w = small_integers((N, 1, H, W), 305), small_integers((K, 1, R, S), 306)
        y_ref, _ = oracle.conv2d_oracle(x, w)
        np.testing.assert_array_equal(run_library(x, w, entry="single").astype(np.float64), y_ref)


def test_cfg1_single_channel(oracle):
    x, w = make_inputs(CONFIGS["cfg1"])
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="single"), y_ref, yabs, FFMA_TOL, "cfg1")


def test_general_entry_with_one_channel_matches_single_channel_entry(oracle):
    x, w = make_inputs(CONFIGS["cfg1"])
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    y_g = run_library(x, w, entry="general", algo=ALGO_FFMA)
    assert_parity(y_g, y_ref, yabs, FFMA_TOL, "cfg1 via general")
    xi, wi = small_integers(x.shape, 307), small_integers(w.shape, 308)
    np.testing.assert_array_equal(run_library(xi, wi, entry="general", algo=ALGO_FFMA),
                                  run_library(xi, wi, entry="single"))


def test_cfg2_full_size_every_output(oracle):
    """Full 4096 x 4096, 32 filters of 5 x 5, in the launch configuration the benchmark times: every output of
    every map, compared map by map so that the reference never holds more than one map in memory."""
    cfg = CONFIGS["cfg2"]
    x, w = make_inputs(cfg)
    y = run_library(x, w, entry="single")
    assert y.shape == (1, 32, 4092, 4092)
    worst = 0.0
    for k in range(cfg.K):
        y_ref, yabs = oracle.conv2d_oracle_range(x, w, k_range=(k, k + 1))
        worst = max(worst, assert_parity(y[:, k:k + 1], y_ref, yabs, FFMA_TOL, f"cfg2 map {k}"))
    print(f"cfg2 max ratio over all {y.size} outputs {worst:.3e}")


# ---------------------------------------------------------------- general case

GENERAL_SHAPES = [
    # N, C, H, W, K, R, S
    (1, 3, 12, 13, 5, 3, 3),
    (2, 17, 20, 21, 70, 3, 3),     # K and C not multiples of the tiles
    (1, 8, 41, 37, 64, 5, 5),
    (2, 6, 15, 44, 9, 7, 7),
    (3, 32, 9, 9, 16, 1, 1),
    (1, 4, 11, 10, 3, 2, 4),       # rectangular taps -> shape-agnostic kernel
    (2, 12, 19, 21, 70, 2, 2),     # 2 x 2 and 4 x 4 taps: the filters a stride-2 rewriting produces
    (1, 12, 23, 40, 33, 4, 4),
    (2, 5, 3, 3, 4, 3, 3),         # one output per map
    (1, 64, 14, 14, 96, 3, 3),     # 96 filters: operand-swap path with zero-padded filters
    (2, 20, 10, 12, 300, 3, 3),    # 300 filters: two filter blocks, partial last channel block
    (1, 40, 16, 16, 130, 1, 7),    # 1 x 7 taps, 130 filters (pixels stay the M operand)
    (5, 33, 7, 9, 128, 3, 3),      # batch*H*W = 315 pixels: ragged last tile, images change inside a tile
    (1, 16, 6, 70, 72, 5, 3),      # wide rows: horizontal wrap inside a tile
    (2, 48, 12, 12, 128, 1, 1),    # 1 x 1 with resident filters
    (1, 24, 9, 10, 1000, 3, 3),    # 1000 filters: eight filter blocks, the last one partial
    (1, 200, 8, 8, 24, 5, 5),      # long contraction, few filters and pixels: stacked taps with a split contraction
    (3, 7, 33, 31, 64, 3, 2),      # odd image width, even tap count per row
]


@pytest.mark.parametrize("dims", GENERAL_SHAPES)
@pytest.mark.parametrize("algo", [ALGO_FFMA, ALGO_AUTO])
def test_general_exact_on_integers(oracle, dims, algo):
    N, C, H, W, K, R, S = dims
    x, w = small_integers((N, C, H, W), 401), small_integers((K, C, R, S), 402)
    y_ref, _ = oracle.conv2d_oracle(x, w)
    y = run_library(x, w, entry="general", algo=algo)
    np.testing.assert_array_equal(y.astype(np.float64), y_ref)


@pytest.mark.parametrize("dims", GENERAL_SHAPES)
def test_general_ffma_within_tolerance(oracle, dims):
    N, C, H, W, K, R, S = dims
    x, w = uniform((N, C, H, W), 403), uniform((K, C, R, S), 404)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="general", algo=ALGO_FFMA), y_ref, yabs, FFMA_TOL, f"ffma {dims}")


def _tf32_available(cfg_dims):
    import paper_1705_10591_b200 as lib
    try:
        return lib.conv2d_fwd_workspace_size(*cfg_dims, ALGO_TF32) > 0
    except lib.Conv2dError:
        return False


@pytest.mark.parametrize("dims", GENERAL_SHAPES)
def test_general_tf32_within_tolerance(oracle, dims):
    if not _tf32_available(dims):
        pytest.skip("no tensor-core instance for this shape")
    import paper_1705_10591_b200 as lib
    from oracle.conv2d_oracle import MODE_TF32_RNA, MODE_TF32_TRUNC
    N, C, H, W, K, R, S = dims
    x, w = uniform((N, C, H, W), 405), uniform((K, C, R, S), 406)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    y = run_library(x, w, entry="general", algo=ALGO_TF32)
    assert_parity(y, y_ref, yabs, TF32_TOL, f"tf32 {dims}")
    # Diagnostic, far tighter than the bar: against the oracle fed TF32 operands only the fp32 accumulation
    # order differs.  The general kernel rounds its operands to nearest when it stages them; the 1 x 1 kernel
    # fed by tensor-map copies hands fp32 bits to the tensor core, which truncates them.
    tma = lib.conv2d_fwd_plan_describe(*dims, ALGO_TF32).get("kernel") == "pointwise_tma"
    y_t, yabs_t = oracle.conv2d_oracle(x, w, mode=MODE_TF32_TRUNC if tma else MODE_TF32_RNA)
    assert_parity(y, y_t, yabs_t, 2e-5, f"tf32 vs TF32-operand oracle {dims}")


FULL = ["cfg3", "cfg4", "cfg5_r1", "cfg5_r3", "cfg5_r5", "cfg5_r7"]


_FULL_REF = {}     # one configuration at a time: (x, w, y_ref, yabs) of the configuration the tests are on


def _full_reference(oracle, name):
    """Oracle outputs of EVERY element of a benchmark configuration (seconds on the host cores), computed once per
    configuration and shared by the algorithms tested on it."""
    if name not in _FULL_REF:
        _FULL_REF.clear()
        cfg = CONFIGS[name]
        x, w = make_inputs(cfg)
        y_ref, yabs = oracle.conv2d_oracle(x, w)
        _FULL_REF[name] = (x, w, y_ref, yabs)
    return _FULL_REF[name]


@pytest.mark.parametrize("algo", [ALGO_FFMA, ALGO_TF32])
@pytest.mark.parametrize("name", FULL)
def test_full_size_configs(oracle, name, algo):
    """Benchmark shapes at full size, in the launch configuration the benchmark times: every output element of
    every (image, map) plane is compared with the oracle."""
    cfg = CONFIGS[name]
    dims = (cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S)
    if algo == ALGO_TF32 and not _tf32_available(dims):
        pytest.skip("no tensor-core instance for this shape")
    x, w, y_ref, yabs = _full_reference(oracle, name)
    y = run_library(x, w, entry="general", algo=algo)
    tol = FFMA_TOL if algo == ALGO_FFMA else TF32_TOL
    worst = assert_parity(y, y_ref, yabs, tol, f"{name} algo={algo}")
    print(f"{name} algo={algo} max ratio over all {y.size} outputs {worst:.3e}")


@pytest.mark.parametrize("algo", [ALGO_FFMA, ALGO_TF32])
def test_full_size_config_exact_on_integers(oracle, algo):
    """One benchmark shape at full size with small-integer inputs: every output bit for bit."""
    cfg = CONFIGS["cfg5_r3"]
    x = small_integers((cfg.N, cfg.C, cfg.H, cfg.W), 441)
    w = small_integers((cfg.K, cfg.C, cfg.R, cfg.S), 442)
    y_ref, _ = oracle.conv2d_oracle(x, w)
    np.testing.assert_array_equal(run_library(x, w, entry="general", algo=algo).astype(np.float64), y_ref)


def test_auto_falls_back_to_fp32_when_no_tensor_core_instance_fits(oracle, monkeypatch):
    """With the flat pixel run only, a very wide image needs a staged halo beyond shared memory: AUTO must still
    give the right answer."""
    import paper_1705_10591_b200 as lib
    monkeypatch.setenv("CONV2D_B200_TF32_PATCH", "0")
    dims = (1, 16, 6, 6000, 8, 5, 5)
    assert not _tf32_available(dims)
    with pytest.raises(lib.Conv2dError) as e:
        lib.conv2d_fwd_workspace_size(*dims, ALGO_TF32)
    assert e.value.status == 5
    N, C, H, W, K, R, S = dims
    x, w = small_integers((N, C, H, W), 421), small_integers((K, C, R, S), 422)
    y_ref, _ = oracle.conv2d_oracle(x, w)
    np.testing.assert_array_equal(run_library(x, w, entry="general", algo=ALGO_AUTO).astype(np.float64), y_ref)


def test_prepacked_filters_flag_reuses_the_workspace(oracle):
    import torch
    import paper_1705_10591_b200 as lib
    N, C, H, W, K, R, S = 2, 32, 12, 12, 128, 3, 3
    x1, x2 = uniform((N, C, H, W), 431), uniform((N, C, H, W), 432)
    w = uniform((K, C, R, S), 433)
    ws = torch.zeros(lib.conv2d_fwd_workspace_size(N, C, H, W, K, R, S, ALGO_TF32), dtype=torch.uint8, device="cuda:0")
    y1 = run_library(x1, w, entry="general", algo=ALGO_TF32, workspace=ws)
    y2 = run_library(x2, w, entry="general", algo=ALGO_TF32, workspace=ws, flags=1)   # filters already re-ordered
    for x, y in ((x1, y1), (x2, y2)):
        y_ref, yabs = oracle.conv2d_oracle(x, w)
        assert_parity(y, y_ref, yabs, TF32_TOL, "prepacked")


def test_relu_zero_windows_give_exact_zero(oracle):
    """Where every product is zero the result must be exactly zero in every path."""
    x = np.zeros((1, 16, 12, 12), np.float32)
    x[:, :, 8:, 8:] = uniform((1, 16, 4, 4), 411)
    w = uniform((32, 16, 3, 3), 412)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    for algo in (ALGO_FFMA, ALGO_AUTO):
        y = run_library(x, w, entry="general", algo=algo)
        assert np.all(y[yabs == 0] == 0)


@pytest.mark.parametrize("tile_px", [64, 96, 160, 224, 288, 352, 448, 512])
def test_general_tf32_every_item_size(oracle, monkeypatch, tile_px):
    """Work items of any multiple of 32 pixels (one or two MMAs per K step, ragged last item, images and rows
    changing inside an item) give the same parity as the planner's own choice."""
    dims = (3, 24, 19, 23, 200, 3, 3)              # 1311 pixels, two filter blocks, filters streamed
    N, C, H, W, K, R, S = dims
    monkeypatch.setenv("CONV2D_B200_TF32_TILE_PX", str(tile_px))
    x, w = uniform((N, C, H, W), 421), uniform((K, C, R, S), 422)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="general", algo=ALGO_TF32), y_ref, yabs, TF32_TOL, f"tile_px {tile_px}")
    xi, wi = small_integers((N, C, H, W), 423), small_integers((K, C, R, S), 424)
    yi_ref, _ = oracle.conv2d_oracle(xi, wi)
    np.testing.assert_array_equal(run_library(xi, wi, entry="general", algo=ALGO_TF32).astype(np.float64), yi_ref)


FEW_CHANNEL_SHAPES = [
    # N, C, H, W, K, R, S      (taps folded into the channel dimension of the tensor-core kernel)
    (2, 1, 20, 24, 40, 3, 3),      # one channel through the general entry: 9 folded channels, no shifts left
    (1, 1, 30, 33, 70, 7, 7),      # 49 folded channels: four channel blocks, the last one nearly empty
    (2, 3, 21, 26, 64, 3, 3),      # RGB first layer: 27 folded channels
    (1, 3, 40, 40, 96, 7, 7),      # 147 folded channels
    (2, 2, 9, 50, 33, 1, 5),       # one row of taps
    (2, 5, 18, 7, 20, 5, 1),       # one column of taps
    (1, 12, 16, 18, 130, 3, 3),    # 12 of 16 channels: folding the columns only (36 channels, 3 row shifts) wins
    (3, 15, 10, 10, 16, 2, 2),
]


@pytest.mark.parametrize("dims", FEW_CHANNEL_SHAPES)
@pytest.mark.parametrize("entry", ["general", "bf16"])
def test_few_channels_folded_taps(oracle, monkeypatch, dims, entry):
    N, C, H, W, K, R, S = dims
    monkeypatch.setenv("CONV2D_B200_TF32_FOLD", "2")           # fold whenever a channel block is not full
    xi, wi = small_integers((N, C, H, W), 431), small_integers((K, C, R, S), 432)
    yi_ref, _ = oracle.conv2d_oracle(xi, wi)
    np.testing.assert_array_equal(run_library(xi, wi, entry=entry, algo=ALGO_TF32).astype(np.float64), yi_ref)
    x, w = uniform((N, C, H, W), 433), uniform((K, C, R, S), 434)
    if entry == "bf16":
        from helpers import bf16_values
        x, w = bf16_values(x)[0], bf16_values(w)[0]
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    y = run_library(x, w, entry=entry, algo=ALGO_TF32)
    assert_parity(y, y_ref, yabs, TF32_TOL if entry == "general" else 1e-5, f"folded {entry} {dims}")
    monkeypatch.setenv("CONV2D_B200_TF32_FOLD", "0")          # same operands, contraction in another order
    y_plain = run_library(x, w, entry=entry, algo=ALGO_TF32)
    assert_parity(y_plain, y_ref, yabs, TF32_TOL if entry == "general" else 1e-5, f"unfolded {entry} {dims}")
    assert_parity(y, y_plain.astype(np.float64), yabs, 2e-5, f"folded vs unfolded {entry} {dims}")


WIDE_SHAPES = [
    # N, C, H, W, K, R, S      (items cut as rectangles of the image: the flat run's halo would be (R-1) image rows)
    (1, 16, 12, 600, 40, 3, 3),      # 128-bit producer loads, ragged last patch column
    (2, 20, 9, 1100, 130, 5, 5),     # two filter blocks; the flat run has no instance at this width
    (1, 8, 30, 260, 64, 7, 7),       # 7 x 7: three quarters of a 32-wide patch row are valid
    (1, 8, 21, 303, 64, 3, 3),       # width not a multiple of 4: one pixel per load
    (3, 33, 5, 520, 16, 1, 3),       # a single row of taps
    (1, 16, 6, 6000, 8, 5, 5),       # extremely wide, few rows
]


@pytest.mark.parametrize("dims", WIDE_SHAPES)
@pytest.mark.parametrize("entry", ["general", "bf16"])
def test_wide_images_patch_addressing(oracle, dims, entry):
    N, C, H, W, K, R, S = dims
    xi, wi = small_integers((N, C, H, W), 451), small_integers((K, C, R, S), 452)
    yi_ref, _ = oracle.conv2d_oracle(xi, wi)
    np.testing.assert_array_equal(run_library(xi, wi, entry=entry, algo=ALGO_TF32).astype(np.float64), yi_ref)
    x, w = uniform((N, C, H, W), 453), uniform((K, C, R, S), 454)
    if entry == "bf16":
        from helpers import bf16_values
        x, w = bf16_values(x)[0], bf16_values(w)[0]
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry=entry, algo=ALGO_TF32), y_ref, yabs,
                  TF32_TOL if entry == "general" else 1e-5, f"patch {entry} {dims}")


@pytest.mark.parametrize("dims", [(2, 17, 20, 21, 70, 3, 3), (1, 64, 14, 14, 96, 3, 3), (5, 33, 7, 9, 128, 3, 3),
                                  (2, 48, 12, 12, 128, 1, 1), (1, 40, 16, 16, 130, 1, 7)])
def test_patch_addressing_forced_on_narrow_images(oracle, monkeypatch, dims):
    """The two addressing modes must agree (same operands, same contraction order per output)."""
    N, C, H, W, K, R, S = dims
    x, w = uniform((N, C, H, W), 455), uniform((K, C, R, S), 456)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    y_flat = run_library(x, w, entry="general", algo=ALGO_TF32)
    monkeypatch.setenv("CONV2D_B200_TF32_PATCH", "2")
    y_patch = run_library(x, w, entry="general", algo=ALGO_TF32)
    assert_parity(y_patch, y_ref, yabs, TF32_TOL, f"patch {dims}")
    assert_parity(y_patch, y_flat.astype(np.float64), yabs, 2e-5, f"patch vs flat {dims}")


STACKED_TAP_SHAPES = [
    # N, C, H, W, K, R, S      (at most 64 filters: horizontally adjacent taps share one 128-row operand)
    (3, 64, 20, 22, 64, 3, 3),       # odd tap count per row: the last tap of a row has an empty upper half
    (2, 40, 17, 19, 50, 5, 5),       # filter count not a multiple of 16; odd image width (one pixel per store)
    (1, 72, 12, 30, 33, 2, 2),       # even taps per row: no empty halves
    (2, 16, 9, 44, 7, 7, 7),         # fewer filters than one lane quarter holds
    (1, 130, 6, 10, 64, 3, 4),       # too few pixels for the machine: split contraction, partial sums added
    (1, 24, 14, 640, 48, 3, 3),      # wide image: items are rectangles, no overlap between items
    (4, 32, 33, 36, 64, 1, 6),       # a single row of taps; several items per block
]


@pytest.mark.parametrize("dims", STACKED_TAP_SHAPES)
@pytest.mark.parametrize("entry", ["general", "bf16"])
def test_stacked_taps_for_few_filters(oracle, monkeypatch, dims, entry):
    """Exact on integers and within tolerance, forced on, and equal to the unstacked kernel's result."""
    N, C, H, W, K, R, S = dims
    monkeypatch.setenv("CONV2D_B200_TF32_PAIR_TAPS", "2")
    xi, wi = small_integers((N, C, H, W), 471), small_integers((K, C, R, S), 472)
    yi_ref, _ = oracle.conv2d_oracle(xi, wi)
    np.testing.assert_array_equal(run_library(xi, wi, entry=entry, algo=ALGO_TF32).astype(np.float64), yi_ref)
    x, w = uniform((N, C, H, W), 473), uniform((K, C, R, S), 474)
    if entry == "bf16":
        from helpers import bf16_values
        x, w = bf16_values(x)[0], bf16_values(w)[0]
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    tol = TF32_TOL if entry == "general" else 1e-5
    y_stacked = run_library(x, w, entry=entry, algo=ALGO_TF32)
    assert_parity(y_stacked, y_ref, yabs, tol, f"stacked taps {entry} {dims}")
    monkeypatch.setenv("CONV2D_B200_TF32_PAIR_TAPS", "0")
    y_plain = run_library(x, w, entry=entry, algo=ALGO_TF32)
    assert_parity(y_plain, y_ref, yabs, tol, f"unstacked {entry} {dims}")
    assert_parity(y_stacked, y_plain.astype(np.float64), yabs, 2e-5, f"stacked vs unstacked {entry} {dims}")


COMPACT_STACK_SHAPES = [
    # N, C, H, W, K, R, S      (at most 64 filters and a bank that stays in shared memory: pairs of taps as 128-row
    #                           slices, a lone last tap of a row as a 64-row slice issued as M = 64)
    (2, 64, 20, 20, 64, 3, 3),       # the early-layer benchmark shape in small: 4 channel blocks, lone third tap
    (2, 16, 10, 10, 64, 3, 2),       # even taps per row: pairs only
    (2, 8, 30, 30, 16, 3, 3),        # half a channel block, 16 filters: one lane quarter's worth
    (3, 20, 15, 17, 40, 3, 3),       # odd image width, 40 filters, partial second channel block
    (1, 16, 12, 40, 64, 1, 3),       # a single row of taps
    (1, 8, 9, 9, 24, 5, 5),          # two pairs and a lone tap per row
    (5, 32, 24, 24, 64, 3, 3),       # several items per block
]


@pytest.mark.parametrize("dims", COMPACT_STACK_SHAPES)
@pytest.mark.parametrize("entry", ["general", "bf16"])
def test_compact_stacked_taps(oracle, monkeypatch, dims, entry):
    """Exact on integers, within tolerance, and equal (up to summation order) to the unstacked kernel."""
    import paper_1705_10591_b200 as lib
    N, C, H, W, K, R, S = dims
    algo_q = ALGO_TF32 if entry == "general" else 3
    monkeypatch.setenv("CONV2D_B200_TF32_PAIR_COMPACT", "1")       # (measured slower on the benchmark shape: off by default)
    assert lib.conv2d_fwd_plan_describe(*dims, algo_q).get("stacked_compact") == 1, "meant to take compact stacking"
    xi, wi = small_integers((N, C, H, W), 481), small_integers((K, C, R, S), 482)
    yi_ref, _ = oracle.conv2d_oracle(xi, wi)
    np.testing.assert_array_equal(run_library(xi, wi, entry=entry, algo=ALGO_TF32).astype(np.float64), yi_ref)
    x, w = uniform((N, C, H, W), 483), uniform((K, C, R, S), 484)
    if entry == "bf16":
        from helpers import bf16_values
        x, w = bf16_values(x)[0], bf16_values(w)[0]
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    tol = TF32_TOL if entry == "general" else 1e-5
    y_compact = run_library(x, w, entry=entry, algo=ALGO_TF32)
    assert_parity(y_compact, y_ref, yabs, tol, f"compact stacking {entry} {dims}")
    monkeypatch.setenv("CONV2D_B200_TF32_PAIR_COMPACT", "0")
    monkeypatch.setenv("CONV2D_B200_TF32_PAIR_TAPS", "0")
    y_plain = run_library(x, w, entry=entry, algo=ALGO_TF32)
    assert_parity(y_compact, y_plain.astype(np.float64), yabs, 2e-5, f"compact vs unstacked {entry} {dims}")

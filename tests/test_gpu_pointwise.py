"""1 x 1 filters on the tensor cores with every operand moved by tensor-map (TMA) copies, against the oracle.

Shapes are chosen so that the library takes that kernel (the plan query says which one it is) and so that its
edges are met: an image whose last 32-pixel atom is ragged, a channel count that is not a multiple of the
32-channel stage or of the 8-channel MMA step, filter counts below and above one 128-filter block, the 64-row
variant, more work items than SMs, items that straddle two images.
"""
import numpy as np
import pytest

from helpers import TF32_TOL, assert_parity, run_library
from workloads import small_integers, uniform

pytestmark = pytest.mark.gpu
ALGO_TF32 = 2

SHAPES = [
    # N, C, H, W, K
    (2, 32, 8, 8, 16),          # two atoms per image, 64-row operand
    (1, 8, 4, 4, 8),            # a single ragged atom (16 pixels), one MMA step
    (1, 64, 12, 10, 200),       # HW = 120: last atom holds 24 pixels; two filter blocks, the second ragged
    (2, 36, 6, 6, 70),          # C = 36: second stage holds 4 channels (half an MMA step: zero-filled rows)
    (5, 100, 10, 10, 64),       # M = 64 rows, ragged atoms, C = 100
    (4, 256, 14, 14, 300),      # most channels the resident bank takes; three filter blocks
    (3, 128, 32, 32, 128),      # the benchmark's per-image shape; items straddle images
    (40, 16, 20, 20, 24),       # 520 atoms: several rounds of items per block
]


def _takes_tma_kernel(dims):
    import paper_1705_10591_b200 as lib
    N, C, H, W, K = dims
    return lib.conv2d_fwd_plan_describe(N, C, H, W, K, 1, 1, ALGO_TF32).get("kernel") == "pointwise_tma"


@pytest.mark.parametrize("dims", SHAPES)
def test_pointwise_exact_on_integers(oracle, dims):
    assert _takes_tma_kernel(dims)
    N, C, H, W, K = dims
    x, w = small_integers((N, C, H, W), 961), small_integers((K, C, 1, 1), 962)
    y_ref, _ = oracle.conv2d_oracle(x, w)
    np.testing.assert_array_equal(run_library(x, w, entry="general", algo=ALGO_TF32).astype(np.float64), y_ref)


@pytest.mark.parametrize("dims", SHAPES)
def test_pointwise_within_tolerance(oracle, dims):
    from oracle.conv2d_oracle import MODE_TF32_TRUNC
    N, C, H, W, K = dims
    x, w = uniform((N, C, H, W), 963), uniform((K, C, 1, 1), 964)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    y = run_library(x, w, entry="general", algo=ALGO_TF32)
    r = assert_parity(y, y_ref, yabs, TF32_TOL, f"pointwise {dims}")
    # the tensor core truncates fp32 operands to TF32: against the oracle fed truncated operands only the order
    # of the fp32 additions differs
    y_t, yabs_t = oracle.conv2d_oracle(x, w, mode=MODE_TF32_TRUNC)
    assert_parity(y, y_t, yabs_t, 2e-5, f"pointwise vs truncated-operand oracle {dims}")
    print(f"pointwise {dims} max ratio {r:.3e}")


def test_pointwise_item_sizes_agree(oracle, monkeypatch):
    """Every item size (atoms per work item) must give the same bits on integer inputs."""
    dims = (3, 40, 16, 12, 96)
    N, C, H, W, K = dims
    x, w = small_integers((N, C, H, W), 965), small_integers((K, C, 1, 1), 966)
    y_ref, _ = oracle.conv2d_oracle(x, w)
    for atoms in (1, 2, 3, 5, 8):
        monkeypatch.setenv("CONV2D_B200_TMA_ATOMS", str(atoms))
        np.testing.assert_array_equal(run_library(x, w, entry="general", algo=ALGO_TF32).astype(np.float64), y_ref)


def test_pointwise_general_kernel_still_serves_the_shape(oracle, monkeypatch):
    """With the tensor-map kernel switched off the general tensor-core kernel takes the same shape."""
    dims = (2, 32, 8, 8, 16)
    monkeypatch.setenv("CONV2D_B200_TF32_TMA", "0")
    assert not _takes_tma_kernel(dims)
    N, C, H, W, K = dims
    x, w = small_integers((N, C, H, W), 967), small_integers((K, C, 1, 1), 968)
    y_ref, _ = oracle.conv2d_oracle(x, w)
    np.testing.assert_array_equal(run_library(x, w, entry="general", algo=ALGO_TF32).astype(np.float64), y_ref)


def test_pointwise_expired_wait_is_reported(oracle, monkeypatch):
    """Host-side injection: one activation stage is armed but never copied and the wait bound is short.  The block
    gives up, frees its tensor memory and returns; the status word reports it and the next call is correct."""
    import torch
    import paper_1705_10591_b200 as lib

    N, C, H, W, K = 2, 64, 16, 16, 128
    x, w = uniform((N, C, H, W), 969), uniform((K, C, 1, 1), 970)
    dev = torch.device("cuda:0")
    xd, wd = torch.from_numpy(x).to(dev), torch.from_numpy(w).to(dev)
    y = torch.zeros((N, K, H, W), device=dev)
    ws_bytes = lib.conv2d_fwd_workspace_size(N, C, H, W, K, 1, 1, ALGO_TF32)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    monkeypatch.setenv("CONV2D_B200_TF32_MAX_POLLS", "2048")
    monkeypatch.setenv("CONV2D_B200_TF32_TEST_DROP_STAGE", "1")
    lib.conv2d_fwd_general(xd.data_ptr(), wd.data_ptr(), y.data_ptr(), N, C, H, W, K, 1, 1, ALGO_TF32,
                           ws.data_ptr(), ws_bytes, 0, stream)
    with pytest.raises(lib.Conv2dError) as e:
        lib.conv2d_get_status(ws.data_ptr(), stream)
    assert e.value.status == 8                       # CONV2D_ERR_DEVICE_TIMEOUT
    torch.cuda.synchronize()
    monkeypatch.delenv("CONV2D_B200_TF32_MAX_POLLS")
    monkeypatch.delenv("CONV2D_B200_TF32_TEST_DROP_STAGE")
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="general", algo=ALGO_TF32), y_ref, yabs, TF32_TOL, "after a time-out")


SHAPES_16BIT = [
    # N, C, H, W, K      (16-bit operands: 64 pixels per atom, 64 channels per stage, K steps of 16)
    (2, 32, 8, 8, 16),          # one atom per image, half a stage of channels, 64-row operand
    (1, 64, 12, 10, 200),       # HW = 120: second atom holds 56 pixels; two filter blocks
    (5, 104, 10, 16, 64),       # C = 104: second stage holds 40 channels (2.5 MMA steps: zero-filled rows)
    (4, 512, 8, 8, 300),        # most channels the resident bank takes; three filter blocks
    (3, 128, 32, 32, 128),      # the benchmark's per-image shape
    (40, 16, 20, 24, 24),       # 320 atoms: several rounds of items per block
]


@pytest.mark.parametrize("kind", ["bf16", "fp16"])
@pytest.mark.parametrize("dims", SHAPES_16BIT)
def test_pointwise_16bit_operands(oracle, dims, kind):
    import paper_1705_10591_b200 as lib
    from helpers import B16_TOL, bf16_values, fp16_values
    N, C, H, W, K = dims
    assert lib.conv2d_fwd_plan_describe(N, C, H, W, K, 1, 1, 3).get("kernel") == "pointwise_tma"
    xi, wi = small_integers((N, C, H, W), 981), small_integers((K, C, 1, 1), 982)
    yi_ref, _ = oracle.conv2d_oracle(xi, wi)
    np.testing.assert_array_equal(run_library(xi, wi, entry=kind).astype(np.float64), yi_ref)
    conv = bf16_values if kind == "bf16" else fp16_values
    x, w = conv(uniform((N, C, H, W), 983))[0], conv(uniform((K, C, 1, 1), 984))[0]
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    r = assert_parity(run_library(x, w, entry=kind), y_ref, yabs, B16_TOL, f"pointwise {kind} {dims}")
    print(f"pointwise {kind} {dims} max ratio {r:.3e}")


# More channels than a resident filter bank holds (256 fp32, 512 16-bit): every ring stage carries its chunk of the
# filters with the pixels, and fp32 filters are first rounded to TF32 by a small kernel.
STREAM_SHAPES = [
    # N, C, H, W, K
    (4, 512, 14, 14, 300),      # three filter blocks, ragged atoms, items tile-major
    (2, 1024, 8, 8, 64),        # 64-row operand, 32 stages per item
    (1, 260, 12, 10, 130),      # C = 260: ninth stage holds 4 channels; second filter block holds 2 filters
    (3, 2048, 7, 8, 128),       # the deepest layers of a residual network
    (20, 320, 16, 16, 256),     # more work items than SMs
]

STREAM_SHAPES_16BIT = [
    (4, 1024, 8, 8, 300),
    (2, 520, 12, 10, 64),       # C = 520: ninth stage holds 8 channels (half an MMA step)
    (3, 2048, 8, 8, 128),
    (20, 640, 16, 16, 256),
]


def _round_to_tf32(a):
    """fp32 -> nearest value with a 10-bit mantissa, ties away from zero (what cvt.rna.tf32.f32 does)."""
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    return ((bits + np.uint32(0x1000)) & np.uint32(0xFFFFE000)).view(np.float32)


@pytest.mark.parametrize("dims", STREAM_SHAPES)
def test_pointwise_streamed_filters(oracle, dims):
    import paper_1705_10591_b200 as lib
    from oracle.conv2d_oracle import MODE_TF32_TRUNC
    N, C, H, W, K = dims
    plan = lib.conv2d_fwd_plan_describe(N, C, H, W, K, 1, 1, ALGO_TF32)
    assert plan.get("kernel") == "pointwise_tma" and plan.get("resident_filters") == 0 and plan.get("filters_rounded_first") == 1
    xi, wi = small_integers((N, C, H, W), 971), small_integers((K, C, 1, 1), 972)
    yi_ref, _ = oracle.conv2d_oracle(xi, wi)
    np.testing.assert_array_equal(run_library(xi, wi, entry="general", algo=ALGO_TF32).astype(np.float64), yi_ref)
    x, w = uniform((N, C, H, W), 973), uniform((K, C, 1, 1), 974)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    y = run_library(x, w, entry="general", algo=ALGO_TF32)
    r = assert_parity(y, y_ref, yabs, TF32_TOL, f"pointwise, streamed filters {dims}")
    # filters rounded to nearest by the library, image truncated by the tensor core: against the oracle fed such
    # operands (truncating a rounded filter changes nothing) only the order of the fp32 additions differs
    y_t, yabs_t = oracle.conv2d_oracle(x, _round_to_tf32(w), mode=MODE_TF32_TRUNC)
    assert_parity(y, y_t, yabs_t, 2e-5, f"pointwise, streamed filters vs TF32-operand oracle {dims}")
    print(f"pointwise streamed {dims} max ratio {r:.3e}")


@pytest.mark.parametrize("kind", ["bf16", "fp16"])
@pytest.mark.parametrize("dims", STREAM_SHAPES_16BIT)
def test_pointwise_streamed_filters_16bit(oracle, dims, kind):
    import paper_1705_10591_b200 as lib
    from helpers import B16_TOL, bf16_values, fp16_values
    N, C, H, W, K = dims
    plan = lib.conv2d_fwd_plan_describe(N, C, H, W, K, 1, 1, 3)
    assert plan.get("kernel") == "pointwise_tma" and plan.get("resident_filters") == 0 and plan.get("filters_rounded_first") == 0
    xi, wi = small_integers((N, C, H, W), 985), small_integers((K, C, 1, 1), 986)
    yi_ref, _ = oracle.conv2d_oracle(xi, wi)
    np.testing.assert_array_equal(run_library(xi, wi, entry=kind).astype(np.float64), yi_ref)
    conv = bf16_values if kind == "bf16" else fp16_values
    x, w = conv(uniform((N, C, H, W), 987))[0], conv(uniform((K, C, 1, 1), 988))[0]
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry=kind), y_ref, yabs, B16_TOL, f"pointwise, streamed filters {kind} {dims}")


def test_pointwise_streamed_filters_prepacked(oracle):
    """CONV2D_FLAG_WEIGHTS_PACKED: the second call finds the rounded filters in the workspace and launches one
    kernel less; the result is the same bits."""
    import torch
    import paper_1705_10591_b200 as lib

    N, C, H, W, K = 2, 512, 8, 8, 96
    x, w = uniform((N, C, H, W), 975), uniform((K, C, 1, 1), 976)
    dev = torch.device("cuda:0")
    xd, wd = torch.from_numpy(x).to(dev), torch.from_numpy(w).to(dev)
    ws_bytes = lib.conv2d_fwd_workspace_size(N, C, H, W, K, 1, 1, ALGO_TF32)
    assert ws_bytes >= 256 + K * C * 4
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    ys = []
    for flags in (0, 1):
        y = torch.zeros((N, K, H, W), device=dev)
        before = lib.conv2d_launch_count()
        lib.conv2d_fwd_general(xd.data_ptr(), wd.data_ptr(), y.data_ptr(), N, C, H, W, K, 1, 1, ALGO_TF32,
                               ws.data_ptr(), ws_bytes, flags, stream)
        lib.conv2d_get_status(ws.data_ptr(), stream)
        assert lib.conv2d_launch_count() - before == 2 - flags
        ys.append(y.cpu().numpy())
    np.testing.assert_array_equal(ys[0], ys[1])
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(ys[1], y_ref, yabs, TF32_TOL, "streamed filters, prepacked")


def test_pointwise_streamed_filters_expired_wait_is_reported(oracle, monkeypatch):
    """The same host-side injection as above on the streamed-filter variant: a stage whose pixels never arrive."""
    import torch
    import paper_1705_10591_b200 as lib

    N, C, H, W, K = 2, 512, 16, 16, 128
    x, w = uniform((N, C, H, W), 977), uniform((K, C, 1, 1), 978)
    dev = torch.device("cuda:0")
    xd, wd = torch.from_numpy(x).to(dev), torch.from_numpy(w).to(dev)
    y = torch.zeros((N, K, H, W), device=dev)
    ws_bytes = lib.conv2d_fwd_workspace_size(N, C, H, W, K, 1, 1, ALGO_TF32)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    monkeypatch.setenv("CONV2D_B200_TF32_MAX_POLLS", "2048")
    monkeypatch.setenv("CONV2D_B200_TF32_TEST_DROP_STAGE", "5")
    lib.conv2d_fwd_general(xd.data_ptr(), wd.data_ptr(), y.data_ptr(), N, C, H, W, K, 1, 1, ALGO_TF32,
                           ws.data_ptr(), ws_bytes, 0, stream)
    with pytest.raises(lib.Conv2dError) as e:
        lib.conv2d_get_status(ws.data_ptr(), stream)
    assert e.value.status == 8                       # CONV2D_ERR_DEVICE_TIMEOUT
    torch.cuda.synchronize()
    monkeypatch.delenv("CONV2D_B200_TF32_MAX_POLLS")
    monkeypatch.delenv("CONV2D_B200_TF32_TEST_DROP_STAGE")
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="general", algo=ALGO_TF32), y_ref, yabs, TF32_TOL, "after a time-out")


# More than 128 filters: two-SM MMAs (cta_group::2) by the two blocks of a cluster, each holding one 128-filter block
# and half of the item's pixels.  CONV2D_B200_TMA_PAIR=2 takes that form wherever it exists, so that the small
# shapes below meet its edges: an odd number of filter blocks (the last pair's second block has no filters), a
# ragged filter count, items that end past the batch (atoms the loads zero-fill and the stores skip), items that
# straddle images, the resident and the streamed filter bank.
PAIR_SHAPES = [
    # N, C, H, W, K
    (2, 32, 8, 8, 256),         # one pair, one ragged item
    (1, 64, 12, 10, 200),       # second block holds 72 filters; HW = 120: ragged atoms
    (4, 256, 14, 14, 300),      # three filter blocks = two pairs; largest resident bank
    (3, 128, 32, 32, 256),      # items straddle images
    (4, 512, 14, 14, 300),      # streamed filters
    (1, 260, 12, 10, 130),      # streamed, ninth stage holds 4 channels, second block holds 2 filters
    (40, 16, 20, 20, 384),      # several rounds of items per pair
    (5, 100, 10, 10, 129),      # second block holds one filter
]


def _two_sm(dims, algo=ALGO_TF32):
    import paper_1705_10591_b200 as lib
    N, C, H, W, K = dims
    plan = lib.conv2d_fwd_plan_describe(N, C, H, W, K, 1, 1, algo)
    return plan.get("kernel") == "pointwise_tma" and plan.get("two_sm") == 1


@pytest.mark.parametrize("dims", PAIR_SHAPES)
def test_pointwise_two_sm(oracle, dims, monkeypatch):
    from oracle.conv2d_oracle import MODE_TF32_TRUNC
    monkeypatch.setenv("CONV2D_B200_TMA_PAIR", "2")
    assert _two_sm(dims)
    N, C, H, W, K = dims
    xi, wi = small_integers((N, C, H, W), 991), small_integers((K, C, 1, 1), 992)
    yi_ref, _ = oracle.conv2d_oracle(xi, wi)
    np.testing.assert_array_equal(run_library(xi, wi, entry="general", algo=ALGO_TF32).astype(np.float64), yi_ref)
    x, w = uniform((N, C, H, W), 993), uniform((K, C, 1, 1), 994)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    y = run_library(x, w, entry="general", algo=ALGO_TF32)
    assert_parity(y, y_ref, yabs, TF32_TOL, f"pointwise, two-SM {dims}")
    w_seen = _round_to_tf32(w) if C > 256 else w          # streamed fp32 filters are rounded first
    y_t, yabs_t = oracle.conv2d_oracle(x, w_seen, mode=MODE_TF32_TRUNC)
    assert_parity(y, y_t, yabs_t, 2e-5, f"pointwise, two-SM vs TF32-operand oracle {dims}")


@pytest.mark.parametrize("kind", ["bf16", "fp16"])
@pytest.mark.parametrize("dims", [(2, 32, 8, 8, 256), (1, 64, 12, 10, 200), (4, 512, 8, 8, 300), (2, 520, 12, 10, 130),
                                  (3, 128, 32, 32, 256)])
def test_pointwise_two_sm_16bit(oracle, dims, kind, monkeypatch):
    from helpers import B16_TOL, bf16_values, fp16_values
    monkeypatch.setenv("CONV2D_B200_TMA_PAIR", "2")
    assert _two_sm(dims, 3)
    N, C, H, W, K = dims
    xi, wi = small_integers((N, C, H, W), 995), small_integers((K, C, 1, 1), 996)
    yi_ref, _ = oracle.conv2d_oracle(xi, wi)
    np.testing.assert_array_equal(run_library(xi, wi, entry=kind).astype(np.float64), yi_ref)
    conv = bf16_values if kind == "bf16" else fp16_values
    x, w = conv(uniform((N, C, H, W), 997))[0], conv(uniform((K, C, 1, 1), 998))[0]
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry=kind), y_ref, yabs, B16_TOL, f"pointwise, two-SM {kind} {dims}")


def test_pointwise_two_sm_item_sizes_agree(oracle, monkeypatch):
    """Every item size of the two-SM form (2, 4, 6, 8 atoms) gives the same bits on integer inputs."""
    dims = (3, 40, 16, 12, 200)
    N, C, H, W, K = dims
    monkeypatch.setenv("CONV2D_B200_TMA_PAIR", "2")
    x, w = small_integers((N, C, H, W), 999), small_integers((K, C, 1, 1), 1000)
    y_ref, _ = oracle.conv2d_oracle(x, w)
    for atoms in (2, 4, 6, 8):
        monkeypatch.setenv("CONV2D_B200_TMA_ATOMS", str(atoms))
        assert _two_sm(dims)
        np.testing.assert_array_equal(run_library(x, w, entry="general", algo=ALGO_TF32).astype(np.float64), y_ref)


def test_pointwise_two_sm_is_the_default_for_deep_wide_layers(oracle):
    """Without any switch the planner takes the two-SM form for a layer with many channels and filters."""
    dims = (16, 512, 16, 16, 512)
    assert _two_sm(dims)
    N, C, H, W, K = dims
    x, w = uniform((N, C, H, W), 1001), uniform((K, C, 1, 1), 1002)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="general", algo=ALGO_TF32), y_ref, yabs, TF32_TOL, f"two-SM by default {dims}")


@pytest.mark.parametrize("dims", [(2, 64, 16, 16, 256), (2, 512, 16, 16, 256)])
def test_pointwise_two_sm_expired_wait_is_reported(oracle, dims, monkeypatch):
    """Host-side injection on the two-SM form (resident and streamed filters): the first block of a pair never
    copies one stage of pixels.  Both blocks of every pair give up within their bounds and meet at the closing
    cluster barrier; the status word reports it; the next call is correct."""
    import torch
    import paper_1705_10591_b200 as lib

    N, C, H, W, K = dims
    monkeypatch.setenv("CONV2D_B200_TMA_PAIR", "2")
    assert _two_sm(dims)
    x, w = uniform((N, C, H, W), 1003), uniform((K, C, 1, 1), 1004)
    dev = torch.device("cuda:0")
    xd, wd = torch.from_numpy(x).to(dev), torch.from_numpy(w).to(dev)
    y = torch.zeros((N, K, H, W), device=dev)
    ws_bytes = lib.conv2d_fwd_workspace_size(N, C, H, W, K, 1, 1, ALGO_TF32)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    monkeypatch.setenv("CONV2D_B200_TF32_MAX_POLLS", "2048")
    monkeypatch.setenv("CONV2D_B200_TF32_TEST_DROP_STAGE", "1")
    lib.conv2d_fwd_general(xd.data_ptr(), wd.data_ptr(), y.data_ptr(), N, C, H, W, K, 1, 1, ALGO_TF32,
                           ws.data_ptr(), ws_bytes, 0, stream)
    with pytest.raises(lib.Conv2dError) as e:
        lib.conv2d_get_status(ws.data_ptr(), stream)
    assert e.value.status == 8                       # CONV2D_ERR_DEVICE_TIMEOUT
    torch.cuda.synchronize()
    monkeypatch.delenv("CONV2D_B200_TF32_MAX_POLLS")
    monkeypatch.delenv("CONV2D_B200_TF32_TEST_DROP_STAGE")
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="general", algo=ALGO_TF32), y_ref, yabs, TF32_TOL, "after a time-out")


# Split contraction: the channel chunks of a tile are shared out to two work items that both add their partial sums
# into a zeroed y with tensor-map reduce copies (a + b = b + a, so the result does not depend on which comes first).
# The planner takes it for very long contractions on few pixels; CONV2D_B200_TMA_KSPLIT=2 forces it wherever a
# shape has two channel chunks.
KSPLIT_SHAPES = [
    # N, C, H, W, K
    (2, 64, 8, 8, 16),          # two chunks, one each; 64-row operand
    (1, 100, 12, 10, 200),      # four chunks (the last holds 4 channels) as 2 + 2; ragged atoms; two filter blocks
    (4, 256, 14, 14, 300),      # resident banks of four chunks
    (3, 288, 16, 16, 128),      # nine chunks as 5 + 4
    (4, 1024, 8, 8, 96),        # 16 + 16 chunks; streamed filters either way
    (2, 2048, 7, 8, 130),       # the planner's own pick
]


@pytest.mark.parametrize("pair", ["0", "2"])
@pytest.mark.parametrize("dims", KSPLIT_SHAPES)
def test_pointwise_split_contraction(oracle, dims, pair, monkeypatch):
    import paper_1705_10591_b200 as lib
    N, C, H, W, K = dims
    monkeypatch.setenv("CONV2D_B200_TMA_KSPLIT", "2")
    monkeypatch.setenv("CONV2D_B200_TMA_PAIR", pair)
    plan = lib.conv2d_fwd_plan_describe(N, C, H, W, K, 1, 1, ALGO_TF32)
    assert plan.get("kernel") == "pointwise_tma" and plan.get("ksplit") == 2
    xi, wi = small_integers((N, C, H, W), 1101), small_integers((K, C, 1, 1), 1102)
    yi_ref, _ = oracle.conv2d_oracle(xi, wi)
    np.testing.assert_array_equal(run_library(xi, wi, entry="general", algo=ALGO_TF32).astype(np.float64), yi_ref)
    x, w = uniform((N, C, H, W), 1103), uniform((K, C, 1, 1), 1104)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    y1 = run_library(x, w, entry="general", algo=ALGO_TF32)
    assert_parity(y1, y_ref, yabs, TF32_TOL, f"pointwise, split contraction {dims}")
    # the same bits every time: neither the order of the two adds nor the timing matters
    np.testing.assert_array_equal(run_library(x, w, entry="general", algo=ALGO_TF32), y1)


@pytest.mark.parametrize("kind", ["bf16", "fp16"])
def test_pointwise_split_contraction_16bit(oracle, kind, monkeypatch):
    from helpers import B16_TOL, bf16_values, fp16_values
    import paper_1705_10591_b200 as lib
    N, C, H, W, K = 3, 320, 8, 8, 200
    monkeypatch.setenv("CONV2D_B200_TMA_KSPLIT", "2")
    assert lib.conv2d_fwd_plan_describe(N, C, H, W, K, 1, 1, 3).get("ksplit") == 2
    xi, wi = small_integers((N, C, H, W), 1105), small_integers((K, C, 1, 1), 1106)
    yi_ref, _ = oracle.conv2d_oracle(xi, wi)
    np.testing.assert_array_equal(run_library(xi, wi, entry=kind).astype(np.float64), yi_ref)
    conv = bf16_values if kind == "bf16" else fp16_values
    x, w = conv(uniform((N, C, H, W), 1107))[0], conv(uniform((K, C, 1, 1), 1108))[0]
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry=kind), y_ref, yabs, B16_TOL, f"pointwise, split contraction {kind}")


def test_pointwise_split_contraction_is_the_planners_pick_for_deep_layers():
    import paper_1705_10591_b200 as lib
    assert lib.conv2d_fwd_plan_describe(32, 2048, 7, 8, 512, 1, 1, ALGO_TF32).get("ksplit") == 2
    assert lib.conv2d_fwd_plan_describe(32, 512, 14, 14, 128, 1, 1, ALGO_TF32).get("ksplit") == 1


@pytest.mark.parametrize("dims", [(2, 32, 8, 8, 256), (1, 64, 12, 10, 200), (4, 512, 14, 14, 300), (3, 128, 32, 32, 256),
                                  (1, 260, 12, 10, 130), (20, 320, 16, 16, 256)])
def test_pointwise_two_sm_wide_items(oracle, dims, monkeypatch):
    """Items of a pair that span two MMA widths of pixels (both accumulator sets for one item): CONV2D_B200_TMA_WIDE=2
    takes them wherever a pair runs, so that ragged items and odd filter-block counts meet this form too."""
    import paper_1705_10591_b200 as lib
    N, C, H, W, K = dims
    monkeypatch.setenv("CONV2D_B200_TMA_PAIR", "2")
    monkeypatch.setenv("CONV2D_B200_TMA_WIDE", "2")
    plan = lib.conv2d_fwd_plan_describe(N, C, H, W, K, 1, 1, ALGO_TF32)
    assert plan.get("two_sm") == 1 and plan.get("acc_sets") == 1 and plan.get("tile_px") == 512
    xi, wi = small_integers((N, C, H, W), 1111), small_integers((K, C, 1, 1), 1112)
    yi_ref, _ = oracle.conv2d_oracle(xi, wi)
    np.testing.assert_array_equal(run_library(xi, wi, entry="general", algo=ALGO_TF32).astype(np.float64), yi_ref)
    x, w = uniform((N, C, H, W), 1113), uniform((K, C, 1, 1), 1114)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="general", algo=ALGO_TF32), y_ref, yabs, TF32_TOL, f"pointwise, wide two-SM items {dims}")
    if (H * W) % 8 == 0 and C % 8 == 0:        # (what the 16-bit operands need for this kernel)
        from helpers import B16_TOL, bf16_values
        assert lib.conv2d_fwd_plan_describe(N, C, H, W, K, 1, 1, 3).get("acc_sets") == 1
        xb, wb = bf16_values(x)[0], bf16_values(w)[0]
        yb_ref, yb_abs = oracle.conv2d_oracle(xb, wb)
        assert_parity(run_library(xb, wb, entry="bf16"), yb_ref, yb_abs, B16_TOL, f"pointwise, wide two-SM items bf16 {dims}")


def test_pointwise_wide_items_are_the_planners_pick_for_long_contractions(oracle):
    import paper_1705_10591_b200 as lib
    dims = (16, 1024, 14, 14, 2048)
    assert lib.conv2d_fwd_plan_describe(*dims, 1, 1, ALGO_TF32).get("acc_sets") == 1
    assert lib.conv2d_fwd_plan_describe(64, 512, 32, 32, 512, 1, 1, ALGO_TF32).get("acc_sets") == 2
    N, C, H, W, K = dims
    x, w = uniform((N, C, H, W), 1115), uniform((K, C, 1, 1), 1116)
    y_ref, yabs = oracle.conv2d_oracle(x, w)
    assert_parity(run_library(x, w, entry="general", algo=ALGO_TF32), y_ref, yabs, TF32_TOL, f"wide items by default {dims}")

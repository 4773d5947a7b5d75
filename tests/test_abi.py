"""CPU-side checks of the C-ABI library: it loads, exports what the header declares, validates arguments."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    from paper_1705_10591_b200 import build, binding
    build.build()
    return binding


def _declared_functions():
    names = set()
    for header in (ROOT / "include").glob("*.h"):
        text = re.sub(r"/\*.*?\*/", "", header.read_text(), flags=re.S)
        names.update(re.findall(r"\b(conv2d_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(lib):
    cdll = lib.load_library()
    declared = _declared_functions()
    assert {"conv2d_fwd_workspace_size", "conv2d_fwd_single_channel", "conv2d_fwd_general"} <= set(declared)
    for name in declared:
        assert hasattr(cdll, name), f"{name} declared in include/ but not exported"
        assert hasattr(lib, name), f"{name} has no Python binding of the same name"


def test_status_strings(lib):
    assert lib.conv2d_status_string(0) == "ok"
    assert len({lib.conv2d_status_string(i) for i in range(9)}) == 9


def test_workspace_query(lib):
    assert lib.conv2d_fwd_workspace_size(1, 1, 64, 64, 8, 3, 3, lib.ALGO_FFMA) == 0
    with pytest.raises(lib.Conv2dError) as e:
        lib.conv2d_fwd_workspace_size(1, 1, 2, 2, 8, 3, 3, lib.ALGO_FFMA)   # filter larger than image
    assert e.value.status == 2
    with pytest.raises(lib.Conv2dError) as e:
        lib.conv2d_fwd_workspace_size(0, 1, 8, 8, 8, 3, 3, lib.ALGO_AUTO)
    assert e.value.status == 2
    cdll = lib.load_library()
    assert cdll.conv2d_fwd_workspace_size(1, 1, 8, 8, 1, 3, 3, 0, None) == 1      # NULL result pointer


def test_argument_errors_come_before_any_device_work(lib):
    ok = 4096  # any 16-byte aligned non-NULL address: validation fails before it is dereferenced
    cases = [
        (dict(x=0), 1), (dict(y=0), 1),
        (dict(x=ok + 4), 3), (dict(y=ok + 8), 3),
        (dict(R=9), 2), (dict(K=0), 2), (dict(H=-1), 2),
        (dict(flags=2), 5),
    ]
    for override, status in cases:
        a = dict(x=ok, w=ok, y=ok, N=1, H=8, W=8, K=2, R=3, S=3, flags=0)
        a.update(override)
        with pytest.raises(lib.Conv2dError) as e:
            lib.conv2d_fwd_single_channel(a["x"], a["w"], a["y"], a["N"], a["H"], a["W"], a["K"], a["R"], a["S"],
                                          0, 0, a["flags"], 0)
        assert e.value.status == status, (override, e.value.status)
        with pytest.raises(lib.Conv2dError) as e:
            lib.conv2d_fwd_general(a["x"], a["w"], a["y"], a["N"], 3, a["H"], a["W"], a["K"], a["R"], a["S"],
                                   lib.ALGO_FFMA, 0, 0, a["flags"] * 2, 0)
        assert e.value.status == status, (override, e.value.status)
    with pytest.raises(lib.Conv2dError) as e:      # explicit TF32 without a workspace
        lib.conv2d_fwd_general(ok, ok, ok, 1, 64, 16, 16, 64, 3, 3, lib.ALGO_TF32, 0, 0, 0, 0)
    assert e.value.status in (1, 5)
    with pytest.raises(lib.Conv2dError) as e:      # unknown algorithm
        lib.conv2d_fwd_general(ok, ok, ok, 1, 3, 8, 8, 2, 3, 3, 7, 0, 0, 0, 0)
    assert e.value.status == 5
    # The padded and strided entries launch a rewriting kernel of their own before the general entry: whatever
    # that entry would reject (misaligned w or y, unknown flag, an algorithm it does not take, too many planes)
    # must be rejected before that kernel.  The launch counter shows that nothing was enqueued.
    big = 1 << 30
    before = lib.conv2d_launch_count()
    padded = [(dict(w=ok + 4), 3), (dict(y=ok + 8), 3), (dict(flags=2), 5), (dict(algo=lib.ALGO_16BIT), 5),
              (dict(algo=7), 5), (dict(N=700, C=100), 5)]
    for override, status in padded:
        a = dict(x=ok, w=ok, y=ok, N=1, C=3, algo=lib.ALGO_FFMA, flags=0)
        a.update(override)
        with pytest.raises(lib.Conv2dError) as e:
            lib.conv2d_fwd_general_padded(a["x"], a["w"], a["y"], a["N"], a["C"], 8, 8, 2, 3, 3, 1, 1, a["algo"],
                                          ok, big, a["flags"], 0)
        assert e.value.status == status, ("padded", override, e.value.status)
        with pytest.raises(lib.Conv2dError) as e:
            lib.conv2d_fwd_general_strided(a["x"], a["w"], a["y"], a["N"], a["C"], 8, 8, 2, 3, 3, 1, 1, 2, a["algo"],
                                           ok, big, a["flags"], 0)
        assert e.value.status == status, ("strided", override, e.value.status)
    assert lib.conv2d_launch_count() == before


def test_no_silent_fallback_without_a_gpu(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(lib.Conv2dError) as e:
        lib.conv2d_fwd_single_channel(4096, 4096, 4096, 1, 8, 8, 2, 3, 3)
    assert e.value.status in (6, 7)


def test_product_package_does_not_touch_the_oracle():
    for path in (ROOT / "paper_1705_10591_b200").rglob("*"):
        if path.suffix in {".py", ".cu", ".cuh", ".h", ".cpp"}:
            assert "oracle" not in path.read_text().lower(), f"{path} mentions the oracle"


def test_workspace_query_over_many_shapes_is_consistent(lib):
    """The tensor-core planner runs on the host: sweep it over odd shapes (no device needed)."""
    import itertools
    seen = 0
    for N, C, HW, K, R in itertools.product((1, 3, 32), (1, 3, 16, 17, 300), (7, 14, 57), (1, 8, 64, 65, 129, 257, 600), (1, 3, 7)):
        if R > HW:
            continue
        try:
            tf32 = lib.conv2d_fwd_workspace_size(N, C, HW, HW, K, R, R, lib.ALGO_TF32)
        except lib.Conv2dError as e:
            assert e.status == 5                      # no instance: must be reported, not guessed
            assert lib.conv2d_fwd_workspace_size(N, C, HW, HW, K, R, R, lib.ALGO_AUTO) == 0
            continue
        seen += 1
        # status block + re-ordered filters: at least one float per real filter tap, padded to whole blocks
        assert tf32 >= 256 + 4 * K * C * R * R
        assert tf32 % 16 == 0
        assert lib.conv2d_fwd_workspace_size(N, C, HW, HW, K, R, R, lib.ALGO_AUTO) == tf32
        assert lib.conv2d_fwd_workspace_size(N, C, HW, HW, K, R, R, lib.ALGO_FFMA) == 0
    assert seen > 100


def test_padded_workspace_query(lib):
    plain = lib.conv2d_fwd_workspace_size(2, 16, 22, 22, 32, 3, 3, lib.ALGO_TF32)
    padded = lib.conv2d_fwd_padded_workspace_size(2, 16, 20, 20, 32, 3, 3, 1, 1, lib.ALGO_TF32)
    assert padded >= plain + 2 * 16 * 22 * 22 * 4          # the general workspace of the extended image + that image
    assert lib.conv2d_fwd_padded_workspace_size(2, 16, 20, 20, 32, 3, 3, 1, 1, lib.ALGO_FFMA) == 256 + 2 * 16 * 22 * 22 * 4
    with pytest.raises(lib.Conv2dError) as e:
        lib.conv2d_fwd_padded_workspace_size(2, 16, 20, 20, 32, 3, 3, -1, 0, lib.ALGO_FFMA)
    assert e.value.status == 2
    # a filter larger than the image becomes legal once the padding makes room for it
    assert lib.conv2d_fwd_padded_workspace_size(1, 4, 3, 3, 8, 5, 5, 1, 1, lib.ALGO_FFMA) > 0
    with pytest.raises(lib.Conv2dError):
        lib.conv2d_fwd_padded_workspace_size(1, 4, 3, 3, 8, 7, 7, 1, 1, lib.ALGO_FFMA)


def test_strided_workspace_query(lib):
    # 224 x 224 RGB, 7 x 7, pad 3, stride 2 -> 112 x 112 outputs; rewritten as 12 channels of 115 x 115 with 4 x 4 filters
    n = lib.conv2d_fwd_strided_workspace_size(2, 3, 224, 224, 64, 7, 7, 3, 3, 2, lib.ALGO_FFMA)
    assert n >= 256 + 2 * 12 * 115 * 115 * 4 + 64 * 12 * 4 * 4 * 4
    for bad in (0, 9, -1):
        with pytest.raises(lib.Conv2dError) as e:
            lib.conv2d_fwd_strided_workspace_size(2, 3, 224, 224, 64, 7, 7, 3, 3, bad, lib.ALGO_FFMA)
        assert e.value.status == 2

"""Pins the CPU oracle to facts that do not come from the oracle itself.

Hand-evaluated fixtures (orientation, channel/map indexing), closed forms,
identities, reductions to library routines and an independently written
brute force.  Each test is chosen so that a plausible slip in the oracle (a
flipped filter, swapped r/s or h/w strides, a dropped channel, a wrong halo
side) fails at least one of them.
"""
from pathlib import Path

import numpy as np
import pytest

from workloads import small_integers, uniform

GOLDEN = Path(__file__).resolve().parent / "golden"


def _read_fixture(path):
    vals = {}
    for line in path.read_text().splitlines():
        line = line.split("#", 1)[0].strip()
        if not line:
            continue
        key, rest = line.split(":", 1)
        vals[key.strip()] = [float(t) for t in rest.split()]
    out = {}
    for key, v in vals.items():
        if key.startswith("shape_"):
            continue
        shape_key = "shape_" + ("y" if key == "yabs" else key)
        out[key] = np.array(v, dtype=np.float64).reshape([int(d) for d in vals[shape_key]])
    return out


@pytest.mark.parametrize("name", ["hand_3x3_ramp", "hand_3x3_corners", "hand_two_channel_rect"])
def test_hand_evaluated_fixture(oracle, name):
    fx = _read_fixture(GOLDEN / f"{name}.txt")
    y, yabs = oracle.conv2d_oracle(fx["x"].astype(np.float32), fx["w"].astype(np.float32))
    np.testing.assert_array_equal(y, fx["y"])
    np.testing.assert_array_equal(yabs, fx["yabs"])


def test_delta_filter_selects_shifted_window(oracle):
    N, C, H, W, K, R, S = 2, 3, 7, 9, 4, 3, 4
    x = uniform((N, C, H, W), 11)
    w = np.zeros((K, C, R, S), np.float32)
    taps = [(0, 0, 0), (1, 2, 3), (2, 1, 0), (1, 0, 2)]  # (c, r, s) per map k
    for k, (c, r, s) in enumerate(taps):
        w[k, c, r, s] = 1.0
    y, yabs = oracle.conv2d_oracle(x, w)
    P, Q = H - R + 1, W - S + 1
    for k, (c, r, s) in enumerate(taps):
        expect = x[:, c, r:r + P, s:s + Q].astype(np.float64)
        np.testing.assert_array_equal(y[:, k], expect)
        np.testing.assert_array_equal(yabs[:, k], np.abs(expect))


def test_delta_image_gives_point_reflected_filter(oracle):
    N, C, H, W, K, R, S = 2, 2, 6, 7, 3, 3, 2
    w = uniform((K, C, R, S), 12)
    n0, c0, h0, w0 = 1, 1, 3, 4
    x = np.zeros((N, C, H, W), np.float32)
    x[n0, c0, h0, w0] = 1.0
    y, _ = oracle.conv2d_oracle(x, w)
    P, Q = H - R + 1, W - S + 1
    expect = np.zeros((N, K, P, Q))
    for k in range(K):
        for p in range(P):
            for q in range(Q):
                r, s = h0 - p, w0 - q
                if 0 <= r < R and 0 <= s < S:
                    expect[n0, k, p, q] = w[k, c0, r, s]
    np.testing.assert_array_equal(y, expect)


def test_linearity_exact_with_small_integers(oracle):
    shape_x, shape_w = (2, 3, 8, 6), (3, 3, 2, 3)
    x1, x2 = small_integers(shape_x, 21), small_integers(shape_x, 22)
    w1, w2 = small_integers(shape_w, 23), small_integers(shape_w, 24)
    a, b = 3.0, -2.0
    y = lambda xx, ww: oracle.conv2d_oracle(xx.astype(np.float32), ww.astype(np.float32))[0]
    np.testing.assert_array_equal(y(a * x1 + b * x2, w1), a * y(x1, w1) + b * y(x2, w1))
    np.testing.assert_array_equal(y(x1, a * w1 + b * w2), a * y(x1, w1) + b * y(x1, w2))


def test_all_ones_counts_the_receptive_field(oracle):
    N, C, H, W, K, R, S = 1, 5, 6, 8, 2, 3, 5
    y, yabs = oracle.conv2d_oracle(np.ones((N, C, H, W), np.float32), np.ones((K, C, R, S), np.float32))
    assert y.shape == (N, K, H - R + 1, W - S + 1)
    assert np.all(y == C * R * S) and np.all(yabs == C * R * S)


def test_affine_image_closed_form(oracle):
    # x[n,c,h,w] = a*h + b*w + d  =>  y = (a*p + b*q + d)*sum(w_k) + a*sum(r*w_k) + b*sum(s*w_k)
    N, C, H, W, K, R, S = 1, 2, 9, 10, 3, 3, 4
    a, b, d = 2.0, -3.0, 5.0
    hh, ww = np.meshgrid(np.arange(H), np.arange(W), indexing="ij")
    x = np.broadcast_to((a * hh + b * ww + d).astype(np.float32), (N, C, H, W)).copy()
    w = small_integers((K, C, R, S), 31)
    y, _ = oracle.conv2d_oracle(x, w)
    P, Q = H - R + 1, W - S + 1
    pp, qq = np.meshgrid(np.arange(P), np.arange(Q), indexing="ij")
    rr = np.arange(R).reshape(1, 1, R, 1)
    ss = np.arange(S).reshape(1, 1, 1, S)
    for k in range(K):
        wk = w[k:k + 1].astype(np.float64)
        expect = (a * pp + b * qq + d) * wk.sum() + a * (rr * wk).sum() + b * (ss * wk).sum()
        np.testing.assert_array_equal(y[0, k], expect)


def test_one_by_one_filter_is_a_matrix_product(oracle):
    N, C, H, W, K = 2, 7, 5, 6, 4
    x, w = uniform((N, C, H, W), 41), uniform((K, C, 1, 1), 42)
    y, _ = oracle.conv2d_oracle(x, w)
    wm = w.reshape(K, C).astype(np.float64)
    for n in range(N):
        expect = wm @ x[n].reshape(C, H * W).astype(np.float64)
        np.testing.assert_allclose(y[n].reshape(K, H * W), expect, rtol=0, atol=1e-13)


def test_full_size_filter_is_a_dot_product(oracle):
    N, C, H, W, K = 3, 2, 4, 5, 2
    x, w = uniform((N, C, H, W), 43), uniform((K, C, H, W), 44)
    y, yabs = oracle.conv2d_oracle(x, w)
    assert y.shape == (N, K, 1, 1)
    for n in range(N):
        for k in range(K):
            prod = x[n].astype(np.float64).ravel() * w[k].astype(np.float64).ravel()
            assert abs(y[n, k, 0, 0] - prod.sum()) < 1e-13
            assert abs(yabs[n, k, 0, 0] - np.abs(prod).sum()) < 1e-13


def test_separable_filter_equals_row_pass_then_column_pass(oracle):
    H, W, R, S = 9, 11, 3, 4
    x = small_integers((1, 1, H, W), 51)
    u, v = small_integers((R,), 52), small_integers((S,), 53)
    w = np.outer(u, v).astype(np.float32).reshape(1, 1, R, S)
    y, _ = oracle.conv2d_oracle(x, w)
    rows = np.zeros((H, W - S + 1))
    for s in range(S):
        rows += v[s] * x[0, 0, :, s:s + W - S + 1].astype(np.float64)
    expect = np.zeros((H - R + 1, W - S + 1))
    for r in range(R):
        expect += u[r] * rows[r:r + H - R + 1]
    np.testing.assert_array_equal(y[0, 0], expect)


def test_shift_equivariance_inside_zero_frame(oracle):
    C, R, S = 2, 3, 3
    core = uniform((1, C, 4, 4), 61)
    w = uniform((2, C, R, S), 62)
    def placed(dy, dx):
        x = np.zeros((1, C, 12, 12), np.float32)
        x[:, :, 3 + dy:7 + dy, 3 + dx:7 + dx] = core
        return oracle.conv2d_oracle(x, w)[0]
    y0, y1 = placed(0, 0), placed(2, 1)
    np.testing.assert_array_equal(y1[:, :, 2:, 1:], y0[:, :, :-2, :-1])


def _gather_brute_force(x, w):
    """Differently written: flattened offsets, one explicit pair list per output."""
    N, C, H, W = x.shape
    K, _, R, S = w.shape
    P, Q = H - R + 1, W - S + 1
    xf, wf = x.astype(np.float64).ravel(), w.astype(np.float64).ravel()
    y = np.zeros(N * K * P * Q)
    ya = np.zeros_like(y)
    tap_x = [c * H * W + r * W + s for c in range(C) for r in range(R) for s in range(S)]
    tap_w = list(range(C * R * S))
    for o in range(y.size):
        q, p, k, n = o % Q, (o // Q) % P, (o // (P * Q)) % K, o // (K * P * Q)
        base_x, base_w = n * C * H * W + p * W + q, k * C * R * S
        prods = [xf[base_x + tx] * wf[base_w + tw] for tx, tw in zip(tap_x, tap_w)]
        y[o] = sum(prods)
        ya[o] = sum(abs(t) for t in prods)
    return y.reshape(N, K, P, Q), ya.reshape(N, K, P, Q)


@pytest.mark.parametrize("dims", [(2, 2, 5, 6, 2, 3, 2), (1, 1, 4, 4, 1, 2, 2), (2, 1, 3, 6, 2, 3, 3), (1, 2, 6, 3, 2, 1, 3)])
def test_brute_force_on_tiny_inputs(oracle, dims):
    N, C, H, W, K, R, S = dims
    x, w = small_integers((N, C, H, W), 71), small_integers((K, C, R, S), 72)
    y, yabs = oracle.conv2d_oracle(x, w)
    by, bya = _gather_brute_force(x, w)
    np.testing.assert_array_equal(y, by)
    np.testing.assert_array_equal(yabs, bya)


def test_against_independent_library_convolution(oracle):
    torch = pytest.importorskip("torch")
    N, C, H, W, K, R, S = 2, 5, 13, 17, 6, 5, 3
    x, w = uniform((N, C, H, W), 81), uniform((K, C, R, S), 82)
    y, _ = oracle.conv2d_oracle(x, w)
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double()).numpy()
    np.testing.assert_allclose(y, ref, rtol=0, atol=1e-12)


def test_magnitude_sum_invariants(oracle):
    x, w = uniform((1, 3, 8, 8), 91), uniform((2, 3, 3, 3), 92)
    y, yabs = oracle.conv2d_oracle(x, w)
    assert np.all(np.abs(y) <= yabs + 1e-15)
    sign = np.where(uniform(x.shape, 93) < 0, -1.0, 1.0).astype(np.float32)
    _, yabs2 = oracle.conv2d_oracle(x * sign, -w)
    np.testing.assert_allclose(yabs2, yabs, rtol=0, atol=1e-13)
    _, yabs3 = oracle.conv2d_oracle(np.abs(x), np.abs(w))
    y3, _ = oracle.conv2d_oracle(np.abs(x), np.abs(w))
    np.testing.assert_allclose(yabs3, yabs, rtol=0, atol=1e-13)
    np.testing.assert_allclose(y3, yabs, rtol=0, atol=1e-13)


def test_sub_range_matches_slices_of_the_whole(oracle):
    x, w = uniform((3, 2, 9, 8), 101), uniform((4, 2, 3, 2), 102)
    y, yabs = oracle.conv2d_oracle(x, w)
    ys, yas = oracle.conv2d_oracle_range(x, w, n_range=(1, 3), k_range=(2, 3), p_range=(4, 7))
    np.testing.assert_array_equal(ys, y[1:3, 2:3, 4:7])
    np.testing.assert_array_equal(yas, yabs[1:3, 2:3, 4:7])


def test_tf32_operand_modes_on_known_bit_patterns(oracle):
    # TF32 keeps 10 explicit mantissa bits: 1 + 2^-11 lies exactly between 1 and 1 + 2^-10.
    from oracle.conv2d_oracle import MODE_TF32_RNA, MODE_TF32_TRUNC
    one = np.ones((1, 1, 1, 1), np.float32)
    for v, rna, trunc in [
        (1.0 + 2.0 ** -11, 1.0 + 2.0 ** -10, 1.0),               # tie: away from zero / down
        (-(1.0 + 2.0 ** -11), -(1.0 + 2.0 ** -10), -1.0),
        (1.0 + 2.0 ** -12, 1.0, 1.0),                             # below half: both down
        (1.0 + 2.0 ** -10 + 2.0 ** -11 + 2.0 ** -23, 1.0 + 2.0 ** -9, 1.0 + 2.0 ** -10),
        (0.75, 0.75, 0.75),                                       # representable: unchanged
    ]:
        x = np.full((1, 1, 1, 1), v, np.float32)
        assert oracle.conv2d_oracle(x, one, mode=MODE_TF32_RNA)[0].item() == rna
        assert oracle.conv2d_oracle(x, one, mode=MODE_TF32_TRUNC)[0].item() == trunc
        assert oracle.conv2d_oracle(one, x, mode=MODE_TF32_RNA)[0].item() == rna
        assert oracle.conv2d_oracle(x, one)[0].item() == np.float32(v)


def test_small_integers_are_unchanged_by_tf32_modes(oracle):
    from oracle.conv2d_oracle import MODE_TF32_RNA, MODE_TF32_TRUNC
    x, w = small_integers((1, 4, 6, 6), 111), small_integers((3, 4, 3, 3), 112)
    y0, _ = oracle.conv2d_oracle(x, w)
    np.testing.assert_array_equal(oracle.conv2d_oracle(x, w, mode=MODE_TF32_RNA)[0], y0)
    np.testing.assert_array_equal(oracle.conv2d_oracle(x, w, mode=MODE_TF32_TRUNC)[0], y0)

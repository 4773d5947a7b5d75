"""The seeded generators: determinism, order independence and the stated distributions."""
import numpy as np

from workloads import CONFIGS, make_inputs, normal, relu_normal, small_integers, uniform


def test_deterministic_and_prefix_stable():
    a, b = uniform((4, 5), 7), uniform((4, 5), 7)
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(uniform((10,), 7), uniform((20,), 7)[:10])   # counter based
    assert not np.array_equal(uniform((20,), 7), uniform((20,), 8))


def test_distributions():
    u = uniform((200000,), 1)
    assert u.dtype == np.float32 and -1.0 <= u.min() and u.max() < 1.0
    assert abs(u.mean()) < 0.01 and abs(u.var() - 1.0 / 3.0) < 0.01
    g = normal((200000,), 2, 0.2)
    assert abs(g.mean()) < 0.005 and abs(g.std() - 0.2) < 0.005
    r = relu_normal((200000,), 3)
    assert r.min() == 0.0 and abs((r == 0).mean() - 0.5) < 0.01
    i = small_integers((100000,), 4)
    assert set(np.unique(i)) == set(float(v) for v in range(-4, 5))


def test_config_shapes_and_weight_scale():
    c3 = CONFIGS["cfg3"]
    x, w = make_inputs(c3, batch=2)
    assert x.shape == (2, 64, 56, 56) and w.shape == (64, 64, 3, 3)
    assert abs(w.std() - (2.0 / 576) ** 0.5) < 2e-3
    assert CONFIGS["cfg2"].flops == 2 * 32 * 25 * 4092 * 4092
    assert CONFIGS["cfg5_r7"].Q == 26
    x5, w5 = make_inputs(CONFIGS["cfg5_r3"], batch=1)
    assert 0.0 <= x5.min() and x5.max() < 1.0 and w5.shape == (128, 128, 3, 3)


def test_bf16_rounding_helper_matches_torch():
    import torch
    from helpers import bf16_values
    from workloads import uniform
    a = uniform((4097,), 431, -3.0, 3.0)
    vals, pat = bf16_values(a)
    t = torch.from_numpy(a).to(torch.bfloat16)
    np.testing.assert_array_equal(vals, t.float().numpy())
    np.testing.assert_array_equal(pat.view(np.int16), t.view(torch.int16).numpy())

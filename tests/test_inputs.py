"""Host logic of the synthetic input generator: determinism, independence of chunking,
distribution moments, bf16 rounding and layout round trips."""
import numpy as np

from paper_2305_11624_b200 import inputs as I


def test_counter_based_values_do_not_depend_on_chunking():
    a = I.uniform01(5, 1, 1000)
    b = np.concatenate([I.uniform01(5, 1, 300), I.uniform01(5, 1, 700, start=300)])
    np.testing.assert_array_equal(a, b)
    assert not np.array_equal(a, I.uniform01(6, 1, 1000))
    assert not np.array_equal(a, I.uniform01(5, 2, 1000))


def test_moments():
    n = 1 << 20
    z = I.normal(11, 1, n).astype(np.float64)
    assert abs(z.mean()) < 5e-3 and abs(z.std() - 1) < 5e-3
    assert abs((z ** 4).mean() - 3) < 0.05
    u = I.uniform(11, 5, n, 0.5, 2.0).astype(np.float64)
    assert u.min() >= 0.5 and u.max() <= 2.0 and abs(u.mean() - 1.25) < 5e-3


def test_bf16_round_to_nearest_even():
    f = lambda bits: np.array([bits], dtype=np.uint32).view(np.float32)
    assert I.f32_to_bf16_bits(f(0x3F800000))[0] == 0x3F80
    assert I.f32_to_bf16_bits(f(0x3F808000))[0] == 0x3F80      # tie -> even (down)
    assert I.f32_to_bf16_bits(f(0x3F818000))[0] == 0x3F82      # tie -> even (up)
    assert I.f32_to_bf16_bits(f(0x3F808001))[0] == 0x3F81
    assert I.f32_to_bf16_bits(f(0xBF80FFFF))[0] == 0xBF81
    x = I.normal(3, 1, 4096)
    r = I.round_bf16(x)
    np.testing.assert_array_equal(I.round_bf16(r), r)
    assert np.max(np.abs(r - x) / np.abs(x)) <= 2.0 ** -8


def test_block_recipe_and_layouts():
    sp = I.CONFIGS[0][0]
    t = I.make_block(sp, I.config_seed(0), (16, 16))
    t2 = I.make_block(sp, I.config_seed(0), (16, 16))
    for k in t:
        np.testing.assert_array_equal(t[k], t2[k])
    assert t["x"].shape == (2, 16, 16, 16) and t["w"].shape == (32, 16, 3, 3)
    assert t["b"] is not None and t["dz"].shape == (2, 32, 16, 16)
    assert 0.5 <= t["var_hat"].min() and t["gamma"].max() <= 1.5
    assert abs(float(t["w"].std()) - np.sqrt(2.0 / 144)) < 0.01
    sp1 = I.CONFIGS[1][1]
    small = I.LayerSpec("s", 1, 8, 5, 6, 4, 3, 3, pad=1)
    u = I.make_block(small, 1, (5, 6))
    assert u["b"] is None
    np.testing.assert_array_equal(I.round_bf16(u["x"]), u["x"])
    nhwc = I.act_to_layout(u["x"], "nhwc")
    assert nhwc.shape == (1, 5, 6, 8) and nhwc[0, 2, 3, 4] == u["x"][0, 4, 2, 3]
    np.testing.assert_array_equal(I.act_from_layout(nhwc, "nhwc", u["x"].shape), u["x"])
    wl = I.weight_to_layout(u["w"], "nhwc")
    assert wl.shape == (4, 3, 3, 8) and wl[1, 2, 0, 5] == u["w"][1, 5, 2, 0]
    np.testing.assert_array_equal(I.weight_from_layout(wl, "nhwc", u["w"].shape), u["w"])
    assert sp1.dims()["pad_h"] == 1 and len(I.CONFIGS) == 5

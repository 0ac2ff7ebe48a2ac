"""Host-side checks of the seeded input generator (no method arithmetic there)."""
import numpy as np

import pike_inputs as G


def test_deterministic_and_counter_based():
    a = G.normal((7, 33), seed=0, tensor_id=5, dtype="f32")
    b = G.normal((7, 33), seed=0, tensor_id=5, dtype="f32")
    assert np.array_equal(a, b)
    # element i depends only on (seed, tensor, i): a longer draw has the same prefix
    long = G.normal((7 * 33 + 100,), seed=0, tensor_id=5, dtype="f32")
    assert np.array_equal(long[: 7 * 33], a.ravel())
    assert not np.array_equal(a, G.normal((7, 33), seed=1, tensor_id=5, dtype="f32"))
    assert not np.array_equal(a, G.normal((7, 33), seed=0, tensor_id=6, dtype="f32"))


def test_uniform_range_and_moments():
    a = 1.0 / 64
    u = G.uniform((1 << 18,), a, seed=0, tensor_id=2, dtype="f32").astype(np.float64)
    assert u.min() >= -a and u.max() <= a      # the fp32 rounding may touch +a
    assert abs(u.mean()) < 4 * a / np.sqrt(3 * u.size)
    assert abs(u.var() - a * a / 3) < 0.02 * a * a / 3


def test_normal_moments():
    z = G.normal((1 << 18,), seed=0, tensor_id=1, dtype="f32").astype(np.float64)
    assert abs(z.mean()) < 4 / np.sqrt(z.size)
    assert abs(z.var() - 1) < 0.02
    assert abs((z ** 4).mean() - 3) < 0.15
    assert np.isfinite(z).all()


def test_bf16_values_are_representable_and_nearest_even():
    z = G.normal((4096,), seed=0, tensor_id=1, dtype="bf16")
    assert (z.view(np.uint32) & 0xFFFF == 0).all()
    f = G.normal((4096,), seed=0, tensor_id=1, dtype="f32")
    assert np.abs(z - f).max() <= np.abs(f).max() * 2.0 ** -8
    # ties go to the even mantissa: 1 + 2^-8 -> 1, 1 + 3*2^-8 -> 1 + 2^-6
    t = np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8], np.float32)
    assert np.array_equal(G.round_to_bf16(t), np.array([1.0, 1 + 2.0 ** -6], np.float32))


def test_f16_values_are_representable_and_nearest_even():
    z = G.normal((4096,), seed=0, tensor_id=1, dtype="f16")
    # a binary16 normal number has 11 significant bits: the low 13 bits of the fp32 mantissa are zero
    normal = np.abs(z) >= 2.0 ** -14
    assert normal.mean() > 0.99 and (z[normal].view(np.uint32) & 0x1FFF == 0).all()
    f = G.normal((4096,), seed=0, tensor_id=1, dtype="f32")
    assert np.abs(z - f).max() <= np.abs(f).max() * 2.0 ** -11
    # ties to even: 1 + 2^-11 -> 1, 1 + 3*2^-11 -> 1 + 2^-9; 2049 -> 2048, 2051 -> 2052
    t = np.array([1 + 2.0 ** -11, 1 + 3 * 2.0 ** -11, 2049, 2051], np.float32)
    assert np.array_equal(G.round_to_f16(t), np.array([1.0, 1 + 2.0 ** -9, 2048, 2052], np.float32))
    # the same draw rounded to bf16 is a different tensor: the two 16-bit recipes are distinct inputs
    assert (G.normal((4096,), seed=0, tensor_id=1, dtype="bf16") != z).mean() > 0.5
    c = G.config3(M=4, D=8, F=16, affine=True, dtype="f16")
    assert np.array_equal(G.round_to_f16(c["gamma"]), c["gamma"]) and np.array_equal(G.round_to_f16(c["w1"]), c["w1"])


def test_config_shapes():
    c1 = G.config1()
    assert c1["x"].shape == (128, 256) and c1["w"].shape == (256, 256) and c1["b"].shape == (256,)
    c2 = G.config2(M=8, K=16, N=24)
    assert c2["x"].shape == (8, 16) and c2["w"].shape == (16, 24) and c2["r"].shape == (8, 24)
    c3 = G.config3(M=4, D=8, F=16, affine=True)
    assert c3["w1"].shape == (8, 16) and c3["w2"].shape == (16, 8)
    assert (c3["gamma"].view(np.uint32) & 0xFFFF == 0).all()
    c5 = G.config5(B=1, H=2, S=4, D=8)
    assert c5["q"].shape == (1, 2, 4, 8)

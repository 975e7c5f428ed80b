"""The seeded generators are deterministic, counter-based and have the stated laws."""
import numpy as np

from workloads import tensors, configs


def test_counter_based_and_deterministic():
    a = tensors.normal(3, 1, 1000)
    b = tensors.normal(3, 1, 1000)
    np.testing.assert_array_equal(a, b)
    # element i does not depend on how many elements are drawn (chunk boundaries included)
    big = tensors.uniform(0, 2, (1 << 22) + 17)
    np.testing.assert_array_equal(big[:100], tensors.uniform(0, 2, 100))
    assert not np.array_equal(tensors.normal(3, 2, 1000), a)
    assert not np.array_equal(tensors.normal(4, 1, 1000), a)


def test_laws():
    n = 1 << 20
    x = tensors.normal(0, 0, n, mean=1.0, std=0.1)
    assert abs(x.mean() - 1.0) < 1e-3 and abs(x.std() - 0.1) < 1e-3
    u = tensors.uniform(0, 1, n, -1.0, 1.0)
    assert u.min() >= -1.0 and u.max() < 1.0 and abs(u.mean()) < 5e-3 and abs(u.var() - 1 / 3) < 5e-3
    k = tensors.integers(0, 2, n, -8, 8)
    assert k.min() == -8 and k.max() == 8 and np.all(k == np.round(k))


def test_bf16_rounding_ties_to_even():
    v = np.array([1.0, 1.00390625, 1.01171875, 1.0078125, -2.5, 3.0e38], dtype=np.float32)
    r = tensors.bf16_bits_to_f32(tensors.round_to_bf16_bits(v))
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7 -> even mantissa (1.0); 1 + 3*2^-8 ties up to 1 + 2^-6
    np.testing.assert_array_equal(r[:5], np.array([1.0, 1.0, 1.015625, 1.0078125, -2.5], dtype=np.float32))
    assert np.isfinite(r[5])


def test_config_inputs_have_declared_shapes():
    spec, laws = configs.get_config("c4_conv_bn_relu_bf16", n=1, h=8, w=8)
    t = configs.draw_inputs(spec, laws, 0)
    assert t["x"].shape == (1, 128, 8, 8) and t["x"].dtype == np.uint16
    assert t["scale"].shape == (128, 1, 1) and t["scale"].dtype == np.float32
    assert 0.5 <= t["scale"].min() and t["scale"].max() < 1.5

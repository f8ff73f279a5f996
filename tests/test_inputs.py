"""The seeded input generator: determinism, bf16 rounding, layouts, recipe statistics."""
import numpy as np
import pytest

from paper_2605_28213_b200 import inputs as gen


def test_same_seed_same_bits_and_different_seed_differs():
    a = gen.make_config("c1", 1)
    b = gen.make_config("c1", 1)
    c = gen.make_config("c1", 2)
    assert np.array_equal(a.A, b.A) and np.array_equal(a.B, b.B)
    assert not np.array_equal(a.A, c.A)
    assert not np.array_equal(a.A, a.B)          # tensors use different streams


def test_bf16_rounding_matches_torch():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(50000), rng.uniform(-1, 1, 50000),
                        [1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, 0.0, -0.0]]).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(gen.f32_to_bf16_bits(x), ref)
    assert np.array_equal(gen.f32_to_bf16_bits(gen.bf16_bits_to_f32(ref)), ref)


def test_config_shapes_layouts_and_padding():
    c2 = gen.make_config("c2", 1)
    assert (c2.M, c2.N, c2.K, c2.lda, c2.ldb, c2.ldc) == (1000, 1001, 999, 999, 1001, 1001)
    assert c2.A.shape == (1000, 999) and c2.B.shape == (999, 1001) and not c2.c_bf16
    p = gen.make_config("c2pad", 1)
    assert p.A.shape == (1000, 1008) and p.B.shape == (999, 1008) and p.ldc == 1004
    assert np.array_equal(p.A[:, :999], c2.A) and np.array_equal(p.B[:, :1001], c2.B)
    assert np.all(p.A[:, 999:] == gen.BF16_NAN_BITS)
    assert np.isnan(gen.bf16_bits_to_f32(p.A[:, 999:])).all()


def test_column_major_b_is_the_transpose_of_the_same_draw():
    r = gen.make_case(8, 24, 16, seed=3, b_col_major=False)
    c = gen.make_case(8, 24, 16, seed=3, b_col_major=True)
    assert c.B.shape == (24, 16) and np.array_equal(c.B, r.B.T) and c.ldb == 16


def test_distributions_follow_the_recipe():
    u = gen.bf16_bits_to_f32(gen.draw((512, 512), "uniform", 1, 0))
    assert u.min() >= -1.0 and u.max() <= 1.0 and abs(u.mean()) < 0.01
    assert abs(u.std() - 3 ** -0.5) < 0.01
    n = gen.bf16_bits_to_f32(gen.draw((512, 512), "normal", 1, 0, 0.02))
    assert abs(n.std() - 0.02) < 0.0005 and abs(n.mean()) < 0.0005
    i = gen.bf16_bits_to_f32(gen.draw((256, 256), "integer", 1, 0))
    assert set(np.unique(i)) == set(float(v) for v in range(-4, 5))


def test_integer_variant_and_algorithmic_bytes():
    c = gen.make_config("c1", 2, integer=True)
    assert c.name == "c1-int"
    assert set(np.unique(gen.bf16_bits_to_f32(c.A))) <= set(float(v) for v in range(-4, 5))
    assert c.algorithmic_bytes == 131072 + 131072 + 262144 and c.flops == 2 * 256 ** 3
    assert gen.config_shape("c5")["M"] == 16 and gen.config_shape("c3")["b_col_major"]

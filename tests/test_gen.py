"""The seeded input generators: determinism, slice independence and the stated distributions."""
import numpy as np

import gen
from gen import rng


def test_streams_are_counter_based():
    a = rng.raw_u64(5, 1, 0, 0, 1000)
    b = rng.raw_u64(5, 1, 0, 400, 100)
    assert np.array_equal(a[400:500], b)
    assert not np.array_equal(a, rng.raw_u64(6, 1, 0, 0, 1000))
    assert not np.array_equal(a, rng.raw_u64(5, 2, 0, 0, 1000))
    assert len(np.unique(a)) == 1000


def test_ternary_density_and_signs():
    t = rng.ternary(1, 1, 400_000, 0.25)
    assert set(np.unique(t)) == {-1, 0, 1}
    assert abs(np.count_nonzero(t) / t.size - 0.25) < 0.005
    assert abs((t == 1).sum() / max(1, np.count_nonzero(t)) - 0.5) < 0.01


def test_normal_and_bf16_rounding():
    g = rng.normal(2, 1, 200_000)
    assert abs(g.mean()) < 0.01 and abs(g.std() - 1.0) < 0.01
    f = g.astype(np.float32)
    bits = rng.f32_to_bf16_bits(f)
    back = rng.bf16_bits_to_f32(bits)
    rel = np.abs(back - f) / np.maximum(np.abs(f), 1e-30)
    assert rel.max() <= 2.0 ** -8
    # ties go to even: 1 + 2^-8 lies halfway between 1 and 1 + 2^-7
    tie = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8], dtype=np.float32)
    assert list(rng.bf16_bits_to_f32(rng.f32_to_bf16_bits(tie))) == [1.0, 1.0 + 2.0 ** -6]


def test_case_builder_matches_spec():
    spec = gen.scaled(gen.CONFIGS["cfg1"])
    c = gen.make_case(spec)
    assert c.U.shape == (256, 256) and c.V.shape == (256, 256) and c.x.shape == (8, 256)
    assert c.S.dtype == np.float32 and np.all(np.diff(c.S) <= 0) and c.S.min() >= 0.01 and c.S.max() <= 1.0
    assert abs(np.count_nonzero(c.U) / c.U.size - 0.3) < 0.02
    # tokens can be generated in slices
    assert np.array_equal(gen.make_x(spec, 3, 2), c.x[3:5])
    s5 = gen.scaled(gen.CONFIGS["cfg5_d20"], M=8, N=512, K=8, B=4)
    x5 = gen.make_x(s5)
    assert x5.dtype == np.int8 and x5.min() >= -127 and x5.max() <= 127
    s2 = gen.scaled(gen.CONFIGS["cfg2"], M=8, N=64, K=8, B=4)
    assert gen.make_x(s2).dtype == np.uint16

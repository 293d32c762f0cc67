"""The synthetic input generators: exact counts, bf16 rounding, Zipf row populations."""
import numpy as np

import mst_inputs as gi


def test_bf16_round_to_nearest_even():
    x = np.array([1.0, 1.00390625, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -2.5, 0.0, 3.14159], dtype=np.float32)
    b = gi.f32_to_bf16_bits(x)
    back = gi.bf16_bits_to_f32(b)
    assert back[0] == 1.0 and back[4] == -2.5 and back[5] == 0.0
    assert back[2] == 1.0                       # tie -> even mantissa (1.0)
    assert back[3] == np.float32(1.0 + 2 ** -6)   # tie -> even mantissa (1.015625)
    assert abs(back[6] - 3.14159) <= 2 ** -7 * 2
    assert np.array_equal(gi.f32_to_bf16_bits(back), b)      # idempotent


def test_uniform_mask_exact_count_and_determinism():
    m = gi.uniform_mask(48, 64, 777, 5, 1)
    assert m.sum() == 777 and m.shape == (48, 64)
    assert np.array_equal(m, gi.uniform_mask(48, 64, 777, 5, 1))
    assert not np.array_equal(m, gi.uniform_mask(48, 64, 777, 6, 1))
    assert gi.uniform_mask(4, 4, 16, 1).all() and not gi.uniform_mask(4, 4, 0, 1).any()


def test_config_layer_counts():
    assert gi.exact_nnz(3072, 768, 0.25) == 589824
    assert [gi.exact_nnz(o, i, 0.1) for _, o, i in gi.block_shapes(1024)] == [314573, 104858, 419430, 419430]
    for lid in range(48):
        assert 0.03 <= gi.config3_density(lid) <= 0.10


def test_zipf_rows():
    O, I, nnz = 768, 768, int(0.06 * 768 * 768)
    c = gi.zipf_row_counts(O, I, nnz, 1.1, 3, 0)
    assert c.sum() == nnz and c.max() <= I
    s = np.sort(c)[::-1]
    assert s[0] == I                                  # the heaviest row saturates at this density
    assert s[0] >= 20 * max(int(np.median(c)), 1)     # heavy skew
    uncapped = s[s < I][:50].astype(float)
    r = np.arange(1, len(uncapped) + 1)
    slope = np.polyfit(np.log(r + (s >= I).sum()), np.log(uncapped), 1)[0]
    assert -1.4 < slope < -0.8                        # ~ rank^-1.1
    m = gi.zipf_mask(64, 96, 900, 1.1, 3, 0)
    assert m.sum() == 900
    assert np.array_equal(m.sum(1), gi.zipf_row_counts(64, 96, 900, 1.1, 3, 0))


def test_layer_problem_bf16_values_are_exact():
    p = gi.uniform_layer("x", 0, 16, 32, 8, "bf16", 0.25, 9)
    assert np.array_equal(gi.f32_to_bf16_bits(p.W), p.W_bits)
    assert np.array_equal(gi.bf16_bits_to_f32(p.X_bits), p.X)
    assert abs(float(p.X.std()) - 1.0) < 0.2 and abs(float(p.W.std()) - 0.02) < 0.01
    assert p.nnz == 128

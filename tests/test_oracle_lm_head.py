"""The oracle's LM-head product (logits = hidden @ weight^T, bf16 in, double accumulation, one
rounding to bf16) against numpy on inputs whose products and sums are exact, and its rounding
against hand-checked cases."""
import numpy as np

import oracle
from helpers import bf16_bits_to_f64, f32_to_bf16_bits


def test_exact_inputs_match_numpy_matmul():
    rng = np.random.default_rng(0)
    h = rng.integers(-3, 4, (37, 96)).astype(np.float32) * np.float32(0.25)
    w = rng.integers(-2, 3, (53, 96)).astype(np.float32)
    got = oracle.lm_head(f32_to_bf16_bits(h), f32_to_bf16_bits(w), threads=3)
    want = h.astype(np.float64) @ w.astype(np.float64).T            # exact: small integers over 4
    assert np.abs(want).max() < 256 * 0.25 * 8
    representable = bf16_bits_to_f64(f32_to_bf16_bits(want.astype(np.float32))) == want
    assert representable.mean() > 0.95                             # nearly all sums fit bf16 exactly
    assert np.array_equal(bf16_bits_to_f64(got)[representable], want[representable])


def test_rounding_is_to_nearest_even_in_one_step():
    # 1 + 2^-8 lies exactly between two bf16 numbers (1 and 1 + 2^-7): ties go to the even one (1.0);
    # 1 + 3 * 2^-8 lies between 1 + 2^-7 and 1 + 2^-6: the even one is 1 + 2^-6.
    # A sum that only a double holds exactly (1 + 2^-8 + 2^-40) must round UP: rounding first to
    # float32 (1 + 2^-8 exactly, then the tie to even) would give 1.0 -- the classic double rounding.
    one = np.float32(1.0)
    def dot(pairs):
        h = f32_to_bf16_bits(np.array([[a for a, _ in pairs]], np.float32))
        w = f32_to_bf16_bits(np.array([[b for _, b in pairs]], np.float32))
        return float(bf16_bits_to_f64(oracle.lm_head(h, w))[0, 0])
    assert dot([(1.0, 1.0), (2.0 ** -8, 1.0)]) == 1.0
    assert dot([(1.0, 1.0), (2.0 ** -8, 1.0), (2.0 ** -8, 2.0)]) == 1.0 + 2.0 ** -6
    assert dot([(1.0, 1.0), (2.0 ** -8, 1.0), (2.0 ** -20, 2.0 ** -20)]) == 1.0 + 2.0 ** -7
    assert dot([(-1.0, 1.0), (2.0 ** -8, -1.0), (2.0 ** -20, -(2.0 ** -20))]) == -(1.0 + 2.0 ** -7)
    assert dot([(0.0, 5.0)]) == 0.0


def test_random_inputs_are_within_half_an_ulp_of_the_exact_product():
    rng = np.random.default_rng(1)
    hb = f32_to_bf16_bits(rng.normal(0, 1, (9, 200)).astype(np.float32))
    wb = f32_to_bf16_bits(rng.normal(0, 1, (31, 200)).astype(np.float32))
    got = bf16_bits_to_f64(oracle.lm_head(hb, wb))
    exact = bf16_bits_to_f64(hb) @ bf16_bits_to_f64(wb).T
    ulp = 2.0 ** (np.floor(np.log2(np.abs(exact))) - 7)
    assert np.all(np.abs(got - exact) <= 0.5 * ulp * (1 + 1e-12))

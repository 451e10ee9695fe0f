"""Pins for the oracle's residual step h_out = round(h_in + y) (fp32 add, bf16 round-to-nearest-even)."""
import numpy as np

from paper_2609_01024_b200 import workloads as wl


def bits(x):
    return wl.f32_to_bf16_bits(np.asarray(x, np.float32))


def test_hand_cases_bf16(oracle):
    # bf16 keeps 8 significant bits: around 1.0 the spacing is 2^-7, so 1 + 2^-8 is a tie (goes to even)
    h = bits([1.0, 1.0, 1.0, 1.0078125, -2.0, 0.0])
    y = np.array([2.0 ** -8, 2.0 ** -8 + 2.0 ** -20, 2.0 ** -9, 2.0 ** -8, 0.5, -0.0], np.float32)
    out = oracle.residual_cast(h, y)
    want = [1.0,            # tie: 1 is even (mantissa ...0), stays
            1.0078125,      # just above the tie: rounds up
            1.0,            # below half a step: stays
            1.015625,       # 1.0078125 is odd: the tie goes up to the even neighbour
            -1.5, 0.0]
    assert np.array_equal(wl.bf16_to_f32(out), np.array(want, np.float32))


def test_fp32_is_the_plain_sum_and_zero_y_is_identity(oracle):
    rng = np.random.default_rng(0)
    h = rng.standard_normal(1000).astype(np.float32)
    y = rng.standard_normal(1000).astype(np.float32)
    assert np.array_equal(oracle.residual_cast(h, y), h + y)
    hb = bits(h)
    assert np.array_equal(oracle.residual_cast(hb, np.zeros(1000, np.float32)), hb)


def test_against_the_generator_rounding(oracle):
    # the input generators' own f32 -> bf16 conversion is an independent implementation of the same rounding
    rng = np.random.default_rng(1)
    h = bits(rng.standard_normal(5000))
    y = (rng.standard_normal(5000) * 0.1).astype(np.float32)
    s = (wl.bf16_to_f32(h) + y).astype(np.float32)
    assert np.array_equal(oracle.residual_cast(h, y), wl.f32_to_bf16_bits(s))

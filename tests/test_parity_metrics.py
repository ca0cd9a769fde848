"""The parity metrics of the GPU tests, checked on the CPU on constructed cases (no GPU, no kernel).

check_out accepts an element beyond max|diff| <= 2e-2 * rms only if the value is one of the two bf16 numbers that
bracket the oracle's unrounded fp32 result (a one-ulp rounding flip).  The bracket must be right at values that
are not powers of two, where one bf16 ulp is 2^-7 of the binade's base, not of the value.
"""
import numpy as np
import pytest

from paper_2609_15627_b200 import inputs
from _gpu_util import bf16_neighbours, check_out, check_y


def _bits(v):
    b = inputs.f32_to_bf16_bits(np.asarray(v, np.float32))
    return b.reshape(np.shape(v))[()]


def test_bf16_neighbours_at_values_that_are_not_powers_of_two():
    # [32, 64): one bf16 ulp is 0.25; [1, 2): 2^-7; negative values mirror; an exact bf16 value brackets itself
    f = np.array([37.3, 63.9, 1.0039, -37.3, 48.0, 2.0 ** -130], np.float32)
    lo, hi = bf16_neighbours(f)
    assert lo.tolist()[:5] == [37.25, 63.75, 1.0, -37.25, 48.0]
    assert hi.tolist()[:5] == [37.5, 64.0, 1.0078125, -37.5, 48.25]
    assert lo[5] <= f[5] <= hi[5] and hi[5] > lo[5]          # subnormal range: still a strict bracket
    # every bracket is tight: lo and hi are adjacent bf16 numbers and contain the value
    rng = np.random.default_rng(0)
    g = (rng.standard_normal(20000) * 20).astype(np.float32)
    lo, hi = bf16_neighbours(g)
    assert np.all(np.abs(lo) <= np.abs(g)) and np.all(np.abs(g) < np.abs(hi))
    lo_b, hi_b = _bits(lo.astype(np.float32)), _bits(hi.astype(np.float32))
    assert np.array_equal(hi_b.astype(np.int64) - lo_b.astype(np.int64), np.ones(g.size, np.int64))


def _case(outlier_f32):
    rng = np.random.default_rng(1)
    ref_f32 = rng.standard_normal(4096).astype(np.float32)        # rms about 1: 2e-2 * rms = 0.02
    ref_f32[100] = outlier_f32
    return ref_f32, _bits(ref_f32)


def test_check_out_accepts_a_one_ulp_flip_upwards_at_a_non_power_of_two():
    ref_f32, ref_bits = _case(37.3)                                # rounds to 37.25; the other neighbour is 37.5
    got = ref_bits.copy()
    got[100] = _bits(37.5)
    r = check_out(got, ref_bits, ref_f32, "flip up")               # |diff| = 0.25 >> 0.02
    assert r["flips"] == 1
    ref_f32, ref_bits = _case(-37.45)                              # rounds to -37.5; the other neighbour is -37.25
    got = ref_bits.copy()
    got[100] = _bits(-37.25)
    assert check_out(got, ref_bits, ref_f32, "flip down")["flips"] == 1


def test_check_out_rejects_two_ulps_and_a_wrong_sign():
    ref_f32, ref_bits = _case(37.3)
    for wrong in (37.75, 37.0, -37.25):
        got = ref_bits.copy()
        got[100] = _bits(wrong)
        with pytest.raises(AssertionError):
            check_out(got, ref_bits, ref_f32, "not a flip")


def test_check_out_and_check_y_enforce_the_frobenius_bounds():
    ref_f32, ref_bits = _case(0.5)
    got_f = inputs.bf16_bits_to_f32(ref_bits) * np.float32(1.0 + 2.0 ** -7)   # every element one ulp off: rel 7.8e-3
    with pytest.raises(AssertionError):
        check_out(_bits(got_f), ref_bits, ref_f32, "rel")
    y = np.random.default_rng(2).standard_normal((64, 256)).astype(np.float32)
    check_y(y * np.float32(1 + 1e-5), y, "close")
    with pytest.raises(AssertionError):
        check_y(y * np.float32(1 + 1e-3), y, "rel 1e-3 > 5e-4")


def test_same_up_to_rounding_allows_one_unit_and_cancelled_values_only():
    from _gpu_util import assert_same_up_to_rounding
    rng = np.random.default_rng(3)
    want = _bits((rng.standard_normal(4096) * 8).astype(np.float32))
    got = want.copy()
    got[5] += 1                                     # one unit up
    got[9] = _bits(np.float32(3e-4)); want[9] = _bits(np.float32(1e-4))   # cancelled to almost nothing: many units, tiny difference
    assert_same_up_to_rounding(got, want, "ok")
    bad = want.copy()
    bad[7] += 2                                     # two units at an ordinary magnitude
    if abs(float(inputs.bf16_bits_to_f32(want[7:8])[0])) > 1.0:
        with pytest.raises(AssertionError):
            assert_same_up_to_rounding(bad, want, "two units")
    many = want.copy()
    many[:400] ^= 1                                 # every tenth element off by one unit: too many
    with pytest.raises(AssertionError):
        assert_same_up_to_rounding(many, want, "many")

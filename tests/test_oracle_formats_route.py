"""Pins for the oracle's scalar formats, routing and permutation (CPU only).

Each expected value comes from the paper's printed facts (tests/golden), from a
closed form, from a library routine (sort, exp) or from brute force, never from
the oracle itself or from the CUDA library.
"""
import math
import os

import numpy as np
import pytest

from _exact import load_numbers
from oracle import moe_oracle as O
from paper_2609_15627_b200 import inputs


# ---- E2M1 / E8M0 / bf16 -----------------------------------------------------------

def test_e2m1_matches_printed_doubled_magnitudes(golden_dir):
    doubled = load_numbers(os.path.join(golden_dir, "e2m1_doubled_magnitudes.txt"))[0]
    assert len(doubled) == 8
    for code in range(8):
        assert 2.0 * O.e2m1_value(code) == float(doubled[code])
        assert 2.0 * O.e2m1_value(code + 8) == -float(doubled[code])
    # code 8 is minus zero: numerically zero, sign bit set (the paper compares numerically)
    assert O.e2m1_value(8) == 0.0 and math.copysign(1.0, O.e2m1_value(8)) == -1.0


def test_e8m0_is_power_of_two():
    for b in range(255):
        assert O.e8m0_value(b) == math.ldexp(1.0, b - 127)
    assert math.isnan(O.e8m0_value(255))
    assert [O.e8m0_value(b) for b in (119, 120, 121, 122)] == [2.0 ** -8, 2.0 ** -7, 2.0 ** -6, 2.0 ** -5]


def test_dequant_exhaustive_codes_times_scales():
    # every code in both nibble positions against every scale byte of the workloads, plus extremes
    for sb in (119, 120, 121, 122, 0, 1, 127, 200):  # 6 * 2^127 would overflow fp32
        codes = np.zeros((1, 16), np.uint8)  # K = 32 -> 16 bytes
        for j in range(16):
            codes[0, j] = (j & 0xF) | (((15 - j) & 0xF) << 4)
        w = O.dequant(codes, np.full((1, 1), sb, np.uint8))
        mags = [0, .5, 1, 1.5, 2, 3, 4, 6]
        for j in range(16):
            lo, hi = j, 15 - j
            for h, c in ((2 * j, lo), (2 * j + 1, hi)):
                want = (-1.0 if c >= 8 else 1.0) * mags[c & 7] * math.ldexp(1.0, sb - 127)
                assert float(w[0, h]) == want, (sb, j, h, c)


def test_dequant_scale_follows_row_and_block():
    # a distinct scale per (row, block): a transposed or shifted scale index changes the result
    rows, K = 4, 128
    codes = np.full((rows, K // 2), 0x22, np.uint8)  # every element is code 2 = 1.0
    scales = inputs.index_scales(rows, K)[0]
    w = O.dequant(codes, scales)
    for r in range(rows):
        for h in range(K):
            assert float(w[r, h]) == math.ldexp(1.0, int(scales[r, h // 32]) - 127)


def test_bf16_rounding_is_nearest_even():
    assert O.f32_to_bf16(1.0) == 0x3F80
    # 1 + 2^-8 is halfway between 1.0 (even) and 1 + 2^-7: ties to even -> 1.0
    assert O.f32_to_bf16(1.0 + 2.0 ** -8) == 0x3F80
    # 1 + 3*2^-8 is halfway between 1+2^-7 (odd) and 1+2^-6 (even) -> up
    assert O.f32_to_bf16(1.0 + 3 * 2.0 ** -8) == 0x3F82
    assert O.f32_to_bf16(1.0 + 2.0 ** -8 + 2.0 ** -20) == 0x3F81
    assert O.f32_to_bf16(-2.5) == 0xC020
    rng = np.random.default_rng(1)
    v = rng.standard_normal(2000).astype(np.float32) * 37.0
    got = np.array([O.f32_to_bf16(float(f)) for f in v], np.uint16)
    back = (got.astype(np.uint32) << 16).view(np.float32)
    # nearest: error at most half a bf16 ulp (2^-8 relative to the binade)
    assert np.all(np.abs(back.astype(np.float64) - v) <= np.abs(v).astype(np.float64) * 2.0 ** -8)
    # the generator's rounding is the same function
    assert np.array_equal(got, inputs.f32_to_bf16_bits(v))
    assert O.bf16_to_f32(0x3F80) == 1.0 and O.bf16_to_f32(0xC020) == -2.5


# ---- the specified exponential ----------------------------------------------------------

def test_exp_spec_against_double_exp():
    assert O.exp_spec(0.0) == 1.0
    d = np.concatenate([np.linspace(-80.0, 0.0, 40001), -np.logspace(-8, 1.9, 4000)]).astype(np.float32)
    worst = 0.0
    for v in d:
        got = O.exp_spec(float(v))
        ref = math.exp(float(v))
        ulp = math.ldexp(1.0, math.frexp(ref)[1] - 24)
        worst = max(worst, abs(got - ref) / ulp)
    assert worst <= 4.0, worst
    # clamp: anything below -80 gives EXP(-80), a normal number
    assert O.exp_spec(-1000.0) == O.exp_spec(-80.0) > 2.0 ** -126


# ---- top-k ------------------------------------------------------------------------------

def _ref_topk(l, k):
    # full stable sort on (-logit): equal logits keep ascending expert id
    order = np.argsort(-l, axis=1, kind="stable")
    return order[:, :k].astype(np.int32)


@pytest.mark.parametrize("T,E,k", [(16, 8, 2), (33, 256, 8), (7, 256, 6), (5, 64, 1), (3, 40, 40)])
def test_topk_matches_full_sort(T, E, k):
    l = inputs.make_logits(T, E, seed=3)
    ids, w, off = O.route(l, k)
    assert np.array_equal(ids, _ref_topk(l, k))
    sel = np.take_along_axis(l, ids, axis=1)
    assert np.all(sel[:, :-1] >= sel[:, 1:])
    assert all(len(set(r)) == k for r in ids.tolist())


def test_topk_ties_take_lower_expert_id():
    E, k = 32, 8
    l = np.zeros((4, E), np.float32)
    l[1, :] = 1.5                      # all equal -> ids 0..k-1
    l[2, ::2] = 0.0
    l[2, 1::2] = -0.0                  # +0 and -0 compare equal -> still 0..k-1
    l[3, [5, 9, 17]] = 2.0             # duplicated maxima then the zeros
    ids, w, _ = O.route(l, k)
    assert ids[0].tolist() == list(range(k))
    assert ids[1].tolist() == list(range(k))
    assert ids[2].tolist() == list(range(k))
    assert ids[3].tolist() == [5, 9, 17, 0, 1, 2, 3, 4]
    # quantised logits with many ties, against the full sort
    rng = np.random.default_rng(5)
    q = rng.integers(-3, 4, size=(64, 256)).astype(np.float32) * 0.25
    ids, _, _ = O.route(q, 8)
    assert np.array_equal(ids, _ref_topk(q, 8))


def test_weights_are_softmax_over_selected():
    l = inputs.make_logits(200, 256, seed=7)
    k = 8
    ids, w, _ = O.route(l, k)
    assert np.all(np.abs(w.astype(np.float64).sum(axis=1) - 1.0) <= k * 2.0 ** -23)
    assert np.all(w[:, :-1] >= w[:, 1:])
    sel = np.take_along_axis(l, ids, axis=1).astype(np.float64)
    ref = np.exp(sel - sel[:, :1])
    ref /= ref.sum(axis=1, keepdims=True)
    assert np.max(np.abs(w - ref) / ref) < 2e-6
    ids1, w1, _ = O.route(l, 1)
    assert np.all(w1 == np.float32(1.0))


def test_weights_bitwise_from_the_written_recipe():
    # re-derive the weights from exp_spec with numpy float32 scalar arithmetic
    l = inputs.make_logits(50, 64, seed=11)
    ids, w, _ = O.route(l, 6)
    for t in range(50):
        sel = l[t, ids[t]]
        ex = [np.float32(O.exp_spec(float(np.float32(v) - np.float32(sel[0])))) for v in sel]
        s = ex[0]
        for e in ex[1:]:
            s = np.float32(s + e)
        for j in range(6):
            assert np.float32(ex[j] / s) == w[t, j]


# ---- offsets and permutation -----------------------------------------------------------------

def test_offsets_and_perm_match_stable_argsort():
    for (T, E, k, seed) in [(16, 8, 2, 0), (257, 256, 8, 1), (64, 256, 8, 2), (100, 16, 4, 3)]:
        l = inputs.make_logits(T, E, seed=seed)
        x = inputs.make_x(T, 64, seed=seed)
        ids, w, off = O.route(l, k)
        cnt = np.bincount(ids.ravel(), minlength=E)
        assert off[0] == 0 and off[E] == T * k
        assert np.array_equal(np.diff(off), cnt)
        x_perm, perm, inv = O.permute(x, ids, off)
        ref = np.argsort(ids.ravel(), kind="stable").astype(np.int32)
        assert np.array_equal(perm, ref)
        assert np.array_equal(inv[perm], np.arange(T * k))
        assert np.array_equal(perm[inv], np.arange(T * k))
        assert np.array_equal(x_perm, x[perm // k])
        # unpermute round trip: every token's row comes back k times
        assert np.array_equal(x_perm[inv].reshape(T, k, -1), np.repeat(x[:, None, :], k, axis=1))
        e_of = ids.ravel()[perm]
        assert np.all(np.diff(e_of) >= 0)
        for e in range(E):
            seg = perm[off[e]:off[e + 1]]
            assert np.all(np.diff(seg) > 0)


def test_printed_block_permutation_and_inverse(golden_dir):
    fwd, inv = load_numbers(os.path.join(golden_dir, "w2_block_permutation.txt"))
    # eight slots alternating between two experts sort into exactly the printed order
    T, E, k = 8, 2, 1
    l = np.zeros((T, E), np.float32)
    for t in range(T):
        l[t, t % 2] = 1.0
    ids, w, off = O.route(l, k)
    assert ids.ravel().tolist() == [0, 1, 0, 1, 0, 1, 0, 1]
    x = inputs.make_x(T, 32, seed=0)
    _, perm, inv_perm = O.permute(x, ids, off)
    assert perm.tolist() == fwd
    assert inv_perm.tolist() == inv
    assert off.tolist() == [0, 4, 8]


def test_printed_rows_per_expert(golden_dir):
    T, k, E, want = load_numbers(os.path.join(golden_dir, "sorter_rows_per_expert.txt"))[0]
    l = np.full((T, E), -1.0, np.float32)
    for t in range(T):
        for j in range(k):
            l[t, (t * k + j) % E] = float(k - j)  # round-robin, slot order fixed by the value
    ids, w, off = O.route(l, k)
    assert np.array_equal(ids, (np.arange(T * k).reshape(T, k) % E))
    assert np.all(np.diff(off) == want)

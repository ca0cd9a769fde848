"""Pins of the oracle's steps either side of the routed path: router projection, shared expert, join
(paper, figure "Execution structure": router scores -> Top-k -> routed experts beside the shared expert -> add
partials).  Each is checked against something other than itself: float64 matrix products with a table typed from the
paper's printed magnitudes, exact integer and exact rational arithmetic, and special cases that collapse the block to a
function already pinned.  No GPU."""
import os
from fractions import Fraction

import numpy as np

from _exact import fma_f32, load_numbers, round_fraction_to_f32
from oracle import moe_oracle as O
from paper_2609_15627_b200 import inputs

bf = inputs.bf16_bits_to_f32


def _table(golden_dir):
    doubled = load_numbers(os.path.join(golden_dir, "e2m1_doubled_magnitudes.txt"))[0]
    mags = np.array(doubled, np.float64) / 2.0
    return np.concatenate([mags, -mags])


def _dequant_np(codes, scales, table):
    lo, hi = codes & 0xF, codes >> 4
    c = np.stack([lo, hi], axis=-1).reshape(*codes.shape[:-1], codes.shape[-1] * 2)
    return table[c] * np.repeat(np.ldexp(1.0, scales.astype(np.int64) - 127), 32, axis=-1)


def test_router_logits_against_float64_and_exact_integers():
    T, H, E = 7, 512, 24                        # T != E: a transposed operand cannot pass
    x, wr = inputs.make_x(T, H, 1), inputs.make_x(E, H, 2)
    lg = O.router_logits(x, wr)
    ref = bf(x).astype(np.float64) @ bf(wr).astype(np.float64).T
    assert lg.shape == (T, E) and lg.dtype == np.float32
    # fp32 running sum of exact products: error below H * 2^-24 * sum |terms|
    bound = H * 2.0 ** -24 * (np.abs(bf(x).astype(np.float64)) @ np.abs(bf(wr).astype(np.float64)).T)
    assert np.all(np.abs(lg - ref) <= bound)
    assert np.abs(lg - ref).max() < 2e-5 * np.sqrt(H)
    # small integers: every partial sum is an integer below 2^24, so the result is exact
    rng = np.random.default_rng(0)
    xi = rng.integers(-8, 9, (T, H)).astype(np.float32)
    wi = rng.integers(-8, 9, (E, H)).astype(np.float32)
    lg = O.router_logits(inputs.f32_to_bf16_bits(xi), inputs.f32_to_bf16_bits(wi))
    assert np.array_equal(lg.astype(np.int64), xi.astype(np.int64) @ wi.astype(np.int64).T)


def test_router_logits_accumulate_in_fp32_in_ascending_h():
    # 2^24 + 1 rounds back to 2^24 in fp32, so ascending order gives 0 where descending order gives 1 and a wider
    # accumulator gives 1 as well
    H = 32
    x = np.ones((1, H), np.float32)
    w = np.zeros((1, H), np.float32)
    w[0, 0], w[0, 1], w[0, 2] = 2.0 ** 24, 1.0, -(2.0 ** 24)
    assert O.router_logits(inputs.f32_to_bf16_bits(x), inputs.f32_to_bf16_bits(w))[0, 0] == 0.0
    w[0, :3] = w[0, 2::-1].copy()
    assert O.router_logits(inputs.f32_to_bf16_bits(x), inputs.f32_to_bf16_bits(w))[0, 0] == 1.0


def test_join_is_the_slot_recurrence_plus_one_addition_in_exact_arithmetic():
    rng = np.random.default_rng(3)
    T, H, k = 5, 8, 3
    y = (rng.standard_normal((T * k, H)) * 20).astype(np.float32)
    ys = (rng.standard_normal((T, H)) * 20).astype(np.float32)
    w = rng.random((T, k)).astype(np.float32)
    inv = rng.permutation(T * k).astype(np.int32)
    out, out_f32 = O.combine_shared(y, inv, w, ys)
    for t in range(T):
        for n in range(H):
            acc = np.float32(0.0)
            for j in range(k):
                acc = fma_f32(w[t, j], y[inv[t * k + j], n], acc)
            acc = round_fraction_to_f32(Fraction(float(acc)) + Fraction(float(ys[t, n])))
            assert out_f32[t, n] == acc
    assert np.array_equal(out, inputs.f32_to_bf16_bits(out_f32))
    # shared rows of zero: exactly the routed combine
    o2, f2 = O.combine_shared(y, inv, w, np.zeros_like(ys))
    o1, f1 = O.combine(y, inv, w)
    assert np.array_equal(o2, o1) and np.array_equal(f2, f1)


def test_shared_expert_is_a_dense_swiglu_mlp_on_every_token(golden_dir):
    table = _table(golden_dir)
    T, H, I = 9, 256, 128
    sw13, ss13, sw2, ss2 = inputs.make_expert_weights(H, I, 1, seed=11)
    ss13[:] = inputs.index_scales(2 * I, H)
    ss2[:] = inputs.index_scales(H, I, lo=117)
    x = inputs.make_x(T, H, seed=11)
    ys = O.shared_expert(x, sw13, ss13, sw2, ss2)
    W13, W2 = _dequant_np(sw13[0], ss13[0], table), _dequant_np(sw2[0], ss2[0], table)
    xf = bf(x).astype(np.float64)
    g, u = xf @ W13[:I].T, xf @ W13[I:].T
    a = bf(inputs.f32_to_bf16_bits((g / (1.0 + np.exp(-g)) * u).astype(np.float32))).astype(np.float64)
    ref = a @ W2.T
    assert ys.shape == (T, H)
    assert np.linalg.norm(ys - ref) / np.linalg.norm(ref) < 2e-3      # a few one-ulp flips of the bf16 intermediate
    assert np.median(np.abs(ys - ref)) < 1e-5 * np.sqrt(np.mean(ref ** 2))


def test_block_collapses_to_its_parts(golden_dir):
    table = _table(golden_dir)
    T, H, I, E, k = 6, 256, 128, 8, 2
    w13, s13, w2, s2 = inputs.make_expert_weights(H, I, E, seed=0)
    sw13, ss13, sw2, ss2 = inputs.make_expert_weights(H, I, 1, seed=21)
    x = inputs.make_x(T, H, 5)
    wr = inputs.f32_to_bf16_bits(bf(inputs.make_x(E, H, 6)) * np.float32(0.05))
    r = O.ffn_block(x, wr, w13, s13, w2, s2, sw13, ss13, sw2, ss2, k)
    # the routed part is the layer on the router's logits
    lg = O.router_logits(x, wr)
    assert np.array_equal(r["logits"], lg)
    staged = O.forward_staged(lg, x, w13, s13, w2, s2, k)
    assert np.array_equal(r["ids"], staged["ids"]) and np.array_equal(r["routed_out"], staged["out"])
    # out = bf16(routed fp32 + shared fp32), element by element
    want = (r["routed_out_f32"].astype(np.float64) + r["y_shared"].astype(np.float64)).astype(np.float32)
    assert np.array_equal(r["out_f32"], want) and np.array_equal(r["out"], inputs.f32_to_bf16_bits(want))
    # a shared expert of zero codes leaves the routed layer; routed experts of zero codes leave the rounded shared expert
    z13, z2 = np.zeros_like(sw13), np.zeros_like(sw2)
    r0 = O.ffn_block(x, wr, w13, s13, w2, s2, z13, ss13, z2, ss2, k)
    assert np.array_equal(r0["out"], staged["out"])
    r1 = O.ffn_block(x, wr, np.zeros_like(w13), s13, np.zeros_like(w2), s2, sw13, ss13, sw2, ss2, k)
    assert np.array_equal(r1["out"], inputs.f32_to_bf16_bits(r["y_shared"]))
    # against float64 end to end (independent dequantisation, dense evaluation of the selected experts)
    xf = bf(x).astype(np.float64)
    ref = np.zeros((T, H))
    for t in range(T):
        for j in range(k):
            e = int(r["ids"][t, j])
            W13, W2 = _dequant_np(w13[e], s13[e], table), _dequant_np(w2[e], s2[e], table)
            g, u = W13[:I] @ xf[t], W13[I:] @ xf[t]
            a = bf(inputs.f32_to_bf16_bits((g / (1 + np.exp(-g)) * u).astype(np.float32))).astype(np.float64)
            ref[t] += float(r["w"][t, j]) * (W2 @ a)
        W13, W2 = _dequant_np(sw13[0], ss13[0], table), _dequant_np(sw2[0], ss2[0], table)
        g, u = W13[:I] @ xf[t], W13[I:] @ xf[t]
        a = bf(inputs.f32_to_bf16_bits((g / (1 + np.exp(-g)) * u).astype(np.float32))).astype(np.float64)
        ref[t] += W2 @ a
    assert np.linalg.norm(r["out_f32"] - ref) / np.linalg.norm(ref) < 2e-3

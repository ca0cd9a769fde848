"""Pins for the oracle's expert FFN, combine and whole-layer forms (CPU only).

Expected values come from numpy float64 linear algebra on matrices dequantised with a
table typed here from the paper's printed list, from exact rational arithmetic, and from
special cases whose answer is known in closed form.
"""
import os

import numpy as np
import pytest

from _exact import fma_f32, load_numbers
from oracle import moe_oracle as O
from paper_2609_15627_b200 import inputs

bf = inputs.bf16_bits_to_f32


def _table(golden_dir):
    doubled = load_numbers(os.path.join(golden_dir, "e2m1_doubled_magnitudes.txt"))[0]
    mags = np.array(doubled, np.float64) / 2.0
    return np.concatenate([mags, -mags])


def _dequant_np(codes, scales, table):
    """Independent dequantisation: codes [.., rows, K/2], scales [.., rows, K/32] -> float64 [.., rows, K]."""
    lo = codes & 0xF
    hi = codes >> 4
    c = np.stack([lo, hi], axis=-1).reshape(*codes.shape[:-1], codes.shape[-1] * 2)
    s = np.ldexp(1.0, scales.astype(np.int64) - 127)
    return table[c] * np.repeat(s, 32, axis=-1)


def _rel_fro(a, b):
    a = a.astype(np.float64)
    b = b.astype(np.float64)
    return np.linalg.norm(a - b) / np.linalg.norm(b)


def _bf16_ulp_distance(a_bits, b_bits):
    def key(u):
        u = u.astype(np.int32)
        return np.where(u & 0x8000, -(u & 0x7FFF), u & 0x7FFF)
    return np.abs(key(a_bits) - key(b_bits))


def test_k1_E1_is_a_dense_swiglu_mlp(golden_dir):
    table = _table(golden_dir)
    T, H, I = 12, 256, 128
    w13, s13, w2, s2 = inputs.make_expert_weights(H, I, 1, seed=4)
    s13[:] = inputs.index_scales(2 * I, H)  # non-constant, index-dependent scales
    s2[:] = inputs.index_scales(H, I, lo=117)
    x = inputs.make_x(T, H, seed=4)
    logits = np.zeros((T, 1), np.float32)
    r = O.forward_staged(logits, x, w13, s13, w2, s2, 1)
    assert np.all(r["w"] == 1.0) and np.all(r["ids"] == 0)
    W13 = _dequant_np(w13[0], s13[0], table)
    W2 = _dequant_np(w2[0], s2[0], table)
    xf = bf(x).astype(np.float64)
    g = xf @ W13[:I].T
    u = xf @ W13[I:].T
    a64 = g / (1.0 + np.exp(-g)) * u
    a_ref = inputs.f32_to_bf16_bits(a64.astype(np.float32))
    d = _bf16_ulp_distance(r["act"], a_ref)
    assert d.max() <= 1 and (d > 0).mean() < 0.01
    # stage 2 in isolation: feed the oracle's own rounded activations to the float64 matmul
    y_ref = bf(r["act"]).astype(np.float64) @ W2.T
    assert _rel_fro(r["y_perm"], y_ref) < 2e-6
    assert np.max(np.abs(r["y_perm"] - y_ref)) < 1e-5 * np.sqrt(np.mean(y_ref ** 2)) * 10
    # k = 1, weight 1.0: out is the rounded y
    assert np.array_equal(r["out"], inputs.f32_to_bf16_bits(r["y_perm"][r["inv_perm"]]))


def test_tiny_layer_against_dense_evaluation_of_every_expert(golden_dir):
    table = _table(golden_dir)
    wl = inputs.WORKLOADS["tiny"]
    d = inputs.make_workload(wl, seed=0)
    r = O.forward_staged(d["logits"], d["x"], d["w13"], d["s13"], d["w2"], d["s2"], wl.k)
    xf = bf(d["x"]).astype(np.float64)
    W13 = _dequant_np(d["w13"], d["s13"], table)  # [E,2I,H]
    W2 = _dequant_np(d["w2"], d["s2"], table)     # [E,H,I]
    g = np.einsum("th,eih->tei", xf, W13[:, :wl.I])
    u = np.einsum("th,eih->tei", xf, W13[:, wl.I:])
    a = bf(inputs.f32_to_bf16_bits((g / (1.0 + np.exp(-g)) * u).astype(np.float32))).astype(np.float64)
    y_all = np.einsum("tei,eni->ten", a, W2)      # every expert for every token
    # routing by a full sort and a float64 softmax, then mask
    order = np.argsort(-d["logits"], axis=1, kind="stable")[:, :wl.k]
    sel = np.take_along_axis(d["logits"], order, axis=1).astype(np.float64)
    p = np.exp(sel - sel[:, :1])
    p /= p.sum(axis=1, keepdims=True)
    out_ref = np.zeros((wl.T, wl.H))
    for t in range(wl.T):
        for j in range(wl.k):
            out_ref[t] += p[t, j] * y_all[t, order[t, j]]
    assert np.array_equal(r["ids"], order.astype(np.int32))
    assert _rel_fro(r["out_f32"], out_ref) < 2e-4
    rms = np.sqrt(np.mean(out_ref ** 2))
    assert np.max(np.abs(r["out_f32"] - out_ref)) < 5e-3 * rms
    assert _rel_fro(bf(r["out"]), out_ref) < 5e-3
    # per-slot rows too
    for t in range(wl.T):
        for j in range(wl.k):
            yp = r["y_perm"][r["inv_perm"][t * wl.k + j]]
            assert _rel_fro(yp, y_all[t, order[t, j]]) < 1e-3


def test_staged_equals_per_token_definition_bitwise():
    for name, seed in (("tiny", 0), ("tiny", 5)):
        wl = inputs.WORKLOADS[name]
        d = inputs.make_workload(wl, seed=seed)
        r = O.forward_staged(d["logits"], d["x"], d["w13"], d["s13"], d["w2"], d["s2"], wl.k)
        b = O.forward_tokens(d["logits"], d["x"], d["w13"], d["s13"], d["w2"], d["s2"], wl.k, np.arange(wl.T))
        assert np.array_equal(b["ids"], r["ids"]) and np.array_equal(b["w"], r["w"])
        assert np.array_equal(b["out"], r["out"])
        assert np.array_equal(b["out_f32"].view(np.uint32), r["out_f32"].view(np.uint32))
        y_unperm = r["y_perm"][r["inv_perm"]].reshape(wl.T, wl.k, wl.H)
        assert np.array_equal(b["y"], y_unperm)
        # a subset of tokens gives the same rows
        sub = np.array([3, 11, 0], np.int32)
        bs = O.forward_tokens(d["logits"], d["x"], d["w13"], d["s13"], d["w2"], d["s2"], wl.k, sub)
        assert np.array_equal(bs["out"], r["out"][sub])


def test_fp64_accumulation_twin_agrees():
    wl = inputs.WORKLOADS["tiny"]
    d = inputs.make_workload(wl, seed=2)
    a = O.forward_staged(d["logits"], d["x"], d["w13"], d["s13"], d["w2"], d["s2"], wl.k, acc64=False)
    b = O.forward_staged(d["logits"], d["x"], d["w13"], d["s13"], d["w2"], d["s2"], wl.k, acc64=True)
    assert _rel_fro(a["y_perm"], b["y_perm"]) < 1e-4
    assert (_bf16_ulp_distance(a["act"], b["act"]) > 1).sum() == 0


def test_zero_codes_give_zero_and_single_weight_gives_one_product():
    H, I, E, k, T = 64, 32, 2, 1, 3
    x = inputs.make_x(T, H, seed=9)
    logits = np.zeros((T, E), np.float32)  # all ties -> expert 0
    w13 = np.zeros((E, 2 * I, H // 2), np.uint8)
    w13[:, :, ::2] = 0x80                # a mix of code 0 (+0) and code 8 (-0)
    s13 = np.full((E, 2 * I, H // 32), 120, np.uint8)
    w2 = np.zeros((E, H, I // 2), np.uint8)
    s2 = np.full((E, H, I // 32), 121, np.uint8)
    r = O.forward_staged(logits, x, w13, s13, w2, s2, k)
    assert np.all(r["y_perm"] == 0.0) and np.all(bf(r["out"]) == 0.0)
    # one gate weight, one up weight, one down weight: every stage is a single exact product
    i0, hg, hu, n0 = 5, 7, 12, 33
    w13[0, i0, hg // 2] = 0x04 << (4 * (hg & 1))         # code 4 = 2.0 at element hg (odd -> high nibble)
    w13[0, I + i0, hu // 2] = 0x0D << (4 * (hu & 1))     # code 13 = -3.0 at element hu (even -> low nibble)
    w2[0, n0, i0 // 2] = 0x03 << (4 * (i0 & 1))          # code 3 = 1.5 at element i0
    r = O.forward_staged(logits, x, w13, s13, w2, s2, k)
    xf = bf(x)
    for t in range(T):
        g = np.float32(2.0 * 2.0 ** -7) * xf[t, hg]
        u = np.float32(-3.0 * 2.0 ** -7) * xf[t, hu]
        a = bf(inputs.f32_to_bf16_bits(np.array([np.float32(g / (np.float32(1) + np.exp(-g))) * u], np.float32)))[0]
        p = r["inv_perm"][t]
        got_a = bf(r["act"][p])
        assert np.count_nonzero(got_a) <= 1
        assert abs(got_a[i0] - a) <= abs(a) * 2.0 ** -7  # libm exp may differ in the last bit
        want_y = np.float32(1.5 * 2.0 ** -6) * got_a[i0]
        assert r["y_perm"][p, n0] == want_y
        assert np.count_nonzero(r["y_perm"][p]) <= 1


def test_w2_scale_plus_one_doubles_y_exactly():
    wl = inputs.WORKLOADS["tiny"]
    d = inputs.make_workload(wl, seed=1)
    a = O.forward_staged(d["logits"], d["x"], d["w13"], d["s13"], d["w2"], d["s2"], wl.k)
    b = O.forward_staged(d["logits"], d["x"], d["w13"], d["s13"], d["w2"], d["s2"] + 1, wl.k)
    assert np.array_equal(b["y_perm"], 2.0 * a["y_perm"])
    assert np.array_equal(b["act"], a["act"])


def test_combine_is_the_fma_recurrence_in_slot_order():
    rng = np.random.default_rng(3)
    T, H, k = 5, 8, 4
    S = T * k
    y = (rng.standard_normal((S, H)) * 20).astype(np.float32)
    inv = rng.permutation(S).astype(np.int32)
    w = rng.random((T, k)).astype(np.float32)
    out, out_f32 = O.combine(y, inv, w)
    for t in range(T):
        for n in range(H):
            acc = np.float32(0.0)
            for j in range(k):
                acc = fma_f32(w[t, j], y[inv[t * k + j], n], acc)
            assert acc == out_f32[t, n]
            assert out[t, n] == inputs.f32_to_bf16_bits(np.array([acc], np.float32))[0]
    # the order matters in floating point: the reversed recurrence differs somewhere
    rev = np.zeros((T, H), np.float32)
    for t in range(T):
        for n in range(H):
            acc = np.float32(0.0)
            for j in reversed(range(k)):
                acc = fma_f32(w[t, j], y[inv[t * k + j], n], acc)
            rev[t, n] = acc
    assert not np.array_equal(rev, out_f32)


def test_relabelling_experts_leaves_the_output_unchanged():
    wl = inputs.WORKLOADS["tiny"]
    d = inputs.make_workload(wl, seed=6)
    a = O.forward_staged(d["logits"], d["x"], d["w13"], d["s13"], d["w2"], d["s2"], wl.k)
    pi = np.random.default_rng(0).permutation(wl.E)  # new id of expert e is pi[e]
    inv = np.argsort(pi)
    logits2 = np.ascontiguousarray(d["logits"][:, inv])
    args2 = [np.ascontiguousarray(d[n][inv]) for n in ("w13", "s13", "w2", "s2")]
    b = O.forward_staged(logits2, d["x"], *args2, wl.k)
    assert np.array_equal(pi[a["ids"]], b["ids"])
    assert np.array_equal(a["out"], b["out"])
    assert np.array_equal(a["out_f32"], b["out_f32"])


def test_generator_statistics_closed_form(golden_dir):
    # Var(weight) = E[v^2] * E[4^e] = 8.5625 * 3.2437e-4 for uniform codes and exponents -8..-5
    table = _table(golden_dir)
    w13, s13, w2, s2 = inputs.make_expert_weights(1024, 512, 2, seed=0)
    W = _dequant_np(w13, s13, table)
    want = (np.mean(table ** 2)) * np.mean(4.0 ** np.arange(-8, -4))
    assert abs(W.var() / want - 1.0) < 0.02 and abs(W.mean()) < 1e-4
    assert set(np.unique(s13)) == {119, 120, 121, 122}
    assert np.array_equal(O.dequant(w13[1], s13[1]).astype(np.float64), W[1])
    x = bf(inputs.make_x(64, 1024, seed=0))
    assert abs(x.std() - 1.0) < 0.02
    # std(g) = sqrt(H * Var(weight)) for unit-variance activations
    g = x.astype(np.float64) @ W[0, :64].T
    assert abs(g.std() / np.sqrt(1024 * want) - 1.0) < 0.1


def test_workload_generator_is_reproducible_and_subsettable():
    a = inputs.make_expert_weights(256, 128, 8, seed=0)
    b = inputs.make_expert_weights(256, 128, 8, seed=0, experts=[2, 5])
    for full, part in zip(a, b):
        assert np.array_equal(full[2], part[2]) and np.array_equal(full[5], part[5])
    l0 = inputs.make_logits(4, 256, seed=0)
    l1 = inputs.make_logits(4, 256, seed=1)
    assert not np.array_equal(l0, l1) and np.array_equal(l0, inputs.make_logits(4, 256, seed=0))
    bias = inputs.zipf_bias(256)
    r = np.arange(1, 257) ** -1.1
    assert np.allclose(np.sort(bias)[::-1], 2 * np.log(r / r.sum()), rtol=1e-6)
    ls = inputs.make_logits(4, 256, seed=0, skew=True)
    assert np.allclose(ls - l0, bias[None, :], atol=1e-5)

"""Helpers for the GPU parity tests: numpy <-> torch marshalling and the parity metrics."""
import numpy as np
import torch

from paper_2609_15627_b200 import inputs, moe


def dev(a):
    """numpy -> cuda tensor; uint16 arrays are bf16 bit patterns."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def bits(t):
    """cuda bf16 tensor -> numpy uint16 bit patterns."""
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def weights_dev(d):
    return tuple(dev(d[n]) for n in ("w13", "s13", "w2", "s2"))


def run_layer(wl, d, wdev=None):
    sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
    buf = moe.LayerBuffers(sh)
    wdev = wdev if wdev is not None else weights_dev(d)
    out = moe.moe_layer(dev(d["logits"]), dev(d["x"]), wdev, buf)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    return buf, out


def bf16_neighbours(f32):
    """The two bf16 values that bracket each (finite) fp32 value: the truncation towards zero and the next bf16
    value away from zero, one unit in the last place of the TRUNCATED value's binade further (bf16 bit patterns of
    one sign are ordered like their magnitudes, so that neighbour is the bit pattern plus one).  Returned as
    float64 arrays; a value that is itself a bf16 number gets (itself, the next one away from zero)."""
    f = np.ascontiguousarray(f32, dtype=np.float32)
    lo_bits = (f.view(np.uint32) >> np.uint32(16)).astype(np.uint16)
    hi_bits = (lo_bits + np.uint16(1)).astype(np.uint16)
    return (inputs.bf16_bits_to_f32(lo_bits).astype(np.float64), inputs.bf16_bits_to_f32(hi_bits).astype(np.float64))


def check_out(got_bits, ref_bits, ref_f32, what=""):
    """The stated tolerance: rel-Frobenius <= 5e-3 and max|diff| <= 2e-2 * rms(reference).

    An element over the max bound is accepted only if the GPU value is one of the two bf16
    neighbours of the oracle's unrounded fp32 result (a rounding flip of one bf16 ulp).
    """
    got = inputs.bf16_bits_to_f32(got_bits).astype(np.float64)
    ref = inputs.bf16_bits_to_f32(ref_bits).astype(np.float64)
    rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
    rms = np.sqrt(np.mean(ref ** 2))
    diff = np.abs(got - ref)
    over = diff > 2e-2 * rms
    flips = 0
    if over.any():
        lo, hi = bf16_neighbours(ref_f32[over])
        g = got[over]
        ok = (g == lo) | (g == hi)
        assert ok.all(), "%s: %d elements beyond 2e-2*rms that are not bf16 rounding flips (max %g, rms %g)" % (
            what, int((~ok).sum()), diff.max(), rms)
        flips = int(over.sum())
    assert rel <= 5e-3, "%s: rel-Frobenius %g" % (what, rel)
    return dict(rel=rel, max_over_rms=float(diff.max() / rms), flips=flips)


def check_y(got, ref, what=""):
    got = got.astype(np.float64)
    ref = ref.astype(np.float64)
    rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
    rms = np.sqrt(np.mean(ref ** 2))
    mx = np.abs(got - ref).max() / max(rms, 1e-30)
    assert rel <= 5e-4 and mx <= 2e-2, "%s: y_perm rel %g max/rms %g" % (what, rel, mx)
    return dict(rel=rel, max_over_rms=float(mx))


def assert_same_up_to_rounding(got_bits, want_bits, what=""):
    """Two bf16 results of the same arithmetic up to the summation order inside fp32 dot products: the fp32 values
    differ in their last bits (by about 1e-6 of the terms they sum), so the bf16 roundings agree except where a value
    sits on a rounding boundary - there by one bf16 unit in the last place - or where the terms cancel to a value far
    below their size, whose own units are smaller than that fp32 difference (allowed: 1e-3 of the result's rms)."""
    a = np.ascontiguousarray(got_bits, dtype=np.uint16).astype(np.int32)
    b = np.ascontiguousarray(want_bits, dtype=np.uint16).astype(np.int32)
    # order-preserving integer of a bf16 bit pattern: distance 1 = neighbouring values (also across zero)
    ka = np.where(a & 0x8000, -(a & 0x7FFF), a & 0x7FFF)
    kb = np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)
    d = np.abs(ka - kb)
    fa = inputs.bf16_bits_to_f32(got_bits).astype(np.float64)
    fb = inputs.bf16_bits_to_f32(want_bits).astype(np.float64)
    rms = np.sqrt(np.mean(fb ** 2))
    bad = (d > 1) & (np.abs(fa - fb) > 1e-3 * rms)
    assert not bad.any(), "%s: %d values more than one bf16 unit and 1e-3 rms apart (worst %g, rms %g)" % (
        what, int(bad.sum()), float(np.abs(fa - fb)[bad].max()), rms)
    assert (d != 0).mean() <= 0.05, "%s: %.3f of the elements differ" % (what, float((d != 0).mean()))

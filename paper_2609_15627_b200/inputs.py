"""Seeded synthetic inputs for the routed FP4 mixture-of-experts layer.

This module only draws inputs.  It holds none of the layer's arithmetic and is
the one module that both the CPU oracle's tests and the CUDA library's tests
and benchmark use, so that both sides see byte-identical buffers.  numpy only.

The inputs stand in for the model checkpoint and the request corpus of the
paper's evaluation (neither is available): shapes and distributions are those
of the five benchmark workloads.

  x       bf16 bit patterns (uint16) [T,H], N(0,1) rounded to nearest-even
  logits  float32 [T,E], N(0,1); the skewed workload adds a per-expert bias
          2*ln(zipf_weight(rank)), zipf exponent 1.1, ranks assigned to expert
          ids by a seeded permutation
  codes   uint8, two E2M1 codes per byte, every code 0..15 equally likely
  scales  uint8 E8M0 bytes, uniform over {119,120,121,122} (2^-8 .. 2^-5)

Every expert's weights come from their own generator keyed by (seed, tensor,
expert), so any subset of experts can be produced without the others.
"""
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    T: int
    H: int
    I: int
    E: int
    k: int
    skew: bool = False

    @property
    def S(self):
        return self.T * self.k


WORKLOADS = {
    "tiny": Workload("tiny", 16, 256, 128, 8, 2),
    "decode_c1": Workload("decode_c1", 1, 4096, 2048, 256, 8),
    "decode_c64": Workload("decode_c64", 64, 4096, 2048, 256, 8),
    "prefill_8k": Workload("prefill_8k", 8192, 4096, 2048, 256, 8),
    "prefill_32k_skewed": Workload("prefill_32k_skewed", 32768, 4096, 2048, 256, 8, skew=True),
}

_TENSOR_X, _TENSOR_LOGITS, _TENSOR_W13, _TENSOR_S13, _TENSOR_W2, _TENSOR_S2, _TENSOR_ZIPF = range(7)


def _rng(seed, tensor, index=0):
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([int(seed), int(tensor), int(index)])))


def f32_to_bf16_bits(a):
    """float32 array -> bf16 bit patterns (uint16), round to nearest even (finite inputs)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    return ((u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(a):
    return (np.ascontiguousarray(a, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def make_x(T, H, seed=0):
    return f32_to_bf16_bits(_rng(seed, _TENSOR_X).standard_normal((T, H), dtype=np.float32))


def zipf_bias(E, seed=0, s=1.1):
    """Per-expert logit bias 2*ln(r^-s / sum_r r^-s); rank r of expert e from a seeded permutation."""
    r = np.arange(1, E + 1, dtype=np.float64)
    wts = r ** (-s)
    wts /= wts.sum()
    rank_of_expert = _rng(seed, _TENSOR_ZIPF).permutation(E)
    return (2.0 * np.log(wts[rank_of_expert])).astype(np.float32)


def make_logits(T, E, seed=0, skew=False):
    l = _rng(seed, _TENSOR_LOGITS).standard_normal((T, E), dtype=np.float32)
    if skew:
        # the bias belongs to the model (its router), not to the batch: it keeps seed 0
        l = l + zipf_bias(E, 0)[None, :]
    return np.ascontiguousarray(l, dtype=np.float32)


def _expert_codes(seed, tensor, e, rows, K):
    return _rng(seed, tensor, e).integers(0, 256, size=(rows, K // 2), dtype=np.uint8)


def _expert_scales(seed, tensor, e, rows, K, lo=119, hi=122):
    return _rng(seed, tensor, e).integers(lo, hi + 1, size=(rows, K // 32), dtype=np.uint8)


def make_expert_weights(H, I, E, seed=0, experts=None, threads=8):
    """(w13 [E,2I,H/2], s13 [E,2I,H/32], w2 [E,H,I/2], s2 [E,H,I/32]) as uint8.

    With `experts` (an iterable of ids) only those experts are filled; the rest stay zero
    codes with scale byte 127, which lets a CPU-side check touch a few experts cheaply.
    """
    w13 = np.zeros((E, 2 * I, H // 2), np.uint8)
    s13 = np.full((E, 2 * I, H // 32), 127, np.uint8)
    w2 = np.zeros((E, H, I // 2), np.uint8)
    s2 = np.full((E, H, I // 32), 127, np.uint8)
    todo = list(range(E)) if experts is None else sorted(set(int(e) for e in experts))

    def fill(e):
        w13[e] = _expert_codes(seed, _TENSOR_W13, e, 2 * I, H)
        s13[e] = _expert_scales(seed, _TENSOR_S13, e, 2 * I, H)
        w2[e] = _expert_codes(seed, _TENSOR_W2, e, H, I)
        s2[e] = _expert_scales(seed, _TENSOR_S2, e, H, I)

    if len(todo) > 4 and threads > 1:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(fill, todo))
    else:
        for e in todo:
            fill(e)
    return w13, s13, w2, s2


def make_workload(wl, seed=0, experts=None):
    """All inputs of one workload: dict(logits, x, w13, s13, w2, s2)."""
    if isinstance(wl, str):
        wl = WORKLOADS[wl]
    w13, s13, w2, s2 = make_expert_weights(wl.H, wl.I, wl.E, seed=0, experts=experts)
    return dict(logits=make_logits(wl.T, wl.E, seed, wl.skew), x=make_x(wl.T, wl.H, seed),
                w13=w13, s13=s13, w2=w2, s2=s2)


# ---- structured fixtures (still inputs only) ---------------------------------

def index_scales(rows, K, E=1, lo=116, span=8):
    """Non-constant scale bytes: each (expert, row, k-block) byte is a distinct function of its
    indices modulo `span`, so a scale read from the wrong row or block changes the result."""
    e = np.arange(E)[:, None, None]
    r = np.arange(rows)[None, :, None]
    b = np.arange(K // 32)[None, None, :]
    return (lo + (3 * e + 5 * r + 7 * b) % span).astype(np.uint8)


def fingerprint_codes(rows, K, E=1, seed=0):
    """Codes in which every row carries its own signature: one seeded random code sequence per expert,
    shared by all its rows, shifted per row by (7*r + 3*(r // 16)) mod 16.  The 16 rows of a tile all
    differ and neighbouring tiles differ, so a kernel that swaps rows or row tiles gives a wrong output."""
    base = _rng(seed, 99).integers(0, 16, size=(E, 1, K), dtype=np.int64)
    r = np.arange(rows, dtype=np.int64)[None, :, None]
    c = ((base + 7 * r + 3 * (r // 16)) % 16).astype(np.uint8)
    return (c[..., 0::2] | (c[..., 1::2] << 4)).astype(np.uint8)

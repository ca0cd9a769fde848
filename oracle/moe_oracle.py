"""numpy front end of the CPU oracle (oracle/moe_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's cpu_baseline / reference legs.  It loads oracle/liboracle_moe.so
(plain C++, built by oracle/build_oracle.py) through ctypes and marshals numpy
arrays; it imports nothing from the CUDA package and the CUDA package imports
nothing from here.

Array conventions (all C-contiguous numpy arrays):
  logits float32 [T,E]; x, x_perm, act, out uint16 (bf16 bit patterns);
  w13 uint8 [E,2I,H/2], s13 uint8 [E,2I,H/32], w2 uint8 [E,H,I/2], s2 uint8 [E,H,I/32];
  ids, perm, inv_perm, offsets int32; topk weights, y_perm float32.
"""
import ctypes as C

import numpy as np

from . import build_oracle

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build_oracle.build())
        L.oracle_e2m1_value.restype = C.c_float
        L.oracle_e2m1_value.argtypes = [C.c_int]
        L.oracle_e8m0_value.restype = C.c_float
        L.oracle_e8m0_value.argtypes = [C.c_int]
        L.oracle_exp_spec.restype = C.c_float
        L.oracle_exp_spec.argtypes = [C.c_float]
        L.oracle_f32_to_bf16.restype = C.c_uint16
        L.oracle_f32_to_bf16.argtypes = [C.c_float]
        L.oracle_bf16_to_f32.restype = C.c_float
        L.oracle_bf16_to_f32.argtypes = [C.c_uint16]
        L.oracle_num_threads.restype = C.c_int
        L.oracle_set_num_threads.argtypes = [C.c_int]
        _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _chk(a, dtype, shape=None):
    assert a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    if shape is not None:
        assert tuple(a.shape) == tuple(shape), (a.shape, shape)
    return a


def num_threads():
    return int(lib().oracle_num_threads())


def set_num_threads(n):
    lib().oracle_set_num_threads(int(n))


def e2m1_value(code):
    return float(lib().oracle_e2m1_value(int(code)))


def e8m0_value(byte):
    return float(lib().oracle_e8m0_value(int(byte)))


def exp_spec(d):
    return float(lib().oracle_exp_spec(C.c_float(float(d))))


def f32_to_bf16(f):
    return int(lib().oracle_f32_to_bf16(C.c_float(float(f))))


def bf16_to_f32(h):
    return float(lib().oracle_bf16_to_f32(int(h)))


def bf16_bits_to_f32(a):
    """uint16 bf16 bit patterns -> float32 array (exact)."""
    return (a.astype(np.uint32) << 16).view(np.float32)


def dequant(codes, scales):
    """[rows, K/2] codes + [rows, K/32] scale bytes -> float32 [rows, K]."""
    rows, kb = codes.shape
    K = kb * 2
    _chk(codes, np.uint8)
    _chk(scales, np.uint8, (rows, K // 32))
    out = np.empty((rows, K), np.float32)
    lib().oracle_dequant(_p(codes), _p(scales), C.c_int64(rows), C.c_int64(K), _p(out))
    return out


def route(logits, k):
    T, E = logits.shape
    _chk(logits, np.float32)
    ids = np.empty((T, k), np.int32)
    w = np.empty((T, k), np.float32)
    offsets = np.empty(E + 1, np.int32)
    lib().oracle_route(_p(logits), T, E, k, _p(ids), _p(w), _p(offsets))
    return ids, w, offsets


def permute(x, ids, offsets):
    T, H = x.shape
    k = ids.shape[1]
    E = offsets.shape[0] - 1
    _chk(x, np.uint16)
    _chk(ids, np.int32, (T, k))
    _chk(offsets, np.int32)
    x_perm = np.empty((T * k, H), np.uint16)
    perm = np.empty(T * k, np.int32)
    inv_perm = np.empty(T * k, np.int32)
    lib().oracle_permute(_p(x), _p(ids), _p(offsets), T, H, E, k, _p(x_perm), _p(perm), _p(inv_perm))
    return x_perm, perm, inv_perm


def expert_ffn(x_perm, offsets, w13, s13, w2, s2, k, acc64=False, want_act=False):
    S, H = x_perm.shape
    E, twoI, _ = w13.shape
    I = twoI // 2
    T = S // k
    _chk(x_perm, np.uint16)
    _chk(offsets, np.int32, (E + 1,))
    _chk(w13, np.uint8, (E, 2 * I, H // 2))
    _chk(s13, np.uint8, (E, 2 * I, H // 32))
    _chk(w2, np.uint8, (E, H, I // 2))
    _chk(s2, np.uint8, (E, H, I // 32))
    y = np.empty((S, H), np.float32)
    act = np.empty((S, I), np.uint16) if want_act else None
    lib().oracle_expert_ffn(_p(x_perm), _p(offsets), _p(w13), _p(s13), _p(w2), _p(s2), T, H, I, E, k,
                            int(bool(acc64)), _p(act), _p(y))
    return (y, act) if want_act else y


def expert_ffn_q(x_perm, offsets, w13, s13, w2, s2, k, acc64=False, want_act=False):
    """The quantised-activation variant of expert_ffn: both contractions consume E2M1 codes with one E8M0 scale per
    32 elements (quant_act) instead of bf16 values; `act` is the bf16 intermediate before its quantisation."""
    S, H = x_perm.shape
    E, twoI, _ = w13.shape
    I = twoI // 2
    T = S // k
    _chk(x_perm, np.uint16)
    _chk(offsets, np.int32, (E + 1,))
    _chk(w13, np.uint8, (E, 2 * I, H // 2))
    _chk(s13, np.uint8, (E, 2 * I, H // 32))
    _chk(w2, np.uint8, (E, H, I // 2))
    _chk(s2, np.uint8, (E, H, I // 32))
    y = np.empty((S, H), np.float32)
    act = np.empty((S, I), np.uint16) if want_act else None
    lib().oracle_expert_ffn_q(_p(x_perm), _p(offsets), _p(w13), _p(s13), _p(w2), _p(s2), T, H, I, E, k,
                              int(bool(acc64)), _p(act), _p(y))
    return (y, act) if want_act else y


def quant_act(v):
    """Rows of bf16 bit patterns [rows, K] -> (packed E2M1 codes [rows, K/2], scale bytes [rows, K/32], decoded
    values [rows, K] float32): the online activation quantisation of the variant, one scale per 32 elements."""
    rows, K = v.shape
    assert K % 32 == 0
    _chk(v, np.uint16)
    packed = np.empty((rows, K // 2), np.uint8)
    scales = np.empty((rows, K // 32), np.uint8)
    deq = np.empty((rows, K), np.float32)
    lib().oracle_quant_act(_p(v), C.c_int64(rows), C.c_int64(K), _p(packed), _p(scales), _p(deq))
    return packed, scales, deq


def combine(y_perm, inv_perm, w):
    S, H = y_perm.shape
    T, k = w.shape
    _chk(y_perm, np.float32)
    _chk(inv_perm, np.int32, (S,))
    _chk(w, np.float32)
    out = np.empty((T, H), np.uint16)
    out_f32 = np.empty((T, H), np.float32)
    lib().oracle_combine(_p(y_perm), _p(inv_perm), _p(w), T, H, k, _p(out), _p(out_f32))
    return out, out_f32


def forward_staged(logits, x, w13, s13, w2, s2, k, acc64=False):
    """route -> permute -> expert_ffn -> combine; returns a dict of every intermediate."""
    ids, w, offsets = route(logits, k)
    x_perm, perm, inv_perm = permute(x, ids, offsets)
    y, act = expert_ffn(x_perm, offsets, w13, s13, w2, s2, k, acc64=acc64, want_act=True)
    out, out_f32 = combine(y, inv_perm, w)
    return dict(ids=ids, w=w, offsets=offsets, x_perm=x_perm, perm=perm, inv_perm=inv_perm, act=act, y_perm=y,
                out=out, out_f32=out_f32)


def forward_tokens(logits, x, w13, s13, w2, s2, k, tokens, acc64=False):
    """The per-token definition on the listed tokens (no permutation involved)."""
    T, E = logits.shape
    H = x.shape[1]
    I = w13.shape[1] // 2
    _chk(logits, np.float32)
    _chk(x, np.uint16, (T, H))
    _chk(w13, np.uint8, (E, 2 * I, H // 2))
    _chk(s13, np.uint8, (E, 2 * I, H // 32))
    _chk(w2, np.uint8, (E, H, I // 2))
    _chk(s2, np.uint8, (E, H, I // 32))
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    n = tokens.shape[0]
    ids = np.empty((n, k), np.int32)
    w = np.empty((n, k), np.float32)
    act = np.empty((n, k, I), np.uint16)
    y = np.empty((n, k, H), np.float32)
    out = np.empty((n, H), np.uint16)
    out_f32 = np.empty((n, H), np.float32)
    lib().oracle_forward_tokens(_p(logits), _p(x), _p(w13), _p(s13), _p(w2), _p(s2), T, H, I, E, k,
                                int(bool(acc64)), _p(tokens), n, _p(ids), _p(w), _p(act), _p(y), _p(out), _p(out_f32))
    return dict(ids=ids, w=w, act=act, y=y, out=out, out_f32=out_f32)


# ---- the steps either side of the routed path: router projection, shared expert, join ----------------------

def router_logits(x, w_router):
    """logits[T,E] float32 = x[T,H] (bf16 bits) times w_router[E,H] (bf16 bits) transposed, fp32 accumulation, h ascending."""
    T, H = x.shape
    E = w_router.shape[0]
    _chk(x, np.uint16)
    _chk(w_router, np.uint16, (E, H))
    logits = np.empty((T, E), np.float32)
    lib().oracle_router_logits(_p(x), _p(w_router), T, H, E, _p(logits))
    return logits


def combine_shared(y_perm, inv_perm, w, y_shared):
    S, H = y_perm.shape
    T, k = w.shape
    _chk(y_perm, np.float32)
    _chk(inv_perm, np.int32, (S,))
    _chk(w, np.float32)
    _chk(y_shared, np.float32, (T, H))
    out = np.empty((T, H), np.uint16)
    out_f32 = np.empty((T, H), np.float32)
    lib().oracle_combine_shared(_p(y_perm), _p(inv_perm), _p(w), _p(y_shared), T, H, k, _p(out), _p(out_f32))
    return out, out_f32


def shared_expert(x, sw13, ss13, sw2, ss2):
    """The shared expert on every token: one expert in the routed experts' weight format (tensors with E = 1), weight 1."""
    T = x.shape[0]
    return expert_ffn(x, np.array([0, T], np.int32), sw13, ss13, sw2, ss2, 1)


def ffn_block(x, w_router, w13, s13, w2, s2, sw13, ss13, sw2, ss2, k, logits=None):
    """Router projection -> Top-k -> routed experts, beside the shared expert -> join.  `logits`: use these instead of
    the oracle's own router projection (to compare the steps after it on logits computed elsewhere)."""
    lg = router_logits(x, w_router) if logits is None else logits
    r = forward_staged(lg, x, w13, s13, w2, s2, k)
    y_shared = shared_expert(x, sw13, ss13, sw2, ss2)
    out, out_f32 = combine_shared(r["y_perm"], r["inv_perm"], r["w"], y_shared)
    r.update(logits=lg, y_shared=y_shared, routed_out=r["out"], routed_out_f32=r["out_f32"], out=out, out_f32=out_f32)
    return r

"""Thin binding over the C-ABI CUDA library (include/moe_b200.h): argument marshalling only.

Every function has the name and meaning of the C entry point it calls; every step of the layer runs
in the library's CUDA kernels.  torch is used for device memory and streams.  There is no CPU path:
if libmoe_b200.so is missing or a call fails, a MoeError is raised.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmoe_b200.so")

EXPORTS = ("moe_workspace_bytes", "moe_status_string", "moe_last_kernel_name", "moe_launch_count", "moe_route",
           "moe_permute", "moe_expert_ffn", "moe_combine", "moe_validate_scales",
           "moe_forward_workspace_bytes", "moe_forward_sync_bytes", "moe_forward",
           "moe_forward_host_workspace_bytes", "moe_forward_host", "moe_expert_ffn_noalloc_max_bytes",
           "moe_expert_ffn_noalloc", "moe_debug_native_cta_share", "moe_debug_read_probe", "moe_prepack_bytes", "moe_prepack",
           "moe_expert_ffn_packed", "moe_forward_packed", "moe_forward_host_packed", "moe_debug_forward_one_launch",
           "moe_debug_expert_ffn_variant", "moe_router_logits", "moe_combine_shared", "moe_ffn_block_workspace_bytes",
           "moe_ffn_block", "moe_expert_ffn_q_workspace_bytes", "moe_expert_ffn_q",
           "moe_ep_permute", "moe_ep_row_table", "moe_ep_expert_ffn")


class MoeError(RuntimeError):
    pass


class Shape(C.Structure):
    _fields_ = [("T", C.c_int32), ("H", C.c_int32), ("I", C.c_int32), ("E", C.c_int32), ("k", C.c_int32)]


_lib = None


def lib():
    """Load the CUDA library once; raise if it was not built (python paper_2609_15627_b200/build_ext.py)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise MoeError("CUDA library not built: %s is missing (run paper_2609_15627_b200/build_ext.py)" % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
        L.moe_workspace_bytes.restype = sz
        L.moe_workspace_bytes.argtypes = [C.POINTER(Shape)]
        L.moe_forward_host_workspace_bytes.restype = sz
        L.moe_forward_host_workspace_bytes.argtypes = [C.POINTER(Shape)]
        L.moe_status_string.restype = C.c_char_p
        L.moe_status_string.argtypes = [C.c_int]
        L.moe_last_kernel_name.restype = C.c_char_p
        L.moe_launch_count.restype = C.c_uint64
        L.moe_route.restype = C.c_int
        L.moe_route.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, sz, vp]
        L.moe_permute.restype = C.c_int
        L.moe_permute.argtypes = [vp, vp, vp, C.POINTER(Shape), vp, vp, vp, vp, sz, vp]
        L.moe_expert_ffn.restype = C.c_int
        L.moe_expert_ffn.argtypes = [vp, vp, vp, vp, vp, vp, C.POINTER(Shape), vp, vp, vp, sz, vp]
        L.moe_expert_ffn_q_workspace_bytes.restype = sz
        L.moe_expert_ffn_q_workspace_bytes.argtypes = [C.POINTER(Shape)]
        L.moe_expert_ffn_q.restype = C.c_int
        L.moe_expert_ffn_q.argtypes = [vp, vp, vp, vp, vp, vp, vp, C.POINTER(Shape), vp, vp, vp, sz, vp]
        L.moe_ep_permute.restype = C.c_int
        L.moe_ep_permute.argtypes = [vp, vp, vp, C.POINTER(Shape), i32, i32, vp, vp, vp, vp, sz, vp]
        L.moe_ep_row_table.restype = C.c_int
        L.moe_ep_row_table.argtypes = [vp, vp, C.POINTER(Shape), i32, i32, vp, i32, vp, vp]
        L.moe_ep_expert_ffn.restype = C.c_int
        L.moe_ep_expert_ffn.argtypes = [vp, vp, vp, vp, vp, vp, C.POINTER(Shape), i32, i32, vp, vp, vp, sz, vp]
        L.moe_combine.restype = C.c_int
        L.moe_combine.argtypes = [vp, vp, vp, C.POINTER(Shape), vp, vp]
        L.moe_validate_scales.restype = C.c_int
        L.moe_validate_scales.argtypes = [vp, sz, vp, vp]
        L.moe_expert_ffn_noalloc_max_bytes.restype = sz
        L.moe_expert_ffn_noalloc.restype = C.c_int
        L.moe_expert_ffn_noalloc.argtypes = [vp, vp, vp, vp, vp, vp, C.POINTER(Shape), vp, vp, vp]
        L.moe_debug_native_cta_share.restype = C.c_int
        L.moe_debug_native_cta_share.argtypes = [i32, i32, i32, i32, i32, C.POINTER(C.c_int32)]
        L.moe_prepack_bytes.restype = sz
        L.moe_prepack_bytes.argtypes = [C.POINTER(Shape)]
        L.moe_prepack.restype = C.c_int
        L.moe_prepack.argtypes = [vp, vp, vp, vp, C.POINTER(Shape), vp, sz, vp]
        L.moe_expert_ffn_packed.restype = C.c_int
        L.moe_expert_ffn_packed.argtypes = [vp, vp, vp, C.POINTER(Shape), vp, vp, vp, sz, vp]
        L.moe_forward_packed.restype = C.c_int
        L.moe_forward_packed.argtypes = [vp, vp, vp, C.POINTER(Shape), vp, vp, vp, vp, vp, sz, vp]
        L.moe_forward_host_packed.restype = C.c_int
        L.moe_forward_host_packed.argtypes = [vp, vp, vp, C.POINTER(Shape), vp, vp, vp, sz, vp]
        L.moe_debug_read_probe.restype = C.c_int
        L.moe_debug_read_probe.argtypes = [vp, sz, vp, sz, vp, vp]
        L.moe_forward_workspace_bytes.restype = sz
        L.moe_forward_workspace_bytes.argtypes = [C.POINTER(Shape)]
        L.moe_forward_sync_bytes.restype = sz
        L.moe_forward_sync_bytes.argtypes = []
        L.moe_forward.restype = C.c_int
        L.moe_forward.argtypes = [vp, vp, vp, vp, vp, vp, C.POINTER(Shape), vp, vp, vp, vp, vp, sz, vp]
        L.moe_debug_forward_one_launch.restype = C.c_int
        L.moe_debug_forward_one_launch.argtypes = L.moe_forward.argtypes
        L.moe_debug_expert_ffn_variant.restype = C.c_int
        L.moe_debug_expert_ffn_variant.argtypes = [vp, vp, vp, vp, vp, vp, C.POINTER(Shape), vp, vp, vp, sz, vp, i32]
        L.moe_router_logits.restype = C.c_int
        L.moe_router_logits.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp]
        L.moe_combine_shared.restype = C.c_int
        L.moe_combine_shared.argtypes = [vp, vp, vp, vp, C.POINTER(Shape), vp, vp]
        L.moe_ffn_block_workspace_bytes.restype = sz
        L.moe_ffn_block_workspace_bytes.argtypes = [C.POINTER(Shape)]
        L.moe_ffn_block.restype = C.c_int
        L.moe_ffn_block.argtypes = [vp] * 10 + [C.POINTER(Shape), vp, vp, vp, vp, vp, sz, vp]
        L.moe_forward_host.restype = C.c_int
        L.moe_forward_host.argtypes = [vp, vp, vp, vp, vp, vp, C.POINTER(Shape), vp, vp, vp, sz, vp]
        _lib = L
    return _lib


def _check(rc, what):
    if rc != 0:
        raise MoeError("%s failed: %s (%d)" % (what, lib().moe_status_string(rc).decode(), rc))


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def shape(T, H, I, E, k):
    return Shape(int(T), int(H), int(I), int(E), int(k))


def moe_workspace_bytes(sh):
    return int(lib().moe_workspace_bytes(C.byref(sh)))


def moe_forward_host_workspace_bytes(sh):
    return int(lib().moe_forward_host_workspace_bytes(C.byref(sh)))


def moe_last_kernel_name():
    return lib().moe_last_kernel_name().decode()


def moe_launch_count():
    return int(lib().moe_launch_count())


def alloc_workspace(sh, device="cuda", host_path=False):
    n = moe_forward_host_workspace_bytes(sh) if host_path else moe_workspace_bytes(sh)
    if n == 0:
        raise MoeError("unsupported shape")
    return torch.empty(n, dtype=torch.uint8, device=device)


def moe_route(logits, k, topk_ids, topk_w, expert_offsets, ws, stream=None):
    T, E = logits.shape
    _check(lib().moe_route(_ptr(logits), T, E, k, _ptr(topk_ids), _ptr(topk_w), _ptr(expert_offsets), _ptr(ws),
                           ws.numel(), _stream(stream)), "moe_route")


def moe_permute(x, topk_ids, expert_offsets, sh, x_perm, perm, inv_perm, ws, stream=None):
    _check(lib().moe_permute(_ptr(x), _ptr(topk_ids), _ptr(expert_offsets), C.byref(sh), _ptr(x_perm), _ptr(perm),
                             _ptr(inv_perm), _ptr(ws), ws.numel(), _stream(stream)), "moe_permute")


def moe_expert_ffn(x_perm, expert_offsets, w13, w13_scale, w2, w2_scale, sh, y_perm, status_word, ws, stream=None):
    _check(lib().moe_expert_ffn(_ptr(x_perm), _ptr(expert_offsets), _ptr(w13), _ptr(w13_scale), _ptr(w2), _ptr(w2_scale),
                                C.byref(sh), _ptr(y_perm), _ptr(status_word), _ptr(ws), ws.numel(), _stream(stream)),
           "moe_expert_ffn")


VARIANT_STREAM, VARIANT_UMMA, VARIANT_NATIVE = 0, 1, 2


def moe_debug_expert_ffn_variant(x_perm, expert_offsets, w13, w13_scale, w2, w2_scale, sh, y_perm, status_word, ws, variant,
                                 stream=None):
    """moe_expert_ffn with the kernel variant named by the caller (see include/moe_b200_debug.h)."""
    _check(lib().moe_debug_expert_ffn_variant(_ptr(x_perm), _ptr(expert_offsets), _ptr(w13), _ptr(w13_scale), _ptr(w2),
                                              _ptr(w2_scale), C.byref(sh), _ptr(y_perm), _ptr(status_word), _ptr(ws),
                                              ws.numel(), _stream(stream), int(variant)), "moe_debug_expert_ffn_variant")


def moe_expert_ffn_noalloc_max_bytes():
    return int(lib().moe_expert_ffn_noalloc_max_bytes())


def moe_expert_ffn_noalloc(x_perm, expert_offsets, w13, w13_scale, w2, w2_scale, sh, y_perm, status_word, stream=None):
    """moe_expert_ffn for callers that cannot allocate: no workspace argument, the intermediate lives in a
    fixed 16 MiB array inside the library (see include/moe_b200.h for the limits and the sharing rules)."""
    _check(lib().moe_expert_ffn_noalloc(_ptr(x_perm), _ptr(expert_offsets), _ptr(w13), _ptr(w13_scale), _ptr(w2),
                                        _ptr(w2_scale), C.byref(sh), _ptr(y_perm), _ptr(status_word), _stream(stream)),
           "moe_expert_ffn_noalloc")


def moe_debug_native_cta_share(n_ctas, cta, n_touched, H, I):
    """(first, end) gate/up items and (first, end) down items of one CTA of the decode-sized expert-FFN kernel."""
    out = (C.c_int32 * 4)()
    _check(lib().moe_debug_native_cta_share(n_ctas, cta, n_touched, H, I, out), "moe_debug_native_cta_share")
    return tuple(out)


def moe_combine(y_perm, inv_perm, topk_w, sh, out, stream=None):
    _check(lib().moe_combine(_ptr(y_perm), _ptr(inv_perm), _ptr(topk_w), C.byref(sh), _ptr(out), _stream(stream)),
           "moe_combine")


def moe_validate_scales(scales, bad_count, stream=None):
    _check(lib().moe_validate_scales(_ptr(scales), scales.numel(), _ptr(bad_count), _stream(stream)),
           "moe_validate_scales")


def moe_prepack_bytes(sh):
    return int(lib().moe_prepack_bytes(C.byref(sh)))


def moe_prepack(w13, w13_scale, w2, w2_scale, sh, stream=None):
    """One-time re-layout of the expert weights; returns the packed buffer (allocation + the call)."""
    n = moe_prepack_bytes(sh)
    if n == 0:
        raise MoeError("unsupported shape")
    packed = torch.empty(n, dtype=torch.uint8, device=w13.device)
    _check(lib().moe_prepack(_ptr(w13), _ptr(w13_scale), _ptr(w2), _ptr(w2_scale), C.byref(sh), _ptr(packed), n,
                             _stream(stream)), "moe_prepack")
    return packed


def moe_expert_ffn_packed(x_perm, expert_offsets, packed, sh, y_perm, status_word, ws, stream=None):
    _check(lib().moe_expert_ffn_packed(_ptr(x_perm), _ptr(expert_offsets), _ptr(packed), C.byref(sh), _ptr(y_perm),
                                       _ptr(status_word), _ptr(ws), ws.numel(), _stream(stream)), "moe_expert_ffn_packed")


def alloc_ffn_q_workspace(sh, device="cuda"):
    n = lib().moe_expert_ffn_q_workspace_bytes(C.byref(sh))
    if n == 0:
        raise MoeError("unsupported shape")
    return torch.empty(n, dtype=torch.uint8, device=device)


def moe_expert_ffn_q(x_perm, expert_offsets, weights, sh, y_perm, status_word, ws, stream=None):
    """The quantised-activation variant; `weights` is the tuple (w13, w13_scale, w2, w2_scale) or the one tensor
    written by moe_prepack."""
    raw = tuple(weights) if isinstance(weights, (tuple, list)) else (None, None, None, None)
    packed = None if isinstance(weights, (tuple, list)) else weights
    _check(lib().moe_expert_ffn_q(_ptr(x_perm), _ptr(expert_offsets), _ptr(raw[0]), _ptr(raw[1]), _ptr(raw[2]), _ptr(raw[3]),
                                  _ptr(packed), C.byref(sh), _ptr(y_perm), _ptr(status_word), _ptr(ws), ws.numel(),
                                  _stream(stream)), "moe_expert_ffn_q")


def moe_ep_permute(x, topk_ids, expert_offsets, sh, e_begin, e_end, x_perm, perm, inv_perm, ws, stream=None):
    _check(lib().moe_ep_permute(_ptr(x), _ptr(topk_ids), _ptr(expert_offsets), C.byref(sh), e_begin, e_end, _ptr(x_perm),
                                _ptr(perm), _ptr(inv_perm), _ptr(ws), ws.numel(), _stream(stream)), "moe_ep_permute")


def moe_ep_row_table(perm, expert_offsets, sh, e_begin, e_end, owner_y, world, row_dst, stream=None):
    """owner_y: int64 device tensor of `world` addresses; row_dst: int64 device tensor [T*k] (receives addresses)."""
    _check(lib().moe_ep_row_table(_ptr(perm), _ptr(expert_offsets), C.byref(sh), e_begin, e_end, _ptr(owner_y), world,
                                  _ptr(row_dst), _stream(stream)), "moe_ep_row_table")


def moe_ep_expert_ffn(x_perm, expert_offsets, w_local, sh, e_begin, e_end, row_dst, status_word, ws, stream=None):
    w13, s13, w2, s2 = w_local
    _check(lib().moe_ep_expert_ffn(_ptr(x_perm), _ptr(expert_offsets), _ptr(w13), _ptr(s13), _ptr(w2), _ptr(s2), C.byref(sh),
                                   e_begin, e_end, _ptr(row_dst), _ptr(status_word), _ptr(ws), ws.numel(), _stream(stream)),
           "moe_ep_expert_ffn")


def moe_forward_packed(logits, x, packed, sh, out, topk_ids, topk_w, status_word, ws, stream=None):
    _check(lib().moe_forward_packed(_ptr(logits), _ptr(x), _ptr(packed), C.byref(sh), _ptr(out), _ptr(topk_ids),
                                    _ptr(topk_w), _ptr(status_word), _ptr(ws), ws.numel(), _stream(stream)),
           "moe_forward_packed")


def moe_forward_host_packed(logits_host, x_host, packed, sh, out_host, status_word, ws, stream=None):
    _check(lib().moe_forward_host_packed(_ptr(logits_host), _ptr(x_host), _ptr(packed), C.byref(sh), _ptr(out_host),
                                         _ptr(status_word), _ptr(ws), ws.numel(), _stream(stream)),
           "moe_forward_host_packed")


class BoundCall:
    """One C-ABI call with its arguments marshalled once: calling the object makes the call again on the same buffers
    (which it keeps alive) - a serving loop that reuses its buffers need not rebuild the argument list every step."""

    def __init__(self, name, fn, args, keep):
        self.name, self.fn, self.args, self.keep = name, fn, args, keep

    def __call__(self):
        rc = self.fn(*self.args)
        if rc != 0:
            _check(rc, self.name)


def bind_forward_host(logits_host, x_host, weights, sh, out_host, status_word, ws, stream=None):
    """moe_forward_host (weights = the four tensors) or moe_forward_host_packed (weights = moe_prepack's tensor) as a
    BoundCall."""
    tensors = (logits_host, x_host, weights, sh, out_host, status_word, ws, stream)
    if isinstance(weights, (tuple, list)):
        args = (_ptr(logits_host), _ptr(x_host), *(_ptr(t) for t in weights), C.byref(sh), _ptr(out_host), _ptr(status_word),
                _ptr(ws), ws.numel(), _stream(stream))
        return BoundCall("moe_forward_host", lib().moe_forward_host, args, tensors)
    args = (_ptr(logits_host), _ptr(x_host), _ptr(weights), C.byref(sh), _ptr(out_host), _ptr(status_word), _ptr(ws),
            ws.numel(), _stream(stream))
    return BoundCall("moe_forward_host_packed", lib().moe_forward_host_packed, args, tensors)


def moe_debug_read_probe(src, sink, status_word, stream=None):
    """Enqueue one read-only pass over the tensor `src` (see the header); time it with events around the call."""
    _check(lib().moe_debug_read_probe(_ptr(src), src.numel() * src.element_size(), _ptr(sink),
                                      sink.numel() * sink.element_size(), _ptr(status_word), _stream(stream)),
           "moe_debug_read_probe")


def moe_forward_workspace_bytes(sh):
    return int(lib().moe_forward_workspace_bytes(C.byref(sh)))


def moe_forward_sync_bytes():
    return int(lib().moe_forward_sync_bytes())


def alloc_forward_workspace(sh, device="cuda"):
    """Workspace of moe_forward with its counter block cleared (the one-time clear the call asks for)."""
    n = moe_forward_workspace_bytes(sh)
    if n == 0:
        raise MoeError("unsupported shape")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    ws[:moe_forward_sync_bytes()].zero_()
    return ws


def moe_forward(logits, x, w13, w13_scale, w2, w2_scale, sh, out, topk_ids, topk_w, status_word, ws, stream=None):
    _check(lib().moe_forward(_ptr(logits), _ptr(x), _ptr(w13), _ptr(w13_scale), _ptr(w2), _ptr(w2_scale), C.byref(sh),
                             _ptr(out), _ptr(topk_ids), _ptr(topk_w), _ptr(status_word), _ptr(ws), ws.numel(),
                             _stream(stream)), "moe_forward")


def moe_debug_forward_one_launch(logits, x, w13, w13_scale, w2, w2_scale, sh, out, topk_ids, topk_w, status_word, ws,
                                 stream=None):
    _check(lib().moe_debug_forward_one_launch(_ptr(logits), _ptr(x), _ptr(w13), _ptr(w13_scale), _ptr(w2), _ptr(w2_scale),
                                              C.byref(sh), _ptr(out), _ptr(topk_ids), _ptr(topk_w), _ptr(status_word),
                                              _ptr(ws), ws.numel(), _stream(stream)), "moe_debug_forward_one_launch")


def moe_forward_host(logits_host, x_host, w13, w13_scale, w2, w2_scale, sh, out_host, status_word, ws, stream=None):
    _check(lib().moe_forward_host(_ptr(logits_host), _ptr(x_host), _ptr(w13), _ptr(w13_scale), _ptr(w2), _ptr(w2_scale),
                                  C.byref(sh), _ptr(out_host), _ptr(status_word), _ptr(ws), ws.numel(), _stream(stream)),
           "moe_forward_host")


def moe_router_logits(x, w_router, logits, status_word=None, stream=None):
    T, H = x.shape
    E = w_router.shape[0]
    _check(lib().moe_router_logits(_ptr(x), _ptr(w_router), T, H, E, _ptr(logits), _ptr(status_word), _stream(stream)),
           "moe_router_logits")


def moe_combine_shared(y_perm, inv_perm, topk_w, y_shared, sh, out, stream=None):
    _check(lib().moe_combine_shared(_ptr(y_perm), _ptr(inv_perm), _ptr(topk_w), _ptr(y_shared), C.byref(sh), _ptr(out),
                                    _stream(stream)), "moe_combine_shared")


def alloc_block_workspace(sh, device="cuda"):
    n = int(lib().moe_ffn_block_workspace_bytes(C.byref(sh)))
    if n == 0:
        raise MoeError("unsupported shape")
    return torch.empty(n, dtype=torch.uint8, device=device)


def moe_ffn_block(x, w_router, routed, shared, sh, out, topk_ids, topk_w, status_word, ws, stream=None):
    """The FFN block: router projection, routed experts, shared expert, join (see include/moe_b200.h).
    `routed` and `shared` are (w13, w13_scale, w2, w2_scale) tuples; the shared tensors have E = 1."""
    _check(lib().moe_ffn_block(_ptr(x), _ptr(w_router), *[_ptr(a) for a in routed], *[_ptr(a) for a in shared], C.byref(sh),
                               _ptr(out), _ptr(topk_ids), _ptr(topk_w), _ptr(status_word), _ptr(ws), ws.numel(),
                               _stream(stream)), "moe_ffn_block")


class LayerBuffers:
    """Device buffers for the four calls on one shape (allocation only, no arithmetic)."""

    def __init__(self, sh, device="cuda"):
        S = sh.T * sh.k
        dev = device
        self.sh = sh
        self.topk_ids = torch.empty((sh.T, sh.k), dtype=torch.int32, device=dev)
        self.topk_w = torch.empty((sh.T, sh.k), dtype=torch.float32, device=dev)
        self.expert_offsets = torch.empty(sh.E + 1, dtype=torch.int32, device=dev)
        self.x_perm = torch.empty((S, sh.H), dtype=torch.bfloat16, device=dev)
        self.perm = torch.empty(S, dtype=torch.int32, device=dev)
        self.inv_perm = torch.empty(S, dtype=torch.int32, device=dev)
        self.y_perm = torch.empty((S, sh.H), dtype=torch.float32, device=dev)
        self.out = torch.empty((sh.T, sh.H), dtype=torch.bfloat16, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.ws = alloc_workspace(sh, dev)


def moe_layer(logits, x, weights, buf, stream=None):
    """route -> permute -> expert_ffn -> combine on device tensors; returns buf.out (enqueue only)."""
    w13, s13, w2, s2 = weights
    sh = buf.sh
    moe_route(logits, sh.k, buf.topk_ids, buf.topk_w, buf.expert_offsets, buf.ws, stream)
    moe_permute(x, buf.topk_ids, buf.expert_offsets, sh, buf.x_perm, buf.perm, buf.inv_perm, buf.ws, stream)
    moe_expert_ffn(buf.x_perm, buf.expert_offsets, w13, s13, w2, s2, sh, buf.y_perm, buf.status, buf.ws, stream)
    moe_combine(buf.y_perm, buf.inv_perm, buf.topk_w, sh, buf.out, stream)
    return buf.out

"""Thin ctypes binding over libcart.so: the same names as include/cart.h, argument marshalling only.

Every step of the attention path runs inside the library's CUDA kernels; this module converts
Python values to C arguments and turns a non-zero cart_status into ``CartError``.  There is no CPU
fallback: if the library has not been built, loading raises.

Device tensors are passed as anything with ``data_ptr()`` (torch tensors) or as integer addresses;
streams as ``torch.cuda.Stream``, an integer ``cudaStream_t`` or None (the legacy default stream).
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libcart.so")

CART_NONE = -1
CART_OK = 0
STATUS_NAMES = ["CART_OK", "CART_ERR_INVALID_ARG", "CART_ERR_SHAPE", "CART_ERR_BAD_HANDLE",
                "CART_ERR_CAPACITY", "CART_ERR_OOM", "CART_ERR_EMPTY", "CART_ERR_IN_USE",
                "CART_ERR_CUDA", "CART_ERR_TIMEOUT", "CART_ERR_EVICTED"]
(CART_ERR_INVALID_ARG, CART_ERR_SHAPE, CART_ERR_BAD_HANDLE, CART_ERR_CAPACITY, CART_ERR_OOM,
 CART_ERR_EMPTY, CART_ERR_IN_USE, CART_ERR_CUDA, CART_ERR_TIMEOUT, CART_ERR_EVICTED) = range(1, 11)
CART_PAGE_TOKENS = 64

# every symbol include/cart.h and include/cart_plan.h declare
EXPORTS = ["cart_scratch_bytes", "cart_create", "cart_destroy", "cart_register_cartridge",
           "cart_compose", "cart_release_cartridge", "cart_request_open", "cart_request_reserve", "cart_request_close",
           "cart_append_kv", "cart_extend_kv", "cart_decode_attention", "cart_decode_step", "cart_prefill_attention", "cart_suffix_len",
           "cart_kv_bytes", "cart_sync_status", "cart_set_timing", "cart_get_timing",
           "cart_set_share_min_readers", "cart_set_piece_cost", "cart_plan_build_shared",
           "cart_set_plan_reuse", "cart_set_prefill_split", "cart_graph_begin", "cart_graph_step", "cart_graph_end", "cart_plan_count", "cart_plan_reusable", "cart_set_side_by_side",
           "cart_request_open_paged", "cart_evict_request", "cart_restore_request", "cart_evict_cartridge",
           "cart_restore_cartridge", "cart_train_attention_fwd", "cart_train_attention_bwd",
           "cart_decode_attention_static", "cart_launch_count", "cart_status_string",
           "cart_last_error", "cart_plan_build"]


class cart_config(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
                ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("max_requests", ctypes.c_int32), ("max_cartridges", ctypes.c_int32),
                ("max_parts", ctypes.c_int32), ("softmax_scale", ctypes.c_float),
                ("arena", ctypes.c_void_p), ("arena_bytes", ctypes.c_uint64),
                ("device", ctypes.c_int32)]


class cart_plan_seg(ctypes.Structure):
    _fields_ = [("k_row", ctypes.c_uint32), ("v_row", ctypes.c_uint32),
                ("head_stride", ctypes.c_uint32), ("layer_stride", ctypes.c_uint32),
                ("n_tok", ctypes.c_uint32), ("flags", ctypes.c_uint32)]


class cart_work_item(ctypes.Structure):
    _fields_ = [("k_row", ctypes.c_uint32), ("v_row", ctypes.c_uint32),
                ("layer_stride", ctypes.c_uint32), ("n_tok", ctypes.c_uint32),
                ("row_group", ctypes.c_uint32), ("flags", ctypes.c_uint32),
                ("slot", ctypes.c_uint32), ("merge", ctypes.c_uint32)]


class cart_merge_item(ctypes.Structure):
    _fields_ = [("row_group", ctypes.c_uint32), ("slot_begin", ctypes.c_uint32),
                ("slot_end", ctypes.c_uint32), ("reserved", ctypes.c_uint32)]


class cart_shared_unit(ctypes.Structure):
    _fields_ = [("k_row", ctypes.c_uint32), ("v_row", ctypes.c_uint32),
                ("layer_stride", ctypes.c_uint32), ("n_tiles", ctypes.c_uint32),
                ("reader_begin", ctypes.c_uint32), ("n_readers", ctypes.c_uint32),
                ("kv_head", ctypes.c_uint16), ("flags", ctypes.c_uint16), ("chunk", ctypes.c_uint32),
                ("lim_base", ctypes.c_int32), ("lim_cap", ctypes.c_int32), ("tr_hi", ctypes.c_uint32),
                ("reserved", ctypes.c_uint32)]


class cart_plan_out(ctypes.Structure):
    _fields_ = [("items", ctypes.POINTER(cart_work_item)), ("items_cap", ctypes.c_int32), ("n_items", ctypes.c_int32),
                ("cta_begin", ctypes.POINTER(ctypes.c_uint32)),
                ("merges", ctypes.POINTER(cart_merge_item)), ("merges_cap", ctypes.c_int32),
                ("n_merges", ctypes.c_int32),
                ("n_cta_used", ctypes.c_int32), ("slots_cap", ctypes.c_int32), ("n_slots", ctypes.c_int32),
                ("total_tiles", ctypes.c_int64), ("piece_cost", ctypes.c_int32),
                ("units", ctypes.POINTER(cart_shared_unit)), ("units_cap", ctypes.c_int32),
                ("n_units", ctypes.c_int32),
                ("unit_cta_begin", ctypes.POINTER(ctypes.c_uint32)), ("n_unit_cta_used", ctypes.c_int32),
                ("readers", ctypes.POINTER(ctypes.c_uint32)), ("readers_cap", ctypes.c_int32),
                ("n_readers", ctypes.c_int32),
                ("reader_slot", ctypes.POINTER(ctypes.c_uint32)),
                ("reader_merge", ctypes.POINTER(ctypes.c_uint32)),
                ("shared_tiles", ctypes.c_int64), ("unit_cost", ctypes.c_int32),
                ("side_by_side", ctypes.c_int32), ("n_shared_ctas", ctypes.c_int32)]


CART_ITEM_BEGIN, CART_ITEM_END, CART_ITEM_DIRECT, CART_ITEM_TAIL, CART_ITEM_SUFFIX, CART_ITEM_PAGED = 1, 2, 4, 8, 16, 32
CART_SEG_SUFFIX, CART_SEG_PAGED = 1, 2
CART_UNIT_SUFFIX, CART_UNIT_PAGED = 1, 2
CART_UNIT_SUFFIX = 1


class CartError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = int(status)
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else "status %d" % status
        super().__init__("%s: %s%s" % (where, name, (" -- " + detail) if detail else ""))


_lib = None


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """Loads libcart.so (built in-tree by ``buildlib.build()``).  Raises if it is missing."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise ImportError("libcart.so not found at %s: build it with "
                          "`python -m paper_2506_06266_b200.buildlib` (there is no CPU fallback)" % p)
    lib = ctypes.CDLL(p)
    vp, i32, u64p = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(ctypes.c_uint64)
    i32p = ctypes.POINTER(ctypes.c_int32)
    lib.cart_scratch_bytes.argtypes = [ctypes.POINTER(cart_config), u64p]
    lib.cart_create.argtypes = [ctypes.POINTER(cart_config), ctypes.POINTER(vp)]
    lib.cart_destroy.argtypes = [vp]
    lib.cart_register_cartridge.argtypes = [vp, vp, vp, i32, vp, i32p]
    lib.cart_compose.argtypes = [vp, i32p, i32, i32p]
    lib.cart_release_cartridge.argtypes = [vp, i32]
    lib.cart_request_open.argtypes = [vp, i32, i32, i32p]
    lib.cart_request_close.argtypes = [vp, i32]
    lib.cart_request_open_paged.argtypes = [vp, i32, i32, i32p]
    lib.cart_evict_request.argtypes = [vp, i32, vp, vp, i32p, vp]
    lib.cart_restore_request.argtypes = [vp, i32, vp, vp, vp]
    lib.cart_evict_cartridge.argtypes = [vp, i32]
    lib.cart_train_attention_fwd.argtypes = [vp, i32, i32p, i32, vp, vp, vp, vp]
    lib.cart_train_attention_bwd.argtypes = [vp, i32, i32p, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.cart_restore_cartridge.argtypes = [vp, i32, vp, vp, vp]
    lib.cart_request_reserve.argtypes = [vp, i32, i32, vp]
    lib.cart_append_kv.argtypes = [vp, i32, i32p, i32, vp, vp, vp]
    lib.cart_extend_kv.argtypes = [vp, i32, i32, vp, vp, i32, vp]
    lib.cart_decode_attention.argtypes = [vp, i32, i32p, i32, vp, vp, vp, vp]
    lib.cart_decode_step.argtypes = [vp, i32, i32p, i32, vp, vp, vp, vp, vp, vp]
    lib.cart_prefill_attention.argtypes = [vp, i32, i32, vp, i32, vp, vp, vp]
    lib.cart_graph_begin.argtypes = [vp, i32p, i32, i32, vp]
    lib.cart_graph_step.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp]
    lib.cart_graph_end.argtypes = [vp, i32]
    lib.cart_suffix_len.argtypes = [vp, i32, i32, i32p]
    lib.cart_kv_bytes.argtypes = [vp, i32, u64p, u64p]
    lib.cart_sync_status.argtypes = [vp, vp]
    lib.cart_set_timing.argtypes = [vp, i32]
    lib.cart_set_share_min_readers.argtypes = [vp, i32]
    lib.cart_set_piece_cost.argtypes = [vp, i32]
    lib.cart_get_timing.argtypes = [vp, ctypes.POINTER(ctypes.c_double), u64p]
    lib.cart_decode_attention_static.argtypes = [vp, vp, i32, i32, i32, i32, ctypes.c_float, vp, vp, i32, vp]
    lib.cart_launch_count.argtypes = [vp]
    lib.cart_launch_count.restype = ctypes.c_uint64
    lib.cart_plan_count.argtypes = [vp]
    lib.cart_plan_count.restype = ctypes.c_uint64
    lib.cart_set_plan_reuse.argtypes = [vp, i32]
    lib.cart_set_prefill_split.argtypes = [vp, i32]
    lib.cart_set_side_by_side.argtypes = [vp, i32]
    lib.cart_plan_reusable.argtypes = [i32p, i32p, i32, i32, i32p]
    lib.cart_status_string.argtypes = [ctypes.c_int]
    lib.cart_status_string.restype = ctypes.c_char_p
    lib.cart_last_error.argtypes = [vp]
    lib.cart_last_error.restype = ctypes.c_char_p
    lib.cart_plan_build.argtypes = [
        ctypes.POINTER(cart_plan_seg), i32p, i32, i32, i32, i32, ctypes.POINTER(cart_work_item), i32,
        i32p, ctypes.POINTER(ctypes.c_uint32), ctypes.POINTER(cart_merge_item), i32, i32p, i32p, i32p,
        ctypes.POINTER(ctypes.c_int64)]
    lib.cart_plan_build_shared.argtypes = [ctypes.POINTER(cart_plan_seg), i32p, i32, i32, i32, i32, i32, i32, i32,
                                           ctypes.POINTER(cart_plan_out)]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name not in ("cart_launch_count", "cart_plan_count", "cart_status_string", "cart_last_error"):
            fn.restype = ctypes.c_int
    if path is None:
        _lib = lib
    return lib


def _ptr(x) -> Optional[int]:
    if x is None:
        return None
    if hasattr(x, "data_ptr"):
        return int(x.data_ptr())
    return int(x)


def _stream(s) -> Optional[int]:
    if s is None:
        return None
    if hasattr(s, "cuda_stream"):
        return int(s.cuda_stream)
    return int(s)


def _ids(xs: Sequence[int]):
    n = len(xs)
    return (ctypes.c_int32 * max(n, 1))(*[int(x) for x in xs]), n


def _check(status: int, where: str, ctx=None) -> None:
    if status != CART_OK:
        detail = ""
        if ctx:
            detail = load_library().cart_last_error(ctx).decode("utf-8", "replace")
        raise CartError(status, where, detail)


def make_config(n_layers: int, n_q_heads: int, n_kv_heads: int, max_requests: int,
                max_cartridges: int, arena=None, arena_bytes: int = 0, device: int = 0,
                head_dim: int = 128, max_parts: int = 0, softmax_scale: float = 0.0) -> cart_config:
    return cart_config(n_layers, n_q_heads, n_kv_heads, head_dim, max_requests, max_cartridges,
                       max_parts, softmax_scale, _ptr(arena), int(arena_bytes), device)


def cart_scratch_bytes(cfg: cart_config) -> int:
    out = ctypes.c_uint64(0)
    _check(load_library().cart_scratch_bytes(ctypes.byref(cfg), ctypes.byref(out)), "cart_scratch_bytes")
    return int(out.value)


def cart_create(cfg: cart_config) -> int:
    out = ctypes.c_void_p(None)
    _check(load_library().cart_create(ctypes.byref(cfg), ctypes.byref(out)), "cart_create")
    return int(out.value)


def cart_destroy(ctx: int) -> None:
    _check(load_library().cart_destroy(ctx), "cart_destroy")


def cart_register_cartridge(ctx: int, k, v, p: int, stream=None) -> int:
    out = ctypes.c_int32(-1)
    _check(load_library().cart_register_cartridge(ctx, _ptr(k), _ptr(v), int(p), _stream(stream),
                                                  ctypes.byref(out)), "cart_register_cartridge", ctx)
    return int(out.value)


def cart_compose(ctx: int, parts: Sequence[int]) -> int:
    arr, n = _ids(parts)
    out = ctypes.c_int32(-1)
    _check(load_library().cart_compose(ctx, arr, n, ctypes.byref(out)), "cart_compose", ctx)
    return int(out.value)


def cart_release_cartridge(ctx: int, cid: int) -> None:
    _check(load_library().cart_release_cartridge(ctx, int(cid)), "cart_release_cartridge", ctx)


def cart_request_open(ctx: int, cartridge: int, suffix_capacity: int) -> int:
    out = ctypes.c_int32(-1)
    _check(load_library().cart_request_open(ctx, int(cartridge), int(suffix_capacity), ctypes.byref(out)),
           "cart_request_open", ctx)
    return int(out.value)


def cart_request_open_paged(ctx: int, cartridge: int, initial_capacity: int = 0) -> int:
    out = ctypes.c_int32(-1)
    _check(load_library().cart_request_open_paged(ctx, int(cartridge), int(initial_capacity), ctypes.byref(out)),
           "cart_request_open_paged", ctx)
    return int(out.value)


def cart_evict_request(ctx: int, req: int, k_out, v_out, stream=None) -> int:
    """Returns n, the number of tokens per (layer, KV head) written to k_out / v_out."""
    n = ctypes.c_int32(0)
    _check(load_library().cart_evict_request(ctx, int(req), _ptr(k_out), _ptr(v_out), ctypes.byref(n), _stream(stream)),
           "cart_evict_request", ctx)
    return int(n.value)


def cart_restore_request(ctx: int, req: int, k_in, v_in, stream=None) -> None:
    _check(load_library().cart_restore_request(ctx, int(req), _ptr(k_in), _ptr(v_in), _stream(stream)),
           "cart_restore_request", ctx)


def cart_evict_cartridge(ctx: int, cid: int) -> None:
    _check(load_library().cart_evict_cartridge(ctx, int(cid)), "cart_evict_cartridge", ctx)


def cart_restore_cartridge(ctx: int, cid: int, k, v, stream=None) -> None:
    _check(load_library().cart_restore_cartridge(ctx, int(cid), _ptr(k), _ptr(v), _stream(stream)),
           "cart_restore_cartridge", ctx)


def cart_train_attention_fwd(ctx: int, layer: int, convs, q, out, lse, stream=None) -> None:
    arr, n = _reqs(convs)
    _check(load_library().cart_train_attention_fwd(ctx, int(layer), arr, n, _ptr(q), _ptr(out), _ptr(lse), _stream(stream)),
           "cart_train_attention_fwd", ctx)


def cart_train_attention_bwd(ctx: int, layer: int, convs, q, out, lse, dout, delta, dq, dk, dv, dzk=None, dzv=None,
                             stream=None) -> None:
    arr, n = _reqs(convs)
    _check(load_library().cart_train_attention_bwd(ctx, int(layer), arr, n, _ptr(q), _ptr(out), _ptr(lse), _ptr(dout),
                                                   _ptr(delta), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dzk), _ptr(dzv),
                                                   _stream(stream)), "cart_train_attention_bwd", ctx)


def cart_request_reserve(ctx: int, req: int, suffix_capacity: int, stream=None) -> None:
    _check(load_library().cart_request_reserve(ctx, int(req), int(suffix_capacity), _stream(stream)),
           "cart_request_reserve", ctx)


def cart_request_close(ctx: int, req: int) -> None:
    _check(load_library().cart_request_close(ctx, int(req)), "cart_request_close", ctx)


class ReqList:
    """A batch of request handles marshalled once, for callers that reuse it every step."""

    def __init__(self, reqs: Sequence[int]):
        self.array, self.n = _ids(reqs)


def _reqs(reqs):
    if isinstance(reqs, ReqList):
        return reqs.array, reqs.n
    return _ids(reqs)


def cart_append_kv(ctx: int, layer: int, reqs, k_new, v_new, stream=None) -> None:
    arr, n = _reqs(reqs)
    _check(load_library().cart_append_kv(ctx, int(layer), arr, n, _ptr(k_new), _ptr(v_new), _stream(stream)),
           "cart_append_kv", ctx)


def cart_extend_kv(ctx: int, layer: int, req: int, k, v, n_tokens: int, stream=None) -> None:
    _check(load_library().cart_extend_kv(ctx, int(layer), int(req), _ptr(k), _ptr(v), int(n_tokens),
                                         _stream(stream)), "cart_extend_kv", ctx)


def cart_decode_attention(ctx: int, layer: int, reqs, q, out, lse=None, stream=None) -> None:
    arr, n = _reqs(reqs)
    _check(load_library().cart_decode_attention(ctx, int(layer), arr, n, _ptr(q), _ptr(out), _ptr(lse),
                                                _stream(stream)), "cart_decode_attention", ctx)


def cart_decode_step(ctx: int, layer: int, reqs, k_new, v_new, q, out, lse=None, stream=None) -> None:
    arr, n = _reqs(reqs)
    _check(load_library().cart_decode_step(ctx, int(layer), arr, n, _ptr(k_new), _ptr(v_new), _ptr(q), _ptr(out),
                                           _ptr(lse), _stream(stream)), "cart_decode_step", ctx)


def cart_graph_begin(ctx: int, reqs, max_steps: int, stream=None) -> None:
    arr, n = _reqs(reqs)
    _check(load_library().cart_graph_begin(ctx, arr, n, int(max_steps), _stream(stream)), "cart_graph_begin", ctx)


def cart_graph_step(ctx: int, layer: int, k_new, v_new, q, out, lse=None, stream=None) -> None:
    _check(load_library().cart_graph_step(ctx, int(layer), _ptr(k_new), _ptr(v_new), _ptr(q), _ptr(out), _ptr(lse),
                                          _stream(stream)), "cart_graph_step", ctx)


def cart_graph_end(ctx: int, steps_run: int) -> None:
    _check(load_library().cart_graph_end(ctx, int(steps_run)), "cart_graph_end", ctx)


def cart_prefill_attention(ctx: int, layer: int, req: int, q, n_new: int, out, lse=None, stream=None) -> None:
    _check(load_library().cart_prefill_attention(ctx, int(layer), int(req), _ptr(q), int(n_new), _ptr(out), _ptr(lse),
                                                 _stream(stream)), "cart_prefill_attention", ctx)


def cart_suffix_len(ctx: int, req: int, layer: int) -> int:
    out = ctypes.c_int32(0)
    _check(load_library().cart_suffix_len(ctx, int(req), int(layer), ctypes.byref(out)), "cart_suffix_len", ctx)
    return int(out.value)


def cart_kv_bytes(ctx: int, req: int) -> Tuple[int, int]:
    a, b = ctypes.c_uint64(0), ctypes.c_uint64(0)
    _check(load_library().cart_kv_bytes(ctx, int(req), ctypes.byref(a), ctypes.byref(b)), "cart_kv_bytes", ctx)
    return int(a.value), int(b.value)


def cart_sync_status(ctx: int, stream=None) -> None:
    _check(load_library().cart_sync_status(ctx, _stream(stream)), "cart_sync_status", ctx)


def cart_set_timing(ctx: int, enable: bool) -> None:
    _check(load_library().cart_set_timing(ctx, 1 if enable else 0), "cart_set_timing", ctx)


def cart_set_share_min_readers(ctx: int, min_readers: int) -> None:
    _check(load_library().cart_set_share_min_readers(ctx, int(min_readers)), "cart_set_share_min_readers", ctx)


def cart_set_piece_cost(ctx: int, tiles_per_piece: int) -> None:
    _check(load_library().cart_set_piece_cost(ctx, int(tiles_per_piece)), "cart_set_piece_cost", ctx)


def cart_set_side_by_side(ctx: int, mode: int) -> None:
    _check(load_library().cart_set_side_by_side(ctx, int(mode)), "cart_set_side_by_side", ctx)


def cart_set_prefill_split(ctx: int, pieces: int) -> None:
    _check(load_library().cart_set_prefill_split(ctx, int(pieces)), "cart_set_prefill_split", ctx)


def cart_set_plan_reuse(ctx: int, max_grow_tokens: int) -> None:
    _check(load_library().cart_set_plan_reuse(ctx, int(max_grow_tokens)), "cart_set_plan_reuse", ctx)


def cart_plan_count(ctx: int) -> int:
    return int(load_library().cart_plan_count(ctx))


def cart_plan_reusable(plan_len: Sequence[int], cur_len: Sequence[int], max_grow: int) -> Optional[int]:
    """Host-only: the common growth d if a plan built at plan_len serves cur_len, else None."""
    n = len(plan_len)
    a = (ctypes.c_int32 * max(n, 1))(*[int(x) for x in plan_len])
    b = (ctypes.c_int32 * max(n, 1))(*[int(x) for x in cur_len])
    d = ctypes.c_int32(-1)
    ok = load_library().cart_plan_reusable(a, b, n, int(max_grow), ctypes.byref(d))
    return int(d.value) if ok else None


def cart_get_timing(ctx: int) -> Tuple[float, int]:
    ms, n = ctypes.c_double(0.0), ctypes.c_uint64(0)
    _check(load_library().cart_get_timing(ctx, ctypes.byref(ms), ctypes.byref(n)), "cart_get_timing", ctx)
    return float(ms.value), int(n.value)


def cart_decode_attention_static(q, kv, n_reqs: int, n_q_heads: int, n_kv_heads: int, n_tokens: int,
                                 out, lse=None, softmax_scale: float = 0.0, device: int = 0, stream=None) -> None:
    """Context-free decode attention whose scratch is a fixed device array inside libcart.so, for
    callers that may not allocate (see include/cart.h).  kv is one buffer: all keys, then all values."""
    _check(load_library().cart_decode_attention_static(
        _ptr(q), _ptr(kv), int(n_reqs), int(n_q_heads), int(n_kv_heads), int(n_tokens), float(softmax_scale),
        _ptr(out), _ptr(lse), int(device), _stream(stream)), "cart_decode_attention_static")


def cart_launch_count(ctx: int) -> int:
    return int(load_library().cart_launch_count(ctx))


def cart_status_string(status: int) -> str:
    return load_library().cart_status_string(int(status)).decode()


def cart_plan_build(segs: Sequence[Sequence[Tuple[int, int, int, int, int]]], n_kv_heads: int, n_cta: int,
                    tile_tokens: int, items_cap: Optional[int] = None):
    """Host-only planner.  segs[i] lists request i's segments as (k_row, v_row, head_stride,
    layer_stride, n_tok).  Returns a dict with items, cta_begin, merges and the counters."""
    lib = load_library()
    flat = [s for r in segs for s in r]
    seg_arr = (cart_plan_seg * max(len(flat), 1))(*[cart_plan_seg(*s) for s in flat])
    begins = [0]
    for r in segs:
        begins.append(begins[-1] + len(r))
    sb = (ctypes.c_int32 * len(begins))(*begins)
    cap = items_cap if items_cap is not None else len(flat) * n_kv_heads + n_cta + 8
    items = (cart_work_item * max(cap, 1))()
    cta_begin = (ctypes.c_uint32 * (n_cta + 1))()
    merges = (cart_merge_item * max(n_cta, 1))()
    n_items, n_merges, n_used, n_slots = (ctypes.c_int32(0) for _ in range(4))
    total = ctypes.c_int64(0)
    st = lib.cart_plan_build(seg_arr, sb, len(segs), n_kv_heads, n_cta, tile_tokens, items, cap,
                             ctypes.byref(n_items), cta_begin, merges, n_cta, ctypes.byref(n_merges),
                             ctypes.byref(n_used), ctypes.byref(n_slots), ctypes.byref(total))
    _check(st, "cart_plan_build")
    return {"items": [items[i] for i in range(n_items.value)], "cta_begin": list(cta_begin),
            "merges": [merges[i] for i in range(n_merges.value)], "n_cta_used": n_used.value,
            "n_slots": n_slots.value, "total_tiles": total.value}


def cart_plan_build_shared(segs: Sequence[Sequence[Tuple[int, int, int, int, int]]], n_kv_heads: int, group: int,
                           n_cta: int, tile_tokens: int, share_min_readers: int, share_tile_tokens: int,
                           slots_cap: int = 1 << 20, piece_cost: int = 0, unit_cost: int = 0,
                           side_by_side: int = 0):
    """Host-only planner with shared segments (see include/cart_plan.h).  Returns a dict with the
    stream plan (items, cta_begin, merges, ...) and the shared part (units, unit_cta_begin, readers,
    reader_slot[entry][head], reader_merge[entry][head])."""
    lib = load_library()
    flat = [s for r in segs for s in r]
    seg_arr = (cart_plan_seg * max(len(flat), 1))(*[cart_plan_seg(*s) for s in flat])
    begins = [0]
    for r in segs:
        begins.append(begins[-1] + len(r))
    sb = (ctypes.c_int32 * len(begins))(*begins)
    n_rg = len(segs) * n_kv_heads
    items_cap = 2 * len(flat) * n_kv_heads + n_cta + 8
    merges_cap = n_rg + n_cta
    readers_cap = max(len(flat), 1)
    units_cap = readers_cap * n_kv_heads + n_cta
    o = cart_plan_out()
    items = (cart_work_item * items_cap)()
    cta_begin = (ctypes.c_uint32 * (n_cta + 1))()
    merges = (cart_merge_item * merges_cap)()
    units = (cart_shared_unit * units_cap)()
    unit_cta_begin = (ctypes.c_uint32 * (n_cta + 1))()
    readers = (ctypes.c_uint32 * readers_cap)()
    reader_slot = (ctypes.c_uint32 * (readers_cap * n_kv_heads))()
    reader_merge = (ctypes.c_uint32 * (readers_cap * n_kv_heads))()
    o.items, o.items_cap, o.cta_begin = items, items_cap, cta_begin
    o.merges, o.merges_cap, o.slots_cap = merges, merges_cap, slots_cap
    o.piece_cost = piece_cost
    o.unit_cost = unit_cost
    o.side_by_side = side_by_side
    o.units, o.units_cap, o.unit_cta_begin = units, units_cap, unit_cta_begin
    o.readers, o.readers_cap, o.reader_slot, o.reader_merge = readers, readers_cap, reader_slot, reader_merge
    st = lib.cart_plan_build_shared(seg_arr, sb, len(segs), n_kv_heads, group, n_cta, tile_tokens,
                                    share_min_readers, share_tile_tokens, ctypes.byref(o))
    _check(st, "cart_plan_build_shared")
    nr = o.n_readers
    return {"items": [items[i] for i in range(o.n_items)], "cta_begin": list(cta_begin),
            "merges": [merges[i] for i in range(o.n_merges)], "n_cta_used": o.n_cta_used,
            "n_slots": o.n_slots, "total_tiles": o.total_tiles,
            "units": [units[i] for i in range(o.n_units)], "unit_cta_begin": list(unit_cta_begin),
            "n_unit_cta_used": o.n_unit_cta_used, "n_shared_ctas": o.n_shared_ctas, "readers": [readers[i] for i in range(nr)],
            "reader_slot": [[reader_slot[e * n_kv_heads + g] for g in range(n_kv_heads)] for e in range(nr)],
            "reader_merge": [[reader_merge[e * n_kv_heads + g] for g in range(n_kv_heads)] for e in range(nr)],
            "shared_tiles": o.shared_tiles}

"""Thin ctypes binding over libspd.so: same names as the C ABI, argument marshalling only.

PyTorch supplies device memory and streams; every step of the path runs in the library's
kernels.  There is no fallback: if the library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import torch

from .build import LIB_PATH

SPD_OK = 0
SPD_F32, SPD_BF16 = 0, 1
SPD_PLAN_PER_CALL, SPD_PLAN_STORE, SPD_PLAN_REUSE = 0, 1, 2
_STATUS_NAMES = {0: "SPD_OK", 1: "SPD_ERR_INVALID_ARG", 2: "SPD_ERR_UNSUPPORTED", 3: "SPD_ERR_WORKSPACE",
                 4: "SPD_ERR_BAD_PAGE", 5: "SPD_ERR_CUDA", 6: "SPD_ERR_TIMEOUT", 7: "SPD_ERR_PLAN"}
_DEVICE_CODES = (SPD_OK, 4, 6, 7)     # what a call that waits for the device may report without raising

EXPORTS = ["spd_workspace_size", "spd_partial_attn", "spd_service_attn_merge", "spd_decode_step",
           "spd_step_blob_layout", "spd_decode_step_host", "spd_query_device_status",
           "spd_kernel_launch_count", "spd_status_string", "spd_profile_begin", "spd_profile_end",
           "spd_decode_step_static", "spd_append_kv",
           "spd_partial_attn_watch", "spd_decode_step_watch", "spd_set_bf16_math", "spd_merge_partials", "spd_prefill_attn",
           "spd_set_prefill_rows", "spd_token_step", "spd_partial_attn_planned", "spd_service_attn_merge_planned",
           "spd_decode_step_planned", "spd_set_split", "spd_set_programmatic_launch", "spd_debug_read_plan",
           "spd_debug_sm_moves", "spd_decode_step_append", "spd_watch_alarm", "spd_service_attn_merge_append"]


class SpdError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {_STATUS_NAMES.get(code, code)} ({status_string(code)})")


class Shape(C.Structure):
    _fields_ = [("batch", C.c_int32), ("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("page_size", C.c_int32), ("dtype", C.c_int32), ("sm_scale", C.c_float)]


class PagedKV(C.Structure):
    _fields_ = [("k_pool", C.c_void_p), ("v_pool", C.c_void_p), ("num_pages", C.c_int32),
                ("page_indptr", C.c_void_p), ("page_indices", C.c_void_p), ("seq_lens", C.c_void_p)]


class Layer(C.Structure):
    _fields_ = [("q", C.c_void_p), ("k_new", C.c_void_p), ("v_new", C.c_void_p), ("priv", PagedKV), ("pub", PagedKV),
                ("out", C.c_void_p)]


class StepBlob(C.Structure):
    _fields_ = [("priv_pages_listed", C.c_int64), ("pub_pages_listed", C.c_int64), ("q", C.c_size_t),
                ("priv_indptr", C.c_size_t), ("priv_lens", C.c_size_t), ("priv_indices", C.c_size_t),
                ("pub_indptr", C.c_size_t), ("pub_lens", C.c_size_t), ("pub_indices", C.c_size_t),
                ("status", C.c_size_t), ("in_bytes", C.c_size_t), ("out", C.c_size_t), ("total_bytes", C.c_size_t)]


class Watch(C.Structure):
    _fields_ = [("tok_lo", C.c_void_p), ("tok_hi", C.c_void_p), ("out", C.c_void_p)]


class Partial(C.Structure):
    _fields_ = [("o", C.c_void_p), ("m", C.c_void_p), ("l", C.c_void_p)]


_lib = None


def lib() -> C.CDLL:
    """Load libspd.so (built in-tree by build.py).  Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} not built: run `python -m paper_2409_19134_b200.build`")
        L = C.CDLL(LIB_PATH)
        vp, sz = C.c_void_p, C.c_size_t
        L.spd_workspace_size.argtypes = [C.POINTER(Shape), C.POINTER(sz)]
        L.spd_partial_attn.argtypes = [C.POINTER(Shape), vp, C.POINTER(PagedKV), Partial, vp, sz, vp]
        L.spd_service_attn_merge.argtypes = [C.POINTER(Shape), vp, C.POINTER(PagedKV), Partial, vp, C.c_int, vp, sz, vp]
        L.spd_decode_step.argtypes = [C.POINTER(Shape), vp, C.POINTER(PagedKV), C.POINTER(PagedKV), vp, C.c_int,
                                      C.c_int32, vp, sz, vp]
        L.spd_step_blob_layout.argtypes = [C.POINTER(Shape), C.c_int64, C.c_int64, C.c_int, C.POINTER(StepBlob)]
        L.spd_decode_step_host.argtypes = [C.POINTER(Shape), C.POINTER(StepBlob), vp, vp, C.POINTER(PagedKV),
                                           C.POINTER(PagedKV), C.c_int, C.POINTER(C.c_int32), vp, sz, vp]
        L.spd_query_device_status.argtypes = [vp, vp, C.POINTER(C.c_int32)]
        L.spd_kernel_launch_count.restype = C.c_int64
        L.spd_status_string.restype = C.c_char_p
        L.spd_status_string.argtypes = [C.c_int]
        L.spd_profile_begin.argtypes = [C.c_int32]
        L.spd_profile_end.argtypes = [C.POINTER(C.c_int32), C.POINTER(C.c_double)]
        L.spd_decode_step_static.argtypes = [C.POINTER(Shape), vp, C.POINTER(PagedKV), C.POINTER(PagedKV), vp, C.c_int,
                                             C.c_int32, C.POINTER(C.c_int32), vp]
        L.spd_partial_attn_watch.argtypes = [C.POINTER(Shape), vp, C.POINTER(PagedKV), Partial, C.POINTER(Watch), vp, sz, vp]
        L.spd_decode_step_watch.argtypes = [C.POINTER(Shape), vp, C.POINTER(PagedKV), C.POINTER(PagedKV), vp, C.c_int,
                                            C.POINTER(Watch), vp, sz, vp]
        L.spd_set_bf16_math.argtypes = [C.c_int32]
        L.spd_set_prefill_rows.argtypes = [C.c_int32]
        L.spd_token_step.argtypes = [C.POINTER(Shape), C.c_int32, C.POINTER(Layer), C.c_int, C.c_int32, vp, sz, vp]
        L.spd_partial_attn_planned.argtypes = [C.POINTER(Shape), vp, C.POINTER(PagedKV), Partial, C.c_int, vp, sz, vp]
        L.spd_service_attn_merge_planned.argtypes = [C.POINTER(Shape), vp, C.POINTER(PagedKV), Partial, vp, C.c_int, C.c_int,
                                                     vp, sz, vp]
        L.spd_decode_step_planned.argtypes = [C.POINTER(Shape), vp, C.POINTER(PagedKV), C.POINTER(PagedKV), vp, C.c_int,
                                              C.c_int32, C.c_int, vp, sz, vp]
        L.spd_decode_step_append.argtypes = [C.POINTER(Shape), vp, vp, vp, C.POINTER(PagedKV), C.POINTER(PagedKV), vp, C.c_int,
                                             C.c_int, vp, sz, vp]
        L.spd_service_attn_merge_append.argtypes = [C.POINTER(Shape), vp, vp, vp, C.POINTER(PagedKV), Partial, vp, C.c_int, C.c_int,
                                                    vp, sz, vp]
        L.spd_watch_alarm.argtypes = [vp, C.c_int32, C.c_int32, vp, C.c_float, vp, vp]
        L.spd_set_split.argtypes = [C.c_int32, C.c_int32]
        L.spd_set_programmatic_launch.argtypes = [C.c_int32]
        L.spd_debug_read_plan.argtypes = [vp, C.c_int32, vp, C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                          C.POINTER(C.c_int32), C.c_int32]
        L.spd_debug_sm_moves.argtypes = [vp, vp, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        L.spd_merge_partials.argtypes = [C.POINTER(Shape), C.c_int32, C.POINTER(Partial), vp, C.c_int, vp]
        L.spd_prefill_attn.argtypes = [C.POINTER(Shape), C.c_int64, vp, vp, vp, vp, vp, vp, C.c_int32, vp, vp, vp, vp,
                                       C.c_int, vp, sz, vp]
        L.spd_append_kv.argtypes = [C.POINTER(Shape), vp, vp, vp, vp, C.c_int32, vp, vp, vp, vp, sz, vp]
        for name in EXPORTS[:7] + EXPORTS[9:]:
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().spd_status_string(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != SPD_OK:
        raise SpdError(code, where)


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.float32:
        return SPD_F32
    if dt == torch.bfloat16:
        return SPD_BF16
    raise TypeError(f"unsupported dtype {dt}")


def make_shape(batch, num_q_heads, num_kv_heads, head_dim, dtype, sm_scale, page_size=16) -> Shape:
    return Shape(batch, num_q_heads, num_kv_heads, head_dim, page_size, _dtype_code(dtype), float(sm_scale))


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None or t.numel() == 0 else t.data_ptr()


def paged_kv(part) -> PagedKV:
    """Marshal an object with k_pool, v_pool, page_indptr, page_indices, seq_lens tensors."""
    for t in (part.k_pool, part.v_pool, part.page_indptr, part.page_indices, part.seq_lens):
        assert t.is_contiguous()
    assert part.page_indptr.dtype == torch.int32 and part.page_indices.dtype == torch.int32
    assert part.seq_lens.dtype == torch.int32
    return PagedKV(_ptr(part.k_pool), _ptr(part.v_pool), int(part.k_pool.shape[0]),
                   part.page_indptr.data_ptr(), _ptr(part.page_indices), part.seq_lens.data_ptr())


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def spd_workspace_size(shape: Shape) -> int:
    n = C.c_size_t(0)
    _check(lib().spd_workspace_size(C.byref(shape), C.byref(n)), "spd_workspace_size")
    return int(n.value)


def alloc_workspace(shape: Shape, device="cuda") -> torch.Tensor:
    """A zeroed workspace tensor of the size the library asks for."""
    return torch.zeros(spd_workspace_size(shape), dtype=torch.uint8, device=device)


def alloc_partial(shape: Shape, device="cuda") -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    B, H, D = shape.batch, shape.num_q_heads, shape.head_dim
    return (torch.empty((B, H, D), dtype=torch.float32, device=device),
            torch.empty((B, H), dtype=torch.float32, device=device),
            torch.empty((B, H), dtype=torch.float32, device=device))


def spd_partial_attn(shape, q, priv, out, ws, stream=None, plan=None) -> None:
    """plan=None calls spd_partial_attn; SPD_PLAN_* calls spd_partial_attn_planned with that mode."""
    kv = paged_kv(priv)
    part = Partial(out[0].data_ptr(), out[1].data_ptr(), out[2].data_ptr())
    if plan is None:
        _check(lib().spd_partial_attn(C.byref(shape), q.data_ptr(), C.byref(kv), part, ws.data_ptr(), ws.numel(),
                                      _stream_ptr(stream)), "spd_partial_attn")
    else:
        _check(lib().spd_partial_attn_planned(C.byref(shape), q.data_ptr(), C.byref(kv), part, int(plan), ws.data_ptr(),
                                              ws.numel(), _stream_ptr(stream)), "spd_partial_attn_planned")


def spd_service_attn_merge(shape, q, pub, partial_in, out, ws, stream=None, plan=None) -> None:
    kv = paged_kv(pub)
    part = Partial(partial_in[0].data_ptr(), partial_in[1].data_ptr(), partial_in[2].data_ptr())
    if plan is None:
        _check(lib().spd_service_attn_merge(C.byref(shape), q.data_ptr(), C.byref(kv), part, out.data_ptr(),
                                            _dtype_code(out.dtype), ws.data_ptr(), ws.numel(), _stream_ptr(stream)),
               "spd_service_attn_merge")
    else:
        _check(lib().spd_service_attn_merge_planned(C.byref(shape), q.data_ptr(), C.byref(kv), part, out.data_ptr(),
                                                    _dtype_code(out.dtype), int(plan), ws.data_ptr(), ws.numel(),
                                                    _stream_ptr(stream)), "spd_service_attn_merge_planned")


def spd_decode_step(shape, q, priv, pub, out, ws, fused=True, stream=None, plan=None) -> None:
    a, b = paged_kv(priv), paged_kv(pub)
    if plan is None:
        _check(lib().spd_decode_step(C.byref(shape), q.data_ptr(), C.byref(a), C.byref(b), out.data_ptr(),
                                     _dtype_code(out.dtype), 1 if fused else 0, ws.data_ptr(), ws.numel(),
                                     _stream_ptr(stream)), "spd_decode_step")
    else:
        _check(lib().spd_decode_step_planned(C.byref(shape), q.data_ptr(), C.byref(a), C.byref(b), out.data_ptr(),
                                             _dtype_code(out.dtype), 1 if fused else 0, int(plan), ws.data_ptr(),
                                             ws.numel(), _stream_ptr(stream)), "spd_decode_step_planned")


def spd_step_blob_layout(shape, priv_pages_listed: int, pub_pages_listed: int, out_dtype) -> StepBlob:
    lay = StepBlob()
    _check(lib().spd_step_blob_layout(C.byref(shape), priv_pages_listed, pub_pages_listed,
                                      _dtype_code(out_dtype), C.byref(lay)), "spd_step_blob_layout")
    return lay


def spd_decode_step_host(shape, layout, host_blob, device_blob, priv_pools, pub_pools, out_dtype, ws,
                         stream=None) -> Tuple[int, int]:
    """host_blob: pinned uint8 host tensor laid out per `layout`; device_blob: uint8 device tensor of
    layout.total_bytes; *_pools: (k_pool, v_pool) device tensors.  Waits for the stream; the output is
    then at host_blob[layout.out:].  Returns (device status, first flagged user or -1)."""
    def kv(pools):
        return PagedKV(_ptr(pools[0]), _ptr(pools[1]), int(pools[0].shape[0]), None, None, None)
    a, b = kv(priv_pools), kv(pub_pools)
    bad = C.c_int32(-1)
    code = lib().spd_decode_step_host(C.byref(shape), C.byref(layout), host_blob.data_ptr(), device_blob.data_ptr(),
                                      C.byref(a), C.byref(b), _dtype_code(out_dtype), C.byref(bad), ws.data_ptr(),
                                      ws.numel(), _stream_ptr(stream))
    if code not in _DEVICE_CODES:
        raise SpdError(code, "spd_decode_step_host")
    return int(code), int(bad.value)


class HostStep:
    """spd_decode_step_host with its arguments marshalled once: for a serving loop that reuses the same
    buffers every step and only rewrites the host blob.  Calling the object runs one step."""

    def __init__(self, shape, layout, host_blob, device_blob, priv_pools, pub_pools, out_dtype, ws, stream=None):
        self._keep = (shape, layout, host_blob, device_blob, priv_pools, pub_pools, ws)   # keep the memory alive
        self._a = PagedKV(_ptr(priv_pools[0]), _ptr(priv_pools[1]), int(priv_pools[0].shape[0]), None, None, None)
        self._b = PagedKV(_ptr(pub_pools[0]), _ptr(pub_pools[1]), int(pub_pools[0].shape[0]), None, None, None)
        self._bad = C.c_int32(-1)
        self._fn = lib().spd_decode_step_host
        self._args = (C.byref(shape), C.byref(layout), C.c_void_p(host_blob.data_ptr()), C.c_void_p(device_blob.data_ptr()),
                      C.byref(self._a), C.byref(self._b), _dtype_code(out_dtype), C.byref(self._bad),
                      C.c_void_p(ws.data_ptr()), C.c_size_t(ws.numel()), C.c_void_p(_stream_ptr(stream)))

    def __call__(self) -> Tuple[int, int]:
        code = self._fn(*self._args)
        if code not in _DEVICE_CODES:
            raise SpdError(code, "spd_decode_step_host")
        return int(code), int(self._bad.value)


def fill_step_blob(layout, host_blob, q, priv, pub) -> None:
    """Copy q and the two partitions' tables (any device) into a host blob at the layout's offsets."""
    def put(off, t):
        src = t.detach().cpu().contiguous().view(torch.uint8).reshape(-1)
        host_blob[off:off + src.numel()] = src
    put(layout.q, q)
    for part, (a, b, c) in ((priv, (layout.priv_indptr, layout.priv_lens, layout.priv_indices)),
                            (pub, (layout.pub_indptr, layout.pub_lens, layout.pub_indices))):
        put(a, part.page_indptr)
        put(b, part.seq_lens)
        put(c, part.page_indices)


def spd_query_device_status(ws, stream=None) -> Tuple[int, int]:
    """Waits for the stream; returns (status code, first flagged user or -1) and clears the flag."""
    bad = C.c_int32(-1)
    code = lib().spd_query_device_status(ws.data_ptr(), _stream_ptr(stream), C.byref(bad))
    return int(code), int(bad.value)


def spd_kernel_launch_count() -> int:
    return int(lib().spd_kernel_launch_count())


def spd_profile_begin(max_calls: int) -> None:
    _check(lib().spd_profile_begin(int(max_calls)), "spd_profile_begin")


def spd_profile_end() -> dict:
    """Returns {'calls', 'kernel_ms'}: calls recorded and their summed kernel time."""
    n, a = C.c_int32(0), C.c_double(0)
    _check(lib().spd_profile_end(C.byref(n), C.byref(a)), "spd_profile_end")
    return dict(calls=int(n.value), kernel_ms=a.value)


STATIC_WS_BYTES = 16 << 20


def spd_decode_step_static(shape, q, priv, pub, out, wait_and_check=True, stream=None) -> Tuple[int, int]:
    """The fused decode step with the workspace held inside the library (nothing is allocated).

    For callers that cannot allocate device memory; the shape must need at most STATIC_WS_BYTES of
    workspace.  Returns (status, first flagged user or -1); status is SPD_OK when not waiting.
    Raises SpdError for host-side rejections such as a shape beyond the limit."""
    a, b = paged_kv(priv), paged_kv(pub)
    bad = C.c_int32(-1)
    code = lib().spd_decode_step_static(C.byref(shape), q.data_ptr(), C.byref(a), C.byref(b), out.data_ptr(),
                                        _dtype_code(out.dtype), 1 if wait_and_check else 0, C.byref(bad),
                                        _stream_ptr(stream))
    if code not in _DEVICE_CODES:
        raise SpdError(code, "spd_decode_step_static")
    return int(code), int(bad.value)


def spd_append_kv(shape, k_new, v_new, part, ws, stream=None) -> None:
    """Append one token per user to the partition `part` (its pools and seq_lens are updated in place)."""
    assert k_new.is_contiguous() and v_new.is_contiguous()
    _check(lib().spd_append_kv(C.byref(shape), k_new.data_ptr(), v_new.data_ptr(), part.k_pool.data_ptr(),
                               part.v_pool.data_ptr(), int(part.k_pool.shape[0]), part.page_indptr.data_ptr(),
                               _ptr(part.page_indices), part.seq_lens.data_ptr(), ws.data_ptr(), ws.numel(),
                               _stream_ptr(stream)), "spd_append_kv")


def spd_decode_step_append(shape, q, k_new, v_new, priv, pub, out, ws, plan=SPD_PLAN_PER_CALL, stream=None) -> None:
    """The append of the new token's rows to `pub` (pools and seq_lens updated in place) and the fused decode step
    over the grown cache, in one launch."""
    assert k_new.is_contiguous() and v_new.is_contiguous()
    a, b = paged_kv(priv), paged_kv(pub)
    _check(lib().spd_decode_step_append(C.byref(shape), q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), C.byref(a),
                                        C.byref(b), out.data_ptr(), _dtype_code(out.dtype), int(plan), ws.data_ptr(),
                                        ws.numel(), _stream_ptr(stream)), "spd_decode_step_append")


def spd_service_attn_merge_append(shape, q, k_new, v_new, pub, partial_in, out, ws, plan=SPD_PLAN_PER_CALL, stream=None) -> None:
    """The service call with the append at its head: `pub` grows by the new token (pools and seq_lens updated in
    place), its partial is merged with `partial_in` and the attention output written, in one launch."""
    assert k_new.is_contiguous() and v_new.is_contiguous()
    kv = paged_kv(pub)
    part = Partial(partial_in[0].data_ptr(), partial_in[1].data_ptr(), partial_in[2].data_ptr())
    _check(lib().spd_service_attn_merge_append(C.byref(shape), q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), C.byref(kv),
                                               part, out.data_ptr(), _dtype_code(out.dtype), int(plan), ws.data_ptr(),
                                               ws.numel(), _stream_ptr(stream)), "spd_service_attn_merge_append")


def spd_token_step(shape, layers, ws, stream=None, same_lengths=False) -> None:
    """layers: a sequence of (q, k_new, v_new, priv, pub, out) per layer; appends to each pub and runs each decode step.
    same_lengths: every layer's lengths equal layer 0's, so its plan is derived once and reused."""
    arr = (Layer * len(layers))()
    for i, (q, k_new, v_new, priv, pub, out) in enumerate(layers):
        assert q.is_contiguous() and k_new.is_contiguous() and v_new.is_contiguous() and out.is_contiguous()
        arr[i] = Layer(q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), paged_kv(priv), paged_kv(pub), out.data_ptr())
    _check(lib().spd_token_step(C.byref(shape), len(layers), arr, _dtype_code(layers[0][5].dtype),
                                1 if same_lengths else 0, ws.data_ptr(), ws.numel(), _stream_ptr(stream)), "spd_token_step")


def _watch(tok_lo, tok_hi, out) -> Watch:
    assert tok_lo.dtype == torch.int32 and tok_hi.dtype == torch.int32 and out.dtype == torch.float32
    return Watch(tok_lo.data_ptr(), tok_hi.data_ptr(), out.data_ptr())


def spd_partial_attn_watch(shape, q, priv, out, tok_lo, tok_hi, watch_out, ws, stream=None) -> None:
    kv, w = paged_kv(priv), _watch(tok_lo, tok_hi, watch_out)
    part = Partial(out[0].data_ptr(), out[1].data_ptr(), out[2].data_ptr())
    _check(lib().spd_partial_attn_watch(C.byref(shape), q.data_ptr(), C.byref(kv), part, C.byref(w), ws.data_ptr(),
                                        ws.numel(), _stream_ptr(stream)), "spd_partial_attn_watch")


def spd_decode_step_watch(shape, q, priv, pub, out, tok_lo, tok_hi, watch_out, ws, stream=None) -> None:
    a, b, w = paged_kv(priv), paged_kv(pub), _watch(tok_lo, tok_hi, watch_out)
    _check(lib().spd_decode_step_watch(C.byref(shape), q.data_ptr(), C.byref(a), C.byref(b), out.data_ptr(),
                                       _dtype_code(out.dtype), C.byref(w), ws.data_ptr(), ws.numel(),
                                       _stream_ptr(stream)), "spd_decode_step_watch")


def spd_watch_alarm(mass, threshold: float, head_mask=None):
    """mass: float32 HOST tensor [batch, heads] from a *_watch call; head_mask: optional bool/uint8 [heads].
    Returns (alarm int32 [batch], score float32 [batch]): score = mean watched mass over the selected heads,
    alarm = 1 where it is below the threshold."""
    assert mass.device.type == "cpu" and mass.dtype == torch.float32 and mass.is_contiguous() and mass.dim() == 2
    B, H = mass.shape
    alarm = torch.zeros(B, dtype=torch.int32)
    score = torch.zeros(B, dtype=torch.float32)
    hm = None if head_mask is None else head_mask.to(torch.uint8).contiguous()
    _check(lib().spd_watch_alarm(mass.data_ptr(), B, H, None if hm is None else hm.data_ptr(), float(threshold),
                                 alarm.data_ptr(), score.data_ptr()), "spd_watch_alarm")
    return alarm, score


def spd_set_bf16_math(path: int) -> None:
    """0 = tensor cores (default), 1 = FMA pipes (comparison arm); process-wide."""
    _check(lib().spd_set_bf16_math(int(path)), "spd_set_bf16_math")


def spd_set_split(min_tiles_per_share: int = 0, uniform_shares: bool = False) -> None:
    """How the tile stream is cut from now on, process-wide: fewest tiles per share (0 = default) and whether
    every CTA weighs the same (the measured rates are ignored; results become repeatable bit for bit)."""
    _check(lib().spd_set_split(int(min_tiles_per_share), 1 if uniform_shares else 0), "spd_set_split")


def spd_set_programmatic_launch(on: bool) -> None:
    _check(lib().spd_set_programmatic_launch(1 if on else 0), "spd_set_programmatic_launch")


def spd_debug_read_plan(ws, which: int = 2, stream=None, capacity: int = 256 * 16 + 1):
    """(tiles, shares, bnd) of the last derived plan of kind `which` (0 private only, 1 public only, 2 both)."""
    T, A = C.c_int32(0), C.c_int32(0)
    bnd = (C.c_int32 * capacity)()
    _check(lib().spd_debug_read_plan(ws.data_ptr(), int(which), _stream_ptr(stream), C.byref(T), C.byref(A), bnd, capacity),
           "spd_debug_read_plan")
    n = min(capacity, A.value + 1)
    return int(T.value), int(A.value), [int(bnd[i]) for i in range(n)]


def spd_debug_sm_moves(ws, stream=None) -> Tuple[int, int]:
    """(launches that could compare, CTAs that ran on another SM than the same CTA index one launch earlier)."""
    a, b = C.c_int64(0), C.c_int64(0)
    _check(lib().spd_debug_sm_moves(ws.data_ptr(), _stream_ptr(stream), C.byref(a), C.byref(b)), "spd_debug_sm_moves")
    return int(a.value), int(b.value)


def spd_set_prefill_rows(rows: int) -> None:
    """Query rows per prefill CTA: 0 = chosen per call from the mean prompt length (default), 128 or 256; process-wide."""
    _check(lib().spd_set_prefill_rows(int(rows)), "spd_set_prefill_rows")


def spd_merge_partials(shape, parts, out, stream=None) -> None:
    """parts: a sequence of (o, m, l) tensor triples; writes the merged, normalised output."""
    arr = (Partial * len(parts))(*[Partial(o.data_ptr(), m.data_ptr(), l.data_ptr()) for o, m, l in parts])
    _check(lib().spd_merge_partials(C.byref(shape), len(parts), arr, out.data_ptr(), _dtype_code(out.dtype),
                                    _stream_ptr(stream)), "spd_merge_partials")


def spd_prefill_attn(shape, q, k, v, tok_indptr, part, out, ws, stream=None) -> None:
    """Causal attention over the prompts (q [T,Hq,D], k, v [T,Hkv,D], tok_indptr int32 [B+1]) into `out`
    [T,Hq,D]; the prompts' K/V rows go into the partition `part` (pools and seq_lens updated in place)."""
    for t in (q, k, v, out):
        assert t.is_contiguous()
    assert tok_indptr.dtype == torch.int32
    _check(lib().spd_prefill_attn(C.byref(shape), int(q.shape[0]), _ptr(q), _ptr(k), _ptr(v), tok_indptr.data_ptr(),
                                  part.k_pool.data_ptr(), part.v_pool.data_ptr(), int(part.k_pool.shape[0]),
                                  part.page_indptr.data_ptr(), _ptr(part.page_indices), part.seq_lens.data_ptr(),
                                  _ptr(out), _dtype_code(out.dtype), ws.data_ptr(), ws.numel(), _stream_ptr(stream)),
           "spd_prefill_attn")

"""ctypes binding of libpie_b200.so: argument marshalling only.

Every function has the name and meaning of the C entry point declared in include/pie_b200.h.
Tensors are torch tensors (device memory and streams come from torch); index arrays are numpy
int32.  There is no fallback: if the shared library cannot be loaded the import fails.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

PIE_DTYPE_BF16, PIE_DTYPE_F32 = 0, 1
PIE_PLAN_FORCE_SIMPLE, PIE_PLAN_NO_TENSOR_TILES, PIE_PLAN_NO_CASCADE, PIE_PLAN_CASCADE_ALWAYS, PIE_PLAN_MASK_BITS = 1, 2, 4, 8, 16
PIE_OK = 0
PIE_ERR_INVALID, PIE_ERR_NO_PAGES, PIE_ERR_BAD_PAGE, PIE_ERR_CONFLICT = -1, -2, -3, -4
PIE_ERR_BATCH_TOO_LARGE, PIE_ERR_MASK, PIE_ERR_CUDA, PIE_ERR_NO_DEVICE = -5, -6, -7, -8
PIE_ERR_UNSUPPORTED, PIE_ERR_DEVICE_TIMEOUT = -9, -10


class pie_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "num_pages", "page_size", "num_q_heads", "num_kv_heads", "head_dim", "dtype",
        "max_requests", "max_query_tokens", "device")] + [("rope_theta", C.c_float)]


class pie_batch_desc(C.Structure):
    _fields_ = [("num_requests", C.c_int32), ("qo_indptr", C.c_void_p), ("page_indptr", C.c_void_p),
                ("page_indices", C.c_void_p), ("last_page_len", C.c_void_p), ("mask_indptr", C.c_void_p),
                ("mask", C.c_void_p), ("flags", C.c_uint32), ("positions", C.c_void_p), ("out_len", C.c_void_p),
                ("no_store", C.c_void_p)]


class pie_plan_info(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "num_requests", "num_query_tokens", "num_split_items", "num_tile_items", "num_simple_rows",
        "num_merge_groups", "launches", "side_by_side_sms", "split_unit_kv_heads", "reserved0")] + [
        (n, C.c_int64) for n in ("kept_pages", "mask_words", "workspace_bytes")]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


def _load():
    path = _build.LIB
    if not _build.is_current():
        _build.build()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing and could not be built: no CUDA path, no fallback")
    lib = C.CDLL(path)
    vp, i32 = C.c_void_p, C.c_int32
    sig = {
        "pie_strerror": (C.c_char_p, [C.c_int]),
        "pie_last_cuda_error": (C.c_char_p, [vp]),
        "pie_create": (C.c_int, [C.POINTER(pie_config), C.POINTER(vp)]),
        "pie_destroy": (C.c_int, [vp]),
        "pie_alloc_kvpages": (C.c_int, [vp, i32, vp]),
        "pie_dealloc_kvpages": (C.c_int, [vp, i32, vp]),
        "pie_num_free_kvpages": (C.c_int, [vp, C.POINTER(i32)]),
        "pie_mask_kvpage": (C.c_int, [vp, i32, vp, vp]),
        "pie_kvpage_write": (C.c_int, [vp, i32, vp, vp, vp, C.c_int, vp]),
        "pie_kvpage_read": (C.c_int, [vp, i32, vp, vp, vp, C.c_int, vp]),
        "pie_copy_kvpage": (C.c_int, [vp, i32, vp, vp, vp, vp, vp, vp]),
        "pie_plan_forward": (C.c_int, [vp, C.POINTER(pie_batch_desc), vp, C.POINTER(vp)]),
        "pie_plan_destroy": (C.c_int, [vp]),
        "pie_plan_get_info": (C.c_int, [vp, C.POINTER(pie_plan_info)]),
        "pie_plan_debug_read": (C.c_int, [vp, C.c_int, vp, C.c_int64, C.POINTER(C.c_int64)]),
        "pie_forward": (C.c_int, [vp, vp, vp, vp, vp, vp, vp, vp]),
        "pie_forward_host": (C.c_int, [vp, C.POINTER(pie_batch_desc), vp, vp, vp, vp, vp, vp]),
        "pie_get_last_device_status": (C.c_int, [vp, vp, C.POINTER(C.c_int)]),
        "pie_forward_static_scratch": (C.c_int, [vp, C.POINTER(pie_batch_desc), vp, vp, vp, vp, vp, vp]),
        "pie_debug_bounded_wait": (C.c_int, [vp, vp]),
        "pie_get_next_dist": (C.c_int, [vp, vp, i32, i32, i32, C.c_int64, i32, vp, vp, vp]),
        "pie_set_option": (C.c_int, [vp, C.c_int, C.c_int]),
        "pie_sched_create": (C.c_int, [i32, C.POINTER(vp)]),
        "pie_sched_destroy": (C.c_int, [vp]),
        "pie_sched_create_queue": (C.c_int, [vp, i32, C.POINTER(i32)]),
        "pie_sched_set_queue_priority": (C.c_int, [vp, i32, i32]),
        "pie_sched_submit": (C.c_int, [vp, i32, i32, i32, vp, C.c_int64, C.c_int64]),
        "pie_sched_pending": (C.c_int, [vp, C.POINTER(i32)]),
        "pie_sched_next_batch": (C.c_int, [vp, C.POINTER(i32), i32, vp, vp, C.POINTER(i32)]),
        "pie_set_kernel_timing": (C.c_int, [vp, C.c_int]),
        "pie_get_kernel_times": (C.c_int, [vp, vp, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)          # AttributeError here = the library lacks a declared symbol
        fn.restype, fn.argtypes = res, args
    return lib


lib = _load()
LIB_PATH = _build.LIB


class PieError(RuntimeError):
    def __init__(self, status, ctx=None):
        self.status = status
        msg = lib.pie_strerror(status).decode()
        if status == PIE_ERR_CUDA and ctx:
            msg += ": " + lib.pie_last_cuda_error(ctx).decode()
        super().__init__(f"pie status {status}: {msg}")


def _check(status, ctx=None):
    if status != PIE_OK:
        raise PieError(status, ctx)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _ptr(a):
    """Address of a numpy array, a torch tensor, or None."""
    if a is None:
        return None
    if isinstance(a, np.ndarray):
        return a.ctypes.data
    return a.data_ptr()


def _stream(stream):
    if stream is not None:
        return stream
    import torch
    return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else None


# ------------------------------------------------------------------ functions, one per C entry
def pie_strerror(status):
    return lib.pie_strerror(status).decode()


def pie_create(num_pages, page_size, num_q_heads, num_kv_heads, head_dim, dtype, max_requests,
               max_query_tokens, device=0, rope_theta=0.0):
    dt = {"bf16": PIE_DTYPE_BF16, "f32": PIE_DTYPE_F32}.get(dtype, dtype)
    cfg = pie_config(num_pages, page_size, num_q_heads, num_kv_heads, head_dim, dt, max_requests,
                     max_query_tokens, device, rope_theta)
    ctx = C.c_void_p()
    _check(lib.pie_create(C.byref(cfg), C.byref(ctx)))
    return ctx


def pie_destroy(ctx):
    _check(lib.pie_destroy(ctx))


def pie_alloc_kvpages(ctx, n):
    out = np.empty(n, dtype=np.int32)
    _check(lib.pie_alloc_kvpages(ctx, n, out.ctypes.data), ctx)
    return out


def pie_dealloc_kvpages(ctx, ids):
    ids = _i32(ids)
    _check(lib.pie_dealloc_kvpages(ctx, len(ids), ids.ctypes.data), ctx)


def pie_num_free_kvpages(ctx):
    out = C.c_int32()
    _check(lib.pie_num_free_kvpages(ctx, C.byref(out)), ctx)
    return out.value


def _on_device(t):
    return 0 if t is None or isinstance(t, np.ndarray) or not t.is_cuda else 1


def pie_kvpage_write(ctx, ids, K, V, stream=None):
    ids = _i32(ids)
    _check(lib.pie_kvpage_write(ctx, len(ids), ids.ctypes.data, _ptr(K), _ptr(V), _on_device(K), _stream(stream)), ctx)


def pie_kvpage_read(ctx, ids, K, V, stream=None):
    ids = _i32(ids)
    _check(lib.pie_kvpage_read(ctx, len(ids), ids.ctypes.data, _ptr(K), _ptr(V), _on_device(K), _stream(stream)), ctx)


def pie_copy_kvpage(ctx, src, dst, src_off, dst_off, ntok, stream=None):
    a = [_i32(x) for x in (src, dst, src_off, dst_off, ntok)]
    _check(lib.pie_copy_kvpage(ctx, len(a[0]), *[x.ctypes.data for x in a], _stream(stream)), ctx)


def _desc(qo_indptr, page_indptr, page_indices, last_page_len, mask_indptr, mask, flags, positions=None, out_len=None,
          no_store=None):
    keep = [_i32(qo_indptr), _i32(page_indptr), _i32(page_indices), _i32(last_page_len)]
    mi = None if mask_indptr is None else np.ascontiguousarray(mask_indptr, dtype=np.int64)
    if mask is not None and (flags & PIE_PLAN_MASK_BITS):
        mk = np.ascontiguousarray(mask, dtype=np.uint32)            # packed rows, mask_indptr counts words
    else:
        mk = None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8)
    ps = None if positions is None else _i32(positions)
    ol = None if out_len is None else _i32(out_len)
    ns = None if no_store is None else np.ascontiguousarray(no_store, dtype=np.uint8)
    keep += [mi, mk, ps, ol, ns]
    d = pie_batch_desc(len(keep[0]) - 1, keep[0].ctypes.data, keep[1].ctypes.data, keep[2].ctypes.data,
                       keep[3].ctypes.data, _ptr(mi), _ptr(mk), flags, _ptr(ps), _ptr(ol), _ptr(ns))
    return d, keep


def pie_plan_forward(ctx, qo_indptr, page_indptr, page_indices, last_page_len, mask_indptr=None,
                     mask=None, flags=0, stream=None, positions=None, out_len=None, no_store=None):
    d, keep = _desc(qo_indptr, page_indptr, page_indices, last_page_len, mask_indptr, mask, flags, positions, out_len, no_store)
    plan = C.c_void_p()
    _check(lib.pie_plan_forward(ctx, C.byref(d), _stream(stream), C.byref(plan)), ctx)
    return plan


def pie_plan_destroy(plan):
    _check(lib.pie_plan_destroy(plan))


def pie_plan_get_info(plan):
    info = pie_plan_info()
    _check(lib.pie_plan_get_info(plan, C.byref(info)))
    return info.as_dict()


def pie_plan_debug_read(plan, which):
    n = C.c_int64()
    _check(lib.pie_plan_debug_read(plan, which, None, 0, C.byref(n)))
    out = np.empty(n.value // 4, dtype=np.uint32 if which == 0 else np.int32)
    if n.value:
        _check(lib.pie_plan_debug_read(plan, which, out.ctypes.data, n.value, C.byref(n)))
    return out


def pie_forward(ctx, plan, q, k_new, v_new, out, lse, stream=None):
    _check(lib.pie_forward(ctx, plan, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _ptr(lse), _stream(stream)), ctx)


def pie_forward_host(ctx, qo_indptr, page_indptr, page_indices, last_page_len, q, k_new, v_new, out,
                     lse, mask_indptr=None, mask=None, flags=0, stream=None, out_len=None, no_store=None):
    d, keep = _desc(qo_indptr, page_indptr, page_indices, last_page_len, mask_indptr, mask, flags, None, out_len, no_store)
    _check(lib.pie_forward_host(ctx, C.byref(d), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _ptr(lse),
                                _stream(stream)), ctx)


def pie_get_next_dist(ctx, logits, top_k, out_ids, out_probs, stream=None):
    """logits: 2-D torch tensor on the device (bf16 or fp32, rows may be strided); out_ids int32 / out_probs
    fp32 tensors [n_rows, top_k]."""
    import torch
    dtype = {torch.bfloat16: PIE_DTYPE_BF16, torch.float32: PIE_DTYPE_F32}[logits.dtype]
    assert logits.dim() == 2 and logits.stride(1) == 1
    _check(lib.pie_get_next_dist(ctx, _ptr(logits), dtype, logits.shape[0], logits.shape[1], logits.stride(0), top_k,
                                 _ptr(out_ids), _ptr(out_probs), _stream(stream)), ctx)


def pie_debug_bounded_wait(ctx, stream=None):
    _check(lib.pie_debug_bounded_wait(ctx, _stream(stream)), ctx)


def pie_get_last_device_status(ctx, stream=None):
    out = C.c_int()
    _check(lib.pie_get_last_device_status(ctx, _stream(stream), C.byref(out)), ctx)
    return out.value


KERNEL_KINDS = ("append", "simple", "split", "tiles", "merge", "copy")


def pie_set_kernel_timing(ctx, enable):
    _check(lib.pie_set_kernel_timing(ctx, int(bool(enable))), ctx)


def pie_get_kernel_times(ctx):
    """{kind: (total ms, launches)} of the kernels recorded since timing was enabled / last read."""
    ms = np.zeros(len(KERNEL_KINDS), dtype=np.float32)
    n = np.zeros(len(KERNEL_KINDS), dtype=np.int32)
    _check(lib.pie_get_kernel_times(ctx, ms.ctypes.data, n.ctypes.data), ctx)
    return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(KERNEL_KINDS)}


def pie_last_cuda_error(ctx):
    return lib.pie_last_cuda_error(ctx).decode()


PIE_STATIC_SCRATCH_BYTES = 16 * 1024 * 1024


def pie_forward_static_scratch(ctx, qo_indptr, page_indptr, page_indices, last_page_len, q, k_new, v_new,
                               out, lse, mask_indptr=None, mask=None, flags=0, stream=None, out_len=None, no_store=None):
    """forward for callers that cannot allocate device memory: plan arrays and split partials go
    to the library's fixed device array (at most PIE_STATIC_SCRATCH_BYTES, else
    PIE_ERR_BATCH_TOO_LARGE).  Tensors are device tensors; calls must not overlap on the GPU."""
    d, keep = _desc(qo_indptr, page_indptr, page_indices, last_page_len, mask_indptr, mask, flags, None, out_len, no_store)
    _check(lib.pie_forward_static_scratch(ctx, C.byref(d), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out),
                                          _ptr(lse), _stream(stream)), ctx)


PIE_OPT_SPLIT_SMS, PIE_OPT_TILE_SMS, PIE_OPT_OVERLAP, PIE_OPT_NO_FUSION = 0, 1, 2, 3


def pie_set_option(ctx, option, value):
    _check(lib.pie_set_option(ctx, option, value), ctx)


def pie_mask_kvpage(ctx, ids, masks):
    """Persistent per-page token masks: bit s of masks[k] set = slot s of page ids[k] visible."""
    ids = _i32(ids)
    m = np.ascontiguousarray(masks, dtype=np.uint32)
    assert len(m) == len(ids)
    _check(lib.pie_mask_kvpage(ctx, len(ids), ids.ctypes.data, m.ctypes.data), ctx)


# ------------------------------------------------------------------ batch scheduler (host only)
def pie_sched_create(max_batch_calls):
    s = C.c_void_p()
    _check(lib.pie_sched_create(max_batch_calls, C.byref(s)))
    return s


def pie_sched_destroy(s):
    _check(lib.pie_sched_destroy(s))


def pie_sched_create_queue(s, priority=0):
    q = C.c_int32()
    _check(lib.pie_sched_create_queue(s, priority, C.byref(q)))
    return q.value


def pie_sched_set_queue_priority(s, queue, priority):
    _check(lib.pie_sched_set_queue_priority(s, queue, priority))


def pie_sched_submit(s, queue, call_type, write_pages, arrival_ns, tag):
    w = _i32(write_pages)
    _check(lib.pie_sched_submit(s, queue, call_type, len(w), w.ctypes.data, arrival_ns, tag))


def pie_sched_pending(s):
    n = C.c_int32()
    _check(lib.pie_sched_pending(s, C.byref(n)))
    return n.value


def pie_sched_next_batch(s, cap=1 << 20):
    """(type, [tags], [queue ids]) of the next batch; (-1, [], []) when nothing is pending."""
    cap = min(cap, 1 << 20)
    tags = np.zeros(cap, dtype=np.int64)
    qs = np.zeros(cap, dtype=np.int32)
    t, n = C.c_int32(), C.c_int32()
    _check(lib.pie_sched_next_batch(s, C.byref(t), cap, tags.ctypes.data, qs.ctypes.data, C.byref(n)))
    return t.value, tags[:n.value].tolist(), qs[:n.value].tolist()

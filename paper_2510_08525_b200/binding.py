"""Thin ctypes binding of librlkv: argument marshalling only, one Python function per C entry point.

Every function takes the same arguments as its C counterpart in ``include/rlkv.h`` (torch tensors
or raw integer addresses for pointers, a torch stream or ``None`` for the stream) and raises
``RlkvError`` on a negative return code.  Nothing here computes anything: all arithmetic runs in the
CUDA kernels of the library.  Importing this module fails loudly if the library cannot be loaded;
there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "librlkv.so")

RLKV_OK, RLKV_EINVAL, RLKV_EFULL, RLKV_EEMPTY, RLKV_ENOMEM, RLKV_ECUDA, RLKV_EKERNEL = 0, -1, -2, -3, -4, -5, -6
RLKV_ESCRATCH = -7

# name -> (restype, argtypes); one entry per symbol declared in include/rlkv.h
_vp, _ci, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
SIGNATURES = {
    "rlkv_cache_size": (_ci, [_ci, _ci, _ci, _ci, _ci, _ci, _vp, _ci, _ci, ctypes.POINTER(_sz)]),
    "rlkv_cache_create": (_ci, [ctypes.POINTER(_vp), _ci, _ci, _ci, _ci, _ci, _ci, _vp, _ci, _ci, _vp, _sz]),
    "rlkv_cache_destroy": (_ci, [_vp]),
    "rlkv_cache_reset": (_ci, [_vp, _vp]),
    "rlkv_append": (_ci, [_vp, _ci, _vp, _vp, _vp]),
    "rlkv_prefill": (_ci, [_vp, _ci, _vp, _vp, _ci, _vp]),
    "rlkv_decode_attention": (_ci, [_vp, _ci, _vp, _vp, _vp]),
    "rlkv_decode_attention_static_scratch": (_ci, [_vp, _ci, _vp, _vp, _vp]),
    "rlkv_append_overlapped": (_ci, [_vp, _ci, _vp, _vp, _vp]),
    "rlkv_decode_attention_overlapped": (_ci, [_vp, _ci, _vp, _vp, _vp]),
    "rlkv_layer_step_overlapped": (_ci, [_vp, _ci, _vp, _vp, _vp, _vp, _vp]),
    "rlkv_debug_standin": (_ci, [_vp, _vp, _sz, _vp, _vp, _vp, _sz, _ci, _vp]),
    "rlkv_static_scratch_bytes": (_sz, []),
    "rlkv_set_output_bf16": (_ci, [_vp, _ci]),
    "rlkv_paged_set_output_bf16": (_ci, [_vp, _ci]),
    "rlkv_paged_set_step_mode": (_ci, [_vp, _ci]),
    "rlkv_decode_mixed_attention": (_ci, [_vp, _ci, _vp, _vp, _vp, _vp]),
    "rlkv_step": (_ci, [_vp, _vp, _vp, _vp, _vp, _vp]),
    "rlkv_step_host": (_ci, [_vp, _vp, _vp, _vp, _vp, _vp]),
    "rlkv_length": (_ci, [_vp, _ci, ctypes.POINTER(_ci)]),
    "rlkv_step_bytes": (_ci, [_vp, _ci, ctypes.POINTER(ctypes.c_uint64)]),
    "rlkv_debug_export_head": (_ci, [_vp, _ci, _ci, _ci, _vp, _vp, ctypes.POINTER(_ci), _vp]),
    "rlkv_kernel_status": (_ci, [_vp, ctypes.POINTER(_ci)]),
    "rlkv_launch_count": (_ci, [_vp, ctypes.POINTER(ctypes.c_uint64)]),
    "rlkv_set_decode_config": (_ci, [_vp, _ci, _ci, _ci, _ci]),
    "rlkv_debug_trace": (_ci, [_vp, _ci, _vp, ctypes.POINTER(_ci)]),
    "rlkv_debug_schedule": (_ci, [_ci, _ci, _ci, _ci, _ci, _ci, _ci, ctypes.POINTER(_ci), ctypes.POINTER(_ci), _vp, _vp, _ci]),
    "rlkv_set_step_mode": (_ci, [_vp, _ci]),
    "rlkv_debug_step_plan": (_ci, [_ci, _ci, _vp, _vp, _vp]),
    "rlkv_debug_claim_order": (_ci, [_ci, _ci, _ci, _ci, _ci, _ci, _ci, _vp, _ci]),
    "rlkv_debug_read_bandwidth": (_ci, [_vp, _sz, _ci, ctypes.POINTER(ctypes.c_float)]),
    "rlkv_strerror": (ctypes.c_char_p, [_ci]),
    "rlkv_paged_size": (_ci, [_ci, _ci, _ci, _ci, _ci, _ci, _ci, _vp, _ci, _ci, ctypes.POINTER(_sz)]),
    "rlkv_paged_create": (_ci, [ctypes.POINTER(_vp), _ci, _ci, _ci, _ci, _ci, _ci, _ci, _vp, _ci, _ci, _vp, _sz]),
    "rlkv_paged_size_fp8": (_ci, [_ci, _ci, _ci, _ci, _ci, _ci, _ci, _vp, _ci, _ci, ctypes.POINTER(_sz)]),
    "rlkv_cache_size_fp8": (_ci, [_ci, _ci, _ci, _ci, _ci, _ci, _vp, _ci, _ci, ctypes.POINTER(_sz)]),
    "rlkv_cache_create_fp8": (_ci, [ctypes.POINTER(_vp), _ci, _ci, _ci, _ci, _ci, _ci, _vp, _ci, _ci, _vp, _vp, _vp, _sz]),
    "rlkv_paged_create_fp8": (_ci, [ctypes.POINTER(_vp), _ci, _ci, _ci, _ci, _ci, _ci, _ci, _vp, _ci, _ci, _vp, _vp, _vp, _sz]),
    "rlkv_paged_destroy": (_ci, [_vp]),
    "rlkv_paged_seq_open": (_ci, [_vp, ctypes.POINTER(_ci)]),
    "rlkv_paged_seq_close": (_ci, [_vp, _ci]),
    "rlkv_paged_append": (_ci, [_vp, _ci, _vp, _ci, _vp, _vp, _vp]),
    "rlkv_paged_prefill": (_ci, [_vp, _ci, _ci, _vp, _vp, _ci, _vp]),
    "rlkv_paged_decode_attention": (_ci, [_vp, _ci, _vp, _ci, _vp, _vp, _vp]),
    "rlkv_paged_step": (_ci, [_vp, _vp, _ci, _vp, _vp, _vp, _vp, _vp]),
    "rlkv_paged_length": (_ci, [_vp, _ci, _ci, ctypes.POINTER(_ci)]),
    "rlkv_paged_pages": (_ci, [_vp, ctypes.POINTER(_ci), ctypes.POINTER(_ci)]),
    "rlkv_paged_step_bytes": (_ci, [_vp, _ci, _vp, _ci, ctypes.POINTER(ctypes.c_uint64)]),
    "rlkv_paged_debug_export_head": (_ci, [_vp, _ci, _ci, _ci, _vp, _vp, ctypes.POINTER(_ci), _vp]),
    "rlkv_paged_kernel_status": (_ci, [_vp, ctypes.POINTER(_ci)]),
    "rlkv_debug_paged_schedule": (_ci, [_vp, _ci, _ci, _ci, _ci, _ci, _ci, ctypes.POINTER(_ci), _vp, _vp, _vp]),
}


class RlkvError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"librlkv error {code}: {text}")
        self.code = code


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2510_08525_b200.build` "
            "(nvcc, sm_100a).  There is no fallback implementation.")
    lib = ctypes.CDLL(LIB_PATH)
    for name, (res, args) in SIGNATURES.items():
        fn = getattr(lib, name)  # AttributeError if the library does not export a declared symbol
        fn.restype, fn.argtypes = res, args
    return lib


lib = _load()


def _check(rc: int) -> None:
    if rc != 0:
        raise RlkvError(rc, lib.rlkv_strerror(rc).decode())


def _ptr(x) -> int:
    """Address of a torch tensor / numpy array, or the integer itself."""
    if x is None:
        return 0
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        if not x.flags["C_CONTIGUOUS"]:
            raise ValueError("array must be contiguous")
        return x.ctypes.data
    if not x.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return x.data_ptr()


def _stream(s) -> int:
    if s is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(s, int):
        return s
    return s.cuda_stream


def _mask(head_is_full) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(head_is_full, dtype=np.uint8).reshape(-1))


def rlkv_cache_size(layers, kv_heads, q_heads, head_dim, batch, max_len, head_is_full, sink, window) -> int:
    m = _mask(head_is_full)
    if m.size != layers * kv_heads:
        raise ValueError("head_is_full must have layers*kv_heads entries")
    out = _sz(0)
    _check(lib.rlkv_cache_size(layers, kv_heads, q_heads, head_dim, batch, max_len, m.ctypes.data, sink, window,
                               ctypes.byref(out)))
    return int(out.value)


def rlkv_cache_create(layers, kv_heads, q_heads, head_dim, batch, max_len, head_is_full, sink, window,
                      device_buf=None, device_buf_bytes=0) -> int:
    """Returns the opaque cache handle (an integer address)."""
    m = _mask(head_is_full)
    if m.size != layers * kv_heads:
        raise ValueError("head_is_full must have layers*kv_heads entries")
    handle = _vp(0)
    _check(lib.rlkv_cache_create(ctypes.byref(handle), layers, kv_heads, q_heads, head_dim, batch, max_len,
                                 m.ctypes.data, sink, window, _ptr(device_buf), device_buf_bytes))
    return int(handle.value)


def rlkv_cache_size_fp8(layers, kv_heads, q_heads, head_dim, batch, max_len, head_is_full, sink, window) -> int:
    m = _mask(head_is_full)
    if m.size != layers * kv_heads:
        raise ValueError("head_is_full must have layers*kv_heads entries")
    out = _sz(0)
    _check(lib.rlkv_cache_size_fp8(layers, kv_heads, q_heads, head_dim, batch, max_len, m.ctypes.data, sink, window,
                                   ctypes.byref(out)))
    return int(out.value)


def rlkv_cache_create_fp8(layers, kv_heads, q_heads, head_dim, batch, max_len, head_is_full, sink, window,
                          k_scale, v_scale, device_buf=None, device_buf_bytes=0) -> int:
    m = _mask(head_is_full)
    ks = np.ascontiguousarray(np.asarray(k_scale, dtype=np.float32).reshape(-1))
    vs = np.ascontiguousarray(np.asarray(v_scale, dtype=np.float32).reshape(-1))
    if m.size != layers * kv_heads or ks.size != m.size or vs.size != m.size:
        raise ValueError("head_is_full, k_scale and v_scale must have layers*kv_heads entries")
    handle = _vp(0)
    _check(lib.rlkv_cache_create_fp8(ctypes.byref(handle), layers, kv_heads, q_heads, head_dim, batch, max_len,
                                     m.ctypes.data, sink, window, ks.ctypes.data, vs.ctypes.data,
                                     _ptr(device_buf), device_buf_bytes))
    return int(handle.value)


def rlkv_cache_destroy(cache) -> None:
    _check(lib.rlkv_cache_destroy(cache))


def rlkv_cache_reset(cache, stream=None) -> None:
    _check(lib.rlkv_cache_reset(cache, _stream(stream)))


def rlkv_append(cache, layer, k, v, stream=None) -> None:
    _check(lib.rlkv_append(cache, layer, _ptr(k), _ptr(v), _stream(stream)))


def rlkv_prefill(cache, layer, k, v, n_tokens, stream=None) -> None:
    _check(lib.rlkv_prefill(cache, layer, _ptr(k), _ptr(v), n_tokens, _stream(stream)))


def rlkv_decode_attention(cache, layer, q, out, stream=None) -> None:
    _check(lib.rlkv_decode_attention(cache, layer, _ptr(q), _ptr(out), _stream(stream)))


def rlkv_append_overlapped(cache, layer, k, v, stream=None) -> None:
    _check(lib.rlkv_append_overlapped(cache, layer, _ptr(k), _ptr(v), _stream(stream)))


def rlkv_decode_attention_overlapped(cache, layer, q, out, stream=None) -> None:
    _check(lib.rlkv_decode_attention_overlapped(cache, layer, _ptr(q), _ptr(out), _stream(stream)))


def rlkv_layer_step_overlapped(cache, layer, k, v, q, out, stream=None) -> None:
    _check(lib.rlkv_layer_step_overlapped(cache, layer, _ptr(k), _ptr(v), _ptr(q), _ptr(out), _stream(stream)))


def rlkv_debug_standin(dst, src, nbytes, after, produce, produce_src, produce_bytes, overlap, stream=None) -> None:
    _check(lib.rlkv_debug_standin(_ptr(dst), _ptr(src), int(nbytes), _ptr(after), _ptr(produce), _ptr(produce_src),
                                  int(produce_bytes), int(overlap), _stream(stream)))


def rlkv_decode_attention_static_scratch(cache, layer, q, out, stream=None) -> None:
    """rlkv_decode_attention with the kernel's work area in the library's static device array;
    the call allocates nothing (see include/rlkv.h for who needs that and for the limits)."""
    _check(lib.rlkv_decode_attention_static_scratch(cache, layer, _ptr(q), _ptr(out), _stream(stream)))


def rlkv_static_scratch_bytes() -> int:
    return int(lib.rlkv_static_scratch_bytes())


def rlkv_decode_mixed_attention(cache, layer, q, alpha, out, stream=None) -> None:
    """Eq. 1: alpha[h] * full attention + (1 - alpha[h]) * sink+window attention over a layer whose
    heads are all full.  alpha: device fp32 [kv_heads]."""
    _check(lib.rlkv_decode_mixed_attention(cache, layer, _ptr(q), _ptr(alpha), _ptr(out), _stream(stream)))


def rlkv_set_output_bf16(cache, on) -> None:
    _check(lib.rlkv_set_output_bf16(cache, int(bool(on))))


def rlkv_paged_set_step_mode(cache, mode) -> None:
    _check(lib.rlkv_paged_set_step_mode(cache, int(mode)))


def rlkv_paged_set_output_bf16(cache, on) -> None:
    _check(lib.rlkv_paged_set_output_bf16(cache, int(bool(on))))


def rlkv_step(cache, k, v, q, out, stream=None) -> None:
    _check(lib.rlkv_step(cache, _ptr(k), _ptr(v), _ptr(q), _ptr(out), _stream(stream)))


def rlkv_step_host(cache, k_host, v_host, q_host, out_host, stream=None) -> None:
    _check(lib.rlkv_step_host(cache, _ptr(k_host), _ptr(v_host), _ptr(q_host), _ptr(out_host), _stream(stream)))


def rlkv_length(cache, layer) -> int:
    out = _ci(0)
    _check(lib.rlkv_length(cache, layer, ctypes.byref(out)))
    return int(out.value)


def rlkv_step_bytes(cache, layer) -> int:
    out = ctypes.c_uint64(0)
    _check(lib.rlkv_step_bytes(cache, layer, ctypes.byref(out)))
    return int(out.value)


def rlkv_debug_export_head(cache, layer, batch_row, kv_head, rows, head_dim):
    """rows = max_len for a full head, sink+window for a compressed head.
    Returns (k uint16[rows][D], v uint16[rows][D], token_of_slot int32[rows])."""
    k = np.empty((rows, head_dim), dtype=np.uint16)
    v = np.empty((rows, head_dim), dtype=np.uint16)
    tok = np.empty(rows, dtype=np.int32)
    got = _ci(0)
    _check(lib.rlkv_debug_export_head(cache, layer, batch_row, kv_head, k.ctypes.data, v.ctypes.data,
                                      ctypes.byref(got), tok.ctypes.data))
    if got.value != rows:
        raise ValueError(f"head has {got.value} rows, caller expected {rows}")
    return k, v, tok


def rlkv_kernel_status(cache) -> int:
    out = _ci(0)
    rc = lib.rlkv_kernel_status(cache, ctypes.byref(out))
    if rc not in (RLKV_OK, RLKV_EKERNEL):
        _check(rc)
    return int(out.value)


def rlkv_launch_count(cache) -> int:
    out = ctypes.c_uint64(0)
    _check(lib.rlkv_launch_count(cache, ctypes.byref(out)))
    return int(out.value)


def rlkv_set_decode_config(cache, ctas_per_sm=0, stages=0, consumer_groups=0, item_tiles=0) -> None:
    _check(lib.rlkv_set_decode_config(cache, ctas_per_sm, stages, consumer_groups, item_tiles))


def rlkv_debug_trace(cache, enable, read=False):
    """Switches the decode kernel's trace on or off; with read=True returns uint64[320][40] of the
    most recent launch (taken before the switch is applied)."""
    words = np.zeros((320, 40), dtype=np.uint64) if read else None
    ctas = _ci(0)
    _check(lib.rlkv_debug_trace(cache, int(enable), _ptr(words), ctypes.byref(ctas)))
    return words


def rlkv_set_step_mode(cache, mode) -> None:
    _check(lib.rlkv_set_step_mode(cache, int(mode)))


def rlkv_debug_schedule(full_units, tiles_full, comp_units, tiles_comp, ctas, item_tiles, tile_map=False, whole_step=False):
    """Returns (starts int32[n_items + 1], n_slots) and, with tile_map=True, also int32[T][4]:
    unit, tile in unit, run, partial record of every flat tile."""
    n, slots = _ci(0), _ci(0)
    args = (full_units, tiles_full, comp_units, tiles_comp, ctas, item_tiles, int(whole_step))
    _check(lib.rlkv_debug_schedule(*args, ctypes.byref(n), ctypes.byref(slots), None, None, 0))
    total = full_units * tiles_full + comp_units * tiles_comp
    starts = np.empty(n.value + 1, dtype=np.int32)
    tmap = np.empty((total, 4), dtype=np.int32) if tile_map else None
    _check(lib.rlkv_debug_schedule(*args, ctypes.byref(n), ctypes.byref(slots), starts.ctypes.data, _ptr(tmap),
                                   max(starts.size, total)))
    return (starts, int(slots.value), tmap) if tile_map else (starts, int(slots.value))


def rlkv_debug_read_bandwidth(buf, nbytes, launches=4) -> float:
    """Mean milliseconds of one read-only pass over nbytes of device memory at buf."""
    ms = ctypes.c_float(0)
    _check(lib.rlkv_debug_read_bandwidth(_ptr(buf), int(nbytes), int(launches), ctypes.byref(ms)))
    return float(ms.value)


def rlkv_debug_claim_order(full_units, tiles_full, comp_units, tiles_comp, ctas, item_tiles, n_items, whole_step=False):
    """int32[n_items]: the item handed to CTA k (k < ctas) / to the (k - ctas)-th claim."""
    order = np.zeros(n_items, dtype=np.int32)
    _check(lib.rlkv_debug_claim_order(full_units, tiles_full, comp_units, tiles_comp, ctas, item_tiles, int(whole_step),
                                      order.ctypes.data, n_items))
    return order


def rlkv_debug_step_plan(n_launches, follows_append=True):
    """Returns (overlap, dep_wait, scratch_copy), int32[n_launches] each."""
    arrs = [np.zeros(n_launches, dtype=np.int32) for _ in range(3)]
    _check(lib.rlkv_debug_step_plan(n_launches, int(follows_append), *[a.ctypes.data for a in arrs]))
    return tuple(arrs)


def rlkv_strerror(code: int) -> str:
    return lib.rlkv_strerror(code).decode()


# ---- the paged, ragged cache -------------------------------------------------------------------
def _slots(slots) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(slots, dtype=np.int32).reshape(-1))


def rlkv_paged_size(layers, kv_heads, q_heads, head_dim, max_seqs, n_pages, max_seq_len, head_is_full, sink, window) -> int:
    m = _mask(head_is_full)
    if m.size != layers * kv_heads:
        raise ValueError("head_is_full must have layers*kv_heads entries")
    out = _sz(0)
    _check(lib.rlkv_paged_size(layers, kv_heads, q_heads, head_dim, max_seqs, n_pages, max_seq_len, m.ctypes.data, sink,
                               window, ctypes.byref(out)))
    return int(out.value)


def rlkv_paged_create(layers, kv_heads, q_heads, head_dim, max_seqs, n_pages, max_seq_len, head_is_full, sink, window,
                      device_buf=None, device_buf_bytes=0) -> int:
    m = _mask(head_is_full)
    if m.size != layers * kv_heads:
        raise ValueError("head_is_full must have layers*kv_heads entries")
    handle = _vp(0)
    _check(lib.rlkv_paged_create(ctypes.byref(handle), layers, kv_heads, q_heads, head_dim, max_seqs, n_pages, max_seq_len,
                                 m.ctypes.data, sink, window, _ptr(device_buf), device_buf_bytes))
    return int(handle.value)


def rlkv_paged_size_fp8(layers, kv_heads, q_heads, head_dim, max_seqs, n_pages, max_seq_len, head_is_full, sink,
                        window) -> int:
    m = _mask(head_is_full)
    if m.size != layers * kv_heads:
        raise ValueError("head_is_full must have layers*kv_heads entries")
    out = _sz(0)
    _check(lib.rlkv_paged_size_fp8(layers, kv_heads, q_heads, head_dim, max_seqs, n_pages, max_seq_len, m.ctypes.data,
                                   sink, window, ctypes.byref(out)))
    return int(out.value)


def rlkv_paged_create_fp8(layers, kv_heads, q_heads, head_dim, max_seqs, n_pages, max_seq_len, head_is_full, sink, window,
                          k_scale, v_scale, device_buf=None, device_buf_bytes=0) -> int:
    m = _mask(head_is_full)
    ks = np.ascontiguousarray(np.asarray(k_scale, dtype=np.float32).reshape(-1))
    vs = np.ascontiguousarray(np.asarray(v_scale, dtype=np.float32).reshape(-1))
    if m.size != layers * kv_heads or ks.size != m.size or vs.size != m.size:
        raise ValueError("head_is_full, k_scale and v_scale must have layers*kv_heads entries")
    handle = _vp(0)
    _check(lib.rlkv_paged_create_fp8(ctypes.byref(handle), layers, kv_heads, q_heads, head_dim, max_seqs, n_pages,
                                     max_seq_len, m.ctypes.data, sink, window, ks.ctypes.data, vs.ctypes.data,
                                     _ptr(device_buf), device_buf_bytes))
    return int(handle.value)


def rlkv_paged_destroy(cache) -> None:
    _check(lib.rlkv_paged_destroy(cache))


def rlkv_paged_seq_open(cache) -> int:
    slot = _ci(-1)
    _check(lib.rlkv_paged_seq_open(cache, ctypes.byref(slot)))
    return int(slot.value)


def rlkv_paged_seq_close(cache, slot) -> None:
    _check(lib.rlkv_paged_seq_close(cache, slot))


def rlkv_paged_append(cache, layer, slots, k, v, stream=None) -> None:
    s = _slots(slots)
    _check(lib.rlkv_paged_append(cache, layer, s.ctypes.data, s.size, _ptr(k), _ptr(v), _stream(stream)))


def rlkv_paged_prefill(cache, layer, slot, k, v, n_tokens, stream=None) -> None:
    _check(lib.rlkv_paged_prefill(cache, layer, slot, _ptr(k), _ptr(v), n_tokens, _stream(stream)))


def rlkv_paged_decode_attention(cache, layer, slots, q, out, stream=None) -> None:
    s = _slots(slots)
    _check(lib.rlkv_paged_decode_attention(cache, layer, s.ctypes.data, s.size, _ptr(q), _ptr(out), _stream(stream)))


def rlkv_paged_step(cache, slots, k, v, q, out, stream=None) -> None:
    s = _slots(slots)
    _check(lib.rlkv_paged_step(cache, s.ctypes.data, s.size, _ptr(k), _ptr(v), _ptr(q), _ptr(out), _stream(stream)))


def rlkv_paged_length(cache, layer, slot) -> int:
    out = _ci(0)
    _check(lib.rlkv_paged_length(cache, layer, slot, ctypes.byref(out)))
    return int(out.value)


def rlkv_paged_pages(cache):
    """(pages on the free list, pages in total)."""
    free, total = _ci(0), _ci(0)
    _check(lib.rlkv_paged_pages(cache, ctypes.byref(free), ctypes.byref(total)))
    return int(free.value), int(total.value)


def rlkv_paged_step_bytes(cache, layer, slots) -> int:
    s = _slots(slots)
    out = ctypes.c_uint64(0)
    _check(lib.rlkv_paged_step_bytes(cache, layer, s.ctypes.data, s.size, ctypes.byref(out)))
    return int(out.value)


def rlkv_paged_debug_export_head(cache, layer, slot, kv_head, max_rows, head_dim):
    """Returns (k, v, token_of_slot) as numpy arrays (uint16 bf16 bits [rows][head_dim], int32 [rows])."""
    k = np.zeros((max_rows, head_dim), dtype=np.uint16)
    v = np.zeros((max_rows, head_dim), dtype=np.uint16)
    tok = np.full(max_rows, -1, dtype=np.int32)
    rows = _ci(0)
    _check(lib.rlkv_paged_debug_export_head(cache, layer, slot, kv_head, k.ctypes.data, v.ctypes.data, ctypes.byref(rows),
                                            tok.ctypes.data))
    n = int(rows.value)
    return k[:n], v[:n], tok[:n]


def rlkv_paged_kernel_status(cache) -> int:
    out = _ci(0)
    _check(lib.rlkv_paged_kernel_status(cache, ctypes.byref(out)))
    return int(out.value)


def rlkv_debug_paged_schedule(lens, n_full, n_comp, cap, ctas, item_tiles):
    """Returns (n_items, delivered, expected, complete), the last three int32 arrays per unit."""
    ln = _slots(lens)
    units = ln.size * (n_full + n_comp)
    delivered, expected, complete = (np.zeros(units, dtype=np.int32) for _ in range(3))
    n_items = _ci(0)
    _check(lib.rlkv_debug_paged_schedule(ln.ctypes.data, ln.size, n_full, n_comp, cap, ctas, item_tiles,
                                         ctypes.byref(n_items), delivered.ctypes.data, expected.ctypes.data,
                                         complete.ctypes.data))
    return int(n_items.value), delivered, expected, complete

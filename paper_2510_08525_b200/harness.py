"""Helpers shared by the benchmark and the GPU tests: a small owner object for a cache handle and
the seeded fill of a cache.  No attention or cache arithmetic happens here -- the fill only moves
generator output into the library through ``rlkv_prefill``.
"""
from __future__ import annotations

import numpy as np
import torch

import synth

from . import binding as rl


class Cache:
    """Owns one rlkv_cache handle; methods forward to the C entry points of the same name."""

    def __init__(self, layers, kv_heads, q_heads, head_dim, batch, max_len, head_is_full, sink, window,
                 device="cuda:0", device_buf=None):
        self.layers, self.kv_heads, self.q_heads, self.head_dim = layers, kv_heads, q_heads, head_dim
        self.batch, self.max_len, self.sink, self.window = batch, max_len, sink, window
        self.head_is_full = np.asarray(head_is_full, dtype=np.uint8).reshape(-1).copy()
        self.device = torch.device(device)
        self._buf = device_buf
        with torch.cuda.device(self.device):
            self.handle = rl.rlkv_cache_create(
                layers, kv_heads, q_heads, head_dim, batch, max_len, self.head_is_full, sink, window,
                device_buf, 0 if device_buf is None else device_buf.numel() * device_buf.element_size())

    def close(self):
        if getattr(self, "handle", None):
            rl.rlkv_cache_destroy(self.handle)
            self.handle = None

    __del__ = close

    def is_full(self, layer, head) -> bool:
        return bool(self.head_is_full[layer * self.kv_heads + head])

    def append(self, layer, k, v):
        rl.rlkv_append(self.handle, layer, k, v)

    def prefill(self, layer, k, v):
        rl.rlkv_prefill(self.handle, layer, k, v, k.shape[0])

    def decode(self, layer, q, out=None):
        if out is None:
            out = torch.empty((self.batch, self.q_heads, self.head_dim), dtype=torch.float32, device=self.device)
        rl.rlkv_decode_attention(self.handle, layer, q, out)
        return out

    def decode_mixed(self, layer, q, alpha, out=None):
        """alpha: fp32 [kv_heads] on the cache's device."""
        if out is None:
            out = torch.empty((self.batch, self.q_heads, self.head_dim), dtype=torch.float32, device=self.device)
        rl.rlkv_decode_mixed_attention(self.handle, layer, q, alpha, out)
        return out

    def length(self, layer) -> int:
        return rl.rlkv_length(self.handle, layer)

    def step_bytes(self, layer) -> int:
        return rl.rlkv_step_bytes(self.handle, layer)

    def export_head(self, layer, b, head):
        rows = self.max_len if self.is_full(layer, head) else self.sink + self.window
        return rl.rlkv_debug_export_head(self.handle, layer, b, head, rows, self.head_dim)

    def status(self) -> int:
        return rl.rlkv_kernel_status(self.handle)


workload_mask = synth.workload_mask


def make_cache(w: synth.Workload, extra_tokens: int = 64, device="cuda:0") -> Cache:
    return Cache(w.layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, w.context + extra_tokens,
                 workload_mask(w), w.sink, w.window, device=device)


def fill_cache(cache: Cache, w: synth.Workload, n_tokens: int, chunk_elems: int = 1 << 24) -> None:
    """Prefill tokens length(layer) .. n_tokens-1 of every layer from the seeded generator."""
    per_token = w.batch * w.kv_heads * w.head_dim
    chunk = max(1, chunk_elems // per_token)
    for layer in range(w.layers):
        t = cache.length(layer)
        while t < n_tokens:
            t1 = min(n_tokens, t + chunk)
            k = synth.rows(w.seed, synth.STREAM_K, layer, t, t1, w.batch, w.kv_heads, w.head_dim, cache.device)
            v = synth.rows(w.seed, synth.STREAM_V, layer, t, t1, w.batch, w.kv_heads, w.head_dim, cache.device)
            cache.prefill(layer, k, v)
            t = t1
    torch.cuda.synchronize(cache.device)


def step_inputs(w: synth.Workload, t: int, device):
    """k, v [layers][B][Hkv][D] and q [layers][B][Hq][D] (bf16) for the decode step that appends token t."""
    k = torch.stack([synth.rows(w.seed, synth.STREAM_K, l, t, t + 1, w.batch, w.kv_heads, w.head_dim, device)[0]
                     for l in range(w.layers)])
    v = torch.stack([synth.rows(w.seed, synth.STREAM_V, l, t, t + 1, w.batch, w.kv_heads, w.head_dim, device)[0]
                     for l in range(w.layers)])
    q = torch.stack([synth.rows(w.seed, synth.STREAM_Q, l, t, t + 1, w.batch, w.q_heads, w.head_dim, device)[0]
                     for l in range(w.layers)])
    return k.contiguous(), v.contiguous(), q.contiguous()


def step_inputs_block(w: synth.Workload, t0: int, t1: int, device):
    """The inputs of the decode steps that append tokens t0 .. t1-1, generated in one go:
    k, v [t1-t0][layers][B][Hkv][D] and q [t1-t0][layers][B][Hq][D]; entry i equals step_inputs(w, t0 + i)."""
    def one(stream_id, heads):
        return torch.stack([synth.rows(w.seed, stream_id, l, t0, t1, w.batch, heads, w.head_dim, device)
                            for l in range(w.layers)], dim=1).contiguous()
    return one(synth.STREAM_K, w.kv_heads), one(synth.STREAM_V, w.kv_heads), one(synth.STREAM_Q, w.q_heads)


class PagedCache:
    """Owns an rlkv_paged handle (request slots with their own lengths, paged full heads)."""

    def __init__(self, layers, kv_heads, q_heads, head_dim, max_seqs, n_pages, max_seq_len, head_is_full, sink, window,
                 device="cuda:0", k_scale=None, v_scale=None):
        self.layers, self.kv_heads, self.q_heads, self.head_dim = layers, kv_heads, q_heads, head_dim
        self.max_seqs, self.n_pages, self.max_seq_len, self.sink, self.window = max_seqs, n_pages, max_seq_len, sink, window
        self.device = torch.device(device)
        self.mask = np.asarray(head_is_full, dtype=np.uint8).reshape(layers, kv_heads)
        with torch.cuda.device(self.device):
            if k_scale is None:
                self.handle = rl.rlkv_paged_create(layers, kv_heads, q_heads, head_dim, max_seqs, n_pages, max_seq_len,
                                                   self.mask, sink, window)
            else:      # every K/V row (pages and rings) as E4M3 codes
                self.handle = rl.rlkv_paged_create_fp8(layers, kv_heads, q_heads, head_dim, max_seqs, n_pages, max_seq_len,
                                                       self.mask, sink, window, k_scale, v_scale)

    def close(self):
        if getattr(self, "handle", None):
            rl.rlkv_paged_destroy(self.handle)
            self.handle = None

    __del__ = close

    def open_seq(self) -> int:
        return rl.rlkv_paged_seq_open(self.handle)

    def close_seq(self, slot) -> None:
        rl.rlkv_paged_seq_close(self.handle, slot)

    def append(self, layer, slots, k, v):
        rl.rlkv_paged_append(self.handle, layer, slots, k, v)

    def prefill(self, layer, slot, k, v):
        rl.rlkv_paged_prefill(self.handle, layer, slot, k, v, k.shape[0])

    def decode(self, layer, slots, q, out=None):
        if out is None:
            out = torch.empty((len(slots), self.q_heads, self.head_dim), dtype=torch.float32, device=self.device)
        rl.rlkv_paged_decode_attention(self.handle, layer, slots, q, out)
        return out

    def length(self, layer, slot) -> int:
        return rl.rlkv_paged_length(self.handle, layer, slot)

    def pages(self):
        return rl.rlkv_paged_pages(self.handle)

    def step_bytes(self, layer, slots) -> int:
        return rl.rlkv_paged_step_bytes(self.handle, layer, slots)

    def export_head(self, layer, slot, head):
        rows = max(self.max_seq_len, self.sink + self.window)
        return rl.rlkv_paged_debug_export_head(self.handle, layer, slot, head, rows, self.head_dim)

    def status(self) -> int:
        return rl.rlkv_paged_kernel_status(self.handle)


def paged_seq_seed(w: synth.Workload, i: int) -> int:
    """Sequence i of a paged batch draws its rows from a generator of its own (batch 1)."""
    return w.seed + 1 + i


def fill_paged(pc: PagedCache, w: synth.Workload, slots, lens, chunk: int = 4096) -> None:
    """Prefill tokens 0 .. lens[i]-1 of every layer of sequence slots[i] from the seeded generator."""
    for i, x in enumerate(lens):
        for layer in range(pc.layers):
            for t0 in range(0, x, chunk):
                t1 = min(x, t0 + chunk)
                kk = synth.rows(paged_seq_seed(w, i), synth.STREAM_K, layer, t0, t1, 1, w.kv_heads, w.head_dim, pc.device)
                vv = synth.rows(paged_seq_seed(w, i), synth.STREAM_V, layer, t0, t1, 1, w.kv_heads, w.head_dim, pc.device)
                pc.prefill(layer, slots[i], kk.reshape(t1 - t0, w.kv_heads, w.head_dim),
                           vv.reshape(t1 - t0, w.kv_heads, w.head_dim))
    torch.cuda.synchronize(pc.device)


def paged_step_inputs(pc: PagedCache, w: synth.Workload, lens):
    """k, v [layers][n][Hkv][D], q [layers][n][Hq][D] (bf16) of the step that appends token lens[i] to sequence i."""
    def stack(stream, heads):
        return torch.stack([torch.cat([synth.rows(paged_seq_seed(w, i), stream, layer, x, x + 1, 1, heads, w.head_dim, pc.device)[0]
                                       for i, x in enumerate(lens)]) for layer in range(pc.layers)]).contiguous()
    return stack(synth.STREAM_K, w.kv_heads), stack(synth.STREAM_V, w.kv_heads), stack(synth.STREAM_Q, w.q_heads)


def paged_spread_lengths(n: int, batch: int):
    """Lengths from a quarter to seven quarters of n, about the same total as batch sequences of n."""
    return [max(1, int(round(n * (0.25 + 1.5 * i / max(1, batch - 1))))) for i in range(batch)]

"""ctypes wrapper around the C oracle (``rlkv_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
benchmark's cpu-baseline / reference legs.  The CUDA library and its Python binding
never import this module.

``Oracle(..., acc="f32")`` is the float build, ``acc="f64"`` the double build of the
very same source (``-DRLKV_ORACLE_ACC=double``).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rlkv_oracle.c")
_LIBS = {"f32": os.path.join(_HERE, "librlkv_oracle_f32.so"),
         "f64": os.path.join(_HERE, "librlkv_oracle_f64.so")}
_loaded: dict = {}


CC = "gcc"
CFLAGS = ["-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-fno-fast-math", "-ffp-contract=off"]


def build(force: bool = False) -> None:
    """Compile both builds of the oracle with gcc (plain C, -O2, OpenMP over (b, q head))."""
    for acc, path in _LIBS.items():
        if not force and os.path.exists(path) and os.path.getmtime(path) >= os.path.getmtime(_SRC):
            continue
        cmd = [CC] + CFLAGS
        if acc == "f64":
            cmd.append("-DRLKV_ORACLE_ACC=double")
        cmd += [_SRC, "-o", path, "-lm"]
        subprocess.run(cmd, check=True)


def _lib(acc: str) -> ctypes.CDLL:
    if acc not in _loaded:
        build()
        lib = ctypes.CDLL(_LIBS[acc])
        vp, ci = ctypes.c_void_p, ctypes.c_int
        lib.rlkv_oracle_create.restype = vp
        lib.rlkv_oracle_create.argtypes = [ci, ci, ci, ci, ci, ci, vp, ci, ci]
        lib.rlkv_oracle_destroy.restype = None
        lib.rlkv_oracle_destroy.argtypes = [vp]
        lib.rlkv_oracle_set_threads.restype = None
        lib.rlkv_oracle_set_threads.argtypes = [vp, ci]
        lib.rlkv_oracle_length.restype = ci
        lib.rlkv_oracle_length.argtypes = [vp, ci]
        lib.rlkv_oracle_append.restype = ci
        lib.rlkv_oracle_append.argtypes = [vp, ci, vp, vp]
        lib.rlkv_oracle_decode.restype = ci
        lib.rlkv_oracle_decode.argtypes = [vp, ci, vp, vp]
        lib.rlkv_oracle_decode_mixed.restype = ci
        lib.rlkv_oracle_decode_mixed.argtypes = [vp, ci, vp, vp, vp]
        lib.rlkv_oracle_retained.restype = ci
        lib.rlkv_oracle_retained.argtypes = [vp, ci, ci]
        lib.rlkv_oracle_export_head.restype = ci
        lib.rlkv_oracle_export_head.argtypes = [vp, ci, ci, ci, vp, vp, vp]
        lib.rlkv_oracle_set_fp8.restype = ci
        lib.rlkv_oracle_set_fp8.argtypes = [vp, vp, vp]
        lib.rlkv_oracle_e4m3_value.restype = ctypes.c_float
        lib.rlkv_oracle_e4m3_value.argtypes = [ctypes.c_uint8]
        lib.rlkv_oracle_e4m3_encode.restype = ctypes.c_uint8
        lib.rlkv_oracle_e4m3_encode.argtypes = [ctypes.c_float]
        lib.rlkv_oracle_max_threads.restype = ci
        lib.rlkv_oracle_acc_bytes.restype = ci
        assert lib.rlkv_oracle_acc_bytes() == (4 if acc == "f32" else 8)
        _loaded[acc] = lib
    return _loaded[acc]


def max_threads() -> int:
    return int(_lib("f32").rlkv_oracle_max_threads())


def e4m3_value(code: int) -> float:
    """Value of an OCP E4M3 code (nan for 0x7f / 0xff)."""
    return float(_lib("f32").rlkv_oracle_e4m3_value(int(code) & 0xff))


def e4m3_encode(x: float) -> int:
    """Nearest E4M3 code of a float32 (ties to even, saturating at +-448, NaN -> 0x7f)."""
    return int(_lib("f32").rlkv_oracle_e4m3_encode(float(np.float32(x))))


def _bits(a) -> np.ndarray:
    """Accept uint16/int16 numpy arrays or torch bf16 tensors; return contiguous uint16."""
    if hasattr(a, "detach"):  # torch tensor
        import torch
        a = a.detach().cpu().contiguous()
        if a.dtype == torch.bfloat16:
            a = a.view(torch.int16)
        a = a.numpy()
    a = np.ascontiguousarray(a)
    if a.dtype == np.int16:
        a = a.view(np.uint16)
    if a.dtype != np.uint16:
        raise TypeError("expected bf16 bit patterns (uint16/int16) or a torch.bfloat16 tensor")
    return a


class Oracle:
    def __init__(self, layers, kv_heads, q_heads, head_dim, batch, max_len, head_is_full,
                 sink, window, acc="f32", threads=1):
        self._lib = _lib(acc)
        self.layers, self.kv_heads, self.q_heads = layers, kv_heads, q_heads
        self.head_dim, self.batch, self.max_len = head_dim, batch, max_len
        self.sink, self.window = sink, window
        mask = np.ascontiguousarray(np.asarray(head_is_full, dtype=np.uint8).reshape(-1))
        if mask.size != layers * kv_heads:
            raise ValueError("head_is_full must have layers*kv_heads entries")
        self.head_is_full = mask
        self._h = self._lib.rlkv_oracle_create(layers, kv_heads, q_heads, head_dim, batch, max_len,
                                               mask.ctypes.data, sink, window)
        if not self._h:
            raise ValueError("rlkv_oracle_create rejected the arguments")
        self.set_threads(threads)

    def close(self):
        if getattr(self, "_h", None):
            self._lib.rlkv_oracle_destroy(self._h)
            self._h = None

    __del__ = close

    def set_threads(self, threads: int) -> None:
        self.threads = int(threads)
        self._lib.rlkv_oracle_set_threads(self._h, int(threads))

    def set_fp8(self, k_scale, v_scale) -> None:
        """Every head stores E4M3 codes from now on (only while the cache is empty).  k_scale,
        v_scale: [layers][kv_heads] positive floats."""
        ks = np.ascontiguousarray(np.asarray(k_scale, dtype=np.float32).reshape(-1))
        vs = np.ascontiguousarray(np.asarray(v_scale, dtype=np.float32).reshape(-1))
        if ks.size != self.layers * self.kv_heads or vs.size != ks.size:
            raise ValueError("k_scale, v_scale must have layers*kv_heads entries")
        rc = self._lib.rlkv_oracle_set_fp8(self._h, ks.ctypes.data, vs.ctypes.data)
        if rc != 0:
            raise RuntimeError(f"rlkv_oracle_set_fp8 failed: {rc}")
        self.fp8 = True

    def length(self, layer: int) -> int:
        return int(self._lib.rlkv_oracle_length(self._h, layer))

    def append(self, layer: int, k, v) -> int:
        k, v = _bits(k), _bits(v)
        want = self.batch * self.kv_heads * self.head_dim
        if k.size != want or v.size != want:
            raise ValueError("k, v must be [batch][kv_heads][head_dim]")
        return int(self._lib.rlkv_oracle_append(self._h, layer, k.ctypes.data, v.ctypes.data))

    def decode(self, layer: int, q) -> np.ndarray:
        q = _bits(q)
        if q.size != self.batch * self.q_heads * self.head_dim:
            raise ValueError("q must be [batch][q_heads][head_dim]")
        out = np.empty((self.batch, self.q_heads, self.head_dim), dtype=np.float32)
        rc = self._lib.rlkv_oracle_decode(self._h, layer, q.ctypes.data, out.ctypes.data)
        if rc != 0:
            raise RuntimeError(f"rlkv_oracle_decode failed: {rc}")
        return out

    def decode_mixed(self, layer: int, q, alpha) -> np.ndarray:
        """Eq. 1: alpha[h] * full attention + (1 - alpha[h]) * sink+window attention; every head of
        the layer must be full.  alpha: [kv_heads] floats in [0, 1]."""
        q = _bits(q)
        if q.size != self.batch * self.q_heads * self.head_dim:
            raise ValueError("q must be [batch][q_heads][head_dim]")
        alpha = np.ascontiguousarray(np.asarray(alpha, dtype=np.float32).reshape(-1))
        if alpha.size != self.kv_heads:
            raise ValueError("alpha must have kv_heads entries")
        out = np.empty((self.batch, self.q_heads, self.head_dim), dtype=np.float32)
        rc = self._lib.rlkv_oracle_decode_mixed(self._h, layer, q.ctypes.data, alpha.ctypes.data, out.ctypes.data)
        if rc != 0:
            raise RuntimeError(f"rlkv_oracle_decode_mixed failed: {rc}")
        return out

    def retained(self, layer: int, head: int) -> int:
        return int(self._lib.rlkv_oracle_retained(self._h, layer, head))

    def export_head(self, layer: int, b: int, head: int):
        full = bool(self.head_is_full[layer * self.kv_heads + head])
        rows = self.max_len if full else self.sink + self.window
        k = np.empty((rows, self.head_dim), dtype=np.uint16)
        v = np.empty((rows, self.head_dim), dtype=np.uint16)
        tok = np.empty(rows, dtype=np.int32)
        got = self._lib.rlkv_oracle_export_head(self._h, layer, b, head, k.ctypes.data,
                                                v.ctypes.data, tok.ctypes.data)
        assert got == rows
        return k, v, tok

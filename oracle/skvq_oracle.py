"""ctypes front end of the SKVQ CPU oracle (``skvq_oracle.c``).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this module.  It never imports the CUDA
package and the CUDA package never imports it.  All arithmetic lives in the C
file; this module only builds it with gcc, allocates numpy arrays in the layout
the C file documents and marshals pointers.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "skvq_oracle.c")
_LIB = os.path.join(_HERE, "libskvq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (IEEE fp32, no contraction, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-Wall", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _Cache(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int), ("Hkv", ctypes.c_int), ("D", ctypes.c_int), ("G", ctypes.c_int),
        ("W", ctypes.c_int), ("cap_q", ctypes.c_int), ("k_bits", ctypes.c_int), ("v_bits", ctypes.c_int),
        ("k_codes", ctypes.c_void_p), ("v_codes", ctypes.c_void_p),
        ("k_meta", ctypes.c_void_p), ("v_meta", ctypes.c_void_p),
        ("k_win", ctypes.c_void_p), ("v_win", ctypes.c_void_p),
        ("lengths", ctypes.c_void_p),
        ("reorder_k", ctypes.c_void_p), ("reorder_v", ctypes.c_void_p),
        ("alpha_k", ctypes.c_void_p), ("alpha_v", ctypes.c_void_p),
        ("n_sink", ctypes.c_int), ("k_sink", ctypes.c_void_p), ("v_sink", ctypes.c_void_p),
        ("meta_fp8", ctypes.c_int),
        ("ng", ctypes.c_int), ("bounds_k", ctypes.c_void_p), ("bounds_v", ctypes.c_void_p),
    ]


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_f16_to_f32.restype = ctypes.c_float
        _lib.orc_f16_to_f32.argtypes = [ctypes.c_uint16]
        _lib.orc_f32_to_f16.restype = ctypes.c_uint16
        _lib.orc_f32_to_f16.argtypes = [ctypes.c_float]
        _lib.orc_quantize_rows.restype = None
        _lib.orc_quantize_rows.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                           ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                                           ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int]
        _lib.orc_dequant_row.restype = None
        _lib.orc_dequant_row.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                         ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int]
        _lib.orc_e4m3_to_f32.restype = ctypes.c_float
        _lib.orc_e4m3_to_f32.argtypes = [ctypes.c_uint8]
        _lib.orc_f32_to_e4m3.restype = ctypes.c_uint8
        _lib.orc_f32_to_e4m3.argtypes = [ctypes.c_float]
        _lib.orc_append.restype = ctypes.c_int
        _lib.orc_append.argtypes = [ctypes.POINTER(_Cache), ctypes.c_void_p, ctypes.c_void_p,
                                    ctypes.c_void_p, ctypes.c_int]
        _lib.orc_attention.restype = None
        _lib.orc_attention.argtypes = [ctypes.POINTER(_Cache), ctypes.c_int, ctypes.c_void_p,
                                       ctypes.c_double, ctypes.c_void_p]
        _lib.orc_num_threads.restype = ctypes.c_int
    return _lib


BITS_TERNARY = 15      # the "1.5-bit" three-level code: five base-3 digits per byte


def row_bytes(D: int, bits: int) -> int:
    """Bytes of one packed row of D codes."""
    return (D + 4) // 5 if bits == BITS_TERNARY else D * bits // 8


def qmax(bits: int) -> int:
    return 2 if bits == BITS_TERNARY else (1 << bits) - 1


def _ptr(a: np.ndarray) -> int:
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data


def num_threads() -> int:
    return int(lib().orc_num_threads())


def f32_to_f16_bits(x: float) -> int:
    return int(lib().orc_f32_to_f16(ctypes.c_float(x)))


def f16_bits_to_f32(b: int) -> float:
    return float(lib().orc_f16_to_f32(ctypes.c_uint16(b)))


def f32_to_e4m3_bits(x: float) -> int:
    return int(lib().orc_f32_to_e4m3(ctypes.c_float(x)))


def e4m3_bits_to_f32(b: int) -> float:
    return float(lib().orc_e4m3_to_f32(ctypes.c_uint8(b)))


def _bounds(bounds, D):
    """Group boundaries as a contiguous int32 array [ng+1] (0 ... D, strictly increasing), or None."""
    if bounds is None:
        return None
    b = np.ascontiguousarray(bounds, dtype=np.int32)
    assert b.ndim == 1 and b[0] == 0 and b[-1] == D and np.all(np.diff(b) > 0)
    return b


def quantize_rows(x: np.ndarray, idx: np.ndarray, alpha: np.ndarray, bits: int, group: int, meta_fp8: bool = False,
                  bounds=None):
    """Reorder + clipped group quantization of independent rows.

    x: float16 [n, D] in original channel order; idx: int32 [D]; alpha: float32 [ng].  Groups are D/group equal runs of
    ``group`` reordered channels, or, with ``bounds`` (int [ng+1], 0 ... D), the runs [bounds[g], bounds[g+1]).
    Returns (codes uint8 [n, D*bits/8], meta float16 [n, ng, 2] = {h, z}); with meta_fp8 the
    meta array holds the E4M3 byte of h and z as uint16 [n, ng, 2].
    """
    x = np.ascontiguousarray(x, dtype=np.float16)
    n, D = x.shape
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    alpha = np.ascontiguousarray(alpha, dtype=np.float32)
    b = _bounds(bounds, D)
    ng = D // group if b is None else len(b) - 1
    assert idx.shape == (D,) and alpha.shape == (ng,) and (bits == BITS_TERNARY or (D * bits) % 8 == 0)
    codes = np.zeros((n, row_bytes(D, bits)), dtype=np.uint8)
    meta = np.zeros((n, ng, 2), dtype=np.uint16 if meta_fp8 else np.float16)
    lib().orc_quantize_rows(_ptr(x), n, _ptr(idx), _ptr(alpha), D, group, bits, int(meta_fp8), _ptr(codes), _ptr(meta),
                            None if b is None else _ptr(b), ng)
    return codes, meta


def dequant_rows(codes: np.ndarray, meta: np.ndarray, bits: int, group: int, meta_fp8: bool = False, bounds=None) -> np.ndarray:
    """fp64 dequantization x^ = h*c + z of packed rows (no rounding)."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    meta = np.ascontiguousarray(meta, dtype=np.uint16 if meta_fp8 else np.float16)
    n = codes.shape[0]
    D = (meta.shape[1] * group if bounds is None else int(np.asarray(bounds)[-1])) if bits == BITS_TERNARY else codes.shape[1] * 8 // bits
    b = _bounds(bounds, D)
    out = np.zeros((n, D), dtype=np.float64)
    for r in range(n):
        lib().orc_dequant_row(_ptr(codes[r]), _ptr(meta[r]), D, group, bits, int(meta_fp8), _ptr(out[r]),
                              None if b is None else _ptr(b), meta.shape[1])
    return out


class OracleCache:
    """Host-side SKVQ cache in the canonical layout, driven by the C oracle."""

    def __init__(self, batch, n_q_heads, n_kv_heads, head_dim, k_bits, v_bits, group_size, window,
                 max_tokens, reorder_k, reorder_v, alpha_k, alpha_v, n_sink=0, meta_fp8=False, bounds_k=None,
                 bounds_v=None):
        self.B, self.Hq, self.Hkv, self.D = batch, n_q_heads, n_kv_heads, head_dim
        self.k_bits, self.v_bits, self.G, self.W = k_bits, v_bits, group_size, window
        self.ng = head_dim // group_size
        # unequal groups: boundaries [Hkv][ng+1] in reordered channel order (None = equal runs of group_size channels)
        self.bounds_k = None if bounds_k is None else np.ascontiguousarray(bounds_k, dtype=np.int32).reshape(n_kv_heads, -1)
        self.bounds_v = None if bounds_v is None else np.ascontiguousarray(bounds_v, dtype=np.int32).reshape(n_kv_heads, -1)
        for bd in (self.bounds_k, self.bounds_v):
            if bd is not None:
                assert np.all(bd[:, 0] == 0) and np.all(bd[:, -1] == head_dim) and np.all(np.diff(bd, axis=1) > 0)
                self.ng = bd.shape[1] - 1
        assert self.bounds_k is None or self.bounds_v is None or self.bounds_k.shape == self.bounds_v.shape
        self.cap_q = max(max_tokens - window, 0)
        B, H, D, W = batch, n_kv_heads, head_dim, window
        self.k_codes = np.zeros((B, H, self.cap_q, row_bytes(D, k_bits)), dtype=np.uint8)
        self.v_codes = np.zeros((B, H, self.cap_q, row_bytes(D, v_bits)), dtype=np.uint8)
        self.meta_fp8 = bool(meta_fp8)      # scale/zero as FP8 E4M3: the arrays then hold the byte of each as uint16
        meta_t = np.uint16 if self.meta_fp8 else np.float16
        self.k_meta = np.zeros((B, H, self.cap_q, self.ng, 2), dtype=meta_t)
        self.v_meta = np.zeros((B, H, self.cap_q, self.ng, 2), dtype=meta_t)
        self.k_win = np.zeros((B, H, W, D), dtype=np.float16)
        self.v_win = np.zeros((B, H, W, D), dtype=np.float16)
        self.n_sink = int(n_sink)
        self.k_sink = np.zeros((B, H, max(self.n_sink, 1), D), dtype=np.float16)
        self.v_sink = np.zeros((B, H, max(self.n_sink, 1), D), dtype=np.float16)
        self.lengths = np.zeros((B,), dtype=np.int32)
        self.reorder_k = np.ascontiguousarray(reorder_k, dtype=np.int32).reshape(H, D)
        self.reorder_v = np.ascontiguousarray(reorder_v, dtype=np.int32).reshape(H, D)
        self.alpha_k = np.ascontiguousarray(alpha_k, dtype=np.float32).reshape(H, self.ng)
        self.alpha_v = np.ascontiguousarray(alpha_v, dtype=np.float32).reshape(H, self.ng)

    def _struct(self) -> _Cache:
        return _Cache(self.B, self.Hkv, self.D, self.G, self.W, self.cap_q, self.k_bits, self.v_bits,
                      _ptr(self.k_codes), _ptr(self.v_codes), _ptr(self.k_meta), _ptr(self.v_meta),
                      _ptr(self.k_win), _ptr(self.v_win), _ptr(self.lengths),
                      _ptr(self.reorder_k), _ptr(self.reorder_v), _ptr(self.alpha_k), _ptr(self.alpha_v),
                      self.n_sink, _ptr(self.k_sink), _ptr(self.v_sink), int(self.meta_fp8), self.ng,
                      None if self.bounds_k is None else _ptr(self.bounds_k),
                      None if self.bounds_v is None else _ptr(self.bounds_v))

    def append(self, k: np.ndarray, v: np.ndarray, n_new=None) -> int:
        """k, v: float16 [B, n, Hkv, D], original channel order; n_new: per-sequence counts or None."""
        k = np.ascontiguousarray(k, dtype=np.float16)
        v = np.ascontiguousarray(v, dtype=np.float16)
        assert k.shape == v.shape and k.shape[0] == self.B and k.shape[2:] == (self.Hkv, self.D)
        n = k.shape[1]
        if n_new is None:
            n_new = np.full((self.B,), n, dtype=np.int32)
        n_new = np.ascontiguousarray(n_new, dtype=np.int32)
        st = self._struct()
        return int(lib().orc_append(ctypes.byref(st), _ptr(k), _ptr(v), _ptr(n_new), n))

    def attention(self, q: np.ndarray, sm_scale: float) -> np.ndarray:
        """q: float16 [B, Hq, D]; returns float64 [B, Hq, D]."""
        q = np.ascontiguousarray(q, dtype=np.float16)
        assert q.shape == (self.B, self.Hq, self.D)
        out = np.zeros((self.B, self.Hq, self.D), dtype=np.float64)
        st = self._struct()
        lib().orc_attention(ctypes.byref(st), self.Hq, _ptr(q), float(np.float32(sm_scale)), _ptr(out))
        return out

"""Thin Python binding of libskvq (see ``include/skvq.h``): argument marshalling only.

Functions carry the names of the C entry points.  Tensors are torch CUDA tensors used purely
as device memory; every computation happens in the library's kernels.  The library is loaded
on first use; if it has not been built the call raises -- there is no fallback.
"""
from __future__ import annotations

import ctypes
import os

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libskvq.so")
_lib = None

SKVQ_OK = 0
SKVQ_ERR_INVALID_ARG, SKVQ_ERR_UNSUPPORTED, SKVQ_ERR_MISALIGNED = -1, -2, -3
SKVQ_ERR_CAPACITY, SKVQ_ERR_WORKSPACE, SKVQ_ERR_CUDA = -4, -5, -6
SKVQ_ERR_SCRATCH_LIMIT = -7
SKVQ_NOALLOC_SCRATCH_BYTES = 8 << 20
SKVQ_STATUS_OVERFLOW = 1
SKVQ_STATUS_COPY_TIMEOUT = 2
SKVQ_STATUS_BOUNDS = 4
SKVQ_TOKEN_ALIGN = 64
SKVQ_GROUP_GRANULE = 32
SKVQ_BITS_TERNARY = 15

EXPORTS = ["skvq_version", "skvq_strerror", "skvq_launch_count", "skvq_check_config", "skvq_quant_capacity",
           "skvq_cache_sizes", "skvq_sink_bytes", "skvq_quantize_append", "skvq_workspace_size", "skvq_decode_attention",
           "skvq_step_staging_size", "skvq_decode_step_host", "skvq_decode_attention_noalloc", "skvq_check_group_bounds"]


class SkvqConfig(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("batch", "n_q_heads", "n_kv_heads", "head_dim", "k_bits", "v_bits",
                                              "group_size", "window", "max_tokens", "n_sink", "meta_fp8")]


class SkvqCacheStruct(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("k_codes", "v_codes", "k_meta", "v_meta", "k_win", "v_win", "lengths",
                                               "reorder_k", "reorder_v", "alpha_k", "alpha_v", "status", "k_sink",
                                               "v_sink", "group_bounds_k", "group_bounds_v")]


class SkvqAttnArgs(ctypes.Structure):
    _fields_ = [("sm_scale", ctypes.c_float), ("max_len_hint", ctypes.c_int32), ("n_splits", ctypes.c_int32),
                ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
                ("ev_begin", ctypes.c_void_p), ("ev_end", ctypes.c_void_p)]


class SkvqError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {skvq_strerror(code)} ({code})")


def use_library(path: str | None) -> None:
    """Make the wrappers call the library at ``path`` from now on (None = the default libskvq.so): the debugging build
    libskvq_checked.so exports the same entry points."""
    global _lib, _LIB_PATH
    _LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libskvq.so") if path is None else path
    _lib = None


def lib() -> ctypes.CDLL:
    """Open libskvq.so (built in-tree by ``build.build_library``); raise if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} not found: build it with paper_2405_06219_b200.build.build_library(); "
                               "there is no fallback path")
        L = ctypes.CDLL(_LIB_PATH)
        P, c_int, c_sz, vp = ctypes.POINTER, ctypes.c_int, ctypes.c_size_t, ctypes.c_void_p
        L.skvq_version.restype = c_int
        L.skvq_strerror.restype = ctypes.c_char_p
        L.skvq_strerror.argtypes = [c_int]
        L.skvq_launch_count.restype = ctypes.c_uint64
        L.skvq_check_config.restype = c_int
        L.skvq_check_config.argtypes = [P(SkvqConfig)]
        L.skvq_check_group_bounds.restype = c_int
        L.skvq_check_group_bounds.argtypes = [P(SkvqConfig), vp]
        L.skvq_quant_capacity.restype = ctypes.c_int32
        L.skvq_quant_capacity.argtypes = [P(SkvqConfig)]
        L.skvq_cache_sizes.restype = c_int
        L.skvq_cache_sizes.argtypes = [P(SkvqConfig), P(c_sz)]
        L.skvq_sink_bytes.restype = c_sz
        L.skvq_sink_bytes.argtypes = [P(SkvqConfig)]
        L.skvq_quantize_append.restype = c_int
        L.skvq_quantize_append.argtypes = [P(SkvqConfig), P(SkvqCacheStruct), vp, vp, vp, ctypes.c_int32, vp]
        L.skvq_workspace_size.restype = c_sz
        L.skvq_workspace_size.argtypes = [P(SkvqConfig), ctypes.c_int32, ctypes.c_int32]
        L.skvq_decode_attention.restype = c_int
        L.skvq_decode_attention.argtypes = [P(SkvqConfig), P(SkvqCacheStruct), vp, vp, P(SkvqAttnArgs), vp]
        L.skvq_step_staging_size.restype = c_sz
        L.skvq_step_staging_size.argtypes = [P(SkvqConfig)]
        L.skvq_decode_step_host.restype = c_int
        L.skvq_decode_step_host.argtypes = [P(SkvqConfig), P(SkvqCacheStruct), vp, vp, vp, vp, vp, P(SkvqAttnArgs), vp]
        L.skvq_decode_attention_noalloc.restype = c_int
        L.skvq_decode_attention_noalloc.argtypes = [P(SkvqConfig), P(SkvqCacheStruct), vp, vp, ctypes.c_float,
                                                    ctypes.c_int32, ctypes.c_int32, vp]
        _lib = L
    return _lib


def _check(code: int, where: str) -> None:
    if code != SKVQ_OK:
        raise SkvqError(code, where)


def _dptr(t) -> int | None:
    return None if t is None else t.data_ptr()


def _stream(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


# ---------------------------------------------------------------- plain wrappers, same names as the C ABI
def skvq_version() -> int:
    return lib().skvq_version()


def skvq_strerror(code: int) -> str:
    return lib().skvq_strerror(code).decode()


def skvq_launch_count() -> int:
    return int(lib().skvq_launch_count())


def skvq_check_config(cfg: SkvqConfig) -> int:
    return lib().skvq_check_config(ctypes.byref(cfg))


def skvq_check_group_bounds(cfg: SkvqConfig, bounds_host) -> int:
    """bounds_host: contiguous int32 numpy array [Hkv, ng+1] in host memory."""
    return lib().skvq_check_group_bounds(ctypes.byref(cfg), bounds_host.ctypes.data)


def skvq_quant_capacity(cfg: SkvqConfig) -> int:
    return lib().skvq_quant_capacity(ctypes.byref(cfg))


def skvq_cache_sizes(cfg: SkvqConfig) -> list[int]:
    out = (ctypes.c_size_t * 6)()
    _check(lib().skvq_cache_sizes(ctypes.byref(cfg), out), "skvq_cache_sizes")
    return list(out)


def skvq_sink_bytes(cfg: SkvqConfig) -> int:
    return int(lib().skvq_sink_bytes(ctypes.byref(cfg)))


def skvq_workspace_size(cfg: SkvqConfig, max_len_hint: int, n_splits: int = 0) -> int:
    return int(lib().skvq_workspace_size(ctypes.byref(cfg), max_len_hint, n_splits))


def skvq_step_staging_size(cfg: SkvqConfig) -> int:
    return int(lib().skvq_step_staging_size(ctypes.byref(cfg)))


def skvq_quantize_append(cfg: SkvqConfig, cache: SkvqCacheStruct, k, v, n_new_per_seq, n_new: int, stream=None) -> None:
    _check(lib().skvq_quantize_append(ctypes.byref(cfg), ctypes.byref(cache), _dptr(k), _dptr(v),
                                      _dptr(n_new_per_seq), n_new, _stream(stream)), "skvq_quantize_append")


def skvq_decode_attention(cfg: SkvqConfig, cache: SkvqCacheStruct, q, out, args: SkvqAttnArgs, stream=None) -> None:
    _check(lib().skvq_decode_attention(ctypes.byref(cfg), ctypes.byref(cache), _dptr(q), _dptr(out),
                                       ctypes.byref(args), _stream(stream)), "skvq_decode_attention")


def skvq_decode_step_host(cfg, cache, k_new_host, v_new_host, q_host, out_host, staging, args, stream=None) -> None:
    _check(lib().skvq_decode_step_host(ctypes.byref(cfg), ctypes.byref(cache), k_new_host.data_ptr(),
                                       v_new_host.data_ptr(), q_host.data_ptr(), out_host.data_ptr(),
                                       _dptr(staging), ctypes.byref(args), _stream(stream)), "skvq_decode_step_host")


def skvq_decode_attention_noalloc(cfg, cache, q, out, sm_scale, max_len_hint, n_splits=0, stream=None) -> None:
    """Decode attention whose split scratch is the library's built-in device array: for callers that cannot
    allocate or lend a workspace.  Shapes beyond SKVQ_NOALLOC_SCRATCH_BYTES raise SkvqError(SKVQ_ERR_SCRATCH_LIMIT)."""
    _check(lib().skvq_decode_attention_noalloc(ctypes.byref(cfg), ctypes.byref(cache), _dptr(q), _dptr(out),
                                               float(sm_scale), int(max_len_hint), int(n_splits), _stream(stream)),
           "skvq_decode_attention_noalloc")


# ---------------------------------------------------------------- device-memory holder
class SkvqCache:
    """Allocates the cache buffers as torch tensors (device memory only) and keeps the C structs.

    reorder_k/_v: int32 [Hkv, D]; alpha_k/_v: float32 [Hkv, D/G] (host arrays or tensors); bounds_k/_v: optional
    int32 [Hkv, D/G + 1] group boundaries (host arrays), checked with skvq_check_group_bounds before the upload.
    """

    def __init__(self, batch, n_q_heads, n_kv_heads, head_dim, k_bits, v_bits, group_size, window, max_tokens,
                 reorder_k, reorder_v, alpha_k, alpha_v, device="cuda:0", n_sink=0, meta_fp8=False, bounds_k=None,
                 bounds_v=None):
        self.cfg = SkvqConfig(batch, n_q_heads, n_kv_heads, head_dim, k_bits, v_bits, group_size, window, max_tokens,
                              n_sink, 1 if meta_fp8 else 0)
        _check(skvq_check_config(self.cfg), "skvq_check_config")
        self.device = torch.device(device)
        self.cap = skvq_quant_capacity(self.cfg)
        self.ng = head_dim // group_size
        sizes = skvq_cache_sizes(self.cfg)
        B, H, W, D = batch, n_kv_heads, window, head_dim
        dev = self.device
        rows = B * H * self.cap
        self.k_codes = torch.zeros((B, H, self.cap, sizes[0] // rows), dtype=torch.uint8, device=dev)
        self.v_codes = torch.zeros((B, H, self.cap, sizes[1] // rows), dtype=torch.uint8, device=dev)
        meta_t = torch.uint8 if meta_fp8 else torch.float16      # {h, z} per (token, group): E4M3 bytes or fp16
        self.k_meta = torch.zeros((B, H, self.cap, self.ng, 2), dtype=meta_t, device=dev)
        self.v_meta = torch.zeros((B, H, self.cap, self.ng, 2), dtype=meta_t, device=dev)
        self.k_win = torch.zeros((B, H, max(W, 1), D), dtype=torch.float16, device=dev)
        self.v_win = torch.zeros((B, H, max(W, 1), D), dtype=torch.float16, device=dev)
        got = [t.numel() * t.element_size() for t in (self.k_codes, self.v_codes, self.k_meta, self.v_meta)]
        assert got == sizes[:4], (got, sizes)
        self.k_sink = torch.zeros((B, H, max(n_sink, 1), D), dtype=torch.float16, device=dev)
        self.v_sink = torch.zeros((B, H, max(n_sink, 1), D), dtype=torch.float16, device=dev)
        assert n_sink == 0 or self.k_sink.numel() * 2 == skvq_sink_bytes(self.cfg)
        self.lengths = torch.zeros((B,), dtype=torch.int32, device=dev)
        self.status = torch.zeros((4,), dtype=torch.int32, device=dev)
        self.reorder_k = torch.as_tensor(reorder_k, dtype=torch.int32).reshape(H, D).contiguous().to(dev)
        self.reorder_v = torch.as_tensor(reorder_v, dtype=torch.int32).reshape(H, D).contiguous().to(dev)
        self.alpha_k = torch.as_tensor(alpha_k, dtype=torch.float32).reshape(H, self.ng).contiguous().to(dev)
        self.alpha_v = torch.as_tensor(alpha_v, dtype=torch.float32).reshape(H, self.ng).contiguous().to(dev)
        self.bounds_k = self._upload_bounds(bounds_k)
        self.bounds_v = self._upload_bounds(bounds_v)
        self.struct = SkvqCacheStruct(*[t.data_ptr() for t in (
            self.k_codes, self.v_codes, self.k_meta, self.v_meta, self.k_win, self.v_win, self.lengths,
            self.reorder_k, self.reorder_v, self.alpha_k, self.alpha_v, self.status, self.k_sink, self.v_sink)],
            _dptr(self.bounds_k), _dptr(self.bounds_v))
        self._workspace = None

    def _upload_bounds(self, bounds):
        if bounds is None:
            return None
        import numpy as np
        b = np.ascontiguousarray(bounds, dtype=np.int32).reshape(self.cfg.n_kv_heads, self.ng + 1)
        _check(skvq_check_group_bounds(self.cfg, b), "skvq_check_group_bounds")
        return torch.from_numpy(b).to(self.device)

    @classmethod
    def for_workload(cls, w, max_tokens=None, device="cuda:0"):
        """Cache for a ``workloads.Workload`` with its reorder index and clip factors."""
        mt = w.context if max_tokens is None else max_tokens
        return cls(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.k_bits, w.v_bits, w.group_size, w.window, mt,
                   w.reorder_index("k"), w.reorder_index("v"), w.alphas(), w.alphas(), device=device, n_sink=w.n_sink,
                   meta_fp8=w.meta_fp8, bounds_k=w.bounds(), bounds_v=w.bounds())

    def nbytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in (self.k_codes, self.v_codes, self.k_meta, self.v_meta,
                                                          self.k_win, self.v_win)) + \
            (2 * self.k_sink.numel() * 2 if self.cfg.n_sink else 0)

    def append(self, k, v, n_new_per_seq=None, stream=None) -> None:
        """k, v: half [B, n, Hkv, D] CUDA tensors; n_new_per_seq: optional int32 [B] CUDA tensor."""
        assert k.is_cuda and v.is_cuda and k.dtype == torch.float16 and k.is_contiguous() and v.is_contiguous()
        assert k.shape == v.shape and k.shape[0] == self.cfg.batch and tuple(k.shape[2:]) == (self.cfg.n_kv_heads,
                                                                                             self.cfg.head_dim)
        skvq_quantize_append(self.cfg, self.struct, k, v, n_new_per_seq, int(k.shape[1]), stream)

    def attn_args(self, sm_scale, max_len_hint, n_splits=0, ev_begin=None, ev_end=None) -> SkvqAttnArgs:
        need = skvq_workspace_size(self.cfg, max_len_hint, n_splits)
        if self._workspace is None or self._workspace.numel() * 4 < need:
            self._workspace = torch.empty((max(need, 16) + 3) // 4, dtype=torch.float32, device=self.device)
        return SkvqAttnArgs(float(sm_scale), int(max_len_hint), int(n_splits), self._workspace.data_ptr(),
                            self._workspace.numel() * 4,
                            None if ev_begin is None else ev_begin.cuda_event,
                            None if ev_end is None else ev_end.cuda_event)

    def attention(self, q, sm_scale, max_len_hint, out=None, n_splits=0, stream=None):
        """q: half [B, Hq, D] CUDA tensor -> half [B, Hq, D]."""
        assert q.is_cuda and q.dtype == torch.float16 and q.is_contiguous()
        if out is None:
            out = torch.empty_like(q)
        skvq_decode_attention(self.cfg, self.struct, q, out, self.attn_args(sm_scale, max_len_hint, n_splits), stream)
        return out

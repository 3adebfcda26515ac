"""Seeded synthetic inputs shaped like long-context decoding workloads.

This module holds no quantization or attention arithmetic: it only draws random
keys, values and queries, and derives the fixed channel-reorder index that the
method treats as an offline-calibrated input.  Both the CUDA tests/benchmark and
the CPU checker consume it, so that they see identical inputs.

Recipe (per workload, numpy Philox streams keyed by (seed, tensor, sequence, chunk)):
  * per (KV head, channel) a key scale sigma = exp(0.5 * n), n ~ N(0, 1); ``n_outliers``
    distinct channels per KV head get their sigma multiplied by ``outlier_scale``;
  * K[b, t, h, c] = fp16(sigma[h, c] * N(0, 1)); V and q are fp16(N(0, 1));
  * reorder index per KV head = stable ascending argsort of the per-channel
    (max - min) over the first ``calib_tokens`` tokens of sequence 0, separately for K and V;
  * one scalar clip factor alpha broadcast to every (head, group);
  * ragged workloads draw per-sequence lengths uniformly from ``ragged`` (inclusive).
Tokens are generated in independent chunks of ``CHUNK`` tokens so any slice of a very
long sequence can be regenerated without producing the rest.
"""
from __future__ import annotations

import dataclasses
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

CHUNK = 4096
_TENSOR_ID = {"k": 1, "v": 2, "q": 3, "sigma": 4, "outliers": 5, "lengths": 6, "k_new": 7, "v_new": 8}


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    context: int                 # tokens per sequence (upper bound when ragged)
    window: int
    k_bits: int
    v_bits: int
    group_size: int
    alpha: float
    n_outliers: int
    outlier_scale: float
    seed: int
    ragged: tuple | None = None  # (lo, hi) inclusive per-sequence length range
    calib_tokens: int = 512
    n_sink: int = 0              # first positions kept fp16 for good (attention sinks; the paper's experiments use 5)
    meta_fp8: bool = False       # scale and zero point stored in FP8 E4M3 instead of fp16
    group_bounds: tuple | None = None   # boundaries of groups of unequal width (0, ..., head_dim), same for every head and
                                        # for keys and values; len - 1 must equal head_dim / group_size

    @property
    def sm_scale(self) -> float:
        return float(np.float32(1.0 / np.sqrt(self.head_dim)))

    def scaled(self, **kw) -> "Workload":
        """Same distributions and quantization settings at other sizes."""
        return dataclasses.replace(self, **kw)

    # ---------------------------------------------------------------- random streams
    def _rng(self, tensor: str, b: int = 0, chunk: int = 0) -> np.random.Generator:
        key = (np.uint64(self.seed) << np.uint64(20)) ^ (np.uint64(_TENSOR_ID[tensor]) << np.uint64(56))
        ctr = (np.uint64(b) << np.uint64(32)) | np.uint64(chunk)
        return np.random.Generator(np.random.Philox(key=int(key), counter=[0, 0, 0, int(ctr)]))

    def key_sigma(self) -> np.ndarray:
        """float32 [Hkv, D] per-channel key scale including the outlier channels."""
        rng = self._rng("sigma")
        sigma = np.exp(0.5 * rng.standard_normal((self.n_kv_heads, self.head_dim))).astype(np.float32)
        rng_o = self._rng("outliers")
        for h in range(self.n_kv_heads):
            ch = rng_o.choice(self.head_dim, size=self.n_outliers, replace=False)
            sigma[h, ch] *= np.float32(self.outlier_scale)
        return sigma

    def lengths(self) -> np.ndarray:
        """int32 [B] tokens per sequence."""
        if self.ragged is None:
            return np.full((self.batch,), self.context, dtype=np.int32)
        lo, hi = self.ragged
        return self._rng("lengths").integers(lo, hi + 1, size=self.batch).astype(np.int32)

    def _chunk(self, tensor: str, b: int, c: int, sigma) -> np.ndarray:
        x = self._rng(tensor, b, c).standard_normal((CHUNK, self.n_kv_heads, self.head_dim), dtype=np.float32)
        if sigma is not None:
            x *= sigma[None]
        return x.astype(np.float16)

    def tokens(self, tensor: str, b: int, t0: int, t1: int) -> np.ndarray:
        """float16 [t1-t0, Hkv, D]: tokens t0..t1-1 of sequence b of tensor 'k' or 'v' (original channel order)."""
        assert tensor in ("k", "v") and 0 <= t0 <= t1
        sigma = self.key_sigma() if tensor == "k" else None
        out = np.empty((t1 - t0, self.n_kv_heads, self.head_dim), dtype=np.float16)
        if t1 == t0:
            return out
        chunks = list(range(t0 // CHUNK, (t1 - 1) // CHUNK + 1))

        def fill(c):
            x = self._chunk(tensor, b, c, sigma)
            lo, hi = max(t0, c * CHUNK), min(t1, (c + 1) * CHUNK)
            out[lo - t0:hi - t0] = x[lo - c * CHUNK:hi - c * CHUNK]

        if len(chunks) == 1:
            fill(chunks[0])
        else:
            with ThreadPoolExecutor(max_workers=min(32, max(8, os.cpu_count() or 8))) as ex:
                list(ex.map(fill, chunks))
        return out

    def prefill(self, tensor: str, n: int | None = None) -> np.ndarray:
        """float16 [B, n, Hkv, D]: the first n tokens (default: context) of every sequence."""
        n = self.context if n is None else n
        return np.stack([self.tokens(tensor, b, 0, n) for b in range(self.batch)], axis=0)

    def new_token(self, tensor: str, step: int) -> np.ndarray:
        """float16 [B, 1, Hkv, D]: the token appended at decode step ``step`` (same distributions)."""
        assert tensor in ("k", "v")
        sigma = self.key_sigma() if tensor == "k" else None
        x = self._rng(tensor + "_new", 0, step).standard_normal(
            (self.batch, 1, self.n_kv_heads, self.head_dim), dtype=np.float32)
        if sigma is not None:
            x *= sigma[None, None]
        return x.astype(np.float16)

    def query(self, step: int = 0) -> np.ndarray:
        """float16 [B, Hq, D]."""
        return self._rng("q", 0, step).standard_normal(
            (self.batch, self.n_q_heads, self.head_dim), dtype=np.float32).astype(np.float16)

    def reorder_index(self, tensor: str) -> np.ndarray:
        """int32 [Hkv, D]: stable ascending argsort of per-channel range over the calibration tokens."""
        x = self.tokens(tensor, 0, 0, self.calib_tokens).astype(np.float32)
        rng_c = x.max(axis=0) - x.min(axis=0)                       # [Hkv, D]
        return np.argsort(rng_c, axis=1, kind="stable").astype(np.int32)

    def bounds(self):
        """int32 [Hkv, ng+1] group boundaries, or None for equal groups."""
        if self.group_bounds is None:
            return None
        assert len(self.group_bounds) - 1 == self.head_dim // self.group_size
        return np.tile(np.asarray(self.group_bounds, dtype=np.int32), (self.n_kv_heads, 1))

    def alphas(self) -> np.ndarray:
        """float32 [Hkv, D/G] clip factors (one scalar broadcast)."""
        return np.full((self.n_kv_heads, self.head_dim // self.group_size), self.alpha, dtype=np.float32)


def configs() -> list[Workload]:
    """The five benchmark workloads (index = configuration number)."""
    s = 20240506
    return [
        Workload("tiny_mha_4k", 1, 32, 32, 128, 4096, 128, 2, 2, 128, 0.9, 4, 15.0, s + 0),
        Workload("llama2_7b_mha_32k", 8, 32, 32, 128, 32768, 128, 2, 2, 128, 0.9, 4, 15.0, s + 1),
        Workload("mistral_7b_gqa_128k", 4, 32, 8, 128, 131072, 128, 2, 2, 32, 0.85, 8, 20.0, s + 2),
        Workload("long_1m", 1, 32, 32, 128, 1048576, 128, 2, 2, 128, 0.9, 4, 15.0, s + 3),
        Workload("serving_mix_4bit", 64, 32, 32, 128, 16384, 256, 4, 4, 64, 0.95, 4, 15.0, s + 4,
                 ragged=(1024, 16384)),
    ]


BITS_TERNARY = 15      # v_bits of the three-level ("1.5-bit") value codes: five base-3 digits per byte


def packed_row_bytes(D: int, bits: int) -> int:
    """Bytes of one packed row of D codes in the cache."""
    return (D + 4) // 5 if bits == BITS_TERNARY else D * bits // 8


def algorithmic_bytes(w: Workload, lengths=None) -> int:
    """Bytes one decode-attention call must move: packed codes + scale/zero of the quantized
    prefix, the fp16 window and sinks, and q/out.  Split scratch is not counted."""
    lengths = w.lengths() if lengths is None else np.asarray(lengths)
    D, ng = w.head_dim, w.head_dim // w.group_size
    mb = 2 if w.meta_fp8 else 4      # bytes of {scale, zero} per (token, group)
    per_tok = (packed_row_bytes(D, w.k_bits) + mb * ng) + (packed_row_bytes(D, w.v_bits) + mb * ng)
    total = 0
    for L in lengths.tolist():
        lq = max(L - w.window, 0)
        ns = min(w.n_sink, lq)
        total += w.n_kv_heads * ((lq - ns) * per_tok + (ns + min(L, w.window)) * D * 2 * 2)
    total += w.batch * w.n_q_heads * D * 2 * 2
    return int(total)


def partition_kernel_bytes(w: Workload, lengths=None) -> int:
    """The share of ``algorithmic_bytes`` that the partition kernel itself must move: packed codes and
    scale/zero of the quantized prefix plus q (the fp16 window and the output belong to the merge kernel)."""
    lengths = w.lengths() if lengths is None else np.asarray(lengths)
    D, ng = w.head_dim, w.head_dim // w.group_size
    mb = 2 if w.meta_fp8 else 4      # bytes of {scale, zero} per (token, group)
    per_tok = (packed_row_bytes(D, w.k_bits) + mb * ng) + (packed_row_bytes(D, w.v_bits) + mb * ng)
    total = sum(w.n_kv_heads * max(L - w.window - w.n_sink, 0) * per_tok for L in lengths.tolist())
    return int(total + w.batch * w.n_q_heads * D * 2)

"""Offline calibration of the inputs the SKVQ cache treats as fixed: channel reorder index, group boundaries
and clip factors (Sec. 3.1; Eq. 3; the prologue of Algorithm 1: get_permutation_matrix, get_group_clipping).

This runs once per model, on the CPU, over a small calibration sample; it is not on the decode path and the
library never calls it.  Its results are plain arrays that go into ``skvq_cache`` (reorder_*, group_bounds_*,
alpha_*).  Everything here is numpy:

  * per channel, the distribution feature is the value range (max - min) over the calibration tokens;
  * channels are clustered by that feature with 1-D k-means into as many clusters as the row has groups; in one
    dimension clusters are runs of the sorted order, so the reorder index is the argsort of the feature and the
    groups are consecutive runs of reordered channels, of unequal width (Sec. 4.2: the number of groups is kept so
    that the average width equals the equal-group setting);
  * the library wants group boundaries on multiples of 32 channels, so the run lengths are rounded to that grid;
  * the clip factor of every group is found by a grid search that minimises the mean squared error of the attention
    output against full-precision attention on the calibration sample (Eq. 3), one group at a time.
"""
from __future__ import annotations

import numpy as np

GRANULE = 32


# ------------------------------------------------------------------------------------------------ grouping
def channel_feature(x: np.ndarray) -> np.ndarray:
    """Range (max - min) of every channel; x: [tokens, D] -> float64 [D]."""
    x = np.asarray(x, dtype=np.float64)
    return x.max(axis=0) - x.min(axis=0)


def kmeans_1d(values: np.ndarray, k: int, iters: int = 100) -> np.ndarray:
    """Lloyd's algorithm on scalars; returns the cluster (0..k-1, ordered by centre) of every value.  The centres start
    at evenly spaced quantiles, so the result is deterministic; an emptied cluster is re-seeded at the value farthest
    from its centre."""
    v = np.asarray(values, dtype=np.float64)
    n = v.size
    k = max(1, min(k, n))
    centres = np.quantile(v, (np.arange(k) + 0.5) / k)
    label = np.zeros(n, dtype=np.int64)
    for _ in range(iters):
        new = np.abs(v[:, None] - centres[None, :]).argmin(axis=1)
        for c in range(k):
            if not np.any(new == c):
                far = np.abs(v - centres[new]).argmax()
                new[far] = c
        moved = not np.array_equal(new, label)
        label = new
        centres = np.array([v[label == c].mean() for c in range(k)])
        if not moved:
            break
    order = np.argsort(centres, kind="stable")
    rank = np.empty(k, dtype=np.int64)
    rank[order] = np.arange(k)
    return rank[label]


def round_bounds(sizes, total: int, granule: int = GRANULE) -> np.ndarray:
    """Boundaries 0 = b_0 < b_1 < ... < b_k = total on multiples of ``granule`` that follow the cumulative cluster
    sizes as closely as the grid allows (every group keeps at least one granule)."""
    k = len(sizes)
    assert total % granule == 0 and k * granule <= total
    cum = np.cumsum(sizes)[:-1].astype(np.float64)
    b = [0]
    for i, c in enumerate(cum):
        lo = b[-1] + granule                           # at least one granule for group i
        hi = total - (k - 1 - i) * granule             # and one for every group still to come
        r = int(round(c / granule)) * granule
        b.append(int(min(max(r, lo), hi)))
    b.append(total)
    return np.asarray(b, dtype=np.int32)


def reorder_and_groups(x: np.ndarray, n_groups: int, granule: int = GRANULE):
    """Reorder index and group boundaries of one KV head from calibration tokens x [tokens, D].

    Returns (idx int32 [D], bounds int32 [n_groups + 1]): stored channel j reads source channel idx[j]
    (stored[j] = src[idx[j]]); group g covers stored channels [bounds[g], bounds[g+1])."""
    f = channel_feature(x)
    idx = np.argsort(f, kind="stable").astype(np.int32)          # clusters of a 1-D k-means are runs of this order
    if n_groups == 1:
        return idx, np.array([0, f.size], dtype=np.int32)
    label = kmeans_1d(f, n_groups)
    sizes = np.bincount(label, minlength=n_groups)
    return idx, round_bounds(sizes, f.size, granule)


# ------------------------------------------------------------------------------------------------ clip factors
def fake_quant(xr: np.ndarray, bounds: np.ndarray, alpha: np.ndarray, bits: int) -> np.ndarray:
    """Quantize and dequantize reordered rows xr [tokens, D] (fp16 values) group by group, in the arithmetic the cache
    uses: lo = alpha*min, hi = alpha*max, h = fp16((hi - lo)/qmax), z = fp16(lo), code = clip(rint((x - z)/h)),
    x^ = h*code + z; fp32 throughout, returned as float64."""
    xr = np.asarray(xr, dtype=np.float16).astype(np.float32)
    qmax = np.float32(2 if bits == 15 else (1 << bits) - 1)      # 15: the three-level code
    out = np.empty(xr.shape, dtype=np.float64)
    for g in range(len(bounds) - 1):
        a, b = int(bounds[g]), int(bounds[g + 1])
        seg = xr[:, a:b]
        al = np.float32(alpha[g])
        lo = al * seg.min(axis=1) + np.float32(0)
        hi = al * seg.max(axis=1) + np.float32(0)
        h = ((hi - lo) / qmax).astype(np.float16).astype(np.float32)
        z = lo.astype(np.float16).astype(np.float32)
        with np.errstate(divide="ignore", invalid="ignore"):
            c = np.rint((seg - z[:, None]) / h[:, None])
        c = np.where(h[:, None] != 0, np.clip(c, 0, qmax), np.float32(0))
        out[:, a:b] = h[:, None].astype(np.float64) * c.astype(np.float64) + z[:, None].astype(np.float64)
    return out


def _attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, sm_scale: float) -> np.ndarray:
    """softmax(sm_scale * q k^T) v for queries q [n_q, D] over one head's k, v [tokens, D] (float64)."""
    s = sm_scale * (q @ k.T)
    s -= s.max(axis=1, keepdims=True)
    p = np.exp(s)
    p /= p.sum(axis=1, keepdims=True)
    return p @ v


def search_alpha(q, k, v, idx_k, idx_v, bounds_k, bounds_v, k_bits: int, v_bits: int, sm_scale: float,
                 grid=None, sweeps: int = 1):
    """Clip factors of one KV head (Eq. 3): alpha* = argmin || Attn(q, K, V) - Attn(q, Q(K), Q(V)) ||^2 over the grid,
    one group at a time (keys first, then values), the other groups at their current best.

    q [n_q, D] are calibration queries of the head(s) that read this KV head, k, v [tokens, D] its calibration tokens,
    all in the model's channel order.  Returns (alpha_k [ng], alpha_v [ng], mse_before, mse_after) where "before" is
    alpha = 1 everywhere."""
    grid = np.round(np.arange(0.70, 1.0001, 0.025), 3) if grid is None else np.asarray(grid, dtype=np.float64)
    q = np.asarray(q, np.float16).astype(np.float64)
    kr = np.asarray(k, np.float16)[:, idx_k]
    vr = np.asarray(v, np.float16)[:, idx_v]
    qk = q[:, idx_k]                                         # the query follows the keys' permutation (Eq. 1)
    ref = _attention(qk, kr.astype(np.float64), vr.astype(np.float64), sm_scale)

    def mse(ak, av):
        out = _attention(qk, fake_quant(kr, bounds_k, ak, k_bits), fake_quant(vr, bounds_v, av, v_bits), sm_scale)
        return float(np.mean((out - ref) ** 2))

    ak = np.ones(len(bounds_k) - 1)
    av = np.ones(len(bounds_v) - 1)
    before = mse(ak, av)
    best = before
    for _ in range(sweeps):
        for arr in (ak, av):
            for g in range(arr.size):
                keep = arr[g]
                for cand in grid:
                    arr[g] = cand
                    m = mse(ak, av)
                    if m < best:
                        best, keep = m, cand
                arr[g] = keep
    return ak.astype(np.float32), av.astype(np.float32), before, best


def calibrate(q, k, v, n_groups: int, k_bits: int, v_bits: int, sm_scale: float, grid=None, granule: int = GRANULE):
    """All heads at once.  q [n_q, Hq, D], k, v [tokens, Hkv, D] calibration tensors (model channel order).

    Returns a dict of arrays ready for the cache: reorder_k/_v int32 [Hkv, D], bounds_k/_v int32 [Hkv, n_groups + 1],
    alpha_k/_v float32 [Hkv, n_groups], and the attention-output MSE per head before (alpha = 1) and after the search."""
    k, v, q = np.asarray(k), np.asarray(v), np.asarray(q)
    hkv, hq = k.shape[1], q.shape[1]
    rep = hq // hkv
    out = {n: [] for n in ("reorder_k", "reorder_v", "bounds_k", "bounds_v", "alpha_k", "alpha_v", "mse_before", "mse_after")}
    for h in range(hkv):
        ik, bk = reorder_and_groups(k[:, h], n_groups, granule)
        iv, bv = reorder_and_groups(v[:, h], n_groups, granule)
        qh = q[:, h * rep:(h + 1) * rep].reshape(-1, q.shape[-1])
        ak, av, m0, m1 = search_alpha(qh, k[:, h], v[:, h], ik, iv, bk, bv, k_bits, v_bits, sm_scale, grid)
        for n, val in zip(out, (ik, iv, bk, bv, ak, av, m0, m1)):
            out[n].append(val)
    return {n: np.stack(val) if n.startswith(("reorder", "bounds", "alpha")) else np.asarray(val) for n, val in out.items()}

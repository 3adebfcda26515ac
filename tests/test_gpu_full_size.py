"""Parity at the benchmark's full sizes, in the launch configuration the benchmark times.

The GPU cache is prefilled chunk by chunk with the library's own quantize_append exactly as ``bench.py`` does
it, a few single-token decode appends follow, and decode attention runs with the default partition.  The CPU
oracle cannot redo a whole configuration in reasonable time, so it redoes SAMPLED (sequence, KV head) pairs in
full: every stored row of those pairs must be bit-exact and the attention output of their query heads within
the tolerance.  Configurations 1 to 4 run at their full sizes (configuration 3 also once with two heads).
"""
import numpy as np
import pytest

from oracle import skvq_oracle as orc
from paper_2405_06219_b200 import workloads

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

ATTN_TOL = 2e-3      # max-abs error of the attention output against the fp64 oracle


def prefill_like_the_benchmark(w, cache, chunk=32768):
    lengths = w.lengths()
    Lmax = int(lengths.max())
    chunk = max(256, min(chunk, (1 << 29) // (w.batch * w.n_kv_heads * w.head_dim * 2) // 256 * 256))
    for t0 in range(0, Lmax, chunk):
        t1 = min(t0 + chunk, Lmax)
        n_b = np.clip(lengths - t0, 0, t1 - t0).astype(np.int32)
        k = np.zeros((w.batch, t1 - t0, w.n_kv_heads, w.head_dim), np.float16)
        v = np.zeros_like(k)
        for b in range(w.batch):
            if n_b[b]:
                k[b, :n_b[b]] = w.tokens("k", b, t0, t0 + int(n_b[b]))
                v[b, :n_b[b]] = w.tokens("v", b, t0, t0 + int(n_b[b]))
        cache.append(torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), torch.from_numpy(n_b).cuda())
        torch.cuda.synchronize()


def oracle_for_pairs(w, b, kv_heads, n_steps):
    """The oracle's cache for sequence b and the listed KV heads only (batch 1), after the same tokens."""
    rep = w.n_q_heads // w.n_kv_heads
    L = int(w.lengths()[b])
    a = w.alphas()[kv_heads]
    oc = orc.OracleCache(1, len(kv_heads) * rep, len(kv_heads), w.head_dim, w.k_bits, w.v_bits, w.group_size, w.window,
                         L + n_steps + 64, w.reorder_index("k")[kv_heads], w.reorder_index("v")[kv_heads], a, a,
                         n_sink=w.n_sink, meta_fp8=w.meta_fp8)
    step = 1 << 16
    for t0 in range(0, L, step):
        t1 = min(t0 + step, L)
        oc.append(np.ascontiguousarray(w.tokens("k", b, t0, t1)[None][:, :, kv_heads]),
                  np.ascontiguousarray(w.tokens("v", b, t0, t1)[None][:, :, kv_heads]))
    return oc


def pick_sequence(lengths, which):
    """An index into the batch: an int as it is, or the longest / shortest / median-length sequence."""
    if isinstance(which, int):
        return which
    order = np.argsort(lengths, kind="stable")
    return int({"longest": order[-1], "shortest": order[0], "median": order[len(order) // 2]}[which])


@pytest.mark.parametrize("cfg_i,kw,picks", [
    (1, dict(), [(7, [0, 31])]),                                    # 32k x batch 8, one query head per KV head
    (2, dict(), [(3, [5])]),                                        # 128k x batch 4, four query heads per KV head, group 32
    (2, dict(n_q_heads=24, meta_fp8=True, n_sink=5), [(1, [2])]),   # the tcgen05 kernel, FP8 parameters, sinks
    (3, dict(n_q_heads=2, n_kv_heads=2), [(0, [1])]),               # one sequence of 1M tokens (two heads instead of 32)
    # configuration 3 as the benchmark runs it: 32 heads, so a CTA's run of the flat partition is 18.5 heads' worth of
    # slots and head boundaries fall inside runs; head 1 starts inside a run, head 18 ends inside one
    (3, dict(), [(0, [1, 18])]),
    # configuration 4 in full: 64 ragged sequences (plan kernel + header in the workspace), 4-bit codes, group 64, window 256
    (4, dict(), [("longest", [0]), ("shortest", [31]), ("median", [13])]),
    # three-level ("1.5-bit") values at full size: rewritten to 2-bit rows inside the integer kernel (configuration 1) and the
    # grouped-query kernel (configuration 2), prefilled by the tile kernel's base-3 packing
    (1, dict(v_bits=15), [(6, [17])]),
    (2, dict(v_bits=15), [(2, [3])]),
])
def test_full_size_sampled_pairs_match_oracle(cfg_i, kw, picks):
    from paper_2405_06219_b200 import binding as B
    w = workloads.configs()[cfg_i].scaled(**kw)
    n_steps = 3
    rep = w.n_q_heads // w.n_kv_heads
    lengths = w.lengths()
    gpu = B.SkvqCache.for_workload(w, int(lengths.max()) + n_steps + 64)
    prefill_like_the_benchmark(w, gpu)
    new_tokens = [(w.new_token("k", s), w.new_token("v", s)) for s in range(n_steps)]
    for kn, vn in new_tokens:                                       # decode steps: one token per sequence
        gpu.append(torch.from_numpy(kn).cuda(), torch.from_numpy(vn).cuda())
    q = w.query(11)
    out = gpu.attention(torch.from_numpy(q).cuda(), w.sm_scale, int(lengths.max()) + n_steps)      # default partition
    torch.cuda.synchronize()
    assert np.isfinite(out.cpu().numpy()).all()
    assert int(gpu.status[0]) == 0

    def bits(t):        # fp16 bit patterns, or one E4M3 byte per parameter (kept in a uint16 by the oracle)
        x = t.cpu().numpy()
        return x.astype(np.uint16) if w.meta_fp8 else x.view(np.uint16)

    for which, kv_heads in picks:
        b = pick_sequence(lengths, which)
        oc = oracle_for_pairs(w, b, kv_heads, n_steps)
        for kn, vn in new_tokens:
            oc.append(np.ascontiguousarray(kn[b:b + 1][:, :, kv_heads]), np.ascontiguousarray(vn[b:b + 1][:, :, kv_heads]))
        L = int(lengths[b]) + n_steps
        assert int(gpu.lengths[b]) == L
        lq, ns = max(L - w.window, 0), min(w.n_sink, max(L - w.window, 0))
        for i, hk in enumerate(kv_heads):
            assert np.array_equal(gpu.k_codes[b, hk, ns:lq].cpu().numpy(), oc.k_codes[0, i, ns:lq]), f"k codes, head {hk}"
            assert np.array_equal(gpu.v_codes[b, hk, ns:lq].cpu().numpy(), oc.v_codes[0, i, ns:lq]), f"v codes, head {hk}"
            assert np.array_equal(bits(gpu.k_meta[b, hk, ns:lq]), oc.k_meta.view(np.uint16)[0, i, ns:lq]), f"k scale/zero, head {hk}"
            assert np.array_equal(bits(gpu.v_meta[b, hk, ns:lq]), oc.v_meta.view(np.uint16)[0, i, ns:lq]), f"v scale/zero, head {hk}"
            assert np.array_equal(gpu.k_sink[b, hk, :ns].cpu().numpy().view(np.uint16), oc.k_sink.view(np.uint16)[0, i, :ns])
            if w.window:
                slots = sorted({t % w.window for t in range(lq, L)})
                assert np.array_equal(gpu.k_win[b, hk][slots].cpu().numpy().view(np.uint16), oc.k_win.view(np.uint16)[0, i][slots])
                assert np.array_equal(gpu.v_win[b, hk][slots].cpu().numpy().view(np.uint16), oc.v_win.view(np.uint16)[0, i][slots])
        q_heads = [hk * rep + r for hk in kv_heads for r in range(rep)]
        want = oc.attention(np.ascontiguousarray(q[b:b + 1][:, q_heads]), w.sm_scale)[0]
        got = out[b, q_heads].cpu().numpy().astype(np.float64)
        assert np.abs(got - want).max() <= ATTN_TOL, f"sequence {b} (length {L}), KV heads {kv_heads}"


@pytest.mark.parametrize("kw", [
    dict(n_q_heads=1, n_kv_heads=1),                       # integer kernel, one head
    dict(n_q_heads=4, n_kv_heads=1, group_size=32),        # grouped-query kernel
    dict(n_q_heads=3, n_kv_heads=1, group_size=64),        # tcgen05 kernel
])
def test_one_cta_streams_a_whole_long_sequence(kw):
    """n_splits = 1 gives the whole sequence to one CTA: each warp then accumulates several hundred thousand tokens,
    far more than the int32 value sums hold between two folds unless the kernels fold on their own."""
    from paper_2405_06219_b200 import binding as B
    w = workloads.configs()[1].scaled(batch=1, context=900_000, **kw)
    gpu = B.SkvqCache.for_workload(w, w.context + 64)
    prefill_like_the_benchmark(w, gpu, chunk=1 << 17)
    oc = oracle_for_pairs(w, 0, [0], 0)
    q = w.query(3)
    out = gpu.attention(torch.from_numpy(q).cuda(), w.sm_scale, w.context + 64, n_splits=1)
    torch.cuda.synchronize()
    want = oc.attention(q, w.sm_scale)
    assert np.abs(out.cpu().numpy().astype(np.float64) - want).max() <= ATTN_TOL
    # q = 0: every token has the same probability, so every token contributes full-size digits to the int32 sums
    # (the worst case for their range); the result is the mean of the dequantized values
    q0 = np.zeros_like(q)
    out0 = gpu.attention(torch.from_numpy(q0).cuda(), w.sm_scale, w.context + 64, n_splits=1)
    torch.cuda.synchronize()
    assert np.abs(out0.cpu().numpy().astype(np.float64) - oc.attention(q0, w.sm_scale)).max() <= ATTN_TOL
    assert int(gpu.status[0]) == 0

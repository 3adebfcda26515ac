"""Pins for the CPU oracle's sliding-window cache and its fp64 attention.

The cache semantics are checked against the paper's statement (latest W tokens stay
fp16, everything older is quantized, single appends equal one bulk append); the
attention against library routines (scipy softmax + einsum, torch SDPA in fp64),
and against properties that hold for any softmax attention.
"""
import numpy as np
import pytest
import scipy.special

from oracle import skvq_oracle as orc
from paper_2405_06219_b200 import workloads
from test_oracle_quantizer import unpack_codes

D = 128


def make_cache(B, Hq, Hkv, W, cap, bits=2, group=128, alpha=0.9, seed=0, identity=False, n_sink=0, meta_fp8=False,
               bounds_k=None, bounds_v=None, v_bits=None):
    rng = np.random.default_rng(seed)
    if identity:
        rk = rv = np.tile(np.arange(D, dtype=np.int32), (Hkv, 1))
    else:
        rk = np.stack([rng.permutation(D) for _ in range(Hkv)]).astype(np.int32)
        rv = np.stack([rng.permutation(D) for _ in range(Hkv)]).astype(np.int32)
    ng = D // group if bounds_k is None else np.asarray(bounds_k).shape[-1] - 1
    a = np.full((Hkv, ng), alpha, np.float32)
    return orc.OracleCache(B, Hq, Hkv, D, bits, bits if v_bits is None else v_bits, group, W, cap, rk, rv, a, a,
                           n_sink=n_sink, meta_fp8=meta_fp8, bounds_k=bounds_k, bounds_v=bounds_v)


def rand_kv(B, n, Hkv, seed):
    rng = np.random.default_rng(seed)
    sigma = np.exp(0.5 * rng.standard_normal((Hkv, D))).astype(np.float32)
    sigma[:, :3] *= 15
    k = (rng.standard_normal((B, n, Hkv, D)).astype(np.float32) * sigma).astype(np.float16)
    v = rng.standard_normal((B, n, Hkv, D)).astype(np.float16)
    return k, v


def cache_state(c):
    return [c.k_codes.copy(), c.v_codes.copy(), c.k_meta.view(np.uint16).copy(), c.v_meta.view(np.uint16).copy(),
            c.k_win.view(np.uint16).copy(), c.v_win.view(np.uint16).copy(), c.lengths.copy()]


def mixed_cache_dense(c, b, hk):
    """Independent numpy reconstruction of K~ and V~ (reordered order) for one (sequence, KV head)."""
    L = int(c.lengths[b])
    Lq = max(L - c.W, 0)
    out = []
    for codes, meta, win, sink, bits, bounds in ((c.k_codes, c.k_meta, c.k_win, c.k_sink, c.k_bits, c.bounds_k),
                                                 (c.v_codes, c.v_meta, c.v_win, c.v_sink, c.v_bits, c.bounds_v)):
        code = unpack_codes(codes[b, hk, :Lq], bits).astype(np.float64)
        widths = np.full(c.ng, c.G) if bounds is None else np.diff(bounds[hk])      # channels per group
        if c.meta_fp8:                               # E4M3 bytes: decoded by a library, not by the oracle
            import torch
            meta = torch.from_numpy(meta[b, hk, :Lq].astype(np.uint8)).view(torch.float8_e4m3fn).to(torch.float64).numpy()
        else:
            meta = meta[b, hk, :Lq]
        h = np.repeat(meta[:, :, 0].astype(np.float64), widths, axis=1)
        z = np.repeat(meta[:, :, 1].astype(np.float64), widths, axis=1)
        dense = np.zeros((L, D))
        dense[:Lq] = h * code + z
        ns = min(c.n_sink, Lq)                       # attention sinks: full-precision rows, never quantized
        dense[:ns] = sink[b, hk, :ns].astype(np.float64)
        for t in range(Lq, L):
            dense[t] = win[b, hk, t % c.W].astype(np.float64)
        out.append(dense)
    return out


def brute_attention(c, q, sm_scale):
    out = np.zeros((c.B, c.Hq, D))
    rep = c.Hq // c.Hkv
    for b in range(c.B):
        if c.lengths[b] == 0:
            continue
        for hq in range(c.Hq):
            hk = hq // rep
            Kt, Vt = mixed_cache_dense(c, b, hk)
            qp = q[b, hq].astype(np.float64)[c.reorder_k[hk]]
            p = scipy.special.softmax(float(np.float32(sm_scale)) * (Kt @ qp))
            o = np.einsum("t,td->d", p, Vt)
            out[b, hq, c.reorder_v[hk]] = o
    return out


# ------------------------------------------------------------------ window semantics (Sec. 3.2, Algorithm 1)
@pytest.mark.parametrize("W,n", [(8, 5), (8, 8), (8, 9), (8, 37), (0, 6), (16, 40)])
def test_window_keeps_last_w_tokens_and_quantizes_the_rest(W, n):
    c = make_cache(2, 4, 2, W, 64, group=32, seed=1)
    k, v = rand_kv(2, n, 2, 2)
    assert c.append(k, v) == 0
    assert np.all(c.lengths == n)
    Lq = max(n - W, 0)
    for b in range(2):
        for h in range(2):
            for t in range(Lq, n):                       # window: reordered fp16, slot t mod W
                assert np.array_equal(c.k_win[b, h, t % W], k[b, t, h][c.reorder_k[h]])
                assert np.array_equal(c.v_win[b, h, t % W], v[b, t, h][c.reorder_v[h]])
            if Lq:
                ck, mk = orc.quantize_rows(k[b, :Lq, h], c.reorder_k[h], c.alpha_k[h], 2, 32)
                cv, mv = orc.quantize_rows(v[b, :Lq, h], c.reorder_v[h], c.alpha_v[h], 2, 32)
                assert np.array_equal(c.k_codes[b, h, :Lq], ck) and np.array_equal(c.v_codes[b, h, :Lq], cv)
                assert np.array_equal(c.k_meta[b, h, :Lq].view(np.uint16), mk.view(np.uint16))
                assert np.array_equal(c.v_meta[b, h, :Lq].view(np.uint16), mv.view(np.uint16))
            assert not c.k_codes[b, h, Lq:].any() and not c.v_meta[b, h, Lq:].view(np.uint16).any()


@pytest.mark.parametrize("W", [0, 8, 16])
def test_single_appends_equal_bulk_and_any_chunking(W):
    n = 45
    k, v = rand_kv(2, n, 2, 3)
    bulk = make_cache(2, 2, 2, W, 64, seed=4)
    bulk.append(k, v)
    one = make_cache(2, 2, 2, W, 64, seed=4)
    for t in range(n):
        one.append(k[:, t:t + 1], v[:, t:t + 1])
    chunked = make_cache(2, 2, 2, W, 64, seed=4)
    t = 0
    for step in (1, 7, 2, 20, 15):
        chunked.append(k[:, t:t + step], v[:, t:t + step])
        t += step
    assert t == n
    for other in (one, chunked):
        for a, b in zip(cache_state(bulk), cache_state(other)):
            assert np.array_equal(a, b)


def test_ragged_append_counts_and_capacity():
    c = make_cache(3, 2, 2, 8, 32, seed=5)
    k, v = rand_kv(3, 30, 2, 6)
    assert c.append(k, v, np.array([30, 0, 11], np.int32)) == 0
    assert c.lengths.tolist() == [30, 0, 11]
    ref = make_cache(1, 2, 2, 8, 32, seed=5)
    ref.append(k[2:3, :11], v[2:3, :11])
    assert np.array_equal(c.k_codes[2], ref.k_codes[0]) and np.array_equal(c.k_win[2], ref.k_win[0])
    before = cache_state(c)
    assert c.append(k[:, :5], v[:, :5], np.array([5, 0, 0], np.int32)) == -1      # 35 > capacity 32
    assert c.lengths.tolist() == [30, 0, 11]
    for a, b in zip(before, cache_state(c)):
        assert np.array_equal(a, b)


# ------------------------------------------------------------------ attention
@pytest.mark.parametrize("Hq,Hkv,bits,group,W,L", [(2, 2, 2, 128, 16, 300), (4, 1, 2, 32, 8, 150),
                                                  (4, 2, 4, 64, 32, 100), (2, 2, 2, 128, 0, 64)])
def test_attention_matches_library_brute_force(Hq, Hkv, bits, group, W, L):
    c = make_cache(2, Hq, Hkv, W, 320, bits=bits, group=group, seed=7)
    k, v = rand_kv(2, L, Hkv, 8)
    c.append(k, v, np.array([L, L - 37], np.int32))
    q = np.random.default_rng(9).standard_normal((2, Hq, D)).astype(np.float16)
    got = c.attention(q, 1 / np.sqrt(D))
    want = brute_attention(c, q, 1 / np.sqrt(D))
    assert np.abs(got - want).max() < 1e-12


def test_all_fp16_window_reduces_to_torch_sdpa():
    """W >= L: nothing is quantized and the call is plain attention; torch's fp64 SDPA is the reference."""
    import torch
    L, Hq, Hkv = 50, 4, 2
    c = make_cache(2, Hq, Hkv, 64, 64, seed=10)
    k, v = rand_kv(2, L, Hkv, 11)
    c.append(k, v)
    assert not c.k_codes.any()
    q = np.random.default_rng(12).standard_normal((2, Hq, D)).astype(np.float16)
    got = c.attention(q, 0.11)
    tq = torch.from_numpy(q.astype(np.float64))[:, :, None, :]                        # [B,Hq,1,D]
    tk = torch.from_numpy(k.astype(np.float64)).permute(0, 2, 1, 3).repeat_interleave(Hq // Hkv, 1)
    tv = torch.from_numpy(v.astype(np.float64)).permute(0, 2, 1, 3).repeat_interleave(Hq // Hkv, 1)
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=float(np.float32(0.11)))[:, :, 0].numpy()
    assert np.abs(got - want).max() < 1e-12


def test_reorder_leaves_attention_unchanged_when_nothing_is_quantized():
    """Eq. 1: permuting q and K channels alike, and un-permuting the V output, changes nothing."""
    L, H = 40, 2
    k, v = rand_kv(1, L, H, 13)
    q = np.random.default_rng(14).standard_normal((1, H, D)).astype(np.float16)
    a = make_cache(1, H, H, 64, 64, seed=15)
    b = make_cache(1, H, H, 64, 64, identity=True)
    a.append(k, v)
    b.append(k, v)
    assert np.abs(a.attention(q, 0.1) - b.attention(q, 0.1)).max() < 1e-13


def test_zero_query_gives_mean_of_values_and_outputs_are_convex():
    c = make_cache(1, 2, 2, 16, 128, seed=16)
    k, v = rand_kv(1, 90, 2, 17)
    c.append(k, v)
    out0 = c.attention(np.zeros((1, 2, D), np.float16), 0.3)
    q = np.random.default_rng(18).standard_normal((1, 2, D)).astype(np.float16)
    out = c.attention(q, 0.3)
    for h in range(2):
        _, Vt = mixed_cache_dense(c, 0, h)
        inv = np.empty(D, np.int64)
        inv[c.reorder_v[h]] = np.arange(D)
        Vorig = Vt[:, inv]                                                          # back to original channel order
        assert np.abs(out0[0, h] - Vorig.mean(0)).max() < 1e-12
        assert np.all(out[0, h] <= Vorig.max(0) + 1e-12) and np.all(out[0, h] >= Vorig.min(0) - 1e-12)


def test_dominant_key_selects_its_value_row_and_score_shift_is_invisible():
    H, L, W = 1, 70, 8
    k, v = rand_kv(1, L, H, 19)
    k = (k.astype(np.float32) * 0.05).astype(np.float16)
    k[:, :, :, 0] = 1.0                      # a channel on which all keys agree
    k[0, 20] = 0
    k[0, 20, 0, 0] = 1.0
    k[0, 20, 0, 1] = 40.0                    # token 20 dominates for a query along channel 1
    c = make_cache(1, H, H, W, 128, alpha=1.0, identity=True)
    c.append(k, v)
    q = np.zeros((1, H, D), np.float16)
    q[0, 0, 1] = 30.0
    out = c.attention(q, 1.0)
    _, Vt = mixed_cache_dense(c, 0, 0)
    assert np.abs(out[0, 0] - Vt[20]).max() < 1e-9
    # adding a multiple of a channel on which all keys agree shifts every score alike (nothing quantized here)
    c2 = make_cache(1, H, H, 128, 128, alpha=1.0, seed=22)
    c2.append(k, v)
    q2 = q.copy()
    q2[0, 0, 0] = 7.0
    q[0, 0, 1] = 0.5
    q2[0, 0, 1] = 0.5
    assert np.abs(c2.attention(q, 1.0) - c2.attention(q2, 1.0)).max() < 1e-9


# ------------------------------------------------------------------ attention sinks (Sec. 3.2 filter rules)
@pytest.mark.parametrize("W,n_sink,n", [(8, 5, 40), (8, 5, 10), (8, 5, 4), (0, 3, 20), (16, 20, 30), (8, 64, 200)])
def test_sinks_keep_exact_rows_and_leave_the_other_tokens_alone(W, n_sink, n):
    """A position below n_sink that has left the window holds the token's exact fp16 values (reordered); every
    other token is quantized exactly as in a cache without sinks; chunked appends give the same state."""
    k, v = rand_kv(2, n, 3, seed=11)
    c = make_cache(2, 3, 3, W, 256, group=32, n_sink=n_sink, seed=5)
    ref = make_cache(2, 3, 3, W, 256, group=32, n_sink=0, seed=5)
    c.append(k, v)
    ref.append(k, v)
    lq = max(n - W, 0)
    ns = min(n_sink, lq)
    for b in range(2):
        for h in range(3):
            assert np.array_equal(c.k_sink[b, h, :ns], k[b, :ns, h][:, c.reorder_k[h]])
            assert np.array_equal(c.v_sink[b, h, :ns], v[b, :ns, h][:, c.reorder_v[h]])
    assert np.array_equal(c.k_codes[:, :, ns:lq], ref.k_codes[:, :, ns:lq])
    assert np.array_equal(c.v_meta.view(np.uint16)[:, :, ns:lq], ref.v_meta.view(np.uint16)[:, :, ns:lq])
    assert np.array_equal(c.k_win.view(np.uint16), ref.k_win.view(np.uint16))
    assert not c.k_codes[:, :, :ns].any()            # the quantized rows of the sinks are never written
    step = make_cache(2, 3, 3, W, 256, group=32, n_sink=n_sink, seed=5)
    t = 0
    for m in (1, 3, 7, 2, 11, 1, 1, 64, 200):
        m = min(m, n - t)
        if m == 0:
            break
        step.append(k[:, t:t + m], v[:, t:t + m])
        t += m
    while t < n:
        step.append(k[:, t:t + 1], v[:, t:t + 1])
        t += 1
    assert np.array_equal(step.k_sink[:, :, :ns], c.k_sink[:, :, :ns]) and np.array_equal(step.v_sink[:, :, :ns], c.v_sink[:, :, :ns])
    assert np.array_equal(step.k_codes[:, :, ns:lq], c.k_codes[:, :, ns:lq])
    assert np.array_equal(step.lengths, c.lengths)


@pytest.mark.parametrize("Hq,Hkv,bits,group,W,n_sink,L", [(4, 2, 2, 32, 16, 5, 150), (2, 2, 4, 64, 8, 3, 9), (2, 1, 2, 128, 0, 4, 33),
                                                      (2, 2, 2, 32, 16, 5, 12)])
def test_sink_attention_matches_library_brute_force(Hq, Hkv, bits, group, W, n_sink, L):
    k, v = rand_kv(1, L, Hkv, seed=21)
    c = make_cache(1, Hq, Hkv, W, 256, bits=bits, group=group, n_sink=n_sink, seed=8)
    c.append(k, v)
    q = np.random.default_rng(3).standard_normal((1, Hq, D)).astype(np.float16)
    got = c.attention(q, 0.088)
    assert np.abs(got - brute_attention(c, q, 0.088)).max() < 1e-12


@pytest.mark.parametrize("Hq,Hkv,bits,group,W,n_sink,L", [(4, 2, 2, 32, 16, 0, 150), (4, 4, 4, 64, 8, 3, 90), (8, 2, 2, 128, 0, 0, 77)])
def test_fp8_parameter_attention_matches_library_brute_force(Hq, Hkv, bits, group, W, n_sink, L):
    """Scale and zero point stored in E4M3: the oracle against numpy/scipy over a cache dequantized with a library's
    E4M3 decoding; and single appends equal one bulk append."""
    k, v = rand_kv(1, L, Hkv, seed=23)
    c = make_cache(1, Hq, Hkv, W, 256, bits=bits, group=group, n_sink=n_sink, seed=12, meta_fp8=True)
    c.append(k, v)
    assert c.k_meta.max() <= 255 and c.k_meta[0, :, n_sink:max(L - W, 0)].any()
    q = np.random.default_rng(4).standard_normal((1, Hq, D)).astype(np.float16)
    got = c.attention(q, 0.088)
    assert np.abs(got - brute_attention(c, q, 0.088)).max() < 1e-12
    c1 = make_cache(1, Hq, Hkv, W, 256, bits=bits, group=group, n_sink=n_sink, seed=12, meta_fp8=True)
    for t in range(L):
        c1.append(k[:, t:t + 1], v[:, t:t + 1])
    assert np.array_equal(c1.k_codes, c.k_codes) and np.array_equal(c1.v_meta, c.v_meta)


def test_all_sinks_and_no_window_is_plain_attention():
    """n_sink >= L with W = 0: nothing is quantized, so the result is softmax attention over the original K, V
    (a library routine, fp64), whatever the reorder index."""
    import torch
    L, Hq, Hkv = 50, 4, 2
    k, v = rand_kv(1, L, Hkv, seed=4)
    c = make_cache(1, Hq, Hkv, 0, 64, group=32, n_sink=64, seed=9)
    c.append(k, v)
    q = np.random.default_rng(6).standard_normal((1, Hq, D)).astype(np.float16)
    got = c.attention(q, 0.088)
    kt = torch.from_numpy(k.astype(np.float64)).permute(0, 2, 1, 3).repeat_interleave(Hq // Hkv, dim=1)
    vt = torch.from_numpy(v.astype(np.float64)).permute(0, 2, 1, 3).repeat_interleave(Hq // Hkv, dim=1)
    qt = torch.from_numpy(q.astype(np.float64))[:, :, None, :]
    want = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, scale=float(np.float32(0.088)))[:, :, 0].numpy()
    assert np.abs(got - want).max() < 1e-12
    assert not c.k_codes.any() and not c.v_codes.any()


def test_empty_sequence_gives_zeros():
    c = make_cache(2, 2, 2, 8, 32, seed=20)
    k, v = rand_kv(2, 12, 2, 21)
    c.append(k, v, np.array([0, 12], np.int32))
    out = c.attention(np.ones((2, 2, D), np.float16), 0.1)
    assert not out[0].any() and out[1].any()


# ------------------------------------------------------------------ workload generator (no method arithmetic)
def test_workload_generator_is_deterministic_and_chunk_invariant():
    w = workloads.configs()[2].scaled(context=10000, batch=2)
    a = w.tokens("k", 1, 4000, 9000)
    b = np.concatenate([w.tokens("k", 1, 4000, 4096), w.tokens("k", 1, 4096, 8192), w.tokens("k", 1, 8192, 9000)])
    assert np.array_equal(a.view(np.uint16), b.view(np.uint16))
    assert not np.array_equal(w.tokens("k", 0, 0, 16), w.tokens("v", 0, 0, 16))
    idx = w.reorder_index("k")
    assert idx.shape == (8, 128) and all(sorted(r.tolist()) == list(range(128)) for r in idx)
    sig = w.key_sigma()
    assert ((sig > 4).sum(1) >= 8).all() and (sig > 4).sum() < 8 * 12
    lens = workloads.configs()[4].lengths()
    assert lens.shape == (64,) and lens.min() >= 1024 and lens.max() <= 16384


def test_algorithmic_bytes_match_stated_sizes():
    cf = workloads.configs()
    assert abs(workloads.algorithmic_bytes(cf[0]) / 1e6 - 11.26) < 0.02
    assert abs(workloads.algorithmic_bytes(cf[1]) / 1e6 - 618.5) < 0.5
    assert abs(workloads.algorithmic_bytes(cf[2]) / 1e6 - 404.4) < 0.5
    assert abs(workloads.algorithmic_bytes(cf[3]) / 1e6 - 2417.7) < 0.5


# ------------------------------------------------------------------ unequal groups and 3-bit codes in the cache
@pytest.mark.parametrize("bits,v_bits,bk,bv", [
    (2, 2, [[0, 32, 128], [0, 96, 128]], [[0, 64, 128], [0, 32, 128]]),      # two groups per row, another split per head and tensor
    (3, 3, None, None),                                                     # 3-bit codes, equal groups
    (3, 2, [[0, 16, 40, 128], [0, 100, 120, 128]], [[0, 8, 64, 128], [0, 32, 64, 128]]),
    (2, 15, None, None),                                                    # 2-bit keys, three-level values (the paper's K2 V1.5)
    (2, 15, [[0, 32, 128], [0, 96, 128]], [[0, 64, 128], [0, 32, 128]]),
])
def test_attention_with_unequal_groups_and_three_bit_codes_matches_brute_force(bits, v_bits, bk, bv):
    """The cache path (append, single-token appends, attention) with group boundaries and 3-bit streams against the
    numpy reconstruction above (library softmax + einsum over an independently unpacked and dequantized cache)."""
    group = 64 if bk is None else 128 // (len(bk[0]) - 1) if 128 % (len(bk[0]) - 1) == 0 else 64
    c = make_cache(2, 4, 2, 8, 96, bits=bits, v_bits=v_bits, group=group, seed=21, bounds_k=bk, bounds_v=bv)
    k, v = rand_kv(2, 60, 2, 22)
    c.append(k[:, :50], v[:, :50])
    for t in range(50, 60):
        c.append(k[:, t:t + 1], v[:, t:t + 1])
    bulk = make_cache(2, 4, 2, 8, 96, bits=bits, v_bits=v_bits, group=group, seed=21, bounds_k=bk, bounds_v=bv)
    bulk.append(k, v)
    for a_, b_ in zip(cache_state(c), cache_state(bulk)):
        assert np.array_equal(a_, b_)
    q = np.random.default_rng(23).standard_normal((2, 4, D)).astype(np.float16)
    got = c.attention(q, 0.0884)
    want = brute_attention(c, q, 0.0884)
    assert np.abs(got - want).max() < 1e-12
    # rows of the quantized segment equal the stand-alone row quantizer with the head's own boundaries
    for h in range(2):
        ck, mk = orc.quantize_rows(k[0, :52, h], c.reorder_k[h], c.alpha_k[h], bits, group, bounds=None if bk is None else bk[h])
        assert np.array_equal(c.k_codes[0, h, :52], ck) and np.array_equal(c.k_meta[0, h, :52].view(np.uint16), mk.view(np.uint16))

"""Shared test plumbing: build the same cache on the CPU oracle and on the GPU library."""
import numpy as np

from oracle import skvq_oracle as orc

ATTN_TOL = 2e-3   # max-abs error of the fp16 attention output against the oracle's fp64 value


def oracle_cache_for(w, max_tokens):
    a = w.alphas()
    return orc.OracleCache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.k_bits, w.v_bits, w.group_size,
                           w.window, max_tokens, w.reorder_index("k"), w.reorder_index("v"), a, a, n_sink=w.n_sink, meta_fp8=w.meta_fp8,
                           bounds_k=w.bounds(), bounds_v=w.bounds())


def assert_cache_bit_exact(gpu, ora, lengths=None):
    """Codes, scales/zeros, ring contents and lengths of the GPU cache equal the oracle's, bit for bit,
    over the rows that hold data (rows beyond the quantized length are unspecified)."""
    import torch
    torch.cuda.synchronize()
    L = ora.lengths if lengths is None else lengths
    assert np.array_equal(gpu.lengths.cpu().numpy(), L)
    W = ora.W
    kc, vc = gpu.k_codes.cpu().numpy(), gpu.v_codes.cpu().numpy()
    if ora.meta_fp8:      # one E4M3 byte per parameter on the GPU, the same byte in a uint16 in the oracle
        km, vm = gpu.k_meta.cpu().numpy().astype(np.uint16), gpu.v_meta.cpu().numpy().astype(np.uint16)
    else:
        km, vm = gpu.k_meta.cpu().numpy().view(np.uint16), gpu.v_meta.cpu().numpy().view(np.uint16)
    kw, vw = gpu.k_win.cpu().numpy().view(np.uint16), gpu.v_win.cpu().numpy().view(np.uint16)
    ks, vs = gpu.k_sink.cpu().numpy().view(np.uint16), gpu.v_sink.cpu().numpy().view(np.uint16)
    ok_meta, ov_meta = ora.k_meta.view(np.uint16), ora.v_meta.view(np.uint16)      # fp16 bits, or one E4M3 byte per uint16
    for b in range(ora.B):
        lq = max(int(L[b]) - W, 0)
        ns = min(ora.n_sink, lq)          # rows of attention sinks: fp16 copies instead of codes
        assert np.array_equal(ks[b, :, :ns], ora.k_sink.view(np.uint16)[b, :, :ns]), f"k sinks differ, sequence {b}"
        assert np.array_equal(vs[b, :, :ns], ora.v_sink.view(np.uint16)[b, :, :ns]), f"v sinks differ, sequence {b}"
        assert np.array_equal(kc[b, :, ns:lq], ora.k_codes[b, :, ns:lq]), f"k codes differ, sequence {b}"
        assert np.array_equal(vc[b, :, ns:lq], ora.v_codes[b, :, ns:lq]), f"v codes differ, sequence {b}"
        assert np.array_equal(km[b, :, ns:lq], ok_meta[b, :, ns:lq]), f"k scale/zero differ, sequence {b}"
        assert np.array_equal(vm[b, :, ns:lq], ov_meta[b, :, ns:lq]), f"v scale/zero differ, sequence {b}"
        if W > 0:
            slots = sorted({t % W for t in range(lq, int(L[b]))})
            assert np.array_equal(kw[b][:, slots], ora.k_win.view(np.uint16)[b][:, slots]), f"k window differs, sequence {b}"
            assert np.array_equal(vw[b][:, slots], ora.v_win.view(np.uint16)[b][:, slots]), f"v window differs, sequence {b}"

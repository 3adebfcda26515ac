"""Out-of-bounds writes: every caller buffer sits between patterned guard regions that must survive the calls.

No memory checker runs with these tests, so the library's kernels are checked the plain way: each device buffer the
C ABI receives (codes, scale/zero, window ring, sink store, lengths, status, workspace, q, out) is carved out of a
larger allocation whose margins, and whose rows past the quantized length, carry a byte pattern.  After prefill,
decode appends and attention the pattern must be intact, and the results must still match the CPU oracle.
"""
import numpy as np
import pytest
import torch

from helpers import ATTN_TOL, assert_cache_bit_exact, oracle_cache_for
from paper_2405_06219_b200 import binding as B
from paper_2405_06219_b200 import build, workloads

pytestmark = pytest.mark.gpu
CF = workloads.configs()
MARGIN = 4096          # bytes in front of and behind every buffer
PATTERN = 0xA5


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build_library()
    B.lib()


class Guarded:
    """A device buffer of `nbytes` bytes with MARGIN patterned bytes on either side."""

    def __init__(self, nbytes, fill=PATTERN):
        self.nbytes = int(nbytes)
        pad = (-self.nbytes) % 256
        self.raw = torch.full((MARGIN + self.nbytes + pad + MARGIN,), PATTERN, dtype=torch.uint8, device="cuda")
        self.body = self.raw[MARGIN:MARGIN + self.nbytes]
        self.body.fill_(fill)
        assert self.body.data_ptr() % 256 == 0

    def view(self, dtype, shape):
        return self.body.view(dtype).view(shape)

    def margins_intact(self):
        r = self.raw.cpu().numpy()
        return bool((r[:MARGIN] == PATTERN).all() and (r[MARGIN + self.nbytes:] == PATTERN).all())


def guarded_cache(w, max_tokens):
    """A SkvqCache whose device buffers were replaced by guarded ones (quantized rows pre-filled with the pattern)."""
    gpu = B.SkvqCache.for_workload(w, max_tokens)
    guards = {}
    for name in ("k_codes", "v_codes", "k_meta", "v_meta", "k_win", "v_win", "k_sink", "v_sink", "lengths", "status"):
        t = getattr(gpu, name)
        g = Guarded(t.numel() * t.element_size(), fill=0 if name in ("lengths", "status") else PATTERN)
        guards[name] = g
        setattr(gpu, name, g.view(t.dtype, t.shape))
    gpu.struct = B.SkvqCacheStruct(*[t.data_ptr() for t in (
        gpu.k_codes, gpu.v_codes, gpu.k_meta, gpu.v_meta, gpu.k_win, gpu.v_win, gpu.lengths,
        gpu.reorder_k, gpu.reorder_v, gpu.alpha_k, gpu.alpha_v, gpu.status, gpu.k_sink, gpu.v_sink)])
    return gpu, guards


@pytest.mark.parametrize("cfg_i,kw,n,lens", [
    (1, dict(context=1500, batch=2, n_q_heads=4, n_kv_heads=4), 1500, [1500, 777]),               # integer kernel, 2-bit g128
    (2, dict(context=1300, batch=2, n_sink=5), 1300, [1300, 129]),                                # grouped-query kernel, g32, sinks
    (4, dict(context=1100, batch=3, ragged=None, n_q_heads=4, n_kv_heads=4), 1100, [1100, 0, 300]),   # 4-bit g64, window 256
    (2, dict(context=900, batch=1, n_q_heads=24), 900, [900]),                                    # tcgen05 kernel
    (4, dict(context=700, batch=1, ragged=None, n_q_heads=8, n_kv_heads=4), 700, [650]),          # 4-bit with 2 heads per KV head: tcgen05 kernel
    (2, dict(context=1000, batch=2, v_bits=15, n_sink=3), 1000, [1000, 333]),                     # three-level values: 26-byte rows, 2-byte aligned
    (1, dict(context=800, batch=1, n_q_heads=4, n_kv_heads=4, k_bits=3, v_bits=3), 800, [800]),   # 3-bit streams: 48-byte rows
])
def test_nothing_is_written_outside_the_buffers(cfg_i, kw, n, lens):
    w = CF[cfg_i].scaled(**kw)
    cap_tokens = n + 40
    gpu, guards = guarded_cache(w, cap_tokens)
    ora = oracle_cache_for(w, cap_tokens)
    k, v = w.prefill("k", n), w.prefill("v", n)
    n_b = np.array(lens, np.int32)
    gpu.append(torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), torch.from_numpy(n_b).cuda())
    ora.append(k, v, n_b)
    steps = 7
    hint = int(n_b.max()) + steps
    need = B.skvq_workspace_size(gpu.cfg, hint, 0)
    ws = Guarded(need)
    qg, og = Guarded(w.batch * w.n_q_heads * w.head_dim * 2, fill=0), Guarded(w.batch * w.n_q_heads * w.head_dim * 2)
    args = B.SkvqAttnArgs(float(w.sm_scale), hint, 0, ws.body.data_ptr(), need, None, None)
    out = og.view(torch.float16, (w.batch, w.n_q_heads, w.head_dim))
    q_dev = qg.view(torch.float16, (w.batch, w.n_q_heads, w.head_dim))
    for s in range(steps):
        kn, vn, q = w.new_token("k", s), w.new_token("v", s), w.query(s)
        gpu.append(torch.from_numpy(kn).cuda(), torch.from_numpy(vn).cuda())
        ora.append(kn, vn)
        q_dev.copy_(torch.from_numpy(q))
        B.skvq_decode_attention(gpu.cfg, gpu.struct, q_dev, out, args)
        torch.cuda.synchronize()
        want = ora.attention(q, w.sm_scale)
        assert np.abs(out.cpu().numpy().astype(np.float64) - want).max() <= ATTN_TOL
    assert_cache_bit_exact(gpu, ora)
    assert int(gpu.status[0].item()) == 0
    for name, g in list(guards.items()) + [("workspace", ws), ("q", qg), ("out", og)]:
        assert g.margins_intact(), f"bytes next to {name} were overwritten"
    # rows of the quantized segment at or beyond the quantized length are never written
    L = ora.lengths
    for name in ("k_codes", "v_codes", "k_meta", "v_meta"):
        t = getattr(gpu, name).cpu().numpy().view(np.uint8)
        for b in range(w.batch):
            lq = max(int(L[b]) - w.window, 0)
            assert (t[b, :, lq:] == PATTERN).all(), f"{name}: rows past the quantized length of sequence {b} were written"

"""Pins for the CPU oracle's quantizer: what the paper and plain mathematics fix.

Each test checks the oracle against something other than itself: numpy's own fp16
conversion, hand-derived closed forms, a brute-force nearest-level search, the
paper's printed average-bit arithmetic, or a property of the definition.
"""
import os

import numpy as np
import pytest

from oracle import skvq_oracle as orc

D = 128
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def unpack_codes(codes: np.ndarray, bits: int) -> np.ndarray:
    """Independent numpy unpack: code j = bits [(j*bits) mod 8, +bits) of byte (j*bits)//8."""
    n, nbytes = codes.shape
    if bits == 15:                                                     # three levels, five base-3 digits per byte
        digits = np.stack([(codes.astype(np.int64) // 3 ** i) % 3 for i in range(5)], axis=2)      # [n, nbytes, 5]
        return digits.reshape(n, nbytes * 5)[:, :D]
    bitsarr = np.unpackbits(codes, axis=1, bitorder="little")          # [n, nbytes*8], LSB first
    bitsarr = bitsarr.reshape(n, nbytes * 8 // bits, bits)
    weights = (1 << np.arange(bits)).astype(np.int64)
    return (bitsarr * weights).sum(axis=2)


def ident():
    return np.arange(D, dtype=np.int32)


# ------------------------------------------------------------------ fp16 conversions
def test_f16_to_f32_all_patterns_match_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    want = bits.view(np.float16).astype(np.float32)
    got = np.array([orc.f16_bits_to_f32(int(b)) for b in bits], dtype=np.float32)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32))


def test_f32_to_f16_matches_numpy_round_to_nearest_even():
    rng = np.random.default_rng(1)
    xs = np.concatenate([
        rng.standard_normal(20000).astype(np.float32) * np.float32(10.0) ** rng.integers(-9, 5, 20000),
        np.array([0.0, -0.0, 65504.0, 65519.9, 65520.0, 70000.0, -65520.0, 2.0 ** -24, 2.0 ** -25,
                  1.5 * 2.0 ** -25, 2.0 ** -14, 6.1e-5, 1.00048828125, 1.000732421875, 2049.0, 2051.0],
                 dtype=np.float32),
        # exact ties between neighbouring halves: (2k+1) * 2^-11 around 1.0
        (1.0 + (2 * np.arange(64) + 1) * 2.0 ** -11).astype(np.float32),
    ]).astype(np.float32)
    with np.errstate(over="ignore"):
        want = xs.astype(np.float16).view(np.uint16)
    got = np.array([orc.f32_to_f16_bits(float(x)) for x in xs], dtype=np.uint16)
    assert np.array_equal(got, want)


# ------------------------------------------------------------------ closed forms
@pytest.mark.parametrize("bits", [2, 3, 4])
def test_lossless_arithmetic_progression(bits):
    """A group holding exactly the 2^bits levels a + k*d (d a power of two), alpha = 1: h = d, z = a, code = k."""
    qmax = (1 << bits) - 1
    a, d = -1.5, 0.25
    ks = np.arange(D) % (qmax + 1)
    x = (a + ks * d).astype(np.float16)[None]
    codes, meta = orc.quantize_rows(x, ident(), np.ones(1, np.float32), bits, D)
    assert np.array_equal(unpack_codes(codes, bits)[0], ks)
    assert float(meta[0, 0, 0]) == d and float(meta[0, 0, 1]) == a
    assert np.array_equal(orc.dequant_rows(codes, meta, bits, D)[0], x[0].astype(np.float64))


def test_pack_layout_golden_bytes():
    """Codes 0,1,2,3 repeated: every 2-bit byte is 0b11100100; 4-bit codes 0..15: bytes 0x10, 0x32, ..."""
    x2 = (np.arange(D) % 4).astype(np.float16)[None]
    codes, _ = orc.quantize_rows(x2, ident(), np.ones(1, np.float32), 2, D)
    assert codes.shape == (1, 32) and np.all(codes == 0xE4)
    x4 = (np.arange(D) % 16).astype(np.float16)[None]
    codes, _ = orc.quantize_rows(x4, ident(), np.ones(1, np.float32), 4, D)
    want = np.array([0x10, 0x32, 0x54, 0x76, 0x98, 0xBA, 0xDC, 0xFE] * 8, dtype=np.uint8)
    assert codes.shape == (1, 64) and np.array_equal(codes[0], want)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_constant_group_is_degenerate(bits):
    x = np.full((1, D), 0.7314, dtype=np.float16)
    codes, meta = orc.quantize_rows(x, ident(), np.full(1, 1.0, np.float32), bits, D)
    assert np.all(codes == 0)
    assert float(meta[0, 0, 0]) == 0.0 and meta[0, 0, 1] == x[0, 0]
    assert np.all(orc.dequant_rows(codes, meta, bits, D) == float(x[0, 0]))


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_two_valued_group_hits_both_ends(bits):
    qmax = (1 << bits) - 1
    rng = np.random.default_rng(3)
    pick = rng.integers(0, 2, D)
    pick[:2] = [0, 1]
    x = np.where(pick == 1, 3.0, -1.5).astype(np.float16)[None]
    codes, _ = orc.quantize_rows(x, ident(), np.ones(1, np.float32), bits, D)
    assert np.array_equal(unpack_codes(codes, bits)[0], pick * qmax)


def test_zero_sign_is_canonical():
    """A group whose minimum is -0 or +0 stores the same (positive) zero point."""
    x = np.zeros((2, D), dtype=np.float16)
    x[0, :] = np.float16(-0.0)
    x[0, 5] = 1.0
    x[1, 5] = 1.0
    x[1, 9] = np.float16(-0.0)
    _, meta = orc.quantize_rows(x, ident(), np.ones(1, np.float32), 2, D)
    assert meta.view(np.uint16)[0, 0, 1] == 0 and meta.view(np.uint16)[1, 0, 1] == 0


# ------------------------------------------------------------------ definition-level properties
def random_rows(n, seed, outliers=True):
    rng = np.random.default_rng(seed)
    sigma = np.exp(0.5 * rng.standard_normal(D)).astype(np.float32)
    if outliers:
        sigma[rng.choice(D, 4, replace=False)] *= 15.0
    return (rng.standard_normal((n, D)).astype(np.float32) * sigma).astype(np.float16)


@pytest.mark.parametrize("bits,group,alpha", [(2, 128, 0.9), (2, 32, 0.85), (4, 64, 0.95), (2, 64, 1.0), (4, 128, 1.0), (3, 64, 0.9)])
def test_stored_parameters_follow_eq2(bits, group, alpha):
    """h = alpha*(max-min)/qmax and z = alpha*min (Eq. 2 / clipping_quant), stored as fp16.
    The expected values are formed in fp64 straight from the definition; fp32 intermediate
    rounding can move the fp16 result by at most one unit in the last place."""
    qmax = (1 << bits) - 1
    x = random_rows(64, 10 + bits + group)
    ng = D // group
    _, meta = orc.quantize_rows(x, ident(), np.full(ng, alpha, np.float32), bits, group)
    xg = x.astype(np.float64).reshape(64, ng, group)
    a = float(np.float32(alpha))
    h_want = (a * (xg.max(2) - xg.min(2)) / qmax)
    z_want = a * xg.min(2)
    h_got, z_got = meta[..., 0].astype(np.float64), meta[..., 1].astype(np.float64)
    ulp_h = np.spacing(np.abs(h_want).astype(np.float16)).astype(np.float64)
    ulp_z = np.spacing(np.abs(z_want).astype(np.float16)).astype(np.float64)
    assert np.all(np.abs(h_got - h_want) <= 0.5 * ulp_h * 1.01 + 1e-12)
    assert np.all(np.abs(z_got - z_want) <= 0.5 * ulp_z * 1.01 + 1e-12)
    exact = (h_got == h_want.astype(np.float16).astype(np.float64)).mean()
    assert exact > 0.99
    assert np.all(h_got >= 0)


@pytest.mark.parametrize("bits,group,alpha", [(2, 128, 0.9), (2, 32, 0.85), (4, 64, 0.95), (2, 128, 1.0), (4, 32, 1.0), (3, 64, 0.9),
                                              (3, 128, 1.0)])
def test_codes_are_nearest_level_brute_force(bits, group, alpha):
    """Brute force over all 2^bits levels: the stored code is (one of) the nearest reconstruction
    levels h*c+z to x, which also gives |x^ - x| <= h/2 inside the clipped range and the end
    point outside it (uniform quantizer of Sec. 3.1)."""
    qmax = (1 << bits) - 1
    x = random_rows(96, 20 + bits + group)
    ng = D // group
    codes, meta = orc.quantize_rows(x, ident(), np.full(ng, alpha, np.float32), bits, group)
    c = unpack_codes(codes, bits)
    assert c.min() >= 0 and c.max() <= qmax
    h = np.repeat(meta[..., 0].astype(np.float64), group, axis=1)
    z = np.repeat(meta[..., 1].astype(np.float64), group, axis=1)
    xd = x.astype(np.float64)
    levels = h[..., None] * np.arange(qmax + 1) + z[..., None]            # [n, D, levels]
    err_all = np.abs(levels - xd[..., None])
    err_got = np.abs(h * c + z - xd)
    slack = 4 * np.finfo(np.float32).eps * (np.abs(xd) + np.abs(z) + qmax * h) + 1e-30
    assert np.all(err_got <= err_all.min(axis=2) + slack)
    inside = (xd >= z) & (xd <= z + qmax * h)
    assert np.all(err_got[inside] <= 0.5 * h[inside] + slack[inside])
    below, above = xd < z, xd > z + qmax * h
    assert np.all(c[below & (h > 0)] == 0) and np.all(c[above & (h > 0)] == qmax)
    if alpha < 1.0:
        assert above.any() or below.any()                                  # clipping really clips
    # dequantization is exactly h*c+z in fp64
    assert np.array_equal(orc.dequant_rows(codes, meta, bits, group), h * c + z)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_alpha_one_full_group_is_textbook_per_token_minmax(bits):
    """alpha = 1, one group per token, identity order: plain per-token asymmetric min-max
    round-to-nearest (the dynamic quantization of Sec. 3.1).  Away from rounding ties the codes
    equal round((x - min) / ((max - min) / qmax)) evaluated in fp64."""
    qmax = (1 << bits) - 1
    x = random_rows(128, 5, outliers=False)
    codes, _ = orc.quantize_rows(x, ident(), np.ones(1, np.float32), bits, D)
    c = unpack_codes(codes, bits)
    xd = x.astype(np.float64)
    mn, mx = xd.min(1, keepdims=True), xd.max(1, keepdims=True)
    u = (xd - mn) / ((mx - mn) / qmax)
    want = np.clip(np.rint(u), 0, qmax).astype(np.int64)
    near_tie = np.abs(u - np.floor(u) - 0.5) < 2e-3 * (qmax + 1)          # fp16 rounding of h moves these
    assert near_tie.mean() < 0.15
    assert np.array_equal(c[~near_tie], want[~near_tie])
    assert np.all(np.abs(c - want)[near_tie] <= 1)
    # the row minimum and maximum land on the end codes
    assert np.all(c[np.arange(128), xd.argmin(1)] == 0) and np.all(c[np.arange(128), xd.argmax(1)] == qmax)


def test_codes_monotone_within_group():
    x = random_rows(32, 7)
    codes, _ = orc.quantize_rows(x, ident(), np.full(4, 0.85, np.float32), 2, 32)
    c = unpack_codes(codes, 2).reshape(32, 4, 32)
    xg = x.astype(np.float64).reshape(32, 4, 32)
    order = np.argsort(xg, axis=2, kind="stable")
    assert np.all(np.diff(np.take_along_axis(c, order, axis=2), axis=2) >= 0)


def test_groups_are_independent_and_contiguous():
    """Changing channels of one group changes only that group's codes and parameters."""
    x = random_rows(4, 8)
    y = x.copy()
    y[:, 32:64] = (y[:, 32:64].astype(np.float32) * 3 + 1).astype(np.float16)
    a = np.full(4, 0.9, np.float32)
    c1, m1 = orc.quantize_rows(x, ident(), a, 2, 32)
    c2, m2 = orc.quantize_rows(y, ident(), a, 2, 32)
    same_bytes = np.ones(32, bool)
    same_bytes[8:16] = False                                              # channels 32..63 = bytes 8..15
    assert np.array_equal(c1[:, same_bytes], c2[:, same_bytes])
    assert np.array_equal(m1[:, [0, 2, 3]], m2[:, [0, 2, 3]]) and not np.array_equal(m1[:, 1], m2[:, 1])


def test_per_group_alpha_is_used_per_group():
    x = random_rows(8, 9)
    a = np.array([1.0, 0.5, 0.75, 0.9], np.float32)
    _, m = orc.quantize_rows(x, ident(), a, 2, 32)
    xg = x.astype(np.float64).reshape(8, 4, 32)
    z_want = (a[None].astype(np.float64) * xg.min(2)).astype(np.float32).astype(np.float16)
    assert np.array_equal(m[..., 1], z_want)


# ------------------------------------------------------------------ reorder
def test_reorder_is_a_gather_by_index():
    """stored[j] = src[idx[j]]: with one group per channel-pair the parameters expose the order."""
    rng = np.random.default_rng(11)
    idx = rng.permutation(D).astype(np.int32)
    x = random_rows(16, 12)
    a = np.full(D // 32, 0.9, np.float32)
    c_re, m_re = orc.quantize_rows(x, idx, a, 4, 32)
    c_id, m_id = orc.quantize_rows(np.ascontiguousarray(x[:, idx]), ident(), a, 4, 32)
    assert np.array_equal(c_re, c_id) and np.array_equal(m_re.view(np.uint16), m_id.view(np.uint16))
    # and it is not the scatter direction
    inv = np.argsort(idx).astype(np.int32)
    c_sc, _ = orc.quantize_rows(np.ascontiguousarray(x[:, inv]), ident(), a, 4, 32)
    assert not np.array_equal(c_re, c_sc)


def test_reorder_with_single_group_only_permutes_codes():
    """With G = D the group statistics ignore order, so reordering permutes the codes and nothing else."""
    rng = np.random.default_rng(13)
    idx = rng.permutation(D).astype(np.int32)
    x = random_rows(16, 14)
    a = np.full(1, 0.9, np.float32)
    c_re, m_re = orc.quantize_rows(x, idx, a, 2, D)
    c_id, m_id = orc.quantize_rows(x, ident(), a, 2, D)
    assert np.array_equal(m_re.view(np.uint16), m_id.view(np.uint16))
    assert np.array_equal(unpack_codes(c_re, 2), unpack_codes(c_id, 2)[:, idx])


# ------------------------------------------------------------------ the paper's storage arithmetic
def test_average_bits_match_paper():
    """bits/element of what the cache stores = N + (bits of h + bits of z) / G; the golden file holds
    the figures the paper prints (ablation text and group-size table)."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "avg_bits.txt")) if l.strip() and not l.startswith("#")]
    for bits, group, param_bits, want in rows:
        bits, group, param_bits, want = int(bits), int(group), int(param_bits), float(want)
        x = random_rows(2, 15)
        codes, meta = orc.quantize_rows(x, ident(), np.ones(D // group, np.float32), bits, group)
        n_params = meta.shape[1] * meta.shape[2]
        stored_bits = codes.shape[1] * 8 + n_params * param_bits          # per row, params at the stated width
        assert stored_bits / D == pytest.approx(want, abs=1e-12)
        if param_bits == 16:                                              # what the oracle really stores
            assert (codes[0].nbytes + meta[0].nbytes) * 8 / D == pytest.approx(want, abs=1e-12)
        else:                                                             # FP8 mode: one byte per parameter
            codes8, meta8 = orc.quantize_rows(x, ident(), np.ones(D // group, np.float32), bits, group, meta_fp8=True)
            assert meta8.max() <= 255
            assert (codes8[0].nbytes + meta8[0].size) * 8 / D == pytest.approx(want, abs=1e-12)


# ------------------------------------------------------------------ FP8 E4M3 parameters (Sec. 4.1, component breakdown)
def _torch_e4m3():
    import torch
    if not hasattr(torch, "float8_e4m3fn"):
        pytest.skip("this torch has no float8_e4m3fn")
    return torch


def test_e4m3_decode_all_bytes_match_library():
    torch = _torch_e4m3()
    want = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    got = np.array([orc.e4m3_bits_to_f32(b) for b in range(256)], np.float32)
    assert np.array_equal(np.isnan(got), np.isnan(want)) and np.isnan(got).sum() == 2       # S.1111.111 only
    ok = ~np.isnan(want)
    assert np.array_equal(got[ok].view(np.uint32), want[ok].view(np.uint32))
    assert got[0x7E] == 448.0 and got[0x01] == 2.0 ** -9 and got[0x08] == 2.0 ** -6 and got[0x38] == 1.0


def test_e4m3_encode_matches_library_round_to_nearest_even():
    """Random values over the whole finite range, every representable value, and every midpoint between two
    neighbours (ties must go to the even mantissa)."""
    torch = _torch_e4m3()
    rng = np.random.default_rng(5)
    grid = np.array([orc.e4m3_bits_to_f32(b) for b in range(0x7F)], np.float64)              # 0 .. 448, ascending
    mids = (grid[:-1] + grid[1:]) / 2
    x = np.concatenate([grid, mids, np.nextafter(mids.astype(np.float32), np.float32(0)).astype(np.float64),
                        np.nextafter(mids.astype(np.float32), np.float32(1e9)).astype(np.float64),
                        rng.uniform(-448, 448, 4000), np.ldexp(rng.uniform(-1, 1, 4000), rng.integers(-14, 9, 4000))])
    x = np.concatenate([x, -x]).astype(np.float32)
    x = x[np.abs(x) <= 448]
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([orc.f32_to_e4m3_bits(float(v)) for v in x], np.uint8)
    assert np.array_equal(got, want)


def test_e4m3_encode_saturates_and_keeps_the_grid():
    for v in (448.5, 463.9, 464.0, 480.0, 1e4, 6.5e4, float("inf")):
        assert orc.f32_to_e4m3_bits(v) == 0x7E and orc.f32_to_e4m3_bits(-v) == 0xFE
    for b in range(0x7F):                                                   # encoding a representable value is the identity
        assert orc.f32_to_e4m3_bits(orc.e4m3_bits_to_f32(b)) == b
    assert orc.f32_to_e4m3_bits(2.0 ** -10) == 0x00 and orc.f32_to_e4m3_bits(3 * 2.0 ** -10) == 0x02    # ties to even


@pytest.mark.parametrize("bits,group", [(2, 32), (2, 128), (4, 64)])
def test_fp8_parameters_are_the_rounded_fp32_ones_and_codes_use_them(bits, group):
    """Eq. 2 with the parameters stored in E4M3: h8 = e4m3(alpha (max - min) / qmax), z8 = e4m3(alpha min), and the
    codes are the nearest levels of the grid those stored values define (brute force in fp64)."""
    qmax = 2 ** bits - 1
    x = random_rows(40, 31)
    alpha = np.full(D // group, 0.9, np.float32)
    codes, meta = orc.quantize_rows(x, ident(), alpha, bits, group, meta_fp8=True)
    c = unpack_codes(codes, bits)
    for r in range(x.shape[0]):
        for g in range(D // group):
            seg = x[r, g * group:(g + 1) * group].astype(np.float32)
            lo, hi = np.float32(0.9) * seg.min(), np.float32(0.9) * seg.max()
            h8, z8 = orc.f32_to_e4m3_bits(float((hi - lo) / np.float32(qmax))), orc.f32_to_e4m3_bits(float(lo))
            assert (int(meta[r, g, 0]), int(meta[r, g, 1])) == (h8, z8)
            h, z = orc.e4m3_bits_to_f32(h8), orc.e4m3_bits_to_f32(z8)
            levels = z + h * np.arange(qmax + 1)
            want = np.abs(seg.astype(np.float64)[:, None] - levels[None, :]).argmin(axis=1)
            got = c[r, g * group:(g + 1) * group]
            # an element may sit within rounding distance of the midpoint between two levels: accept either there
            d = np.abs(seg.astype(np.float64) - levels[got]) - np.abs(seg.astype(np.float64) - levels[want])
            assert np.all(d <= 1e-6 * max(h, 1e-30) + 1e-12)
    xhat = orc.dequant_rows(codes, meta, bits, group, meta_fp8=True)
    h_all = np.repeat(np.vectorize(orc.e4m3_bits_to_f32)(meta[:, :, 0].astype(np.uint8)), group, axis=1)
    z_all = np.repeat(np.vectorize(orc.e4m3_bits_to_f32)(meta[:, :, 1].astype(np.uint8)), group, axis=1)
    assert np.array_equal(xhat, h_all.astype(np.float64) * c + z_all.astype(np.float64))
    inside = (x >= z_all) & (x <= z_all + qmax * h_all)                    # inside the stored grid the error is half a step
    assert np.all(np.abs(x.astype(np.float64) - xhat)[inside] <= 0.5 * h_all[inside] * (1 + 1e-6))


# ------------------------------------------------------------------ 3-bit codes (the 3-bit column of the KVQuant comparison, Sec. 4.3)
def test_three_bit_pack_layout_golden_bytes():
    """A row is a little-endian bit stream of 3-bit fields: codes 0..7 in order occupy three bytes
    0x88 0xC6 0xFA (bits 000 100 010 110 001 101 011 111 read least significant first); eight codes per 3 bytes,
    32 codes per 12 bytes, a 128-channel row is 48 bytes."""
    x = (np.arange(D) % 8).astype(np.float16)[None]
    codes, meta = orc.quantize_rows(x, ident(), np.ones(1, np.float32), 3, D)
    assert codes.shape == (1, 48)
    assert np.array_equal(codes[0], np.array([0x88, 0xC6, 0xFA] * 16, dtype=np.uint8))
    assert float(meta[0, 0, 0]) == 1.0 and float(meta[0, 0, 1]) == 0.0
    # the width-generic numpy unpack (bit j*3 .. j*3+2 of the stream) reads the same codes back
    assert np.array_equal(unpack_codes(codes, 3)[0], np.arange(D) % 8)
    # a code that straddles a byte boundary: only code 2 (bits 6..8) set to 7 -> 0xC0 0x01
    y = np.zeros((1, D), np.float16)
    y[0, 2] = 7.0
    y[0, 127] = 7.0      # keeps max = 7 wherever code 2 sits; last code occupies bits 381..383 = top of byte 47
    codes, _ = orc.quantize_rows(y, ident(), np.ones(1, np.float32), 3, D)
    assert codes[0, 0] == 0xC0 and codes[0, 1] == 0x01 and codes[0, 47] == 0xE0 and not codes[0, 2:47].any()


# ------------------------------------------------------------------ unequal groups (split_groups of Algorithm 1; Sec. 4.2)
def test_equal_boundaries_reproduce_equal_groups_bit_for_bit():
    x = random_rows(32, 40)
    rng = np.random.default_rng(41)
    idx = rng.permutation(D).astype(np.int32)
    for bits, group in ((2, 32), (4, 64), (3, 64), (2, 128)):
        ng = D // group
        a = (0.8 + 0.05 * np.arange(ng)).astype(np.float32)
        c_eq, m_eq = orc.quantize_rows(x, idx, a, bits, group)
        c_bd, m_bd = orc.quantize_rows(x, idx, a, bits, group, bounds=np.arange(ng + 1) * group)
        assert np.array_equal(c_eq, c_bd) and np.array_equal(m_eq.view(np.uint16), m_bd.view(np.uint16))
        assert np.array_equal(orc.dequant_rows(c_eq, m_eq, bits, group),
                              orc.dequant_rows(c_bd, m_bd, bits, group, bounds=np.arange(ng + 1) * group))


@pytest.mark.parametrize("bits,bounds", [(2, [0, 32, 128]), (2, [0, 96, 128]), (4, [0, 16, 48, 128]), (3, [0, 8, 72, 100, 128]),
                                         (2, [0, 1, 128])])
def test_unequal_groups_use_their_own_slice(bits, bounds):
    """Every group [b_g, b_{g+1}) is quantized exactly like a stand-alone row of that width would be: parameters
    from its own min and max (Eq. 2, recomputed here in fp64 on the slice), codes nearest to its own levels, and
    nothing of a group depends on the channels outside it."""
    qmax = (1 << bits) - 1
    x = random_rows(48, 50 + bits + len(bounds))
    ng = len(bounds) - 1
    alpha = (0.85 + 0.05 * np.arange(ng)).clip(max=1.0).astype(np.float32)
    codes, meta = orc.quantize_rows(x, ident(), alpha, bits, D, bounds=bounds)
    assert meta.shape == (48, ng, 2) and codes.shape == (48, D * bits // 8)
    c = unpack_codes(codes, bits)
    xd = x.astype(np.float64)
    deq = orc.dequant_rows(codes, meta, bits, D, bounds=bounds)
    for g in range(ng):
        lo, hi = bounds[g], bounds[g + 1]
        a = float(alpha[g])
        h_want, z_want = a * (xd[:, lo:hi].max(1) - xd[:, lo:hi].min(1)) / qmax, a * xd[:, lo:hi].min(1)
        h, z = meta[:, g, 0].astype(np.float64), meta[:, g, 1].astype(np.float64)
        assert np.all(np.abs(h - h_want) <= 0.5 * np.spacing(np.abs(h_want).astype(np.float16)).astype(np.float64) * 1.01 + 1e-12)
        assert np.all(np.abs(z - z_want) <= 0.5 * np.spacing(np.abs(z_want).astype(np.float16)).astype(np.float64) * 1.01 + 1e-12)
        levels = h[:, None, None] * np.arange(qmax + 1) + z[:, None, None]
        err = np.abs(h[:, None] * c[:, lo:hi] + z[:, None] - xd[:, lo:hi])
        slack = 4 * np.finfo(np.float32).eps * (np.abs(xd[:, lo:hi]) + np.abs(z[:, None]) + qmax * h[:, None]) + 1e-30
        assert np.all(err <= np.abs(levels - xd[:, lo:hi, None]).min(axis=2) + slack)
        assert np.array_equal(deq[:, lo:hi], h[:, None] * c[:, lo:hi] + z[:, None])
        # the same channels quantized on their own (one group spanning a row that repeats the slice) give the same codes
        if (hi - lo) in (32, 64, 128):
            rep = np.tile(x[:, lo:hi], (1, D // (hi - lo)))
            c_alone, m_alone = orc.quantize_rows(rep, ident(), np.full(D // (hi - lo), alpha[g], np.float32), bits, hi - lo)
            assert np.array_equal(unpack_codes(c_alone, bits)[:, :hi - lo], c[:, lo:hi])
            assert np.array_equal(m_alone[:, 0].view(np.uint16), meta[:, g].view(np.uint16))


def test_one_channel_group_is_lossless():
    """An outlier channel in a group of its own: min = max, so h = 0, z = the value (alpha = 1), and it comes back exactly."""
    rng = np.random.default_rng(60)
    x = rng.standard_normal((16, D)).astype(np.float16)
    x[:, 0] = (40 + rng.standard_normal(16)).astype(np.float16)           # one outlier channel
    codes, meta = orc.quantize_rows(x, ident(), np.ones(2, np.float32), 2, D, bounds=[0, 1, D])
    deq = orc.dequant_rows(codes, meta, 2, D, bounds=[0, 1, D])
    assert np.array_equal(deq[:, 0], x[:, 0].astype(np.float64))
    assert np.all(meta[:, 0, 0] == 0) and np.array_equal(meta[:, 0, 1], x[:, 0])
    # and the rest of the row no longer pays for the outlier: its scale is that of the 127 ordinary channels
    _, meta_one = orc.quantize_rows(x, ident(), np.ones(1, np.float32), 2, D)
    assert np.all(meta[:, 1, 0].astype(np.float64) <= meta_one[:, 0, 0].astype(np.float64))
    assert np.median(meta[:, 1, 0].astype(np.float64) / meta_one[:, 0, 0].astype(np.float64)) < 0.5


def test_unequal_groups_cost_what_their_average_size_costs():
    """The paper keeps the NUMBER of groups fixed so that the average group size, and with it the average bits, equals
    the equal-group setting it compares with (Sec. 4.2): 2 groups of 32 + 96 channels store what 2 x 64 store."""
    x = random_rows(4, 61)
    c_u, m_u = orc.quantize_rows(x, ident(), np.ones(2, np.float32), 2, D, bounds=[0, 32, 128], meta_fp8=True)
    c_e, m_e = orc.quantize_rows(x, ident(), np.ones(2, np.float32), 2, 64, meta_fp8=True)
    assert c_u.shape == c_e.shape and m_u.shape == m_e.shape
    assert (c_u[0].nbytes + m_u[0].size) * 8 / D == pytest.approx(2.25)      # the paper's figure for group 64, FP8 parameters


# ------------------------------------------------------------------ the three-level ("1.5-bit") value code (abstract, Sec. 4.2)
def test_three_level_code_golden_bytes_and_closed_forms():
    """Five codes per byte in base 3: codes 0,1,2,0,1 -> 0 + 1*3 + 2*9 + 0*27 + 1*81 = 102, and so on with the pattern
    j mod 3 continuing across bytes; 128 codes take 26 bytes (the last byte holds codes 125, 126, 127 and two zero digits)."""
    x = (np.arange(D) % 3).astype(np.float16)[None]
    codes, meta = orc.quantize_rows(x, ident(), np.ones(1, np.float32), 15, D)
    assert codes.shape == (1, 26) and orc.row_bytes(D, 15) == 26 and orc.qmax(15) == 2
    want = [sum(((5 * b + i) % 3) * 3 ** i for i in range(5) if 5 * b + i < D) for b in range(26)]
    assert codes[0].tolist() == want and want[0] == 102
    assert float(meta[0, 0, 0]) == 1.0 and float(meta[0, 0, 1]) == 0.0            # h = (2 - 0) / 2, z = 0
    assert np.array_equal(unpack_codes(codes, 15)[0], np.arange(D) % 3)
    assert np.array_equal(orc.dequant_rows(codes, meta, 15, D)[0], x[0].astype(np.float64))      # three exact levels: lossless
    # a two-valued group sits on codes 0 and 2; a constant group is degenerate (h = 0)
    y = np.where(np.arange(D) % 2 == 0, -1.5, 3.0).astype(np.float16)[None]
    c2, _ = orc.quantize_rows(y, ident(), np.ones(1, np.float32), 15, D)
    assert np.array_equal(unpack_codes(c2, 15)[0], (np.arange(D) % 2) * 2)
    c3, m3 = orc.quantize_rows(np.full((1, D), 0.37, np.float16), ident(), np.ones(1, np.float32), 15, D)
    assert not c3.any() and float(m3[0, 0, 0]) == 0.0


@pytest.mark.parametrize("group,alpha,bounds", [(128, 1.0, None), (64, 0.9, None), (32, 0.85, None), (64, 0.9, [0, 32, 128])])
def test_three_level_codes_are_nearest_level_and_parameters_follow_eq2(group, alpha, bounds):
    """h = alpha (max - min) / 2, z = alpha min; the code is the nearest of the three levels z, z + h, z + 2h."""
    x = random_rows(64, 70 + group)
    ng = D // group
    codes, meta = orc.quantize_rows(x, ident(), np.full(ng, alpha, np.float32), 15, group, bounds=bounds)
    c = unpack_codes(codes, 15)
    assert c.min() >= 0 and c.max() <= 2
    widths = np.full(ng, group) if bounds is None else np.diff(bounds)
    h = np.repeat(meta[..., 0].astype(np.float64), widths, axis=1)
    z = np.repeat(meta[..., 1].astype(np.float64), widths, axis=1)
    xd = x.astype(np.float64)
    err = np.abs(h * c + z - xd)
    best = np.abs(h[..., None] * np.arange(3) + z[..., None] - xd[..., None]).min(axis=2)
    slack = 4 * np.finfo(np.float32).eps * (np.abs(xd) + np.abs(z) + 2 * h) + 1e-30
    assert np.all(err <= best + slack)
    edges = np.concatenate([[0], np.cumsum(widths)])
    a = float(np.float32(alpha))
    for g in range(ng):
        seg = xd[:, edges[g]:edges[g + 1]]
        h_want = a * (seg.max(1) - seg.min(1)) / 2
        assert np.all(np.abs(meta[:, g, 0].astype(np.float64) - h_want) <= 0.5 * np.spacing(np.abs(h_want).astype(np.float16)).astype(np.float64) * 1.01 + 1e-12)
    assert np.array_equal(orc.dequant_rows(codes, meta, 15, group, bounds=bounds), h * c + z)
    # storage: 26 bytes for 128 codes = 1.625 bits per code (the paper's nominal figure is 1.5)
    assert codes.shape[1] * 8 / D == 1.625

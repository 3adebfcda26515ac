// skvq_quantize_append: channel reorder, group-wise clipped dynamic asymmetric quantization,
// 2/3/4-bit and three-level packing and sliding-window bookkeeping (Sec. 3.1 Eq. 2, Sec. 3.2, Algorithm 1).
//
// Work decomposition.  For sequence b with L0 tokens before and L1 = L0 + n_b after the call:
//   "evict" items   tokens t in [max(L0-W,0), min(L0, L1-W)): still in the fp16 ring (already in
//                   reordered order).  The owner quantizes ring slot t % W into row t and then
//                   refills the same slot with the one new token t' = t (mod W) that ends up inside
//                   the final window, so the read and the overwrite of a slot never race.
//   "new" items     tokens t in [L0, L1): quantized straight from the input if t < L1-W, else
//                   written to the ring unless an evict item refills that slot.
// Bulk appends (prefill) send every whole, 64-aligned run of tokens that goes straight from the input to the
// quantized segment through the tile kernel (skvq_append_tc.cu: reorder on the tensor core, one thread per token
// row); append_kernel takes the rest: evictions from the ring, ring writes and the ragged ends.
// Eight lanes own one 128-channel row (16 channels each); a warp handles two tokens at a time,
// K rows on lanes 0-7/16-23 and V rows on lanes 8-15/24-31.  Group statistics are reduced with
// xor-shuffles over G/16 lanes.  All quantizer arithmetic uses explicitly rounded fp32 intrinsics
// so the codes, scales and zeros do not depend on compiler contraction.

#include "skvq_append_common.cuh"

namespace skvq {
namespace {

constexpr int kItemsPerCta = 64;
constexpr int kAppendThreads = 128;

// The codes of 16 elements by the defining formula (IEEE division, rintf): it runs only for the few row segments
// that have a quotient next to a rounding boundary, and for 3-bit codes.  Inlined on purpose: as a separate function
// it takes the 16 values through local memory, which every caller then pays for on the fast path too (measured:
// 1.88 -> 2.13 TB/s of prefill input).  The 16 fields are a little-endian bit stream of 16 * BITS bits in words[0],
// words[1]; the three-level codes come out as 16 two-bit fields (the caller packs them in base 3).
template <int BITS>
__device__ __forceinline__ void quantize16_exact(const float (&x)[16], float zf, float hf, uint32_t (&words)[2])
{
    constexpr int qmax = code_max(BITS), FIELD = BITS == kTernary ? 2 : BITS;
    unsigned long long stream = 0ull;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        float c = rintf(__fdiv_rn(__fsub_rn(x[j], zf), hf));
        c = fminf(fmaxf(c, 0.0f), (float)qmax);
        stream |= (unsigned long long)(uint32_t)(int)c << (j * FIELD);
    }
    words[0] = (uint32_t)stream;
    words[1] = (uint32_t)(stream >> 32);
}

// Quantize the 16 channels held by this lane; `lanes_per_group` lanes share the group statistics.
// Writes what is stored per (token, group): a half2 {h, z}, or its two E4M3 bytes in the low 16 bits of hz_bits.
// LPG > 0: lanes per group known at compile time (the shuffle rounds unroll); 0: taken from lanes_per_group.
// lanes_per_group == 0 (with LPG == 0): the group is the lanes [lane_lo, lane_hi) of the row's 8 (groups of unequal width).
template <int BITS, int LPG = 0>
__device__ __forceinline__ void quantize16(const float (&x)[16], float alpha, int lanes_per_group, bool meta_fp8,
                                           uint32_t (&words)[2], uint32_t &hz_bits, int lane_lo = 0, int lane_hi = 0)
{
    // The 8 lanes that own one row always take the same path, so they are the shuffle's member set
    // (K and V rows may use different bit widths and therefore different instantiations).
    const uint32_t seg_mask = 0xFFu << ((threadIdx.x & 31) & 24);
    constexpr int qmax = code_max(BITS);
    float mn = x[0], mx = x[0];
#pragma unroll
    for (int j = 1; j < 16; ++j) {
        mn = fminf(mn, x[j]);
        mx = fmaxf(mx, x[j]);
    }
    if constexpr (LPG > 0) {
#pragma unroll
        for (int m = 1; m < LPG; m <<= 1) {
            mn = fminf(mn, __shfl_xor_sync(seg_mask, mn, m));
            mx = fmaxf(mx, __shfl_xor_sync(seg_mask, mx, m));
        }
    } else if (lanes_per_group > 0) {
        for (int m = 1; m < lanes_per_group; m <<= 1) {
            mn = fminf(mn, __shfl_xor_sync(seg_mask, mn, m));
            mx = fmaxf(mx, __shfl_xor_sync(seg_mask, mx, m));
        }
    } else {
        // a run of lanes that need not be a power of two nor aligned: look at all eight, keep those of the run
        const int base = (threadIdx.x & 31) & 24;
        float a = mn, b = mx;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float vj = __shfl_sync(seg_mask, mn, base + j), wj = __shfl_sync(seg_mask, mx, base + j);
            if (j >= lane_lo && j < lane_hi) { a = fminf(a, vj); b = fmaxf(b, wj); }
        }
        mn = a;
        mx = b;
    }
    // Clip both ends (Eq. 2 / clipping_quant); "+ 0" turns a negative zero into +0.
    const float lo = __fadd_rn(__fmul_rn(alpha, mn), 0.0f);
    const float hi = __fadd_rn(__fmul_rn(alpha, mx), 0.0f);
    const float h32 = __fdiv_rn(__fsub_rn(hi, lo), (float)qmax);
    __half2 hz;      // the stored parameters: the codes are computed against these
    if (meta_fp8) {
        const uint16_t b = to_e4m3x2(h32, lo);
        hz = from_e4m3x2(b);
        hz_bits = b;
    } else {
        hz = __halves2half2(__float2half_rn(h32), __float2half_rn(lo));
        hz_bits = *reinterpret_cast<const uint32_t *>(&hz);
    }
    const float hf = __low2float(hz);
    const float zf = __high2float(hz);
    words[0] = 0u;
    words[1] = 0u;
    if constexpr (BITS == 3 || BITS == kTernary) {
        // 3-bit fields do not tile a 32-bit word, three-level codes are packed across lanes afterwards; these widths
        // take the defining formula directly
        if (hf != 0.0f) quantize16_exact<BITS>(x, zf, hf, words);
    } else if (hf != 0.0f) {
        // The code is clamp(rint(RN((x - z) / h)), 0, qmax) with IEEE division.  One division per element makes
        // this path bound by the special-function unit, so the quotient is first formed as d * RN(1/h): that is
        // within 3 * 2^-24 relative of the IEEE quotient, so wherever every value within 2^-18 relative of it
        // rounds to the same integer, that integer is the code.  The test is two FMAs onto 1.5 * 2^23 (the
        // mantissa's low bits are then the rounded integer, ties to even, like rintf) that must agree.  A lane
        // with any element in doubt (a quotient next to k + 0.5, including exact ties) redoes its 16 elements with
        // the division itself.  The packed word is summed modulo 2^32 with the constant bits of 1.5 * 2^23
        // taken out at the end.
        constexpr float MAGIC = 12582912.0f;                       // 0x4B400000
        constexpr float UP = 1.0f + 3.814697265625e-06f, DN = 1.0f - 3.814697265625e-06f;
        constexpr int PER_WORD = 32 / BITS;
        uint32_t kconst = 0u;
#pragma unroll
        for (int j = 0; j < PER_WORD; ++j) kconst += 0x4B400000u << (j * BITS);
        const float r = __frcp_rn(hf);
        uint32_t doubt = 0u, w0 = 0u, w1 = 0u;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const float q = __fmul_rn(__fsub_rn(x[j], zf), r);
            const float qc = fminf(fmaxf(q, 0.0f), (float)qmax);
            const uint32_t ta = __float_as_uint(__fmaf_rn(qc, DN, MAGIC));
            const uint32_t tb = __float_as_uint(__fmaf_rn(qc, UP, MAGIC));
            doubt |= ta ^ tb;
            if ((j * BITS) < 32) w0 += ta << ((j * BITS) & 31);
            else w1 += ta << ((j * BITS) & 31);
        }
        if (doubt == 0u) {
            words[0] = w0 - kconst;
            if (BITS == 4) words[1] = w1 - kconst;
        } else {
            quantize16_exact<BITS>(x, zf, hf, words);
        }
    }
}

__global__ void __launch_bounds__(kAppendThreads) append_kernel(AppendArgs a)
{
    asm volatile("griddepcontrol.launch_dependents;");      // the bookkeeping kernel may be launched; it waits for this grid
    const Shape &s = a.s;
    const int b = blockIdx.z, h = blockIdx.y;
    const int W = s.W;
    const int L0 = a.c.lengths[b];
    const int n_b = seq_new_count(a, b);
    const int L1 = L0 + n_b;
    if (n_b == 0 || L1 > s.max_tokens) return;   // overflow is reported by the bookkeeping kernel
    const int q_end = max(L1 - W, 0);            // tokens below this index are quantized after the call
    const int t_lo = max(L0 - W, 0);
    const int n_evict = max(min(L0, q_end) - t_lo, 0);
    int f0, f1;
    bulk_range(L0, s.n_sink, q_end, f0, f1);
    const int n_bulk = a.use_bulk ? f1 - f0 : 0;   // new tokens the tile kernel takes: skipped here
    const int n_items = n_evict + n_b - n_bulk;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane & 7;
    const bool is_v = (lane >> 3) & 1;
    const int tok_sel = lane >> 4;

    const int bits = is_v ? s.v_bits : s.k_bits;
    const int row_bytes = packed_row_bytes(bits);
    const size_t bh = (size_t)b * s.Hkv + h;
    uint8_t *codes = (is_v ? a.c.v_codes : a.c.k_codes) + bh * (size_t)s.cap * row_bytes;
    __half2 *meta = (is_v ? a.c.v_meta : a.c.k_meta);      // two bytes per (token, group) with FP8 parameters
    const size_t meta0 = bh * (size_t)s.cap * s.ng;
    const bool f8 = s.meta_fp8 != 0;
    __half *win = (is_v ? a.c.v_win : a.c.k_win) + bh * (size_t)W * kHeadDim;
    const __half *src = (is_v ? a.v : a.k) + ((size_t)b * a.n_new * s.Hkv + h) * kHeadDim;   // token stride Hkv*D
    const size_t src_tok_stride = (size_t)s.Hkv * kHeadDim;
    const float *alpha_head = (is_v ? a.c.alpha_v : a.c.alpha_k) + (size_t)h * s.ng;
    const int32_t *bounds = is_v ? a.c.bounds_v : a.c.bounds_k;      // groups of unequal width, or NULL
    if (bounds) bounds += (size_t)h * (s.ng + 1);

    // This lane's 16 gather indices (stored[j] = source[idx[j]], j = 16*sub .. 16*sub+15).
    int idx[16];
    {
        const int32_t *ip = (is_v ? a.c.reorder_v : a.c.reorder_k) + (size_t)h * kHeadDim + (sub << 4);
#pragma unroll
        for (int j = 0; j < 16; ++j) idx[j] = ip[j] & (kHeadDim - 1);
    }

    const int item_base = blockIdx.x * kItemsPerCta;
    for (int it = warp * 2; it < kItemsPerCta; it += (kAppendThreads / 32) * 2) {
        const int item = item_base + it + tok_sel;
        // Warp-uniform exit: both halves of the warp are past the end.
        if (item_base + it >= n_items) break;
        const bool active = item < n_items;
        // Lanes of an inactive half still take part in the shuffles below with dummy data.
        float x[16];
        __half xh[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) { x[j] = 0.0f; xh[j] = __float2half(0.0f); }

        int t = 0;
        bool from_ring = false, do_quant = false, do_ring_write = false;
        int ring_token = 0;   // token whose (gathered) input row goes to the ring
        if (active) {
            if (item < n_evict) {
                t = t_lo + item;
                from_ring = true;
                do_quant = true;
                // the new token with the same slot that ends inside the final window
                const int k_steps = (q_end - t + W - 1) / W;
                ring_token = t + k_steps * W;
                do_ring_write = true;
            } else {
                t = L0 + (item - n_evict);
                if (n_bulk > 0 && t >= f0) t += n_bulk;
                if (t < q_end) {
                    do_quant = true;
                } else if (W > 0) {
                    const bool occupied = (L0 >= W) || ((t % W) < L0);
                    do_ring_write = !occupied;
                    ring_token = t;
                }
            }
        }
        if (do_quant) {
            if (from_ring) {
                const uint4 *p = reinterpret_cast<const uint4 *>(win + (size_t)(t % W) * kHeadDim + (sub << 4));
                uint4 v0 = p[0], v1 = p[1];
                const __half *hv0 = reinterpret_cast<const __half *>(&v0);
                const __half *hv1 = reinterpret_cast<const __half *>(&v1);
#pragma unroll
                for (int j = 0; j < 8; ++j) { x[j] = __half2float(hv0[j]); x[8 + j] = __half2float(hv1[j]); }
            } else {
                const __half *row = src + (size_t)(t - L0) * src_tok_stride;
#pragma unroll
                for (int j = 0; j < 16; ++j) x[j] = __half2float(row[idx[j]]);
            }
        }
        // Every lane of a row's 8-lane segment executes the shuffles inside; inactive rows store nothing.
        {
            int lanes_per_group = s.G >> 4;
            int g = (sub << 4) / s.G;
            int lane_lo = g * lanes_per_group, lane_hi = lane_lo + lanes_per_group;
            if (bounds) {      // groups of unequal width: this lane's 16 channels lie inside one of them (boundaries are multiples of 32)
                g = 0;
                for (int i = 1; i < s.ng; ++i) g += ((sub << 4) >= bounds[i]) ? 1 : 0;
                lane_lo = bounds[g] >> 4;
                lane_hi = bounds[g + 1] >> 4;
                lanes_per_group = 0;
            }
            const float alpha = alpha_head[g];
            uint32_t words[2];
            uint32_t hz;
            if (bits == 2) quantize16<2>(x, alpha, lanes_per_group, f8, words, hz, lane_lo, lane_hi);
            else if (bits == 3) quantize16<3>(x, alpha, lanes_per_group, f8, words, hz, lane_lo, lane_hi);
            else if (bits == kTernary) quantize16<kTernary>(x, alpha, lanes_per_group, f8, words, hz, lane_lo, lane_hi);
            else quantize16<4>(x, alpha, lanes_per_group, f8, words, hz, lane_lo, lane_hi);
            uint32_t tern = 0u;      // three-level codes: bytes 4*sub .. 4*sub+3 of the row
            if (bits == kTernary) {
                // Byte n carries codes 5n .. 5n+4 as base-3 digits.  They lie in the two-bit fields of at most two
                // neighbouring lanes of the row; all 8 lanes of the row take part in the shuffles.
                const uint32_t seg_mask = 0xFFu << (lane & 24);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int first = 5 * (4 * sub + k);                  // first code of the byte; beyond the row for bytes >= 26
                    const int src = min(first >> 4, 7);
                    const uint32_t lo = __shfl_sync(seg_mask, words[0], (lane & 24) + src);
                    uint32_t hi = __shfl_sync(seg_mask, words[0], (lane & 24) + min(src + 1, 7));
                    if (src == 7) hi = 0u;                                // codes past channel 127 do not exist: digits 0
                    const uint32_t f = (uint32_t)((((unsigned long long)hi << 32) | lo) >> (2 * (first & 15))) & 0x3FFu;
                    const uint32_t byte = (f & 3u) + 3u * ((f >> 2) & 3u) + 9u * ((f >> 4) & 3u) + 27u * ((f >> 6) & 3u) + 81u * ((f >> 8) & 3u);
                    tern |= byte << (8 * k);
                }
            }
            if (do_quant && !SKVQ_IN_BOUNDS(t >= 0 && t < s.cap && (from_ring || (t - L0 >= 0 && t - L0 < a.n_new)), a.c.status)) do_quant = false;
            if (do_quant && t < s.n_sink) {
                // an attention sink (Sec. 3.2 filter rule): its reordered fp16 row is kept as it is
                __align__(16) __half xh16[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) xh16[j] = __float2half_rn(x[j]);      // exact: x came from fp16
                uint4 *p = reinterpret_cast<uint4 *>((is_v ? a.c.v_sink : a.c.k_sink) +
                                                     (bh * s.n_sink + t) * (size_t)kHeadDim + (sub << 4));
                p[0] = *reinterpret_cast<const uint4 *>(&xh16[0]);
                p[1] = *reinterpret_cast<const uint4 *>(&xh16[8]);
            } else if (do_quant) {
                uint8_t *codes_row = codes + (size_t)t * row_bytes;
                if (bits == 2) {
                    reinterpret_cast<uint32_t *>(codes_row)[sub] = words[0];
                } else if (bits == 3) {      // 48 bits per lane: the row stream continues without padding
                    uint16_t *p = reinterpret_cast<uint16_t *>(codes_row) + 3 * sub;
                    p[0] = (uint16_t)words[0];
                    p[1] = (uint16_t)(words[0] >> 16);
                    p[2] = (uint16_t)words[1];
                } else if (bits == kTernary) {      // 26 bytes per row, rows 2-byte aligned: lanes 0-5 hold four bytes, lane 6 two
                    uint16_t *p = reinterpret_cast<uint16_t *>(codes_row) + 2 * sub;
                    if (sub < 7) p[0] = (uint16_t)tern;
                    if (sub < 6) p[1] = (uint16_t)(tern >> 16);
                } else {
                    reinterpret_cast<uint2 *>(codes_row)[sub] = make_uint2(words[0], words[1]);
                }
                if (sub == lane_lo) {
                    const size_t mi = meta0 + (size_t)t * s.ng + g;
                    if (f8) reinterpret_cast<uint16_t *>(meta)[mi] = (uint16_t)hz;
                    else reinterpret_cast<uint32_t *>(meta)[mi] = hz;
                }
            }
        }
        if (do_ring_write && !SKVQ_IN_BOUNDS(W > 0 && ring_token - L0 >= 0 && ring_token - L0 < a.n_new, a.c.status)) do_ring_write = false;
        if (do_ring_write) {
            const __half *row = src + (size_t)(ring_token - L0) * src_tok_stride;
#pragma unroll
            for (int j = 0; j < 16; ++j) xh[j] = row[idx[j]];
            uint4 *p = reinterpret_cast<uint4 *>(win + (size_t)(ring_token % W) * kHeadDim + (sub << 4));
            p[0] = *reinterpret_cast<const uint4 *>(&xh[0]);
            p[1] = *reinterpret_cast<const uint4 *>(&xh[8]);
        }
    }
}

constexpr int kBulkTok = 64;      // the smallest append that goes through the tile kernel

// lengths[b] += n_b, or flag an overflow and leave the sequence alone.
__global__ void append_bookkeeping_kernel(AppendArgs a)
{
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");      // every append CTA has read the old lengths
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= a.s.B) return;
    const int n_b = seq_new_count(a, b);
    const int L1 = a.c.lengths[b] + n_b;
    if (L1 > a.s.max_tokens) {
        if (a.c.status) atomicOr(a.c.status, SKVQ_STATUS_OVERFLOW);
    } else {
        a.c.lengths[b] = L1;
    }
}

}  // namespace

cudaError_t launch_append(const Shape &s, const CachePtrs &c, const __half *k, const __half *v,
                          const int32_t *n_new_per_seq, int n_new, cudaStream_t stream)
{
    if (n_new <= 0) return cudaSuccess;
    const bool bulk = n_new >= kBulkTok;
    AppendArgs a{s, c, k, v, n_new_per_seq, n_new, bulk ? 1 : 0};
    // what append_kernel keeps: evictions (at most W), and new tokens outside the bulk tiles (fewer than W + 128
    // when there are bulk tiles, all of them otherwise)
    const int n_evict_max = s.W < n_new ? s.W : n_new;
    const int n_rest_max = bulk ? (n_new < s.W + 127 ? n_new : s.W + 127) : n_new;
    const int max_items = n_evict_max + n_rest_max;
    int launched = 0;
    if (bulk) {
        cudaError_t e = launch_append_tiles(a, stream);
        if (e != cudaSuccess) return e;
        ++launched;
    }
    dim3 grid((max_items + kItemsPerCta - 1) / kItemsPerCta, s.Hkv, s.B);
    append_kernel<<<grid, kAppendThreads, 0, stream>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    {
        // launched while append_kernel still runs (it waits for that grid before it touches the lengths)
        cudaLaunchConfig_t lc = {};
        lc.gridDim = dim3((s.B + 127) / 128);
        lc.blockDim = dim3(128);
        lc.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = attr;
        lc.numAttrs = 1;
        e = cudaLaunchKernelEx(&lc, append_bookkeeping_kernel, a);
        if (e != cudaSuccess) return e;
    }
    count_launch(launched + 2);
    return cudaGetLastError();
}

}  // namespace skvq

// skvq_quantize_append: channel reorder, group-wise clipped dynamic asymmetric quantization,
// 2/4-bit packing and sliding-window bookkeeping (Sec. 3.1 Eq. 2, Sec. 3.2, Algorithm 1).
//
// Work decomposition.  For sequence b with L0 tokens before and L1 = L0 + n_b after the call:
//   "evict" items   tokens t in [max(L0-W,0), min(L0, L1-W)): still in the fp16 ring (already in
//                   reordered order).  The owner quantizes ring slot t % W into row t and then
//                   refills the same slot with the one new token t' = t (mod W) that ends up inside
//                   the final window, so the read and the overwrite of a slot never race.
//   "new" items     tokens t in [L0, L1): quantized straight from the input if t < L1-W, else
//                   written to the ring unless an evict item refills that slot.
// Eight lanes own one 128-channel row (16 channels each); a warp handles two tokens at a time,
// K rows on lanes 0-7/16-23 and V rows on lanes 8-15/24-31.  Group statistics are reduced with
// xor-shuffles over G/16 lanes.  All quantizer arithmetic uses explicitly rounded fp32 intrinsics
// so the codes, scales and zeros do not depend on compiler contraction.
#include "skvq_internal.cuh"

namespace skvq {
namespace {

constexpr int kItemsPerCta = 64;
constexpr int kAppendThreads = 128;

struct AppendArgs {
    Shape s;
    CachePtrs c;
    const __half *k, *v;
    const int32_t *n_new_per_seq;
    int n_new;
};

__device__ __forceinline__ int seq_new_count(const AppendArgs &a, int b)
{
    int n = a.n_new_per_seq ? a.n_new_per_seq[b] : a.n_new;
    return min(max(n, 0), a.n_new);
}

// Quantize the 16 channels held by this lane; `lanes_per_group` lanes share the group statistics.
template <int BITS>
__device__ __forceinline__ void quantize16(const float (&x)[16], float alpha, int lanes_per_group, uint32_t (&words)[2],
                                           __half2 &hz)
{
    // The 8 lanes that own one row always take the same path, so they are the shuffle's member set
    // (K and V rows may use different bit widths and therefore different instantiations).
    const uint32_t seg_mask = 0xFFu << ((threadIdx.x & 31) & 24);
    constexpr int qmax = (1 << BITS) - 1;
    float mn = x[0], mx = x[0];
#pragma unroll
    for (int j = 1; j < 16; ++j) {
        mn = fminf(mn, x[j]);
        mx = fmaxf(mx, x[j]);
    }
    for (int m = 1; m < lanes_per_group; m <<= 1) {
        mn = fminf(mn, __shfl_xor_sync(seg_mask, mn, m));
        mx = fmaxf(mx, __shfl_xor_sync(seg_mask, mx, m));
    }
    // Clip both ends (Eq. 2 / clipping_quant); "+ 0" turns a negative zero into +0.
    const float lo = __fadd_rn(__fmul_rn(alpha, mn), 0.0f);
    const float hi = __fadd_rn(__fmul_rn(alpha, mx), 0.0f);
    const float h32 = __fdiv_rn(__fsub_rn(hi, lo), (float)qmax);
    const __half h16 = __float2half_rn(h32);
    const __half z16 = __float2half_rn(lo);
    const float hf = __half2float(h16);
    const float zf = __half2float(z16);
    hz = __halves2half2(h16, z16);
    words[0] = 0u;
    words[1] = 0u;
    if (hf != 0.0f) {
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            float r = rintf(__fdiv_rn(__fsub_rn(x[j], zf), hf));
            r = fminf(fmaxf(r, 0.0f), (float)qmax);
            const uint32_t code = (uint32_t)(int)r;
            words[(j * BITS) >> 5] |= code << ((j * BITS) & 31);
        }
    }
}

__global__ void __launch_bounds__(kAppendThreads) append_kernel(AppendArgs a)
{
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
    const int n_items = n_evict + n_b;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane & 7;
    const bool is_v = (lane >> 3) & 1;
    const int tok_sel = lane >> 4;

    const int bits = is_v ? s.v_bits : s.k_bits;
    const int row_bytes = kHeadDim * bits / 8;
    const size_t bh = (size_t)b * s.Hkv + h;
    uint8_t *codes = (is_v ? a.c.v_codes : a.c.k_codes) + bh * (size_t)s.cap * row_bytes;
    __half2 *meta = (is_v ? a.c.v_meta : a.c.k_meta) + bh * (size_t)s.cap * s.ng;
    __half *win = (is_v ? a.c.v_win : a.c.k_win) + bh * (size_t)W * kHeadDim;
    const __half *src = (is_v ? a.v : a.k) + ((size_t)b * a.n_new * s.Hkv + h) * kHeadDim;   // token stride Hkv*D
    const size_t src_tok_stride = (size_t)s.Hkv * kHeadDim;
    const float *alpha_head = (is_v ? a.c.alpha_v : a.c.alpha_k) + (size_t)h * s.ng;

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
            const int lanes_per_group = s.G >> 4;
            const int g = (sub << 4) / s.G;
            const float alpha = alpha_head[g];
            uint32_t words[2];
            __half2 hz;
            if (bits == 2) quantize16<2>(x, alpha, lanes_per_group, words, hz);
            else quantize16<4>(x, alpha, lanes_per_group, words, hz);
            if (do_quant) {
                uint8_t *codes_row = codes + (size_t)t * row_bytes;
                if (bits == 2) reinterpret_cast<uint32_t *>(codes_row)[sub] = words[0];
                else reinterpret_cast<uint2 *>(codes_row)[sub] = make_uint2(words[0], words[1]);
                if ((sub & (lanes_per_group - 1)) == 0) meta[(size_t)t * s.ng + g] = hz;
            }
        }
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

// lengths[b] += n_b, or flag an overflow and leave the sequence alone.
__global__ void append_bookkeeping_kernel(AppendArgs a)
{
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
    AppendArgs a{s, c, k, v, n_new_per_seq, n_new};
    const int max_items = (s.W < n_new ? s.W : n_new) + n_new;
    dim3 grid((max_items + kItemsPerCta - 1) / kItemsPerCta, s.Hkv, s.B);
    append_kernel<<<grid, kAppendThreads, 0, stream>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    append_bookkeeping_kernel<<<(s.B + 127) / 128, 128, 0, stream>>>(a);
    count_launch(2);
    return cudaGetLastError();
}

}  // namespace skvq

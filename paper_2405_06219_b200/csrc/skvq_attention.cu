// skvq_decode_attention: softmax(q K~^T) V~ of one query per sequence over
// [packed quantized prefix || fp16 window] (Eq. 1, Algorithm 1), split along the sequence
// (flash-decoding) with a log-sum-exp merge.  Dequantization happens in registers.
//
// Per (sequence, KV head, split) one CTA serves all rep = Hq/Hkv query heads that share the
// KV head.  It never forms h*code+z per element for the scores: with q' the permuted query,
//   q'.K~_t = sum_g h_{t,g} (sum_{j in g} q'_j c_{t,j}) + sum_g z_{t,g} (sum_{j in g} q'_j)
// so the zero points cost one multiply-add per group.  Scores live in the log2 domain
// (sm_scale*log2(e) folded into q').  The split that owns the tail also walks the fp16 ring.
// Partials (o'[128], m, l) go to the caller's workspace; merge_kernel combines them, divides
// by the softmax denominator, undoes the value permutation and writes fp16.
#include <math_constants.h>

#include "skvq_internal.cuh"

namespace skvq {
namespace {

constexpr int kThreads = 128;
constexpr int kTile = 128;   // tokens per tile = threads

struct AttnArgs {
    Shape s;
    CachePtrs c;
    const __half *q;
    __half *out;
    float scale_log2;   // sm_scale * log2(e)
    SplitPlan plan;
    float *ws;
};

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, m));
    return v;
}
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
    return v;
}

// Scalar partition kernel (configurations the tensor-core kernel does not cover: 4-bit codes, mixed
// widths, 8 query heads per KV head): one thread per token for the scores, one per channel for P.V.
template <int KBITS, int VBITS>
__global__ void __launch_bounds__(kThreads) partition_kernel(AttnArgs a)
{
    const Shape &s = a.s;
    const int split = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rep = s.rep, G = s.G, ng = s.ng, W = s.W;
    const int L = a.c.lengths[b];
    const int Lq = max(L - W, 0);
    const bool owns_window = (split == a.plan.n_splits);      // the last part is the fp16 window
    const int q_begin = owns_window ? Lq : min(split * a.plan.split_len, Lq);
    const int q_end = owns_window ? Lq : min(q_begin + a.plan.split_len, Lq);
    const int n_parts = a.plan.n_splits + 1;

    __shared__ float sq[kMaxRep][kHeadDim];        // permuted query, times sm_scale*log2(e)
    __shared__ float sqsum[kMaxRep][4];            // per-group sums of the above
    __shared__ float sp[kMaxRep][kTile];           // probabilities of the current tile
    __shared__ float sred[kMaxRep][kThreads / 32];

    const size_t bh = (size_t)b * s.Hkv + hk;
    const int32_t *idx_k = a.c.reorder_k + (size_t)hk * kHeadDim;
    for (int r = 0; r < rep; ++r) {
        const __half *qrow = a.q + ((size_t)b * s.Hq + hk * rep + r) * kHeadDim;
        sq[r][tid] = __half2float(qrow[idx_k[tid] & (kHeadDim - 1)]) * a.scale_log2;
    }
    __syncthreads();
    if (tid < rep * ng) {
        const int r = tid / ng, g = tid % ng;
        float acc = 0.f;
        for (int j = g * G; j < (g + 1) * G; ++j) acc += sq[r][j];
        sqsum[r][g] = acc;
    }
    __syncthreads();

    constexpr int KROW = kHeadDim * KBITS / 8, VROW = kHeadDim * VBITS / 8;
    constexpr int KQMAX = (1 << KBITS) - 1, VQMAX = (1 << VBITS) - 1;
    const uint8_t *k_codes = a.c.k_codes + bh * (size_t)s.cap * KROW;
    const uint8_t *v_codes = a.c.v_codes + bh * (size_t)s.cap * VROW;
    const __half2 *k_meta = a.c.k_meta + bh * (size_t)s.cap * ng;
    const __half2 *v_meta = a.c.v_meta + bh * (size_t)s.cap * ng;
    const __half *k_win = a.c.k_win + bh * (size_t)W * kHeadDim;
    const __half *v_win = a.c.v_win + bh * (size_t)W * kHeadDim;

    float m_run[kMaxRep], l_thread[kMaxRep], acc[kMaxRep];
#pragma unroll
    for (int r = 0; r < kMaxRep; ++r) { m_run[r] = -CUDART_INF_F; l_thread[r] = 0.f; acc[r] = 0.f; }

    // Two passes over "segments": the quantized range of this split, then (for the owner) the window.
    for (int seg = 0; seg < 2; ++seg) {
        const bool quant = (seg == 0);
        if (!quant && !owns_window) break;
        const int t_begin = quant ? q_begin : Lq;
        const int t_end = quant ? q_end : L;
        for (int tile0 = t_begin; tile0 < t_end; tile0 += kTile) {
            const int t = tile0 + tid;
            const bool valid = t < t_end;
            float sc[kMaxRep];
#pragma unroll
            for (int r = 0; r < kMaxRep; ++r) sc[r] = -CUDART_INF_F;
            if (valid) {
#pragma unroll
                for (int r = 0; r < kMaxRep; ++r) sc[r] = 0.f;
                if (quant) {
                    const uint32_t *row = reinterpret_cast<const uint32_t *>(k_codes + (size_t)t * KROW);
                    constexpr int PER_WORD = 32 / KBITS;
                    for (int g = 0; g < ng; ++g) {
                        float part[kMaxRep];
#pragma unroll
                        for (int r = 0; r < kMaxRep; ++r) part[r] = 0.f;
                        for (int w = g * G / PER_WORD; w < (g + 1) * G / PER_WORD; ++w) {
                            const uint32_t word = __ldg(row + w);
#pragma unroll
                            for (int i = 0; i < PER_WORD; ++i) {
                                const float code = (float)((word >> (i * KBITS)) & KQMAX);
                                const int j = w * PER_WORD + i;
#pragma unroll
                                for (int r = 0; r < kMaxRep; ++r)
                                    if (r < rep) part[r] = fmaf(sq[r][j], code, part[r]);
                            }
                        }
                        const float2 hz = __half22float2(k_meta[(size_t)t * ng + g]);
#pragma unroll
                        for (int r = 0; r < kMaxRep; ++r)
                            if (r < rep) sc[r] += hz.x * part[r] + hz.y * sqsum[r][g];
                    }
                } else {
                    const __half2 *row = reinterpret_cast<const __half2 *>(k_win + (size_t)(t % W) * kHeadDim);
                    for (int j2 = 0; j2 < kHeadDim / 2; ++j2) {
                        const float2 kv = __half22float2(row[j2]);
#pragma unroll
                        for (int r = 0; r < kMaxRep; ++r)
                            if (r < rep) sc[r] = fmaf(sq[r][2 * j2], kv.x, fmaf(sq[r][2 * j2 + 1], kv.y, sc[r]));
                    }
                }
            }
            // Online softmax update per query head.
            float corr[kMaxRep];
#pragma unroll
            for (int r = 0; r < kMaxRep; ++r) {
                corr[r] = 1.f;
                if (r < rep) {
                    const float wm = warp_max(sc[r]);
                    if (lane == 0) sred[r][warp] = wm;
                }
            }
            __syncthreads();
#pragma unroll
            for (int r = 0; r < kMaxRep; ++r) {
                if (r < rep) {
                    float tm = sred[r][0];
#pragma unroll
                    for (int w = 1; w < kThreads / 32; ++w) tm = fmaxf(tm, sred[r][w]);
                    const float m_new = fmaxf(m_run[r], tm);    // finite: the tile has a valid token
                    corr[r] = exp2f(m_run[r] - m_new);          // exp2(-inf) = 0 on the first tile
                    const float p = valid ? exp2f(sc[r] - m_new) : 0.f;
                    sp[r][tid] = p;
                    l_thread[r] = l_thread[r] * corr[r] + p;
                    m_run[r] = m_new;
                    acc[r] *= corr[r];
                }
            }
            __syncthreads();
            // P.V: this thread owns (reordered) channel tid.
            const int n_tok = min(kTile, t_end - tile0);
            if (quant) {
                constexpr int PER_WORD = 32 / VBITS;
                const int g = tid / G;
                const int w = tid / PER_WORD, sh = (tid % PER_WORD) * VBITS;
                for (int tt = 0; tt < n_tok; ++tt) {
                    const size_t row = (size_t)(tile0 + tt);
                    const uint32_t word = __ldg(reinterpret_cast<const uint32_t *>(v_codes + row * VROW) + w);
                    const float2 hz = __half22float2(v_meta[row * ng + g]);
                    const float val = fmaf(hz.x, (float)((word >> sh) & VQMAX), hz.y);
#pragma unroll
                    for (int r = 0; r < kMaxRep; ++r)
                        if (r < rep) acc[r] = fmaf(sp[r][tt], val, acc[r]);
                }
            } else {
                for (int tt = 0; tt < n_tok; ++tt) {
                    const float val = __half2float(v_win[(size_t)((tile0 + tt) % W) * kHeadDim + tid]);
#pragma unroll
                    for (int r = 0; r < kMaxRep; ++r)
                        if (r < rep) acc[r] = fmaf(sp[r][tt], val, acc[r]);
                }
            }
            __syncthreads();   // sp and sred are rewritten by the next tile
        }
    }

    // Write the partial: o'[d], m, l per query head.
#pragma unroll
    for (int r = 0; r < kMaxRep; ++r) {
        if (r < rep) {
            const float ws_ = warp_sum(l_thread[r]);
            if (lane == 0) sred[r][warp] = ws_;
        }
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < kMaxRep; ++r) {
        if (r < rep) {
            float *part = a.ws + (((size_t)b * s.Hq + hk * rep + r) * n_parts + split) * kPartialStride;
            part[tid] = acc[r];
            if (tid == 0) {
                float l = 0.f;
                for (int w = 0; w < kThreads / 32; ++w) l += sred[r][w];
                part[kHeadDim] = m_run[r];
                part[kHeadDim + 1] = l;
            }
        }
    }
}

// Combine the split partials of one (sequence, query head): thread d owns reordered channel d.
__global__ void __launch_bounds__(kHeadDim) merge_kernel(AttnArgs a)
{
    const int hq = blockIdx.x, b = blockIdx.y, d = threadIdx.x;
    const Shape &s = a.s;
    const int hk = hq / s.rep;
    const int S = a.plan.n_splits + 1;
    const float *part = a.ws + ((size_t)b * s.Hq + hq) * S * kPartialStride;
    float M = -CUDART_INF_F;
    for (int i = 0; i < S; ++i) M = fmaxf(M, part[(size_t)i * kPartialStride + kHeadDim]);
    float o = 0.f, l = 0.f;
    if (M > -CUDART_INF_F) {
        for (int i = 0; i < S; ++i) {
            const float *p = part + (size_t)i * kPartialStride;
            const float w = exp2f(p[kHeadDim] - M);
            o = fmaf(p[d], w, o);
            l = fmaf(p[kHeadDim + 1], w, l);
        }
    }
    const float res = l > 0.f ? o / l : 0.f;
    const int dst = a.c.reorder_v[(size_t)hk * kHeadDim + d] & (kHeadDim - 1);
    a.out[((size_t)b * s.Hq + hq) * kHeadDim + dst] = __float2half_rn(res);
}

}  // namespace

SplitPlan plan_splits(const Shape &s, int max_len, int requested_splits)
{
    const int lq = max_len - s.W > 0 ? max_len - s.W : 0;
    SplitPlan p;
    long split_len;
    if (requested_splits > 0) {
        split_len = (lq + requested_splits - 1) / requested_splits;
        split_len = (split_len + SKVQ_TOKEN_ALIGN - 1) / SKVQ_TOKEN_ALIGN * SKVQ_TOKEN_ALIGN;
    } else {
        // About 8 CTAs per resident slot (148 SMs x 3 CTAs), between 1024 and 8192 tokens per split,
        // in multiples of 256 tokens (4 warps x 64-token tiles).
        const long total = (long)lq * s.B * s.Hkv;
        split_len = (total + 148L * 3 * 8 - 1) / (148L * 3 * 8);
        if (split_len < 1024) split_len = 1024;
        if (split_len > 8192) split_len = 8192;
        split_len = (split_len + 255) / 256 * 256;
    }
    if (split_len < SKVQ_TOKEN_ALIGN) split_len = SKVQ_TOKEN_ALIGN;
    p.split_len = (int)split_len;
    p.n_splits = (int)((lq + split_len - 1) / split_len);
    if (p.n_splits < 1) p.n_splits = 1;
    return p;
}

cudaError_t launch_attention(const Shape &s, const CachePtrs &c, const __half *q, __half *out, float sm_scale,
                             const SplitPlan &plan, float *workspace, cudaEvent_t ev_begin, cudaEvent_t ev_end,
                             cudaStream_t stream)
{
    AttnArgs a{s, c, q, out, sm_scale * 1.4426950408889634f, plan, workspace};
    dim3 grid(plan.n_splits + 1, s.Hkv, s.B);
    if (ev_begin) cudaEventRecord(ev_begin, stream);
    bool handled = false;
    cudaError_t em = launch_partition_mma(s, c, q, a.scale_log2, plan, workspace, stream, &handled);
    if (em != cudaSuccess) return em;
    if (!handled) {
        em = launch_partition_gqa(s, c, q, a.scale_log2, plan, workspace, stream, &handled);
        if (em != cudaSuccess) return em;
    }
    if (handled) { /* tensor-core kernel launched */ }
    else if (s.k_bits == 2 && s.v_bits == 2) partition_kernel<2, 2><<<grid, kThreads, 0, stream>>>(a);
    else if (s.k_bits == 4 && s.v_bits == 4) partition_kernel<4, 4><<<grid, kThreads, 0, stream>>>(a);
    else if (s.k_bits == 4 && s.v_bits == 2) partition_kernel<4, 2><<<grid, kThreads, 0, stream>>>(a);
    else partition_kernel<2, 4><<<grid, kThreads, 0, stream>>>(a);
    if (ev_end) cudaEventRecord(ev_end, stream);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    merge_kernel<<<dim3(s.Hq, s.B), kHeadDim, 0, stream>>>(a);
    count_launch(2);
    return cudaGetLastError();
}

}  // namespace skvq

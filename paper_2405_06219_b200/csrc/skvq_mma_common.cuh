// Pieces shared by the tensor-core partition kernels of skvq_decode_attention: launch arguments, PTX
// wrappers (mma.sync, ldmatrix, cp.async.bulk + mbarrier with bounded polling) and the scalar code for
// the fp16 window part.
#pragma once
#include <math_constants.h>

#include "skvq_internal.cuh"

namespace skvq {
namespace mmak {

constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr int kTileTok = 64;                 // tokens per warp tile
constexpr int kRowBytes = 32;                // 128 channels x 2 bits
constexpr uint32_t kWaitLimit = 1u << 22;    // bounded mbarrier polling

struct MmaArgs {
    Shape s;
    CachePtrs c;
    const __half *q;
    float scale_log2;
    SplitPlan plan;
    float *ws;
};

// ---------------------------------------------------------------- small PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t mask, uint32_t magic)
{
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(a), "r"(mask), "r"(magic));
    return r;
}

__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void imma16832(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void imma16832_uu(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Two 16x16 byte matrices, transposed: lanes 0-15 give the row addresses of the first, lanes 16-31 of the
// second.  Lane (g,t) receives r0 = bytes (rows 4t..4t+3, column g), r1 = (rows 4t..4t+3, column g+8) of the
// first matrix and r2, r3 likewise of the second: exactly the A fragment of mma.m16n8k32 with rows = byte
// columns and k = matrix rows.
__device__ __forceinline__ void ldmatrix_b8_trans_x2(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m16n16.x2.trans.shared.b8 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Poll with an iteration limit; false means the copy never completed (reported, never spun on forever).
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity)
{
    for (uint32_t i = 0; i < kWaitLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// Bulk asynchronous copy global -> this CTA's shared memory; 16-byte aligned addresses, size % 16 == 0.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

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

// Scalar path for the fp16 window part (at most W tokens; a few percent of the bytes).
template <int R>
__device__ void window_part(const MmaArgs &a, int b, int hk, uint8_t *smem_raw)
{
    const Shape &s = a.s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int W = s.W;
    const int L = a.c.lengths[b];
    const int Lq = max(L - W, 0);
    float (*sq)[kHeadDim] = reinterpret_cast<float (*)[kHeadDim]>(smem_raw);                 // [R][128]
    float (*sp)[kThreads] = reinterpret_cast<float (*)[kThreads]>(smem_raw + R * kHeadDim * 4);   // [R][128]
    float (*sred)[kWarps] = reinterpret_cast<float (*)[kWarps]>(smem_raw + 2 * R * kHeadDim * 4);  // [R][4]
    const size_t bh = (size_t)b * s.Hkv + hk;
    const int32_t *idx_k = a.c.reorder_k + (size_t)hk * kHeadDim;
#pragma unroll
    for (int r = 0; r < R; ++r)
        sq[r][tid] = __half2float(a.q[((size_t)b * s.Hq + hk * R + r) * kHeadDim + (idx_k[tid] & (kHeadDim - 1))]) * a.scale_log2;
    __syncthreads();
    const __half *k_win = a.c.k_win + bh * (size_t)W * kHeadDim;
    const __half *v_win = a.c.v_win + bh * (size_t)W * kHeadDim;
    float m_run[R], l_thread[R], acc[R];
#pragma unroll
    for (int r = 0; r < R; ++r) { m_run[r] = -CUDART_INF_F; l_thread[r] = 0.f; acc[r] = 0.f; }
    for (int tile0 = Lq; tile0 < L; tile0 += kThreads) {
        const int t = tile0 + tid;
        const bool valid = t < L;
        float sc[R];
#pragma unroll
        for (int r = 0; r < R; ++r) sc[r] = valid ? 0.f : -CUDART_INF_F;
        if (valid) {
            const uint4 *row = reinterpret_cast<const uint4 *>(k_win + (size_t)(t % W) * kHeadDim);
#pragma unroll 4
            for (int j8 = 0; j8 < kHeadDim / 8; ++j8) {
                const uint4 u = __ldg(row + j8);
                const __half2 *h2 = reinterpret_cast<const __half2 *>(&u);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 kv = __half22float2(h2[i]);
#pragma unroll
                    for (int r = 0; r < R; ++r)
                        sc[r] = fmaf(sq[r][8 * j8 + 2 * i], kv.x, fmaf(sq[r][8 * j8 + 2 * i + 1], kv.y, sc[r]));
                }
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const float wm = warp_max(sc[r]);
            if (lane == 0) sred[r][warp] = wm;
        }
        __syncthreads();
#pragma unroll
        for (int r = 0; r < R; ++r) {
            float tm = sred[r][0];
#pragma unroll
            for (int w = 1; w < kWarps; ++w) tm = fmaxf(tm, sred[r][w]);
            const float m_new = fmaxf(m_run[r], tm);
            const float corr = exp2f(m_run[r] - m_new);
            const float p = valid ? exp2f(sc[r] - m_new) : 0.f;
            sp[r][tid] = p;
            l_thread[r] = l_thread[r] * corr + p;
            m_run[r] = m_new;
            acc[r] *= corr;
        }
        __syncthreads();
        const int n_tok = min(kThreads, L - tile0);
        for (int tt = 0; tt < n_tok; ++tt) {
            const float val = __half2float(v_win[(size_t)((tile0 + tt) % W) * kHeadDim + tid]);
#pragma unroll
            for (int r = 0; r < R; ++r) acc[r] = fmaf(sp[r][tt], val, acc[r]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const float wsum = warp_sum(l_thread[r]);
        if (lane == 0) sred[r][warp] = wsum;
    }
    __syncthreads();
    const int part_idx = a.plan.n_splits;   // the window is the last part
    const int n_parts = a.plan.n_splits + 1;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        float *part = a.ws + (((size_t)b * s.Hq + hk * R + r) * n_parts + part_idx) * kPartialStride;
        part[tid] = acc[r];
        if (tid == 0) {
            float l = 0.f;
            for (int w = 0; w < kWarps; ++w) l += sred[r][w];
            part[kHeadDim] = m_run[r];
            part[kHeadDim + 1] = l;
        }
    }
}

}  // namespace mmak
}  // namespace skvq

// Tensor-core partition kernel of skvq_decode_attention for 2-bit K and V (Eq. 1, Algorithm 1).
//
// Why tensor cores on an HBM-bound path: at 2 bits a cache element costs 0.28 bytes, so streaming
// at several TB/s leaves fewer than two issue slots per element on the scalar pipes.  The 2-bit
// codes are therefore turned into fp16 operands with ONE logic op per two codes and contracted
// with mma.sync.m16n8k16 (fp32 accumulate); scale and zero point never touch individual elements:
//   q'.K~_t   = sum_g h_{t,g} (sum_{j in g} q'_j c_{t,j}) + sum_g z_{t,g} (sum_{j in g} q'_j)
//   sum_t p_t V~_{t,d} = sum_t (p_t h_{t,g(d)}) c_{t,d} + sum_t p_t z_{t,g(d)}
// Unpack trick: OR-ing a 2-bit field that sits at mantissa bits [p, p+2) of an fp16 lane with an
// exponent pattern gives the half value  base + weight*code  (base = 2^E, weight = 2^(E+p-10)).
// The constant base contributes base * sum(B operand), which is subtracted in fp32 afterwards;
// the weight is folded into the other operand (K side) or divided out at the end (V side).
//
// One CTA = 4 independent warps on one (sequence, KV head, split); each warp streams 64-token
// tiles of codes + scale/zero through its own ring of shared-memory stages filled by
// cp.async.bulk (mbarrier completion), keeps its own online-softmax state, and the 4 states are
// merged in shared memory before one partial per query head is written to the workspace.
// The fp16 window is a separate, small "part" handled by scalar code.
#include <math_constants.h>

#include "skvq_internal.cuh"

namespace skvq {
namespace {

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
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
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

// ---------------------------------------------------------------- compile-time layout
template <int G, int R>
struct Cfg {
    static constexpr int NG = kHeadDim / G;
    static constexpr int PIECES = (R * NG * 2 <= 8) ? 2 : 1;             // P split into hi+lo halves when columns allow
    static constexpr int NCV = R * NG * PIECES;                          // V-side columns: (head, group, piece)
    static constexpr int NTV = (NCV + 7) / 8;
    static constexpr int NCVP = NTV * 8;
    static constexpr int kCodeTile = kTileTok * kRowBytes;               // 2048 B
    static constexpr int kMetaTile = kTileTok * NG * 4;                  // 256 B * NG
    static constexpr int kStageBytes = 2 * kCodeTile + 2 * kMetaTile;
    static constexpr int kStages = 3;
    static constexpr int kScBytes = kTileTok * R * NG * 4;               // per-group raw scores
    static constexpr int kPBytes = 4 * NCVP * 16 * 2;                    // P operand tile
    static constexpr int kWarpBytes = kStages * kStageBytes + kScBytes + kPBytes + 64;   // + mbarriers
    static constexpr int kQBytes = (R * kHeadDim * 4 + 2 * R * NG * 4 + 127) / 128 * 128;
    static constexpr int kSmemBytes = kQBytes + kWarps * kWarpBytes;
    static_assert(kStages * kStageBytes >= NCV * kHeadDim * 4 + R * kPartialStride * 4, "stage area is reused for the final merge");
};

// V-side field weights: field f of a 16-bit half lands at mantissa position 4, 6 or 8 of (x<<4, x, x>>6).
__device__ __forceinline__ float v_weight_inv(int f)
{
    // weights {1,4,16,4,16,1,4,16}
    const int sel = (f == 0 || f == 5) ? 0 : ((f == 1 || f == 3 || f == 6) ? 1 : 2);
    return sel == 0 ? 1.0f : (sel == 1 ? 0.25f : 0.0625f);
}

// Eight half2 operands (value 64 + w_f*code) from a word made of two 16-bit halves of eight 2-bit fields each.
__device__ __forceinline__ void unpack_v(uint32_t x, uint32_t (&o)[8])
{
    constexpr uint32_t MAGIC = 0x54005400u, M4 = 0x00300030u, M6 = 0x00C000C0u, M8 = 0x03000300u;
    const uint32_t s0 = x << 4, s2 = x >> 6;
    o[0] = and_or(s0, M4, MAGIC);
    o[1] = and_or(s0, M6, MAGIC);
    o[2] = and_or(s0, M8, MAGIC);
    o[3] = and_or(x, M6, MAGIC);
    o[4] = and_or(x, M8, MAGIC);
    o[5] = and_or(s2, M4, MAGIC);
    o[6] = and_or(s2, M6, MAGIC);
    o[7] = and_or(s2, M8, MAGIC);
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

template <int G, int R>
__global__ void __launch_bounds__(kThreads) partition_mma_kernel(MmaArgs a)
{
    using C = Cfg<G, R>;
    constexpr int NG = C::NG;
    extern __shared__ __align__(128) uint8_t smem[];
    const Shape &s = a.s;
    const int part = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
    if (part == a.plan.n_splits) {
        window_part<R>(a, b, hk, smem);
        return;
    }
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int L = a.c.lengths[b];
    const int Lq = max(L - s.W, 0);
    const int q_begin = min(part * a.plan.split_len, Lq);
    const int q_end = min(q_begin + a.plan.split_len, Lq);
    const int n_parts = a.plan.n_splits + 1;

    // ---- CTA-wide prologue: permuted query, per-(head, group) constants
    float *qs = reinterpret_cast<float *>(smem);                       // [R][128] q' (exact fp16 values)
    float *koff = qs + R * kHeadDim;                                   // [R][NG] scale * 16 * sum of the B operand
    float *sqs = koff + R * NG;                                        // [R][NG] scale * sum_j q'_j
    uint8_t *warp_base = smem + C::kQBytes + warp * C::kWarpBytes;
    {
        const int32_t *idx_k = a.c.reorder_k + (size_t)hk * kHeadDim;
        const int src = idx_k[tid] & (kHeadDim - 1);
#pragma unroll
        for (int r = 0; r < R; ++r)
            qs[r * kHeadDim + tid] = __half2float(a.q[((size_t)b * s.Hq + hk * R + r) * kHeadDim + src]);
    }
    __syncthreads();
    if (tid < R * NG) {
        const int r = tid / NG, gg = tid % NG;
        float sb = 0.f, sq = 0.f;
        for (int j = gg * G; j < (gg + 1) * G; ++j) {
            const float qv = qs[r * kHeadDim + j];
            // channel j sits in field (j & 7) of its word; odd fields carry weight 4 (see the K unpack below)
            const float bq = __half2float(__float2half_rn((j & 1) ? qv * 0.25f : qv));
            sb += bq;
            sq += qv;
        }
        koff[tid] = 16.0f * sb * a.scale_log2;
        sqs[tid] = sq * a.scale_log2;
    }
    __syncthreads();

    // B operand of the score MMAs: k-step s contracts the 16 channels of code word s.
    //   b0 = (q'[16s+2t], q'[16s+8+2t])          weight 1
    //   b1 = (q'[16s+2t+1], q'[16s+9+2t]) / 4    weight 4
    uint32_t bq[8][2];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        __half2 v0 = __floats2half2_rn(0.f, 0.f), v1 = v0;
        if (g < R) {
            const float *qr = qs + g * kHeadDim + 16 * ks + 2 * t;
            v0 = __floats2half2_rn(qr[0], qr[8]);
            v1 = __floats2half2_rn(qr[1] * 0.25f, qr[9] * 0.25f);
        }
        bq[ks][0] = *reinterpret_cast<uint32_t *>(&v0);
        bq[ks][1] = *reinterpret_cast<uint32_t *>(&v1);
    }

    // ---- per-warp pipeline state
    uint8_t *stage_base = warp_base;
    float *Sc = reinterpret_cast<float *>(warp_base + C::kStages * C::kStageBytes);      // [64][R*NG]
    __half *Pt = reinterpret_cast<__half *>(warp_base + C::kStages * C::kStageBytes + C::kScBytes);
    uint64_t *bars = reinterpret_cast<uint64_t *>(warp_base + C::kStages * C::kStageBytes + C::kScBytes + C::kPBytes);
    const uint32_t bar0 = smem_u32(bars);
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < C::kStages; ++i) mbar_init(bar0 + 8 * i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();

    const size_t bh = (size_t)b * s.Hkv + hk;
    const uint8_t *k_codes = a.c.k_codes + bh * (size_t)s.cap * kRowBytes;
    const uint8_t *v_codes = a.c.v_codes + bh * (size_t)s.cap * kRowBytes;
    const __half2 *k_meta = a.c.k_meta + bh * (size_t)s.cap * NG;
    const __half2 *v_meta = a.c.v_meta + bh * (size_t)s.cap * NG;

    const int n_tiles = (q_end - q_begin + kTileTok - 1) / kTileTok;            // tiles of this split
    const int n_my = n_tiles > warp ? (n_tiles - warp + kWarps - 1) / kWarps : 0;   // tiles warp, warp+4, ...

    auto issue = [&](int i) {   // lane 0 only: start the copies of this warp's i-th tile
        const int st = i % C::kStages;
        const int tok0 = q_begin + (warp + i * kWarps) * kTileTok;                // multiple of 64: 16-byte aligned sources
        const uint32_t dst = smem_u32(stage_base + st * C::kStageBytes);
        const uint32_t bar = bar0 + 8 * st;
        mbar_expect_tx(bar, C::kStageBytes);
        bulk_g2s(dst, k_codes + (size_t)tok0 * kRowBytes, C::kCodeTile, bar);
        bulk_g2s(dst + C::kCodeTile, v_codes + (size_t)tok0 * kRowBytes, C::kCodeTile, bar);
        bulk_g2s(dst + 2 * C::kCodeTile, k_meta + (size_t)tok0 * NG, C::kMetaTile, bar);
        bulk_g2s(dst + 2 * C::kCodeTile + C::kMetaTile, v_meta + (size_t)tok0 * NG, C::kMetaTile, bar);
    };
    if (lane == 0) {
        for (int i = 0; i < C::kStages && i < n_my; ++i) issue(i);
    }

    // online-softmax state (per warp; m is warp-uniform, the sums are per-lane partials)
    float m_run[R], l_part[R], s_part[R][NG], z_part[R][NG];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        m_run[r] = -CUDART_INF_F;
        l_part[r] = 0.f;
#pragma unroll
        for (int gg = 0; gg < NG; ++gg) { s_part[r][gg] = 0.f; z_part[r][gg] = 0.f; }
    }
    float cv[C::NTV][8][4];
#pragma unroll
    for (int nt = 0; nt < C::NTV; ++nt)
#pragma unroll
        for (int f = 0; f < 8; ++f)
#pragma unroll
            for (int i = 0; i < 4; ++i) cv[nt][f][i] = 0.f;

    bool failed = false;
    const int krot = (4 * t - 6) & 31;   // rotate right so that fields 2t, 2t+1 land on mantissa bits 6..9

    for (int i = 0; i < n_my; ++i) {
        const int st = i % C::kStages;
        const uint32_t parity = (uint32_t)(i / C::kStages) & 1u;
        if (!mbar_wait_bounded(bar0 + 8 * st, parity)) { failed = true; break; }
        const uint8_t *Kc = stage_base + st * C::kStageBytes;
        const uint8_t *Vc = Kc + C::kCodeTile;
        const __half2 *Km = reinterpret_cast<const __half2 *>(Kc + 2 * C::kCodeTile);
        const __half2 *Vm = reinterpret_cast<const __half2 *>(Kc + 2 * C::kCodeTile + C::kMetaTile);
        const int tok0 = q_begin + (warp + i * kWarps) * kTileTok;

        // ---------------- scores: C[token][head] per group
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) {
            const uint4 *r0 = reinterpret_cast<const uint4 *>(Kc + (16 * mt + g) * kRowBytes);
            const uint4 *r1 = reinterpret_cast<const uint4 *>(Kc + (16 * mt + g + 8) * kRowBytes);
            const uint4 x0a = r0[0], x0b = r0[1], x1a = r1[0], x1b = r1[1];
            const uint32_t w0[8] = {x0a.x, x0a.y, x0a.z, x0a.w, x0b.x, x0b.y, x0b.z, x0b.w};
            const uint32_t w1[8] = {x1a.x, x1a.y, x1a.z, x1a.w, x1b.x, x1b.y, x1b.z, x1b.w};
            float acc[NG][4];
#pragma unroll
            for (int gg = 0; gg < NG; ++gg)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[gg][e] = 0.f;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                constexpr uint32_t MAGIC = 0x4C004C00u, M6 = 0x00C000C0u, M8 = 0x03000300u;   // 16 + code, 16 + 4*code
                const uint32_t rot0 = __funnelshift_r(w0[ks], w0[ks], krot);
                const uint32_t rot1 = __funnelshift_r(w1[ks], w1[ks], krot);
                mma16816(acc[(16 * ks) / G], and_or(rot0, M6, MAGIC), and_or(rot1, M6, MAGIC), and_or(rot0, M8, MAGIC),
                         and_or(rot1, M8, MAGIC), bq[ks][0], bq[ks][1]);
            }
            // lane (g,t) holds heads 2t, 2t+1 of tokens 16mt+g and 16mt+g+8
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) {
                if (2 * t < R) {
                    Sc[(16 * mt + g) * (R * NG) + (2 * t) * NG + gg] = acc[gg][0];
                    Sc[(16 * mt + g + 8) * (R * NG) + (2 * t) * NG + gg] = acc[gg][2];
                }
                if (2 * t + 1 < R) {
                    Sc[(16 * mt + g) * (R * NG) + (2 * t + 1) * NG + gg] = acc[gg][1];
                    Sc[(16 * mt + g + 8) * (R * NG) + (2 * t + 1) * NG + gg] = acc[gg][3];
                }
            }
        }
        __syncwarp();

        // ---------------- softmax bookkeeping: lane owns tokens lane and lane+32 of the tile
        float sc[2][R];
        bool valid[2];
        float hv[2][NG], zv[2][NG];
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            const int tau = lane + 32 * hf;
            valid[hf] = (tok0 + tau) < q_end;
            float hk_[NG], zk_[NG];
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) {
                const float2 kz = __half22float2(Km[tau * NG + gg]);
                const float2 vz = __half22float2(Vm[tau * NG + gg]);
                hk_[gg] = kz.x; zk_[gg] = kz.y;
                hv[hf][gg] = vz.x; zv[hf][gg] = vz.y;
            }
#pragma unroll
            for (int r = 0; r < R; ++r) {
                float sv = 0.f;
#pragma unroll
                for (int gg = 0; gg < NG; ++gg) {
                    const float u = fmaf(Sc[tau * (R * NG) + r * NG + gg], a.scale_log2, -koff[r * NG + gg]);
                    sv = fmaf(hk_[gg], u, sv);
                    sv = fmaf(zk_[gg], sqs[r * NG + gg], sv);
                }
                sc[hf][r] = valid[hf] ? sv : -CUDART_INF_F;
            }
        }
        float corr[R];
        bool rescale = false;
        float p[2][R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const float tm = warp_max(fmaxf(sc[0][r], sc[1][r]));     // finite: the tile holds a valid token
            const float m_new = fmaxf(m_run[r], tm);
            corr[r] = exp2f(m_run[r] - m_new);
            rescale |= (m_new > m_run[r]);
            m_run[r] = m_new;
            p[0][r] = valid[0] ? exp2f(sc[0][r] - m_new) : 0.f;
            p[1][r] = valid[1] ? exp2f(sc[1][r] - m_new) : 0.f;
            l_part[r] = fmaf(l_part[r], corr[r], p[0][r] + p[1][r]);
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) { s_part[r][gg] *= corr[r]; z_part[r][gg] *= corr[r]; }
        }
        // P operand: value (p*h) per (head, group), split into fp16 hi (+ lo) pieces.
        //   k index of the PV MMAs: k=2t'<->token t', 2t'+1<->t'+4, 2t'+8<->t'+8, 2t'+9<->t'+12 within a 16-token block
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            const int tau = lane + 32 * hf;
            const int kb = tau >> 4, tt = tau & 3, ii = (tau & 15) >> 2;
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int gg = 0; gg < NG; ++gg) {
                    const float ph = valid[hf] ? p[hf][r] * hv[hf][gg] : 0.f;
                    const float pz = valid[hf] ? p[hf][r] * zv[hf][gg] : 0.f;
                    const __half hi = __float2half_rn(ph);
                    float used = __half2float(hi);
                    const int col = (r * NG + gg) * C::PIECES;
                    Pt[((kb * C::NCVP + col) * 4 + tt) * 4 + ii] = hi;
                    if (C::PIECES == 2) {
                        const __half lo = __float2half_rn(ph - used);
                        used += __half2float(lo);
                        Pt[((kb * C::NCVP + col + 1) * 4 + tt) * 4 + ii] = lo;
                    }
                    s_part[r][gg] += used;
                    z_part[r][gg] += pz;
                }
        }
        if (rescale) {   // warp-uniform
#pragma unroll
            for (int nt = 0; nt < C::NTV; ++nt) {
                // this lane's two columns and the heads they belong to
                const int c0 = 8 * nt + 2 * t, c1 = c0 + 1;
                float f0 = 1.f, f1 = 1.f;
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    if (c0 / (NG * C::PIECES) == r) f0 = corr[r];
                    if (c1 / (NG * C::PIECES) == r) f1 = corr[r];
                }
#pragma unroll
                for (int f = 0; f < 8; ++f) {
                    cv[nt][f][0] *= f0; cv[nt][f][2] *= f0;
                    cv[nt][f][1] *= f1; cv[nt][f][3] *= f1;
                }
            }
        }
        __syncwarp();

        // ---------------- P.V: rows = channels (lane g reads code word g), k = tokens
#pragma unroll
        for (int kb = 0; kb < 4; ++kb) {
            const uint32_t *vrow = reinterpret_cast<const uint32_t *>(Vc + (16 * kb + t) * kRowBytes) + g;
            const uint32_t x0 = vrow[0], x1 = vrow[4 * 8], x2 = vrow[8 * 8], x3 = vrow[12 * 8];   // tokens t, t+4, t+8, t+12
            uint32_t A0[8], A1[8], A2[8], A3[8];
            unpack_v(__byte_perm(x0, x1, 0x5410), A0);   // low halves: channels 16g+f,   tokens (t, t+4)
            unpack_v(__byte_perm(x0, x1, 0x7632), A1);   // high halves: channels 16g+8+f
            unpack_v(__byte_perm(x2, x3, 0x5410), A2);   // tokens (t+8, t+12)
            unpack_v(__byte_perm(x2, x3, 0x7632), A3);
#pragma unroll
            for (int nt = 0; nt < C::NTV; ++nt) {
                const uint2 pb = *reinterpret_cast<const uint2 *>(Pt + ((kb * C::NCVP + 8 * nt + g) * 4 + t) * 4);
#pragma unroll
                for (int f = 0; f < 8; ++f) mma16816(cv[nt][f], A0[f], A1[f], A2[f], A3[f], pb.x, pb.y);
            }
        }
        __syncwarp();   // every lane is done with this stage, Sc and Pt
        if (lane == 0 && i + C::kStages < n_my) issue(i + C::kStages);
    }

    if (failed) {
        // Drain (bounded) whatever copies are still in flight into this warp's stages, then report.
        for (int i2 = 0; i2 < n_my; ++i2) {
            const int st = i2 % C::kStages;
            (void)mbar_wait_bounded(bar0 + 8 * st, (uint32_t)(i2 / C::kStages) & 1u);
        }
        if (lane == 0 && a.c.status) atomicOr(a.c.status, 2);
#pragma unroll
        for (int r = 0; r < R; ++r) { m_run[r] = -CUDART_INF_F; l_part[r] = 0.f; }
    }

    // ---- per-warp result: o'[head][channel] in the (now idle) stage area
    float *Ot = reinterpret_cast<float *>(stage_base);                       // [NCV][128]
    float *Ow = Ot + C::NCV * kHeadDim;                                      // [R][132]: o', m, l
    __syncwarp();
#pragma unroll
    for (int nt = 0; nt < C::NTV; ++nt) {
        const int c0 = 8 * nt + 2 * t;
#pragma unroll
        for (int f = 0; f < 8; ++f) {
            if (c0 < C::NCV) {
                Ot[c0 * kHeadDim + 16 * g + f] = cv[nt][f][0];
                Ot[c0 * kHeadDim + 16 * g + 8 + f] = cv[nt][f][2];
            }
            if (c0 + 1 < C::NCV) {
                Ot[(c0 + 1) * kHeadDim + 16 * g + f] = cv[nt][f][1];
                Ot[(c0 + 1) * kHeadDim + 16 * g + 8 + f] = cv[nt][f][3];
            }
        }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
        l_part[r] = warp_sum(l_part[r]);
#pragma unroll
        for (int gg = 0; gg < NG; ++gg) { s_part[r][gg] = warp_sum(s_part[r][gg]); z_part[r][gg] = warp_sum(z_part[r][gg]); }
    }
    __syncwarp();
#pragma unroll
    for (int q4 = 0; q4 < 4; ++q4) {
        const int d = lane + 32 * q4;
        const float winv = v_weight_inv(d & 7);
#pragma unroll
        for (int r = 0; r < R; ++r) {
            float sg = 0.f, zg = 0.f;
#pragma unroll
            for (int gg = 0; gg < NG; ++gg)
                if (d / G == gg) { sg = s_part[r][gg]; zg = z_part[r][gg]; }
            const int col = (r * NG + d / G) * C::PIECES;
            float o = Ot[col * kHeadDim + d];
            if (C::PIECES == 2) o += Ot[(col + 1) * kHeadDim + d];
            // remove the constant 64 carried by every unpacked code, undo the field weight, add the zero points
            o = (o - 64.0f * sg) * winv + zg;
            Ow[r * kPartialStride + d] = failed ? 0.f : o;
        }
    }
    if (lane < R) {
        float mm = -CUDART_INF_F, ll = 0.f;
#pragma unroll
        for (int r = 0; r < R; ++r)
            if (lane == r) { mm = m_run[r]; ll = l_part[r]; }
        Ow[lane * kPartialStride + kHeadDim] = mm;
        Ow[lane * kPartialStride + kHeadDim + 1] = ll;
    }
    __syncthreads();

    // ---- merge the four warps and write one partial per query head
#pragma unroll
    for (int r = 0; r < R; ++r) {
        float M = -CUDART_INF_F;
        const float *ow[kWarps];
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            ow[w] = reinterpret_cast<const float *>(smem + C::kQBytes + w * C::kWarpBytes) + C::NCV * kHeadDim + r * kPartialStride;
            M = fmaxf(M, ow[w][kHeadDim]);
        }
        float o = 0.f, l = 0.f;
        if (M > -CUDART_INF_F) {
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                const float wgt = exp2f(ow[w][kHeadDim] - M);
                o = fmaf(ow[w][tid], wgt, o);
                l = fmaf(ow[w][kHeadDim + 1], wgt, l);
            }
        }
        float *dst = a.ws + (((size_t)b * s.Hq + hk * R + r) * n_parts + part) * kPartialStride;
        dst[tid] = o;
        if (tid == 0) { dst[kHeadDim] = M; dst[kHeadDim + 1] = l; }
    }
}

template <int G, int R>
cudaError_t launch_one(const MmaArgs &a, cudaStream_t stream)
{
    using C = Cfg<G, R>;
    static bool configured = false;
    auto kern = partition_mma_kernel<G, R>;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    dim3 grid(a.plan.n_splits + 1, a.s.Hkv, a.s.B);
    kern<<<grid, kThreads, C::kSmemBytes, stream>>>(a);
    return cudaGetLastError();
}

template <int G>
cudaError_t launch_g(const MmaArgs &a, cudaStream_t stream, bool *handled)
{
    *handled = true;
    switch (a.s.rep) {
        case 1: return launch_one<G, 1>(a, stream);
        case 2: return launch_one<G, 2>(a, stream);
        case 4: return launch_one<G, 4>(a, stream);
        default: *handled = false; return cudaSuccess;
    }
}

}  // namespace

// Launches the tensor-core partition kernel when the configuration is covered (2-bit K and V,
// 1, 2 or 4 query heads per KV head); *handled tells the caller whether it did.
cudaError_t launch_partition_mma(const Shape &s, const CachePtrs &c, const __half *q, float scale_log2,
                                 const SplitPlan &plan, float *workspace, cudaStream_t stream, bool *handled)
{
    *handled = false;
    if (s.k_bits != 2 || s.v_bits != 2) return cudaSuccess;
    MmaArgs a{s, c, q, scale_log2, plan, workspace};
    switch (s.G) {
        case 128: return launch_g<128>(a, stream, handled);
        case 64: return launch_g<64>(a, stream, handled);
        case 32: return launch_g<32>(a, stream, handled);
        default: return cudaSuccess;
    }
}

}  // namespace skvq

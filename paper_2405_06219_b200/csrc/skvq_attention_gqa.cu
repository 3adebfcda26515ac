// Tensor-core partition kernel of skvq_decode_attention for 2-bit K and V with several query heads per
// KV head and/or fine groups (Eq. 1, Algorithm 1): up to 4 query heads share every cache element, and each
// (token, group) has its own scale and zero point, so the per-element work and the per-(token, head, group)
// work both have to be small.
//
//   q'.K~_t            = sum_g h_{t,g} (sum_{j in g} q'_j c_{t,j}) + sum_g z_{t,g} (sum_{j in g} q'_j)
//   sum_t p_t V~_{t,d} = sum_t (p_t h_{t,g(d)}) c_{t,d} + sum_t p_t z_{t,g(d)}
//
// Scores (fp16 MMA m16n8k16, tokens are the M rows, query heads the N columns): one lop3 plants a 2-bit field
// that sits at mantissa bits [p, p+2) of an fp16 lane into the constant 64.0, giving 64 + 4^i*code; the
// weight 4^i is divided out of the query operand and the constant 64 is removed together with the zero-point
// term by ONE extra MMA whose A operand is the token's {h, z} words exactly as they lie in the cache and
// whose B operand holds (-64*sum q'/w, sum q') per (head, group) as fp16 hi + lo pairs.  The accumulators are
// already per (token, head); the group sums are combined with h in registers.
// Values (u8 MMA m16n8k32, the M rows are (head, byte digit)): ldmatrix.trans.b8 turns the V tile into
// "four tokens of one byte column" registers, one AND leaves 4^j*code bytes, and p*h per group goes on a
// 32-bit fixed-point grid whose four bytes are four A rows.  The integer accumulators are exact; they are
// folded into fp32 (shared memory) only when the softmax reference or the bound on h moves, and the
// reference only moves when a score exceeds it by 2^8, which after the first tile is rare.
// sum_t p_t z_{t,g} is one more small fp16 MMA per 16 tokens.
//
// One CTA = 4 independent warps on one (sequence, KV head, split); tiles of 64 tokens arrive through a per-warp
// ring of shared-memory stages filled by cp.async.bulk (mbarrier completion, bounded polling).
#include "skvq_mma_common.cuh"

namespace skvq {
namespace {

using namespace mmak;

constexpr int kHeadSlots = 4;           // query heads per KV head this kernel serves (rows = head x 4 digits)
constexpr float kRefSlack = 8.0f;       // the softmax reference moves only when a score exceeds it by this (log2)

template <int G>
struct GCfg {
    static constexpr int NG = kHeadDim / G;
    static constexpr int kCodeTile = kTileTok * kRowBytes;               // 2048 B
    static constexpr int kMetaTile = kTileTok * NG * 4;
    static constexpr int kStageBytes = 2 * kCodeTile + 2 * kMetaTile;
    static constexpr int kStages = 2;
    static constexpr int kPStride = 68;                                  // floats per head row of the P tile (bank spread)
    static constexpr int kPBytes = kHeadSlots * kPStride * 4;
    static constexpr int kHBytes = kTileTok * NG * 4;                    // h_v * fixed-point scale per (token, group)
    static constexpr int kOBytes = kHeadSlots * kHeadDim * 4;            // folded P.V sums
    static constexpr int kZBytes = kHeadSlots * 4 * 4;                   // sum p*z per (head, group)
    static constexpr int kWarpBytes = kStages * kStageBytes + kPBytes + kHBytes + kOBytes + kZBytes + 64;
    static constexpr int kQFloats = kHeadSlots * kHeadDim + 2 * kHeadSlots * 4 + 2 * kHeadSlots + kWarps * kHeadSlots;
    static constexpr int kQBytes = (kQFloats * 4 + 127) / 128 * 128;
    static constexpr int kSmemBytes = kQBytes + kWarps * kWarpBytes;
    static_assert(kStages * kStageBytes >= kHeadSlots * kPartialStride * 4, "stage area is reused for the warp result");
};

// Weight 4^i that the score unpack leaves on field f (0..7) of a 16-bit half: positions 4, 6, 8 of the mantissa.
__device__ __forceinline__ float field_weight_inv(int f)
{
    const int sel = (f == 0 || f == 5) ? 0 : ((f == 1 || f == 3 || f == 6) ? 1 : 2);
    return sel == 0 ? 1.0f : (sel == 1 ? 0.25f : 0.0625f);
}

__device__ __forceinline__ uint32_t pack_half2(float lo, float hi)
{
    const __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h);
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}

__device__ __forceinline__ uint32_t to_fixed_u32(float x)
{
    uint32_t r;
    asm("cvt.rni.sat.u32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return r;
}

template <int G, int R>
__global__ void __launch_bounds__(kThreads, 3) partition_gqa_kernel(MmaArgs a)
{
    using C = GCfg<G>;
    constexpr int NG = C::NG;
    static_assert(R <= kHeadSlots, "rows of the P.V MMAs are 4 heads x 4 digits");
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

    // ---- CTA-wide prologue: permuted query on a per-head power-of-two scale, per-(head, group) constants
    float *qs = reinterpret_cast<float *>(smem);                   // [4][128] q' * F_r (exact), 0 for absent heads
    float *cst = qs + kHeadSlots * kHeadDim;                       // [4][4]  -64 * sum_j q'_j F_r / w_j
    float *sqs = cst + kHeadSlots * 4;                             // [4][4]  sum_j q'_j F_r
    float *csc = sqs + kHeadSlots * 4;                             // [4]     sm_scale*log2(e) / F_r
    int *fexp = reinterpret_cast<int *>(csc + kHeadSlots);         // [4]
    float *redmax = reinterpret_cast<float *>(fexp + kHeadSlots);  // [4 warps][4]
    uint8_t *warp_base = smem + C::kQBytes + warp * C::kWarpBytes;
    {
        const int32_t *idx_k = a.c.reorder_k + (size_t)hk * kHeadDim;
        const int src = idx_k[tid] & (kHeadDim - 1);
#pragma unroll
        for (int r = 0; r < kHeadSlots; ++r) {
            const float qv = r < R ? __half2float(a.q[((size_t)b * s.Hq + hk * R + r) * kHeadDim + src]) : 0.f;
            qs[r * kHeadDim + tid] = qv;
            const float wm = warp_max(fabsf(qv));
            if (lane == 0) redmax[warp * kHeadSlots + r] = wm;
        }
    }
    __syncthreads();
    if (tid < kHeadSlots) {
        float qmax = 0.f;
        for (int w = 0; w < kWarps; ++w) qmax = fmaxf(qmax, redmax[w * kHeadSlots + tid]);
        int e = 0;
        if (qmax > 0.f) (void)frexpf(qmax, &e);            // qmax = m * 2^e, 0.5 <= m < 1: q' * 2^-e lies in (-1, 1)
        fexp[tid] = e;
        csc[tid] = ldexpf(a.scale_log2, e);
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < kHeadSlots; ++r) qs[r * kHeadDim + tid] = ldexpf(qs[r * kHeadDim + tid], -fexp[r]);
    __syncthreads();
    if (tid < kHeadSlots * NG) {
        const int r = tid / NG, gg = tid % NG;
        float sq = 0.f, sw = 0.f;
        for (int j = gg * G; j < (gg + 1) * G; ++j) {
            const float v = qs[r * kHeadDim + j];
            sq += v;
            sw += v * field_weight_inv(j & 7);
        }
        sqs[r * 4 + gg] = sq;
        cst[r * 4 + gg] = -64.0f * sw;
    }
    __syncthreads();

    // B operand of the score MMAs, 8 k-steps of 16 channels.  Lane t = (word w1 = t >> 1, half u = t & 1) of a
    // 32-channel word pair unpacks four registers from its word: fields {0,1,2,3} (u = 0) or {5,6,7,4} (u = 1),
    // each with the field eight places up in the register's high half.  k-step 2p+s of pair p uses registers
    // 2s (k = 2t, 2t+1) and 2s+1 (k = 2t+8, 2t+9).  Column n = g is query head g.
    const int w1 = t >> 1, u = t & 1;
    uint32_t bK[8][2];
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int sx = 0; sx < 2; ++sx)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int reg = 2 * sx + j;
                const int fld = u ? (((reg + 1) & 3) + 4) : reg;
                const int ch = 32 * p + 16 * w1 + fld;
                const float wi = field_weight_inv(fld);
                const float lo = g < kHeadSlots ? qs[g * kHeadDim + ch] * wi : 0.f;
                const float hi = g < kHeadSlots ? qs[g * kHeadDim + ch + 8] * wi : 0.f;
                bK[2 * p + sx][j] = pack_half2(lo, hi);
            }
    // B operand of the {h, z} MMA: k = 2t <-> h of group t, k = 2t+1 <-> z of group t; fp16 hi parts in k < 8,
    // lo parts in k >= 8 (the A operand repeats the same words there).
    uint32_t bZ[2] = {0u, 0u};
    if (g < kHeadSlots && t < NG) {
        const float c0 = cst[g * 4 + t], c1 = sqs[g * 4 + t];
        const float c0h = __half2float(__float2half_rn(c0)), c1h = __half2float(__float2half_rn(c1));
        bZ[0] = pack_half2(c0h, c1h);
        bZ[1] = pack_half2(c0 - c0h, c1 - c1h);
    }
    // this lane's two score columns are heads 2t and 2t+1
    const float cs0 = (2 * t < kHeadSlots) ? csc[2 * t] : 0.f;
    const float cs1 = (2 * t + 1 < kHeadSlots) ? csc[2 * t + 1] : 0.f;

    // ---- per-warp shared memory
    uint8_t *stage_base = warp_base;
    float *Pt = reinterpret_cast<float *>(warp_base + C::kStages * C::kStageBytes);                 // [4][68]
    float *Hf = reinterpret_cast<float *>(warp_base + C::kStages * C::kStageBytes + C::kPBytes);    // [64][NG]
    float *Os = reinterpret_cast<float *>(warp_base + C::kStages * C::kStageBytes + C::kPBytes + C::kHBytes);   // [4][128]
    float *Zs = Os + kHeadSlots * kHeadDim;                                                         // [4][4]
    uint64_t *bars = reinterpret_cast<uint64_t *>(reinterpret_cast<uint8_t *>(Zs) + C::kZBytes);
    const uint32_t bar0 = smem_u32(bars);
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < C::kStages; ++i) mbar_init(bar0 + 8 * i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
#pragma unroll
    for (int i = 0; i < kHeadSlots * kHeadDim / 32; ++i) Os[lane + 32 * i] = 0.f;
    __syncwarp();

    const size_t bh = (size_t)b * s.Hkv + hk;
    const uint8_t *k_codes = a.c.k_codes + bh * (size_t)s.cap * kRowBytes;
    const uint8_t *v_codes = a.c.v_codes + bh * (size_t)s.cap * kRowBytes;
    const __half2 *k_meta = a.c.k_meta + bh * (size_t)s.cap * NG;
    const __half2 *v_meta = a.c.v_meta + bh * (size_t)s.cap * NG;

    const int n_tiles = (q_end - q_begin + kTileTok - 1) / kTileTok;
    const int n_my = n_tiles > warp ? (n_tiles - warp + kWarps - 1) / kWarps : 0;

    auto issue = [&](int i) {   // lane 0 only
        const int st = i % C::kStages;
        const int tok0 = q_begin + (warp + i * kWarps) * kTileTok;
        const uint32_t dst = smem_u32(stage_base + st * C::kStageBytes);
        const uint32_t bar = bar0 + 8 * st;
        mbar_expect_tx(bar, C::kStageBytes);
        bulk_g2s(dst, k_codes + (size_t)tok0 * kRowBytes, C::kCodeTile, bar);
        bulk_g2s(dst + C::kCodeTile, v_codes + (size_t)tok0 * kRowBytes, C::kCodeTile, bar);
        bulk_g2s(dst + 2 * C::kCodeTile, k_meta + (size_t)tok0 * NG, C::kMetaTile, bar);
        bulk_g2s(dst + 2 * C::kCodeTile + C::kMetaTile, v_meta + (size_t)tok0 * NG, C::kMetaTile, bar);
    };
    if (lane == 0)
        for (int i = 0; i < C::kStages && i < n_my; ++i) issue(i);

    // ---- running state
    // softmax references of heads 2t, 2t+1 (log2 domain); lanes whose columns are no head never ask for a move
    float m_ref0 = t < kHeadSlots / 2 ? -CUDART_INF_F : 0.f, m_ref1 = m_ref0;
    float l0 = 0.f, l1 = 0.f;                                  // partial sums of p over this lane's token rows
    float zacc[4] = {0.f, 0.f, 0.f, 0.f};                      // sum_t p z: rows = group g, columns = heads 2t, 2t+1
    int acc[16][4];                                            // P.V: rows (head g&3, digit g>>2 [+2]), columns = channels
#pragma unroll
    for (int i = 0; i < 16; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0;
    float h_bound = 6.103515625e-05f;                          // power of two above every value scale seen so far
    bool acc_live = false, failed = false;

    // lane constants of the unpack and of the digit gather
    const uint32_t rot_amt = u ? 26u : 4u;                     // rotate left: x << 4, or x >> 6
    const uint32_t mask_x = u ? 0x03000300u : 0x00C000C0u;     // register 3 comes from the unrotated word
    const int hd = g & 3, d0 = g >> 2;                         // this lane's P.V rows: head hd, digits d0 and d0 + 2
    const uint32_t sel_dig = d0 ? 0x7351u : 0x6240u;           // bytes d0 of two words, then bytes d0+2 of the same

    // Brings the integer sums into the fp32 sums in shared memory and rescales those by 2^(old ref - new ref).
    auto fold = [&](float corr_hd) {
        const float sa = h_bound * (d0 ? 1.52587890625e-05f : 5.9604644775390625e-08f);   // h_bound * 2^8 * 2^-32 * 256^d0
        const float sb = sa * 65536.0f;
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) {
            float x0 = fmaf((float)acc[nt][2], sb, (float)acc[nt][0] * sa);
            float x1 = fmaf((float)acc[nt][3], sb, (float)acc[nt][1] * sa);
            x0 += __shfl_xor_sync(0xffffffffu, x0, 16);
            x1 += __shfl_xor_sync(0xffffffffu, x1, 16);
            if (g < 4) {
                // n-tile nt = (hh, half, j): byte columns 16hh + 8half + n, channel 4*(byte column) + j
                const int ch = 4 * (16 * (nt >> 3) + 8 * ((nt >> 2) & 1) + 2 * t) + (nt & 3);
                float *o = Os + hd * kHeadDim + ch;
                o[0] = (o[0] + x0) * corr_hd;      // both terms are relative to the old reference
                o[4] = (o[4] + x1) * corr_hd;
            }
            acc[nt][0] = 0; acc[nt][1] = 0; acc[nt][2] = 0; acc[nt][3] = 0;
        }
    };

    for (int i = 0; i < n_my; ++i) {
        const int st = i % C::kStages;
        const uint32_t parity = (uint32_t)(i / C::kStages) & 1u;
        if (!mbar_wait_bounded(bar0 + 8 * st, parity)) { failed = true; break; }
        uint8_t *Kc = stage_base + st * C::kStageBytes;
        uint8_t *Vc = Kc + C::kCodeTile;
        uint32_t *Km = reinterpret_cast<uint32_t *>(Kc + 2 * C::kCodeTile);       // [64][NG] words {h, z}
        uint32_t *Vm = reinterpret_cast<uint32_t *>(Kc + 2 * C::kCodeTile + C::kMetaTile);
        const int tok0 = q_begin + (warp + i * kWarps) * kTileTok;
        const int n_valid = min(kTileTok, q_end - tok0);
        if (n_valid < kTileTok) {
            // rows past the end hold unspecified bytes: give their scale/zero words a defined value
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const int tau = lane + 32 * hf;
                if (tau >= n_valid) {
#pragma unroll
                    for (int gg = 0; gg < NG; ++gg) { Km[tau * NG + gg] = 0u; Vm[tau * NG + gg] = 0u; }
                }
            }
            __syncwarp();
        }

        // ---------------- scores: lane (g, t) ends with tokens 16mt+g, 16mt+g+8 x heads 2t, 2t+1
        float sraw[4][4];
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) {
            const uint32_t *row0 = reinterpret_cast<const uint32_t *>(Kc + (16 * mt + g) * kRowBytes) + w1;
            const uint32_t *row1 = row0 + 8 * (kRowBytes / 4);
            float ak[NG][4];
#pragma unroll
            for (int gg = 0; gg < NG; ++gg)
#pragma unroll
                for (int e = 0; e < 4; ++e) ak[gg][e] = 0.f;
#pragma unroll
            for (int p = 0; p < 4; ++p) {
                constexpr uint32_t MAGIC = 0x54005400u, M4 = 0x00300030u, M6 = 0x00C000C0u, M8 = 0x03000300u;
                const uint32_t xa = row0[2 * p], xb = row1[2 * p];
                const uint32_t ra = __funnelshift_l(xa, xa, rot_amt), rb = __funnelshift_l(xb, xb, rot_amt);
                const uint32_t a00 = and_or(ra, M4, MAGIC), a01 = and_or(ra, M6, MAGIC);
                const uint32_t a02 = and_or(ra, M8, MAGIC), a03 = and_or(xa, mask_x, MAGIC);
                const uint32_t a10 = and_or(rb, M4, MAGIC), a11 = and_or(rb, M6, MAGIC);
                const uint32_t a12 = and_or(rb, M8, MAGIC), a13 = and_or(xb, mask_x, MAGIC);
                mma16816(ak[(32 * p) / G], a00, a10, a01, a11, bK[2 * p][0], bK[2 * p][1]);
                mma16816(ak[(32 * p) / G], a02, a12, a03, a13, bK[2 * p + 1][0], bK[2 * p + 1][1]);
            }
            // {h, z} words of the two tokens: A operand of the constant/zero-point MMA, and h for the group sums
            const uint32_t *m0 = Km + (16 * mt + g) * NG, *m1 = m0 + 8 * NG;
            uint32_t mw0[NG], mw1[NG];
            if constexpr (NG == 4) {
                const uint4 x0 = *reinterpret_cast<const uint4 *>(m0), x1 = *reinterpret_cast<const uint4 *>(m1);
                mw0[0] = x0.x; mw0[1] = x0.y; mw0[2] = x0.z; mw0[3] = x0.w;
                mw1[0] = x1.x; mw1[1] = x1.y; mw1[2] = x1.z; mw1[3] = x1.w;
            } else if constexpr (NG == 2) {
                const uint2 x0 = *reinterpret_cast<const uint2 *>(m0), x1 = *reinterpret_cast<const uint2 *>(m1);
                mw0[0] = x0.x; mw0[1] = x0.y; mw1[0] = x1.x; mw1[1] = x1.y;
            } else {
                mw0[0] = m0[0]; mw1[0] = m1[0];
            }
            const uint32_t za = t < NG ? m0[t < NG ? t : 0] : 0u;
            const uint32_t zb = t < NG ? m1[t < NG ? t : 0] : 0u;
            float az[4] = {0.f, 0.f, 0.f, 0.f};
            mma16816(az, za, zb, za, zb, bZ[0], bZ[1]);
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) {
                const float h0 = __low2float(*reinterpret_cast<const __half2 *>(&mw0[gg]));
                const float h1 = __low2float(*reinterpret_cast<const __half2 *>(&mw1[gg]));
                az[0] = fmaf(h0, ak[gg][0], az[0]);
                az[1] = fmaf(h0, ak[gg][1], az[1]);
                az[2] = fmaf(h1, ak[gg][2], az[2]);
                az[3] = fmaf(h1, ak[gg][3], az[3]);
            }
            sraw[mt][0] = az[0]; sraw[mt][1] = az[1]; sraw[mt][2] = az[2]; sraw[mt][3] = az[3];
        }

        // ---------------- value scales of tokens lane, lane+32; does the reference or the bound have to move?
        float hv[2][NG];
        bool moved = false;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            const int tau = lane + 32 * hf;
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) {
                hv[hf][gg] = __low2float(*reinterpret_cast<const __half2 *>(Vm + tau * NG + gg));
                moved |= (hv[hf][gg] >= h_bound);
            }
        }
        float arg[4][4];
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) {
            const bool v0 = (16 * mt + g) < n_valid, v1 = (16 * mt + g + 8) < n_valid;
            arg[mt][0] = v0 ? fmaf(sraw[mt][0], cs0, -m_ref0) : -CUDART_INF_F;
            arg[mt][1] = v0 ? fmaf(sraw[mt][1], cs1, -m_ref1) : -CUDART_INF_F;
            arg[mt][2] = v1 ? fmaf(sraw[mt][2], cs0, -m_ref0) : -CUDART_INF_F;
            arg[mt][3] = v1 ? fmaf(sraw[mt][3], cs1, -m_ref1) : -CUDART_INF_F;
            moved |= (fmaxf(fmaxf(arg[mt][0], arg[mt][1]), fmaxf(arg[mt][2], arg[mt][3])) > kRefSlack);
        }
        if (__any_sync(0xffffffffu, moved)) {
            // Raise the references to the running maxima (and the bound on h), fold what was accumulated so far.
            float tm0 = -CUDART_INF_F, tm1 = -CUDART_INF_F;
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) {
                const bool v0 = (16 * mt + g) < n_valid, v1 = (16 * mt + g + 8) < n_valid;
                if (v0) { tm0 = fmaxf(tm0, sraw[mt][0] * cs0); tm1 = fmaxf(tm1, sraw[mt][1] * cs1); }
                if (v1) { tm0 = fmaxf(tm0, sraw[mt][2] * cs0); tm1 = fmaxf(tm1, sraw[mt][3] * cs1); }
            }
#pragma unroll
            for (int msk = 4; msk < 32; msk <<= 1) {
                tm0 = fmaxf(tm0, __shfl_xor_sync(0xffffffffu, tm0, msk));
                tm1 = fmaxf(tm1, __shfl_xor_sync(0xffffffffu, tm1, msk));
            }
            const float n0 = fmaxf(m_ref0, tm0), n1 = fmaxf(m_ref1, tm1);
            const float c0 = ex2_approx(m_ref0 - n0), c1 = ex2_approx(m_ref1 - n1);   // 0 on the first tile
            m_ref0 = n0; m_ref1 = n1;
            l0 *= c0; l1 *= c1;
            zacc[0] *= c0; zacc[1] *= c1; zacc[2] *= c0; zacc[3] *= c1;
            // the correction of head hd lives in the lanes with t = hd >> 1
            const float ca = __shfl_sync(0xffffffffu, c0, hd >> 1), cb = __shfl_sync(0xffffffffu, c1, hd >> 1);
            const float corr_hd = (hd & 1) ? cb : ca;
            if (acc_live) fold(corr_hd);
            float hm = 0.f;
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) hm = fmaxf(hm, fmaxf(hv[0][gg], hv[1][gg]));
            hm = warp_max(hm);
            if (hm >= h_bound) h_bound = __int_as_float(((__float_as_int(hm) >> 23) + 1) << 23);
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) {
                const bool v0 = (16 * mt + g) < n_valid, v1 = (16 * mt + g + 8) < n_valid;
                arg[mt][0] = v0 ? fmaf(sraw[mt][0], cs0, -m_ref0) : -CUDART_INF_F;
                arg[mt][1] = v0 ? fmaf(sraw[mt][1], cs1, -m_ref1) : -CUDART_INF_F;
                arg[mt][2] = v1 ? fmaf(sraw[mt][2], cs0, -m_ref0) : -CUDART_INF_F;
                arg[mt][3] = v1 ? fmaf(sraw[mt][3], cs1, -m_ref1) : -CUDART_INF_F;
            }
        }
        // probabilities (at most 2^8) -> P tile [head][token]; value scales on the fixed-point grid -> Hf
        if (t < kHeadSlots / 2) {
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) {
                const float p0 = ex2_approx(arg[mt][0]), p1 = ex2_approx(arg[mt][1]);
                const float p2 = ex2_approx(arg[mt][2]), p3 = ex2_approx(arg[mt][3]);
                l0 += p0 + p2;
                l1 += p1 + p3;
                float *pr = Pt + (2 * t) * C::kPStride + 16 * mt + g;
                pr[0] = p0; pr[C::kPStride] = p1; pr[8] = p2; pr[C::kPStride + 8] = p3;
            }
        }
        {
            const float hscale = 16777216.0f / h_bound;      // 2^32 / (h_bound * 2^8)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const int tau = lane + 32 * hf;
#pragma unroll
                for (int gg = 0; gg < NG; ++gg) Hf[tau * NG + gg] = hv[hf][gg] * hscale;   // 0 for rows past the end
            }
        }
        __syncwarp();

        // ---------------- sum_t p_t z_{t,g}: rows = groups, columns = heads, k = 16 tokens
#pragma unroll
        for (int kb = 0; kb < 4; ++kb) {
            const int ta = 16 * kb + 2 * t;
            uint32_t a0 = 0u, a2 = 0u, b0 = 0u, b1 = 0u;
            if (g < NG) {
                a0 = prmt(Vm[ta * NG + g], Vm[(ta + 1) * NG + g], 0x7632u);
                a2 = prmt(Vm[(ta + 8) * NG + g], Vm[(ta + 9) * NG + g], 0x7632u);
            }
            if (g < kHeadSlots) {
                const float2 pa = *reinterpret_cast<const float2 *>(Pt + g * C::kPStride + ta);
                const float2 pb = *reinterpret_cast<const float2 *>(Pt + g * C::kPStride + ta + 8);
                b0 = pack_half2(pa.x, pa.y);
                b1 = pack_half2(pb.x, pb.y);
            }
            mma16816(zacc, a0, 0u, a2, 0u, b0, b1);
        }

        // ---------------- P.V: A rows (head hd, digits d0 / d0+2), k = 32 tokens, columns = 8 channels of one group
        const uint32_t vaddr = smem_u32(Vc) + lane * kRowBytes;
#pragma unroll
        for (int kk = 0; kk < 2; ++kk) {
            uint32_t Ag[NG][4];
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int tk = 32 * kk + 16 * half + 4 * t;
                const float4 p4 = *reinterpret_cast<const float4 *>(Pt + hd * C::kPStride + tk);
                const float pv[4] = {p4.x, p4.y, p4.z, p4.w};
                uint32_t uu[4][NG];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float hrow[NG];
                    if constexpr (NG == 4) {
                        const float4 h4 = *reinterpret_cast<const float4 *>(Hf + (tk + j) * 4);
                        hrow[0] = h4.x; hrow[1] = h4.y; hrow[2] = h4.z; hrow[3] = h4.w;
                    } else if constexpr (NG == 2) {
                        const float2 h2 = *reinterpret_cast<const float2 *>(Hf + (tk + j) * 2);
                        hrow[0] = h2.x; hrow[1] = h2.y;
                    } else {
                        hrow[0] = Hf[tk + j];
                    }
#pragma unroll
                    for (int gg = 0; gg < NG; ++gg) uu[j][gg] = to_fixed_u32(pv[j] * hrow[gg]);
                }
#pragma unroll
                for (int gg = 0; gg < NG; ++gg) {
                    const uint32_t t01 = prmt(uu[0][gg], uu[1][gg], sel_dig), t23 = prmt(uu[2][gg], uu[3][gg], sel_dig);
                    Ag[gg][2 * half] = prmt(t01, t23, 0x5410u);
                    Ag[gg][2 * half + 1] = prmt(t01, t23, 0x7632u);
                }
            }
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                uint32_t rr[4];
                ldmatrix_b8_trans_x2(rr, vaddr + kk * 32 * kRowBytes + hh * 16);
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int gg = (64 * hh + 32 * half) / G;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t m = 0x03030303u << (2 * j);
                        imma16832_uu(acc[hh * 8 + half * 4 + j], Ag[gg][0], Ag[gg][1], Ag[gg][2], Ag[gg][3], rr[half] & m,
                                     rr[2 + half] & m);
                    }
                }
            }
        }
        acc_live = true;
        __syncwarp();   // every lane is done with this stage, the P tile and Hf
        if (lane == 0 && i + C::kStages < n_my) issue(i + C::kStages);
    }

    if (failed) {
        for (int i2 = 0; i2 < n_my; ++i2) {
            const int st = i2 % C::kStages;
            (void)mbar_wait_bounded(bar0 + 8 * st, (uint32_t)(i2 / C::kStages) & 1u);
        }
        if (lane == 0 && a.c.status) atomicOr(a.c.status, 2);
    }

    // ---- per-warp result
    if (acc_live) fold(1.0f);
    if (g < NG && t < kHeadSlots / 2) {
        Zs[(2 * t) * 4 + g] = zacc[0];
        Zs[(2 * t + 1) * 4 + g] = zacc[1];
    }
#pragma unroll
    for (int msk = 4; msk < 32; msk <<= 1) {
        l0 += __shfl_xor_sync(0xffffffffu, l0, msk);
        l1 += __shfl_xor_sync(0xffffffffu, l1, msk);
    }
    __syncwarp();
    float *Ow = reinterpret_cast<float *>(stage_base);                       // [R][132]: o', m, l
#pragma unroll
    for (int r = 0; r < R; ++r) {
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
            const int d = lane + 32 * q4;
            const int j = d & 3;                                             // channel d carries the weight 4^j
            const float winv = j == 0 ? 1.0f : (j == 1 ? 0.25f : (j == 2 ? 0.0625f : 0.015625f));
            const float o = Os[r * kHeadDim + d] * winv + Zs[r * 4 + d / G];
            Ow[r * kPartialStride + d] = (failed || !acc_live) ? 0.f : o;
        }
    }
    if (g == 0 && t < kHeadSlots / 2) {
        if (2 * t < R) {
            Ow[(2 * t) * kPartialStride + kHeadDim] = (failed || !acc_live) ? -CUDART_INF_F : m_ref0;
            Ow[(2 * t) * kPartialStride + kHeadDim + 1] = (failed || !acc_live) ? 0.f : l0;
        }
        if (2 * t + 1 < R) {
            Ow[(2 * t + 1) * kPartialStride + kHeadDim] = (failed || !acc_live) ? -CUDART_INF_F : m_ref1;
            Ow[(2 * t + 1) * kPartialStride + kHeadDim + 1] = (failed || !acc_live) ? 0.f : l1;
        }
    }
    __syncthreads();

    // ---- merge the four warps and write one partial per query head
#pragma unroll
    for (int r = 0; r < R; ++r) {
        float M = -CUDART_INF_F;
        const float *ow[kWarps];
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            ow[w] = reinterpret_cast<const float *>(smem + C::kQBytes + w * C::kWarpBytes) + r * kPartialStride;
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
    using C = GCfg<G>;
    static bool configured = false;
    auto kern = partition_gqa_kernel<G, R>;
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

// Launches the kernel above when the configuration is covered (2-bit K and V, 1, 2 or 4 query heads per KV
// head); *handled tells the caller whether it did.
cudaError_t launch_partition_gqa(const Shape &s, const CachePtrs &c, const __half *q, float scale_log2,
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

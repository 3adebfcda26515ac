// Tensor-core partition kernel of skvq_decode_attention for 2-bit K and V (Eq. 1, Algorithm 1).
//
// Why tensor cores on an HBM-bound path: at 2 bits a cache element costs 0.28 bytes, so streaming
// at several TB/s leaves fewer than two issue slots per element, and the logic pipe that does the
// bit work retires half a warp instruction per clock.  The codes are therefore turned into MMA
// operands with as few logic ops as possible and contracted on the tensor cores; scale and zero
// point never touch individual elements:
//   q'.K~_t            = sum_g h_{t,g} (sum_{j in g} q'_j c_{t,j}) + sum_g z_{t,g} (sum_{j in g} q'_j)
//   sum_t p_t V~_{t,d} = sum_t (p_t h_{t,g(d)}) c_{t,d} + sum_t p_t z_{t,g(d)}
// Scores (integer MMA, exact): `word & (0x03030303 << 2t)` leaves four codes of a packed word as
// bytes worth 4^t * code -- one AND per four codes, no shift -- which feed mma.m16n8k32.u8.s8.
// The query is put on a power-of-two fixed-point grid, divided by 4^t and split into four signed
// byte digits that sit in four B columns, so sum_j q'_j c_j is formed exactly in int32.
// Values (fp16 MMA): OR-ing a 2-bit field that sits at mantissa bits [p, p+2) of an fp16 lane with
// an exponent pattern gives the half value 64 + weight*code; the constant 64 contributes
// 64 * sum(P), subtracted in fp32 at the end, and the weight is divided out per channel.
// P = p*h is split into fp16 hi + lo pieces (two B columns) when the column budget allows.
//
// One CTA = 4 independent warps on one (sequence, KV head, split); each warp streams 64-token
// tiles of codes + scale/zero through its own ring of shared-memory stages filled by
// cp.async.bulk (mbarrier completion), keeps its own online-softmax state, and the 4 states are
// merged in shared memory before one partial per query head is written to the workspace.
// The fp16 window is handled by the merge kernel.
#include "skvq_mma_common.cuh"

namespace skvq {
namespace {

using namespace mmak;

// ---------------------------------------------------------------- compile-time layout
template <int G, int R>
struct Cfg {
    static constexpr int NG = kHeadDim / G;
    // Integer P.V path: one query head and at most two groups, so that (group, byte digit) fits the 8 MMA columns.
    static constexpr bool VINT8 = (R == 1 && NG <= 2);
    static constexpr int PIECES = (R * NG * 2 <= 8) ? 2 : 1;             // fp16 path: P split into hi+lo halves when columns allow
    static constexpr int NCV = R * NG * PIECES;                          // V-side columns: (head, group, piece)
    static constexpr int NTV = (NCV + 7) / 8;
    static constexpr int NCVP = NTV * 8;
    static constexpr int kCodeTile = kTileTok * kRowBytes;               // 2048 B
    static constexpr int kMetaTile = kTileTok * NG * 4;                  // 256 B * NG
    static constexpr int kStageBytes = 2 * kCodeTile + 2 * kMetaTile;
    static constexpr int kStages = 2;
    static constexpr int NTK = (4 * R + 7) / 8;                          // K-side n-tiles: 4 byte digits per head
    static constexpr int kScBytes = kTileTok * R * NG * 8;               // per (token, group, head): low and high digit pairs
    static constexpr int kPBytes = VINT8 ? 2 * 8 * 32 : 4 * NCVP * 16 * 2;   // P operand tile
    static constexpr int kWarpBytes = kStages * kStageBytes + kScBytes + kPBytes + 64;   // + mbarriers
    static constexpr int kQBytes = (R * kHeadDim * 4 + R * NG * 4 + 2 * R * 4 + 64 + 127) / 128 * 128;
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

template <int G, int R>
__global__ void __launch_bounds__(kThreads) partition_mma_kernel(MmaArgs a)
{
    using C = Cfg<G, R>;
    constexpr int NG = C::NG;
    extern __shared__ __align__(128) uint8_t smem[];
    const Shape &s = a.s;
    const int part = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int L = a.c.lengths[b];
    const int Lq = max(L - s.W, 0);
    const int q_begin = min(part * a.plan.split_len, Lq);
    const int q_end = min(q_begin + a.plan.split_len, Lq);
    const int n_parts = a.plan.n_splits;

    // ---- CTA-wide prologue: permuted query, its fixed-point grid and per-(head, group) sums
    float *qs = reinterpret_cast<float *>(smem);                       // [R][128] q' (exact fp16 values)
    float *sqs = qs + R * kHeadDim;                                    // [R][NG] scale * sum_j q'_j
    float *cF = sqs + R * NG;                                          // [R] scale / F_r, F_r = 2^kexp[r]
    int *kexp = reinterpret_cast<int *>(cF + R);                       // [R]
    float *redmax = reinterpret_cast<float *>(kexp + R);               // [4][R]
    uint8_t *warp_base = smem + C::kQBytes + warp * C::kWarpBytes;
    {
        const int32_t *idx_k = a.c.reorder_k + (size_t)hk * kHeadDim;
        const int src = idx_k[tid] & (kHeadDim - 1);
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const float qv = __half2float(a.q[((size_t)b * s.Hq + hk * R + r) * kHeadDim + src]);
            qs[r * kHeadDim + tid] = qv;
            const float wm = warp_max(fabsf(qv));
            if (lane == 0) redmax[warp * R + r] = wm;
        }
    }
    __syncthreads();
    if (tid < R) {
        // F = 2^k with |q'_j| * F <= 2^30: every q'_j * F / 4^t is then an integer (or rounds at 2^-24 relative)
        float qmax = 0.f;
        for (int w = 0; w < kWarps; ++w) qmax = fmaxf(qmax, redmax[w * R + tid]);
        int k = 0;
        if (qmax > 0.f) {
            int e;
            const float m = frexpf(qmax, &e);          // qmax = m * 2^e, 0.5 <= m < 1
            k = 30 - ((m == 0.5f) ? e - 1 : e);
        }
        kexp[tid] = k;
        cF[tid] = ldexpf(a.scale_log2, -k);
    }
    if (tid >= 32 && tid < 32 + R * NG) {
        const int r = (tid - 32) / NG, gg = (tid - 32) % NG;
        float sq = 0.f;
        for (int j = gg * G; j < (gg + 1) * G; ++j) sq += qs[r * kHeadDim + j];
        sqs[r * NG + gg] = sq * a.scale_log2;
    }
    __syncthreads();

    // B operand of the score MMAs (s8): k-step ks contracts the 32 channels of code words 2ks, 2ks+1;
    // byte b of register `reg` = digit (col & 3) of round(q'[32ks + 16reg + 4b + t] * F / 4^t), column col = head*4 + digit.
    // Thread tid owns channel tid: it writes the four digits of that channel as bytes straight into the
    // register image bimg[head][digit][ks][reg][t] (byte b), which the lanes then load word by word.
    uint8_t *bimg0 = smem + C::kQBytes;   // [R][4][4][2][4] words = R*512 bytes in warp 0's stage area, idle until the pipeline starts
    {
        const int ks = tid >> 5, reg = (tid >> 4) & 1, bb = (tid >> 2) & 3, tt = tid & 3;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            // q' * 2^(k - 2t): an exact power-of-two scaling done on the exponent field
            int v = __float2int_rn(qs[r * kHeadDim + tid] * __int_as_float((127 + kexp[r] - 2 * tt) << 23));
#pragma unroll
            for (int i = 0; i < 4; ++i) {      // balanced base-256 digits, least significant first
                const int di = (i < 3) ? (int)(int8_t)(v & 0xFF) : v;
                v = (v - di) >> 8;
                bimg0[(((((r * 4 + i) * 4 + ks) * 2 + reg) * 4 + tt) << 2) + bb] = (uint8_t)(di & 0xFF);
            }
        }
    }
    __syncthreads();
    uint32_t bq[C::NTK][4][2];
#pragma unroll
    for (int nt = 0; nt < C::NTK; ++nt) {
        const int col = 8 * nt + g, r = col >> 2, dig = col & 3;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
#pragma unroll
            for (int reg = 0; reg < 2; ++reg)
                bq[nt][ks][reg] = (r < R) ? reinterpret_cast<const uint32_t *>(bimg0)[((((r * 4 + dig) * 4 + ks) * 2 + reg) * 4 + t)] : 0u;
    }
    __syncthreads();   // the image lives in the stage area: everyone has read it before any copy lands there
    float cFr[R], sqr[R][NG];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        cFr[r] = cF[r];
#pragma unroll
        for (int gg = 0; gg < NG; ++gg) sqr[r][gg] = sqs[r * NG + gg];
    }

    // ---- per-warp pipeline state
    uint8_t *stage_base = warp_base;
    float *Sc = reinterpret_cast<float *>(warp_base + C::kStages * C::kStageBytes);      // [64][NG][R][2]
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
    // fp16 P.V path: float accumulators cv.  Integer path: int accumulators iacc (exact while the softmax
    // reference and the scale bound stay put) that are folded into fv whenever either one moves.
    constexpr int NACC = C::VINT8 ? 1 : C::NTV;
    float cv[NACC][8][4];
    int iacc[C::VINT8 ? 8 : 1][4];
#pragma unroll
    for (int nt = 0; nt < NACC; ++nt)
#pragma unroll
        for (int f = 0; f < 8; ++f)
#pragma unroll
            for (int i = 0; i < 4; ++i) cv[nt][f][i] = 0.f;
#pragma unroll
    for (int f = 0; f < (C::VINT8 ? 8 : 1); ++f)
#pragma unroll
        for (int i = 0; i < 4; ++i) iacc[f][i] = 0;
    float h_bound = 6.103515625e-05f;   // 2^-14: every scale seen so far is below this power of two (integer path)

    bool failed = false;
    const uint32_t kmask = 0x03030303u << (2 * t);
    uint8_t *Pb = reinterpret_cast<uint8_t *>(Pt);   // integer path: [2 k-blocks][8 columns][4 t][2 halves][4 tokens] bytes

    for (int i = 0; i < n_my; ++i) {
        const int st = i % C::kStages;
        const uint32_t parity = (uint32_t)(i / C::kStages) & 1u;
        if (!mbar_wait_bounded(bar0 + 8 * st, parity)) { failed = true; break; }
        const uint8_t *Kc = stage_base + st * C::kStageBytes;
        const uint8_t *Vc = Kc + C::kCodeTile;
        const __half2 *Km = reinterpret_cast<const __half2 *>(Kc + 2 * C::kCodeTile);
        const __half2 *Vm = reinterpret_cast<const __half2 *>(Kc + 2 * C::kCodeTile + C::kMetaTile);
        const int tok0 = q_begin + (warp + i * kWarps) * kTileTok;

        // ---------------- scores: exact integer dot products sum_j q'_j c_j per (token, head, group)
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) {
            const uint4 *r0 = reinterpret_cast<const uint4 *>(Kc + (16 * mt + g) * kRowBytes);
            const uint4 *r1 = reinterpret_cast<const uint4 *>(Kc + (16 * mt + g + 8) * kRowBytes);
            const uint4 x0a = r0[0], x0b = r0[1], x1a = r1[0], x1b = r1[1];
            const uint32_t w0[8] = {x0a.x, x0a.y, x0a.z, x0a.w, x0b.x, x0b.y, x0b.z, x0b.w};
            const uint32_t w1[8] = {x1a.x, x1a.y, x1a.z, x1a.w, x1b.x, x1b.y, x1b.z, x1b.w};
            int acc[C::NTK][NG][4];
#pragma unroll
            for (int nt = 0; nt < C::NTK; ++nt)
#pragma unroll
                for (int gg = 0; gg < NG; ++gg)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[nt][gg][e] = 0;
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                // byte b of (word & kmask) = 4^t * code(4b + t): four channels per AND, no shift
                const uint32_t a0 = w0[2 * ks] & kmask, a1 = w1[2 * ks] & kmask;
                const uint32_t a2 = w0[2 * ks + 1] & kmask, a3 = w1[2 * ks + 1] & kmask;
#pragma unroll
                for (int nt = 0; nt < C::NTK; ++nt) imma16832(acc[nt][(32 * ks) / G], a0, a1, a2, a3, bq[nt][ks][0], bq[nt][ks][1]);
            }
            // lane (g,t) holds columns 2t, 2t+1 = two adjacent digits of one head for tokens 16mt+g and 16mt+g+8
#pragma unroll
            for (int nt = 0; nt < C::NTK; ++nt) {
                const int r = (8 * nt + 2 * t) >> 2;
                if (r < R) {
#pragma unroll
                    for (int gg = 0; gg < NG; ++gg) {
                        const float lo = fmaf((float)acc[nt][gg][1], 256.0f, (float)acc[nt][gg][0]);
                        const float hi = fmaf((float)acc[nt][gg][3], 256.0f, (float)acc[nt][gg][2]);
                        Sc[(((16 * mt + g) * NG + gg) * R + r) * 2 + (t & 1)] = lo;
                        Sc[(((16 * mt + g + 8) * NG + gg) * R + r) * 2 + (t & 1)] = hi;
                    }
                }
            }
        }
        __syncwarp();

        // ---------------- softmax bookkeeping: lane owns tokens lane and lane+32 of the tile
        float sc[2][R];
        bool valid[2];
        float hv[2][NG], zv[2][NG];
        bool moved = false;   // does any score exceed the running maximum, or any scale the running bound?
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
                hv[hf][gg] = valid[hf] ? vz.x : 0.f;      // rows past the end hold unspecified bytes
                zv[hf][gg] = valid[hf] ? vz.y : 0.f;
                if (C::VINT8) moved |= (hv[hf][gg] >= h_bound);
            }
#pragma unroll
            for (int r = 0; r < R; ++r) {
                float sv = 0.f;
#pragma unroll
                for (int gg = 0; gg < NG; ++gg) {
                    const float2 lh = *reinterpret_cast<const float2 *>(Sc + ((tau * NG + gg) * R + r) * 2);
                    const float u = fmaf(lh.y, 65536.0f, lh.x) * cFr[r];      // scale * sum_j q'_j c_j
                    sv = fmaf(hk_[gg], u, sv);
                    sv = fmaf(zk_[gg], sqr[r][gg], sv);
                }
                sc[hf][r] = valid[hf] ? sv : -CUDART_INF_F;
                moved |= (sc[hf][r] > m_run[r]);
            }
        }
        if (__any_sync(0xffffffffu, moved)) {
            // Rare after the first tiles: raise the references and bring every running sum onto them.
            float corr[R];
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float m_new = fmaxf(m_run[r], warp_max(fmaxf(sc[0][r], sc[1][r])));
                corr[r] = ex2_approx(m_run[r] - m_new);      // 0 on the first tile (m_run = -inf)
                m_run[r] = m_new;
                l_part[r] *= corr[r];
#pragma unroll
                for (int gg = 0; gg < NG; ++gg) { s_part[r][gg] *= corr[r]; z_part[r][gg] *= corr[r]; }
            }
            if constexpr (C::VINT8) {
                float hm = 0.f;
#pragma unroll
                for (int gg = 0; gg < NG; ++gg) hm = fmaxf(hm, fmaxf(hv[0][gg], hv[1][gg]));
                hm = warp_max(hm);
                // fold the integer sums into fv: value = iacc * 256^digit * h_bound * 2^-32, columns 2t, 2t+1 = digits 2(t&1), +1
                const float f0 = h_bound * ((t & 1) ? 1.52587890625e-05f : 2.3283064365386963e-10f);   // 2^-16 : 2^-32
                const float f1 = f0 * 256.0f;
#pragma unroll
                for (int f = 0; f < 8; ++f) {
                    cv[0][f][0] = fmaf((float)iacc[f][0], f0, cv[0][f][0]) * corr[0];
                    cv[0][f][1] = fmaf((float)iacc[f][1], f1, cv[0][f][1]) * corr[0];
                    cv[0][f][2] = fmaf((float)iacc[f][2], f0, cv[0][f][2]) * corr[0];
                    cv[0][f][3] = fmaf((float)iacc[f][3], f1, cv[0][f][3]) * corr[0];
                    iacc[f][0] = 0; iacc[f][1] = 0; iacc[f][2] = 0; iacc[f][3] = 0;
                }
                if (hm >= h_bound) h_bound = __int_as_float(((__float_as_int(hm) >> 23) + 1) << 23);   // next power of two above hm
            } else {
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
        }
        float p[2][R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            p[0][r] = ex2_approx(sc[0][r] - m_run[r]);      // exp2(-inf) = 0 for tokens past the end
            p[1][r] = ex2_approx(sc[1][r] - m_run[r]);
            l_part[r] += p[0][r] + p[1][r];
        }
        if constexpr (C::VINT8) {
            // P operand (u8): p*h on a 32-bit fixed-point grid below h_bound; the four bytes of that integer are
            // the four digit columns of the token.  Token tau is k index (tau & 31) of k-block tau >> 5.
            const float hscale = 4294967296.0f / h_bound;
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                uint8_t *dst = Pb + (hf * 8 * 4 + ((lane >> 2) & 3)) * 8 + (lane >> 4) * 4 + (lane & 3);
#pragma unroll
                for (int gg = 0; gg < NG; ++gg) {
                    uint32_t fx;
                    asm("cvt.rni.sat.u32.f32 %0, %1;" : "=r"(fx) : "f"(p[hf][0] * hv[hf][gg] * hscale));
                    z_part[0][gg] = fmaf(p[hf][0], zv[hf][gg], z_part[0][gg]);
#pragma unroll
                    for (int dg = 0; dg < 4; ++dg) dst[(gg * 4 + dg) * 32] = (uint8_t)(fx >> (8 * dg));
                }
            }
        } else {
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
                        const float ph = p[hf][r] * hv[hf][gg];
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
                        z_part[r][gg] = fmaf(p[hf][r], zv[hf][gg], z_part[r][gg]);
                    }
            }
        }
        __syncwarp();

        if constexpr (C::VINT8) {
            // ---------------- P.V in int8: rows = channels 4*(byte column) + j, k = 32 tokens per MMA
            const uint32_t vaddr = smem_u32(Vc) + lane * kRowBytes;   // lanes 0-15: tokens 0-15, lanes 16-31: tokens 16-31
#pragma unroll
            for (int kk = 0; kk < 2; ++kk) {
                const uint2 pb = *reinterpret_cast<const uint2 *>(Pb + ((kk * 8 + g) * 4 + t) * 8);
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    uint32_t rr[4];
                    ldmatrix_b8_trans_x2(rr, vaddr + kk * 32 * kRowBytes + hh * 16);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t m = 0x03030303u << (2 * j);
                        imma16832_uu(iacc[hh * 4 + j], rr[0] & m, rr[1] & m, rr[2] & m, rr[3] & m, pb.x, pb.y);
                    }
                }
            }
        } else {
            // ---------------- P.V in fp16: rows = channels (lane g reads code word g), k = tokens
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
        }
        __syncwarp();   // every lane is done with this stage, Sc and the P tile
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
    for (int r = 0; r < R; ++r) {
        l_part[r] = warp_sum(l_part[r]);
#pragma unroll
        for (int gg = 0; gg < NG; ++gg) { s_part[r][gg] = warp_sum(s_part[r][gg]); z_part[r][gg] = warp_sum(z_part[r][gg]); }
    }
    if constexpr (C::VINT8) {
        // last fold of the integer sums, then add the four digit columns of each group: a lane pair (t, t^1) holds them
        const float f0 = h_bound * ((t & 1) ? 1.52587890625e-05f : 2.3283064365386963e-10f);
        const float f1 = f0 * 256.0f;
#pragma unroll
        for (int f = 0; f < 8; ++f) {
            float lo = fmaf((float)iacc[f][0], f0, cv[0][f][0]) + fmaf((float)iacc[f][1], f1, cv[0][f][1]);   // byte column (f>>2)*16+g
            float hi = fmaf((float)iacc[f][2], f0, cv[0][f][2]) + fmaf((float)iacc[f][3], f1, cv[0][f][3]);   // byte column +8
            lo += __shfl_xor_sync(0xffffffffu, lo, 1);
            hi += __shfl_xor_sync(0xffffffffu, hi, 1);
            // lanes t = 0,1 carry group 0, lanes t = 2,3 group 1; the even lane of each pair stores
            const int gg = t >> 1;
            if ((t & 1) == 0 && gg < NG) {
                const int bc = (f >> 2) * 16 + g, j = f & 3;
                Ot[gg * kHeadDim + 4 * bc + j] = lo;
                Ot[gg * kHeadDim + 4 * (bc + 8) + j] = hi;
            }
        }
        __syncwarp();
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
            const int d = lane + 32 * q4;
            const int j = d & 3;                                      // channel d = 4*(byte column) + j carries weight 4^j
            const float winv = j == 0 ? 1.0f : (j == 1 ? 0.25f : (j == 2 ? 0.0625f : 0.015625f));
            float zg = 0.f;
#pragma unroll
            for (int gg = 0; gg < NG; ++gg)
                if (d / G == gg) zg = z_part[0][gg];
            const float o = Ot[(d / G) * kHeadDim + d] * winv + zg;
            Ow[d] = failed ? 0.f : o;
        }
    } else {
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
    dim3 grid(a.plan.n_splits, a.s.Hkv, a.s.B);
    kern<<<grid, kThreads, C::kSmemBytes, stream>>>(a);
    return cudaGetLastError();
}

template <int G>
cudaError_t launch_g(const MmaArgs &a, cudaStream_t stream, bool *handled)
{
    *handled = true;
    switch (a.s.rep) {
        case 1: return launch_one<G, 1>(a, stream);
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
    if (s.k_bits != 2 || s.v_bits != 2 || s.rep != 1) return cudaSuccess;
    MmaArgs a{s, c, q, scale_log2, plan, workspace};
    switch (s.G) {
        case 128: return launch_g<128>(a, stream, handled);
        case 64: return launch_g<64>(a, stream, handled);
        default: return cudaSuccess;
    }
}

}  // namespace skvq

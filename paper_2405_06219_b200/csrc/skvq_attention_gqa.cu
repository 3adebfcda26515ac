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
// reference only moves when a score exceeds it by 12 in the log2 domain (a factor 4096: the 32-bit grid then still
// resolves 2^-20 of the largest p*h), which after the first tiles is rare.
// sum_t p_t z_{t,g} is one more small fp16 MMA per 16 tokens.
//
// One CTA = 4 independent warps on one (sequence, KV head, split); tiles of 64 tokens arrive through a per-warp
// ring of shared-memory stages filled by cp.async.bulk (mbarrier completion, bounded polling).
#include "skvq_mma_common.cuh"

namespace skvq {
namespace {

using namespace mmak;

constexpr int kHeadSlots = 4;           // query heads per KV head this kernel serves (rows = head x 4 digits)
constexpr int kRefSlackLog2 = 12;       // the softmax reference moves only when a score exceeds it by this (log2)
constexpr float kRefSlack = (float)kRefSlackLog2;

// TERN: three-level V rows (five base-3 digits per byte, 26 bytes) arrive as they are stored and are rewritten per tile, by
// the warp, as rows of 2-bit fields in a buffer of their own; from there on they are 2-bit rows.
template <int G, bool F8, bool TERN>
struct GCfg {
    static constexpr int NG = kHeadDim / G;
    static constexpr int kCodeTile = kTileTok * kRowBytes;               // 2048 B
    static constexpr int kMetaBytes = F8 ? 2 : 4;                        // {scale, zero} per (token, group): two E4M3 bytes or a half2
    static constexpr int kMetaTile = kTileTok * NG * kMetaBytes;
    static constexpr int kVRaw = TERN ? packed_row_bytes(kTernary) : kRowBytes;      // bytes per V row in the cache
    static constexpr int kVCopy = kTileTok * kVRaw;                      // bytes of V codes copied per tile (the slot keeps its size)
    static constexpr int kStageBytes = 2 * kCodeTile + 2 * kMetaTile;
    static constexpr int kVdBytes = TERN ? kCodeTile : 0;                // the rewritten V tile
    static constexpr int kStages = 2;
    static constexpr int kXBytes = NG * 2 * 32 * 8;                      // digit registers on their way to the A fragments
    static constexpr int kOBytes = kHeadSlots * kHeadDim * 4;            // folded P.V sums
    static constexpr int kZBytes = kHeadSlots * 4 * 4;                   // sum p*z per (head, group)
    static constexpr int kWarpBytes = kStages * kStageBytes + kXBytes + kOBytes + kZBytes + 64 + kVdBytes;
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

// Eight half2 operands (value 64 + w_f*code, w = {1,4,16,4,16,1,4,16}) from one packed word: register f holds
// field f of the low half (channel f of the word) and of the high half (channel f + 8).
__device__ __forceinline__ void unpack16(uint32_t x, uint32_t (&o)[8])
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

// Four 8x8 b16 matrices (rows of 16 bytes): lane (g, t) receives word t of row g of each matrix.
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

template <int NG>
__device__ __forceinline__ void load_words(const uint32_t *p, uint32_t (&w)[NG])
{
    if constexpr (NG == 4) {
        const uint4 x = *reinterpret_cast<const uint4 *>(p);
        w[0] = x.x; w[1] = x.y; w[2] = x.z; w[3] = x.w;
    } else if constexpr (NG == 2) {
        const uint2 x = *reinterpret_cast<const uint2 *>(p);
        w[0] = x.x; w[1] = x.y;
    } else {
        w[0] = p[0];
    }
}

// One E4M3 byte pair {h, z} -> the same pair as fp16 (every E4M3 value is an fp16 value).
__device__ __forceinline__ uint32_t e4m3x2_to_half2(uint16_t b)
{
    uint32_t r;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(b));
    return r;
}
// The NG {h, z} words of token tok of a scale/zero tile, as fp16 pairs.
template <int NG, bool F8>
__device__ __forceinline__ void load_meta(const uint8_t *tile, int tok, uint32_t (&w)[NG])
{
    if constexpr (F8) {
        uint16_t b[NG];
        if constexpr (NG == 4) {
            const uint2 x = *reinterpret_cast<const uint2 *>(tile + tok * 8);
            b[0] = (uint16_t)x.x; b[1] = (uint16_t)(x.x >> 16); b[2] = (uint16_t)x.y; b[3] = (uint16_t)(x.y >> 16);
        } else if constexpr (NG == 2) {
            const uint32_t x = *reinterpret_cast<const uint32_t *>(tile + tok * 4);
            b[0] = (uint16_t)x; b[1] = (uint16_t)(x >> 16);
        } else {
            b[0] = *reinterpret_cast<const uint16_t *>(tile + tok * 2);
        }
#pragma unroll
        for (int i = 0; i < NG; ++i) w[i] = e4m3x2_to_half2(b[i]);
    } else {
        load_words<NG>(reinterpret_cast<const uint32_t *>(tile) + tok * NG, w);
    }
}
// Word g (not a compile-time index) of the same.
template <int NG, bool F8>
__device__ __forceinline__ uint32_t load_meta_word(const uint8_t *tile, int tok, int g)
{
    if constexpr (F8) return e4m3x2_to_half2(reinterpret_cast<const uint16_t *>(tile)[tok * NG + g]);
    else return reinterpret_cast<const uint32_t *>(tile)[tok * NG + g];
}

__device__ __forceinline__ float lo_half(uint32_t w) { return __low2float(*reinterpret_cast<const __half2 *>(&w)); }
__device__ __forceinline__ float hi_half(uint32_t w) { return __high2float(*reinterpret_cast<const __half2 *>(&w)); }

// Token ownership inside a 64-token tile.  The tile is two blocks of 32 tokens (kk), a block four octets (q);
// lane group g owns token 32kk + 8q + ((g + q) & 7) of every octet.  The skew keeps both ldmatrix patterns
// (8 score rows of one octet, 4 tokens of one owner for the values) at two rows per shared-memory bank group.
__device__ __forceinline__ int owned_token(int kk, int q, int gg) { return 32 * kk + 8 * q + ((gg + q) & 7); }

// Two CTAs per SM (up to 255 registers per thread) measured faster than three (168 registers): the compiler needs
// the registers to overlap the four 16-token score blocks and the two value blocks of a tile.
// UNEQ: two groups of unequal width per row (boundaries on multiples of 32 channels, read from the cache); the group of
// a 32-channel block then comes from a map instead of from its position.
template <int G, int R, bool F8, bool UNEQ, bool TERN>
__global__ void __launch_bounds__(kThreads, 2) partition_gqa_kernel(MmaArgs a)
{
    using C = GCfg<G, F8, TERN>;
    constexpr int NG = C::NG;
    static_assert(!UNEQ || NG == 2, "unequal groups: two per row");
    static_assert(R <= kHeadSlots, "rows of the P.V MMAs are 4 heads x 4 digits");
    extern __shared__ __align__(128) uint8_t smem[];
    const Shape &s = a.s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    // Order matters: the merge kernel reads the lengths, the sinks and the window BEFORE its own wait, so it may only be
    // scheduled once everything in front of this grid (append, bookkeeping, plan) has completed and is visible.  Waiting
    // first and triggering afterwards gives exactly that; the merge kernel still runs under this kernel's body.
    asm volatile("griddepcontrol.wait;" ::: "memory");      // the lengths, and the plan kernel's header when there is one
    asm volatile("griddepcontrol.launch_dependents;");      // the merge kernel may start its window part now

    __shared__ __align__(16) Segment seg_sh;
    __shared__ int more_sh;
    __shared__ SlotWalker walk;      // only thread 0 touches it; shared memory keeps it out of everybody's registers
    __shared__ __align__(16) int hdr_sh[kPlanSmemInts];
    __shared__ uint16_t digits_sh[TERN ? 256 : 1];      // byte value -> its five base-3 digits as 2-bit fields
    if constexpr (TERN) {
        for (int v = tid; v < 256; v += kThreads)
            digits_sh[v] = (uint16_t)((v % 3) | ((v / 3 % 3) << 2) | ((v / 9 % 3) << 4) | ((v / 27 % 3) << 6) | ((v / 81) << 8));
    }
    if (a.plan.in_kernel) {
        if (warp == 0) plan_in_warp(a.c.lengths, s.B, s.Hkv, s.W, a.plan.lq_cap, a.plan.n_slots, hdr_sh);
        __syncthreads();
    }
    if (tid == 0)
        more_sh = walk.start(a.plan.in_kernel ? hdr_sh : reinterpret_cast<const int *>(a.ws), !a.plan.in_kernel, s.B, s.Hkv,
                             blockIdx.x) ? 1 : 0;
    __syncthreads();
    if (!more_sh) return;
    float *partials = a.ws + a.plan.hdr_ints;

    // per-warp pipeline state that outlives a segment: the stage barriers and how many tiles have gone through them
    uint8_t *warp_base = smem + C::kQBytes + warp * C::kWarpBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(warp_base + C::kStages * C::kStageBytes + C::kXBytes + C::kOBytes + C::kZBytes);
    const uint32_t bar0 = smem_u32(bars);
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < C::kStages; ++i) mbar_init(bar0 + 8 * i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    uint32_t tiles_done = 0;
    bool failed = false;

    for (;;) {
    if (tid == 0) seg_sh = walk.next(a.c.lengths, s.W, a.plan.lq_cap);
    __syncthreads();
    const int b = seg_sh.b, hk = seg_sh.hk, q_begin = seg_sh.tok_begin, q_end = seg_sh.tok_end, part = seg_sh.part;
    if (!segment_in_bounds(seg_sh, s, a.plan, a.c.status)) break;      // checked build only; uniform: every thread reads the same segment
    const int n_parts = a.plan.s_max;

    uint8_t *stage_base = warp_base;
    const size_t bh = (size_t)b * s.Hkv + hk;
    const uint8_t *k_codes = a.c.k_codes + bh * (size_t)s.cap * kRowBytes;
    const uint8_t *v_codes = a.c.v_codes + bh * (size_t)s.cap * C::kVRaw;
    const uint8_t *k_meta = reinterpret_cast<const uint8_t *>(a.c.k_meta) + bh * (size_t)s.cap * NG * C::kMetaBytes;
    const uint8_t *v_meta = reinterpret_cast<const uint8_t *>(a.c.v_meta) + bh * (size_t)s.cap * NG * C::kMetaBytes;

    const int n_tiles = (q_end - q_begin + kTileTok - 1) / kTileTok;
    const int n_my = (n_tiles > warp && !failed) ? (n_tiles - warp + kWarps - 1) / kWarps : 0;

    auto issue = [&](int i) {   // lane 0 only
        const int st = (tiles_done + i) % C::kStages;
        const int tok0 = q_begin + (warp + i * kWarps) * kTileTok;
        const uint32_t dst = smem_u32(stage_base + st * C::kStageBytes);
        const uint32_t bar = bar0 + 8 * st;
        mbar_expect_tx(bar, C::kStageBytes - C::kCodeTile + C::kVCopy);
        bulk_g2s(dst, k_codes + (size_t)tok0 * kRowBytes, C::kCodeTile, bar);
        bulk_g2s(dst + C::kCodeTile, v_codes + (size_t)tok0 * C::kVRaw, C::kVCopy, bar);
        bulk_g2s(dst + 2 * C::kCodeTile, k_meta + (size_t)tok0 * NG * C::kMetaBytes, C::kMetaTile, bar);
        bulk_g2s(dst + 2 * C::kCodeTile + C::kMetaTile, v_meta + (size_t)tok0 * NG * C::kMetaBytes, C::kMetaTile, bar);
    };
    if (lane == 0) {      // the first copies are in flight while the query is prepared
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the stages held the previous segment's result
        for (int i = 0; i < C::kStages && i < n_my; ++i) issue(i);
    }


    // ---- CTA-wide prologue: permuted query on a per-head power-of-two scale, per-(head, group) constants
    float *qs = reinterpret_cast<float *>(smem);                   // [4][128] q' * F_r (exact), 0 for absent heads
    float *cst = qs + kHeadSlots * kHeadDim;                       // [4][4]  -64 * sum_j q'_j F_r / w_j
    float *sqs = cst + kHeadSlots * 4;                             // [4][4]  sum_j q'_j F_r
    float *csc = sqs + kHeadSlots * 4;                             // [4]     sm_scale*log2(e) / F_r
    int *fexp = reinterpret_cast<int *>(csc + kHeadSlots);         // [4]
    float *redmax = reinterpret_cast<float *>(fexp + kHeadSlots);  // [4 warps][4]
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
        int j0 = gg * G, j1 = (gg + 1) * G;
        if (UNEQ && a.c.bounds_k) {
            j0 = a.c.bounds_k[(size_t)hk * (NG + 1) + gg] & ~(kGranule - 1);
            j1 = min(a.c.bounds_k[(size_t)hk * (NG + 1) + gg + 1] & ~(kGranule - 1), kHeadDim);
        }
        for (int j = j0; j < j1; ++j) {
            const float v = qs[r * kHeadDim + j];
            sq += v;
            sw += v * field_weight_inv(j & 7);
        }
        sqs[r * 4 + gg] = sq;
        cst[r * 4 + gg] = -64.0f * sw;
    }
    __syncthreads();

    // group of every 32-channel block (two bits each) for keys and values
    const uint32_t kmap = UNEQ ? granule_groups(a.c.bounds_k, hk, G, NG) : 0u, vmap = UNEQ ? granule_groups(a.c.bounds_v, hk, G, NG) : 0u;

    // B operands of the score MMAs.  ldmatrix hands lane t words t and 4+t of a token row; all sixteen fields of a
    // word are used, so k-step sx of channel half hf covers, in lane t, fields 2sx and 2sx+1 (+8) of word 4hf+t.
    // The words of lanes t = 0,1 and t = 2,3 lie in different 32-channel blocks, so column n = (head n>>1,
    // block parity n&1) carries the query only on the k rows of its own block: the two columns of a head hold the
    // partial sums of the two blocks apart, and the lane that owns columns 2t, 2t+1 owns head t.
    uint32_t bK[2][4][2];
    {
        const int hdn = g >> 1, par = g & 1;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf)
#pragma unroll
            for (int sx = 0; sx < 4; ++sx)
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const int fld = 2 * sx + j;
                    const int ch = 16 * (4 * hf + t) + fld;
                    const float wi = field_weight_inv(fld);
                    const bool on = (par == (t >> 1));
                    const float lo = on ? qs[hdn * kHeadDim + ch] * wi : 0.f;
                    const float hi = on ? qs[hdn * kHeadDim + ch + 8] * wi : 0.f;
                    bK[hf][sx][j] = pack_half2(lo, hi);
                }
    }
    // B operand of the {h, z} MMA: k = 2t <-> h of group t, k = 2t+1 <-> z of group t; fp16 hi parts in k < 8,
    // lo parts in k >= 8 (the A operand repeats the same words there).  Only the even column of a head is used.
    uint32_t bZ[2] = {0u, 0u};
    if ((g & 1) == 0 && t < NG) {
        const float c0 = cst[(g >> 1) * 4 + t], c1 = sqs[(g >> 1) * 4 + t];
        const float c0h = __half2float(__float2half_rn(c0)), c1h = __half2float(__float2half_rn(c1));
        bZ[0] = pack_half2(c0h, c1h);
        bZ[1] = pack_half2(c0 - c0h, c1 - c1h);
    }
    const float cs = csc[t];                                     // this lane's score columns belong to head t

    // ---- per-warp shared memory
    uint2 *Xs = reinterpret_cast<uint2 *>(warp_base + C::kStages * C::kStageBytes);                  // [NG][2][32]
    float *Os = reinterpret_cast<float *>(warp_base + C::kStages * C::kStageBytes + C::kXBytes);     // [4][128]
    float *Zs = Os + kHeadSlots * kHeadDim;                                                          // [4][4]
#pragma unroll
    for (int i = 0; i < kHeadSlots * kHeadDim / 32; ++i) Os[lane + 32 * i] = 0.f;
    __syncwarp();

    // ---- running state (this lane: head t, the eight tokens per tile that lane group g owns)
    float m_ref = -CUDART_INF_F;                               // softmax reference of head t (log2 domain)
    float l_sum = 0.f;                                         // partial sum of p over this lane's tokens
    float zp[NG];                                              // partial sums of p * z_v per group
#pragma unroll
    for (int gg = 0; gg < NG; ++gg) zp[gg] = 0.f;
    int acc[16][4];                                            // P.V: rows (head g&3, digit g>>2 [+2]), columns = channels
#pragma unroll
    for (int i = 0; i < 16; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0;
    float h_bound = 6.103515625e-05f;                          // power of two above every value scale seen so far
    int tiles_since_fold = 0;                                  // a token adds at most 255 * 192 to an int32 sum: fold at least every 32768 tokens
    uint32_t h_thr = 0x0400u;                                  // the same bound as an fp16 bit pattern (2^-14)
    bool acc_live = false;

    // lane constants
    const int hd = g & 3, d0 = g >> 2;                         // this lane's P.V rows: head hd, digits d0 and d0 + 2
    // ldmatrix row addresses (byte offsets inside a stage).  Scores: matrices {octet 2jj, octet 2jj+1} x {bytes 0-15,
    // 16-31}, lane supplies row lane&7 of matrix lane>>3.  Values: lanes 0-15 rows 4t'+j = token j of owner t',
    // lanes 16-31 the same for owners t'+4.
    uint32_t offK[2];
#pragma unroll
    for (int jj = 0; jj < 2; ++jj) {
        const int mi = lane >> 3, r = lane & 7, qq = 2 * jj + (mi & 1);
        offK[jj] = (uint32_t)(owned_token(0, qq, r) * kRowBytes + 16 * (mi >> 1));
    }
    const uint32_t offV = (uint32_t)(owned_token(0, lane & 3, ((lane & 15) >> 2) + 4 * (lane >> 4)) * kRowBytes);
    int own[4];                                                // owned token of octet q inside a 32-token block
#pragma unroll
    for (int q = 0; q < 4; ++q) own[q] = owned_token(0, q, g);
    const uint2 *xrd = Xs + d0 * 32;                           // digit pairs (d0, d0+2) of the owners this lane reads

    // Brings the integer sums into the fp32 sums in shared memory; everything there is then multiplied by corr_hd.
    auto fold = [&](float corr_hd) {
        const float sa = h_bound * (d0 ? 256.0f : 1.0f) * (1.0f / (float)(1u << (32 - kRefSlackLog2)));   // h_bound * 2^slack * 2^-32 * 256^d0
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
            tiles_since_fold = 0;
        }
    };

    for (int i = 0; i < n_my; ++i) {
        const int st = (tiles_done + i) % C::kStages;
        const uint32_t parity = ((tiles_done + i) / C::kStages) & 1u;
        if (!mbar_wait_bounded(bar0 + 8 * st, parity)) { failed = true; break; }
        uint8_t *Kc = stage_base + st * C::kStageBytes;
        uint8_t *Vc = Kc + C::kCodeTile;
        if constexpr (TERN) {
            // a lane takes tokens lane and lane + 32: a byte's five digits come from the table as ten bits and are ORed
            // into the row's stream of 2-bit fields
            uint8_t *Vd = warp_base + C::kWarpBytes - C::kVdBytes;
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const uint16_t *raw = reinterpret_cast<const uint16_t *>(Vc + (lane + 32 * hf) * C::kVRaw);      // rows are 2-byte aligned
                uint32_t w[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
#pragma unroll
                for (int n2 = 0; n2 < C::kVRaw / 2; ++n2) {
                    const uint32_t two = raw[n2];
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        const int pos = 10 * (2 * n2 + k), wi = pos >> 5, sh = pos & 31;      // ten bits from bit pos of the row on
                        const uint32_t e = digits_sh[k ? (two >> 8) : (two & 255u)];
                        w[wi] |= e << sh;
                        if (sh > 22 && wi + 1 < 8) w[wi + 1] |= e >> (32 - sh);
                    }
                }
                uint4 *o = reinterpret_cast<uint4 *>(Vd + (lane + 32 * hf) * kRowBytes);
                o[0] = make_uint4(w[0], w[1], w[2], w[3]);
                o[1] = make_uint4(w[4], w[5], w[6], w[7]);
            }
            Vc = Vd;      // visible to the other lanes behind the __syncwarp() calls in front of the value MMAs
        }
        uint8_t *Km = Kc + 2 * C::kCodeTile;                        // [64][NG] {h, z}
        uint8_t *Vm = Kc + 2 * C::kCodeTile + C::kMetaTile;
        const int tok0 = q_begin + (warp + i * kWarps) * kTileTok;
        const int n_valid = min(kTileTok, q_end - tok0);
        const int n_skip = max(s.n_sink - tok0, 0);      // rows of attention sinks: the merge kernel reads their fp16 copies
        if (n_valid < kTileTok || n_skip > 0) {
            // rows past the end (and rows of sinks) hold unspecified bytes: give their scale/zero words a defined value
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const int tau = lane + 32 * hf;
                if (tau >= n_valid || tau < n_skip) {
#pragma unroll
                    for (int gg = 0; gg < NG; ++gg) {
                        if constexpr (F8) {
                            reinterpret_cast<uint16_t *>(Km)[tau * NG + gg] = 0;
                            reinterpret_cast<uint16_t *>(Vm)[tau * NG + gg] = 0;
                        } else {
                            reinterpret_cast<uint32_t *>(Km)[tau * NG + gg] = 0u;
                            reinterpret_cast<uint32_t *>(Vm)[tau * NG + gg] = 0u;
                        }
                    }
                }
            }
            __syncwarp();
        }

        // ---------------- scores of head t for the eight owned tokens: sraw[2kk+jj][0/1] = octets 2jj, 2jj+1
        const uint32_t kaddr = smem_u32(Kc);
        float sraw[4][2];
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) {
            const int kk = mt >> 1, jj = mt & 1;
            uint32_t rw[4];
            ldmatrix_x4(rw, kaddr + kk * 32 * kRowBytes + offK[jj]);
            float ak[2][4];
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                uint32_t u0[8], u1[8];
                unpack16(rw[2 * hf], u0);          // row g     (octet 2jj)
                unpack16(rw[2 * hf + 1], u1);      // row g + 8 (octet 2jj+1)
                ak[hf][0] = 0.f; ak[hf][1] = 0.f; ak[hf][2] = 0.f; ak[hf][3] = 0.f;
#pragma unroll
                for (int sx = 0; sx < 4; ++sx)
                    mma16816(ak[hf], u0[2 * sx], u1[2 * sx], u0[2 * sx + 1], u1[2 * sx + 1], bK[hf][sx][0], bK[hf][sx][1]);
            }
            // {h, z} words of the two tokens: A operand of the constant/zero-point MMA, and h for the group sums
            const int tk0 = 32 * kk + own[2 * jj], tk1 = 32 * kk + own[2 * jj + 1];
            uint32_t mw0[NG], mw1[NG];
            load_meta<NG, F8>(Km, tk0, mw0);
            load_meta<NG, F8>(Km, tk1, mw1);
            const uint32_t za = t < NG ? load_meta_word<NG, F8>(Km, tk0, t < NG ? t : 0) : 0u;
            const uint32_t zb = t < NG ? load_meta_word<NG, F8>(Km, tk1, t < NG ? t : 0) : 0u;
            float az[4] = {0.f, 0.f, 0.f, 0.f};
            mma16816(az, za, zb, za, zb, bZ[0], bZ[1]);
            float s0 = az[0], s1 = az[2];
#pragma unroll
            for (int hf = 0; hf < 2; ++hf)
#pragma unroll
                for (int par = 0; par < 2; ++par) {
                    if constexpr (UNEQ) {
                        const bool g1 = (kmap >> (2 * (2 * hf + par))) & 1u;
                        s0 = fmaf(lo_half(g1 ? mw0[1] : mw0[0]), ak[hf][par], s0);
                        s1 = fmaf(lo_half(g1 ? mw1[1] : mw1[0]), ak[hf][2 + par], s1);
                    } else {
                        const int gg = (64 * hf + 32 * par) / G;
                        s0 = fmaf(lo_half(mw0[gg]), ak[hf][par], s0);
                        s1 = fmaf(lo_half(mw1[gg]), ak[hf][2 + par], s1);
                    }
                }
            sraw[mt][0] = s0;
            sraw[mt][1] = s1;
        }

        // ---------------- does the softmax reference, or the bound on the value scales, have to move?
        uint32_t hmax_bits;
        {
            uint32_t wa[NG], wb[NG];
            load_meta<NG, F8>(Vm, lane, wa);
            load_meta<NG, F8>(Vm, lane + 32, wb);
            uint32_t mx = __vmaxu2(wa[0], wb[0]);
#pragma unroll
            for (int gg = 1; gg < NG; ++gg) mx = __vmaxu2(mx, __vmaxu2(wa[gg], wb[gg]));
            hmax_bits = mx & 0xFFFFu;                          // scales are non-negative: fp16 order = integer order
        }
        bool moved = hmax_bits >= h_thr || ++tiles_since_fold * kTileTok >= 32768;
        const bool whole = n_valid == kTileTok && n_skip == 0;      // all but the first and last tiles of a segment
        float arg[4][2];
        float amax = -CUDART_INF_F;
        if (whole) {
#pragma unroll
            for (int mt = 0; mt < 4; ++mt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    arg[mt][e] = fmaf(sraw[mt][e], cs, -m_ref);
                    amax = fmaxf(amax, arg[mt][e]);
                }
        } else {
#pragma unroll
            for (int mt = 0; mt < 4; ++mt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int tok_in = 32 * (mt >> 1) + own[2 * (mt & 1) + e];
                    const bool valid = tok_in < n_valid && tok_in >= n_skip;
                    arg[mt][e] = valid ? fmaf(sraw[mt][e], cs, -m_ref) : -CUDART_INF_F;
                    amax = fmaxf(amax, arg[mt][e]);
                }
        }
        moved |= amax > kRefSlack;
        if (__any_sync(0xffffffffu, moved)) {
            // Raise the reference of every head to its running maximum (and the bound on h); fold what was accumulated.
            float tm = -CUDART_INF_F;
#pragma unroll
            for (int mt = 0; mt < 4; ++mt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int tok_in = 32 * (mt >> 1) + own[2 * (mt & 1) + e];
                    const bool valid = tok_in < n_valid && tok_in >= n_skip;
                    if (valid) tm = fmaxf(tm, sraw[mt][e] * cs);
                }
#pragma unroll
            for (int msk = 4; msk < 32; msk <<= 1) tm = fmaxf(tm, __shfl_xor_sync(0xffffffffu, tm, msk));
            const float m_new = fmaxf(m_ref, tm);
            const float corr = m_new == -CUDART_INF_F ? 1.f : ex2_approx(m_ref - m_new);      // 0 on the first tile with a token
            m_ref = m_new;
            l_sum *= corr;
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) zp[gg] *= corr;
            const float corr_hd = __shfl_sync(0xffffffffu, corr, hd);  // lane hd = (g 0, t hd) holds head hd
            if (acc_live) fold(corr_hd);
            const uint32_t hm = __reduce_max_sync(0xffffffffu, hmax_bits);
            if (hm >= h_thr) {
                const float hmf = __half2float(__ushort_as_half((unsigned short)hm));
                h_bound = __int_as_float(((__float_as_int(hmf) >> 23) + 1) << 23);    // next power of two above
                h_thr = h_bound > 32768.0f ? 0x7C00u : (uint32_t)__half_as_ushort(__float2half_rn(h_bound));
            }
#pragma unroll
            for (int mt = 0; mt < 4; ++mt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int tok_in = 32 * (mt >> 1) + own[2 * (mt & 1) + e];
                    const bool valid = tok_in < n_valid && tok_in >= n_skip;
                    arg[mt][e] = valid ? fmaf(sraw[mt][e], cs, -m_ref) : -CUDART_INF_F;
                }
        }
        const float hscale = (float)(1u << (32 - kRefSlackLog2)) / h_bound;      // 2^32 / (h_bound * 2^slack)

        // ---------------- per 32-token block: probabilities, p*h on the fixed-point grid, digits -> A fragments, MMAs
        const uint32_t vaddr = smem_u32(Vc) + offV;
#pragma unroll
        for (int kk = 0; kk < 2; ++kk) {
            uint32_t uu[4][NG];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float p = ex2_approx(arg[2 * kk + (q >> 1)][q & 1]);      // at most 2^slack; 0 past the end
                l_sum += p;
                uint32_t vw[NG];
                load_meta<NG, F8>(Vm, 32 * kk + own[q], vw);
                const float ps = p * hscale;
#pragma unroll
                for (int gg = 0; gg < NG; ++gg) {
                    uu[q][gg] = to_fixed_u32(ps * lo_half(vw[gg]));
                    zp[gg] = fmaf(p, hi_half(vw[gg]), zp[gg]);
                }
            }
            // byte transpose: digit d of the four owned tokens in one register; pairs (0,2) and (1,3) are what the
            // two reader lanes of a head want
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) {
                const uint32_t t01 = prmt(uu[0][gg], uu[1][gg], 0x5140u), t23 = prmt(uu[2][gg], uu[3][gg], 0x5140u);
                const uint32_t h01 = prmt(uu[0][gg], uu[1][gg], 0x7362u), h23 = prmt(uu[2][gg], uu[3][gg], 0x7362u);
                Xs[(gg * 2 + 0) * 32 + lane] = make_uint2(prmt(t01, t23, 0x5410u), prmt(h01, h23, 0x5410u));   // digits 0, 2
                Xs[(gg * 2 + 1) * 32 + lane] = make_uint2(prmt(t01, t23, 0x7632u), prmt(h01, h23, 0x7632u));   // digits 1, 3
            }
            __syncwarp();
            // A fragments: k = 4t+j <-> token j of owner t (slot 4t + hd), k = 16+4t+j <-> owner t+4
            uint32_t Ag[NG][4];
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) {
                const uint2 xa = xrd[gg * 64 + 4 * t + hd], xb = xrd[gg * 64 + 4 * (t + 4) + hd];
                Ag[gg][0] = xa.x; Ag[gg][1] = xa.y; Ag[gg][2] = xb.x; Ag[gg][3] = xb.y;
            }
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                uint32_t rr[4];
                ldmatrix_b8_trans_x2(rr, vaddr + kk * 32 * kRowBytes + hh * 16);
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t A0, A1, A2, A3;      // the digits of this 32-channel block's group
                    if constexpr (UNEQ) {
                        const bool g1 = (vmap >> (2 * (2 * hh + half))) & 1u;
                        A0 = g1 ? Ag[1][0] : Ag[0][0]; A1 = g1 ? Ag[1][1] : Ag[0][1];
                        A2 = g1 ? Ag[1][2] : Ag[0][2]; A3 = g1 ? Ag[1][3] : Ag[0][3];
                    } else {
                        const int gg = (64 * hh + 32 * half) / G;
                        A0 = Ag[gg][0]; A1 = Ag[gg][1]; A2 = Ag[gg][2]; A3 = Ag[gg][3];
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t m = 0x03030303u << (2 * j);
                        imma16832_uu(acc[hh * 8 + half * 4 + j], A0, A1, A2, A3, rr[half] & m, rr[2 + half] & m);
                    }
                }
            }
            __syncwarp();   // the exchange buffer is rewritten by the next block
        }
        acc_live = true;
        if (lane == 0 && i + C::kStages < n_my) issue(i + C::kStages);
    }

    if (failed) {
        for (int i2 = 0; i2 < n_my; ++i2) {
            const int st = (tiles_done + i2) % C::kStages;
            (void)mbar_wait_bounded(bar0 + 8 * st, ((tiles_done + i2) / C::kStages) & 1u);
        }
        if (lane == 0 && a.c.status) atomicOr(a.c.status, SKVQ_STATUS_COPY_TIMEOUT);
    }

    // ---- per-warp result
    if (acc_live) fold(1.0f);
#pragma unroll
    for (int msk = 4; msk < 32; msk <<= 1) {
        l_sum += __shfl_xor_sync(0xffffffffu, l_sum, msk);
#pragma unroll
        for (int gg = 0; gg < NG; ++gg) zp[gg] += __shfl_xor_sync(0xffffffffu, zp[gg], msk);
    }
    if (g == 0) {
#pragma unroll
        for (int gg = 0; gg < NG; ++gg) Zs[t * 4 + gg] = zp[gg];
    }
    __syncwarp();
    const bool dead = failed || !acc_live;
    float *Ow = reinterpret_cast<float *>(stage_base);                       // [R][132]: o', m, l
#pragma unroll
    for (int r = 0; r < R; ++r) {
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
            const int d = lane + 32 * q4;
            const int j = d & 3;                                             // channel d carries the weight 4^j
            const float winv = j == 0 ? 1.0f : (j == 1 ? 0.25f : (j == 2 ? 0.0625f : 0.015625f));
            const float o = Os[r * kHeadDim + d] * winv + Zs[r * 4 + (UNEQ ? (int)((vmap >> (2 * (d >> 5))) & 1u) : d / G)];
            Ow[r * kPartialStride + d] = dead ? 0.f : o;
        }
    }
    if (g == 0 && t < R) {
        Ow[t * kPartialStride + kHeadDim] = dead ? -CUDART_INF_F : m_ref;
        Ow[t * kPartialStride + kHeadDim + 1] = dead ? 0.f : l_sum;
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
        float *dst = partials + (((size_t)b * s.Hq + hk * R + r) * n_parts + part) * kPartialStride;
        dst[tid] = o;
        if (tid == 0) { dst[kHeadDim] = M; dst[kHeadDim + 1] = l; }
    }
    tiles_done += n_my;
    __syncthreads();          // the segment's shared data is dead; thread 0 decides whether there is another one
    if (tid == 0) more_sh = walk.done() ? 0 : 1;
    __syncthreads();
    if (!more_sh) break;
    }
}

template <int G, int R, bool F8, bool UNEQ, bool TERN>
cudaError_t launch_t(const MmaArgs &a, cudaStream_t stream, bool overlap)
{
    using C = GCfg<G, F8, TERN>;
    static unsigned long long configured = 0;      // one bit per device
    auto kern = partition_gqa_kernel<G, R, F8, UNEQ, TERN>;
    const cudaError_t ec = configure_smem_once(kern, C::kSmemBytes, configured);
    if (ec != cudaSuccess) return ec;
    return launch_dependent(kern, dim3(a.plan.n_slots), dim3(kThreads), C::kSmemBytes, stream, overlap, a);
}

template <int G, int R, bool F8, bool UNEQ>
cudaError_t launch_one(const MmaArgs &a, cudaStream_t stream, bool overlap)
{
    return a.s.v_bits == kTernary ? launch_t<G, R, F8, UNEQ, true>(a, stream, overlap) : launch_t<G, R, F8, UNEQ, false>(a, stream, overlap);
}

template <int G, bool F8, bool UNEQ>
cudaError_t launch_g(const MmaArgs &a, cudaStream_t stream, bool overlap, bool *handled)
{
    *handled = true;
    switch (a.s.rep) {
        case 1: return launch_one<G, 1, F8, UNEQ>(a, stream, overlap);
        case 2: return launch_one<G, 2, F8, UNEQ>(a, stream, overlap);
        case 4: return launch_one<G, 4, F8, UNEQ>(a, stream, overlap);
        default: *handled = false; return cudaSuccess;
    }
}

}  // namespace

// Launches the kernel above when the configuration is covered (2-bit K, 2-bit or three-level V, 1, 2 or 4 query heads per KV
// head; groups of unequal width with two groups per row); *handled tells the caller whether it did.
cudaError_t launch_partition_gqa(const Shape &s, const CachePtrs &c, const __half *q, float scale_log2,
                                 const SplitPlan &plan, float *workspace, cudaStream_t stream, bool overlap, bool *handled)
{
    *handled = false;
    if (s.k_bits != 2 || (s.v_bits != 2 && s.v_bits != kTernary)) return cudaSuccess;
    if (s.bounded && s.G != 64) return cudaSuccess;
    MmaArgs a{s, c, q, scale_log2, plan, workspace};
    if (s.bounded) return s.meta_fp8 ? launch_g<64, true, true>(a, stream, overlap, handled) : launch_g<64, false, true>(a, stream, overlap, handled);
    if (s.meta_fp8) {
        switch (s.G) {
            case 128: return launch_g<128, true, false>(a, stream, overlap, handled);
            case 64: return launch_g<64, true, false>(a, stream, overlap, handled);
            case 32: return launch_g<32, true, false>(a, stream, overlap, handled);
            default: return cudaSuccess;
        }
    }
    switch (s.G) {
        case 128: return launch_g<128, false, false>(a, stream, overlap, handled);
        case 64: return launch_g<64, false, false>(a, stream, overlap, handled);
        case 32: return launch_g<32, false, false>(a, stream, overlap, handled);
        default: return cudaSuccess;
    }
}

}  // namespace skvq

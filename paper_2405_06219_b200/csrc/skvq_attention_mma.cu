// Integer tensor-core partition kernel of skvq_decode_attention for one query head per KV head and at most two
// groups per row (G = 64 or 128), 2- or 4-bit K and V in any combination, or three-level V (Eq. 1, Algorithm 1).
//
// Why tensor cores on an HBM-bound path: at 2 bits a cache element costs 0.28 bytes, so streaming at several
// TB/s leaves fewer than two issue slots per element, and the logic pipe that does the bit work retires half
// a warp instruction per clock.  The codes are therefore turned into MMA operands with one AND per four codes
// and contracted on the tensor cores; scale and zero point never touch individual elements:
//   q'.K~_t            = sum_g h_{t,g} (sum_{j in g} q'_j c_{t,j}) + sum_g z_{t,g} (sum_{j in g} q'_j)
//   sum_t p_t V~_{t,d} = sum_t (p_t h_{t,g(d)}) c_{t,d} + sum_t p_t z_{t,g(d)}
// Scores (mma.m16n8k32.u8.s8, exact): `word & mask` leaves four codes of a packed word as bytes worth
// w * code -- masks 0x03030303 << 2i (w = 4^i) for 2-bit codes, 0x0F0F0F0F << 4i (w = 16^i) for 4-bit codes, no
// shift.  The query is put on a power-of-two fixed-point grid, divided by w and split into four signed byte
// digits that sit in four B columns, so sum_j q'_j c_j is formed exactly in int32.
// Values (mma.m16n8k32.u8.u8, exact): ldmatrix.trans.b8 transposes the V tile so that a register holds one byte
// column of four tokens, the same masks leave w * code, and p*h goes on a 32-bit fixed-point grid below a
// running power-of-two bound on h whose four bytes are the four digit columns of a group.  The integer
// accumulators are folded into fp32 whenever the softmax reference or that bound moves.
//
// One CTA = 4 independent warps on one (sequence, KV head, split); each warp streams tiles of codes + scale/zero
// (64 tokens; 32 when both K and V are 4-bit, so that a tile has the same bytes) through its own ring of
// shared-memory stages filled by cp.async.bulk (mbarrier completion, bounded polling), keeps its own
// online-softmax state, and the 4 states are merged in shared memory before one partial is written to the
// workspace.  The fp16 window is handled by the merge kernel.
#include "skvq_mma_common.cuh"

namespace skvq {
namespace {

using namespace mmak;

// ---------------------------------------------------------------- compile-time layout
template <int G, int KB, int VB, bool F8>
struct Cfg {
    static constexpr int NG = kHeadDim / G;
    static_assert(NG <= 2, "(group, byte digit) has to fit the 8 MMA columns");
    static constexpr int T = (KB == 4 && VB == 4) ? 32 : 64;             // tokens per warp tile
    // Three-level V rows (VB = kTernary: five base-3 digits per byte) arrive as they are stored and are rewritten per
    // tile, by the warp, as rows of 2-bit fields in a buffer of their own; from there on they are 2-bit rows (VBE).
    static constexpr bool kTern = VB == kTernary;
    static constexpr int VBE = kTern ? 2 : VB;
    static constexpr int KROW = kHeadDim * KB / 8, VROW = kHeadDim * VBE / 8;  // bytes per token row in shared memory
    static constexpr int VRAW = packed_row_bytes(VB);                     // bytes per V row in the cache
    static constexpr int VCPB = 8 / VBE;                                  // codes per byte = masks per register
    static constexpr int kKTile = T * KROW, kVTile = T * VRAW;
    static constexpr int kVdBytes = kTern ? T * VROW : 0;                 // the rewritten V tile
    static constexpr int kMetaBytes = F8 ? 2 : 4;      // {scale, zero} per (token, group): two E4M3 bytes or a half2
    static constexpr int kMetaTile = T * NG * kMetaBytes;
    static constexpr int kStageBytes = kKTile + kVTile + 2 * kMetaTile;
    static constexpr int kStages = 2;
    static constexpr int kScBytes = T * NG * 8;                           // per (token, group): low and high digit pairs
    static constexpr int kPBytes = (T / 32) * 8 * 32;                     // P operand tile: [k-block][8 columns][32 tokens] bytes
    static constexpr int kWarpBytes = kStages * kStageBytes + kScBytes + kPBytes + 64 + kVdBytes;   // + mbarriers (+ the rewritten V tile)
    static constexpr int kQBytes = (kHeadDim * 4 + NG * 4 + 2 * 4 + 64 + 127) / 128 * 128 + 512;   // + the B operand image
    static constexpr int kSmemBytes = kQBytes + kWarps * kWarpBytes;
    static constexpr int kCtasPerSm = (KB == VB) ? 4 : 3;      // three measured slower for the equal-width kernels
    static_assert(kStages * kStageBytes >= NG * kHeadDim * 4 + kPartialStride * 4, "stage area is reused for the final merge");
    static_assert(kKTile % 16 == 0 && kVTile % 16 == 0 && kMetaTile % 16 == 0, "bulk copies move multiples of 16 bytes");
};

// UNEQ: two groups of unequal width per row (boundaries on multiples of 32 channels, read from the cache); the group of
// a 32-channel block then comes from a map instead of from its position.
template <int G, int KB, int VB, bool F8, bool UNEQ>
__global__ void __launch_bounds__(kThreads, Cfg<G, KB, VB, F8>::kCtasPerSm) partition_mma_kernel(MmaArgs a)
{
    using C = Cfg<G, KB, VB, F8>;
    static_assert(!UNEQ || C::NG == 2, "unequal groups: two per row");
    constexpr int NG = C::NG, KROW = C::KROW, VROW = C::VROW, T = C::T, VBE = C::VBE;
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
    __shared__ uint16_t digits_sh[C::kTern ? 256 : 1];      // byte value -> its five base-3 digits as 2-bit fields
    if constexpr (C::kTern) {
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
    uint64_t *bars = reinterpret_cast<uint64_t *>(warp_base + C::kStages * C::kStageBytes + C::kScBytes + C::kPBytes);
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
    const uint8_t *k_codes = a.c.k_codes + bh * (size_t)s.cap * KROW;
    const uint8_t *v_codes = a.c.v_codes + bh * (size_t)s.cap * C::VRAW;
    const uint8_t *k_meta = reinterpret_cast<const uint8_t *>(a.c.k_meta) + bh * (size_t)s.cap * NG * C::kMetaBytes;
    const uint8_t *v_meta = reinterpret_cast<const uint8_t *>(a.c.v_meta) + bh * (size_t)s.cap * NG * C::kMetaBytes;

    const int n_tiles = (q_end - q_begin + T - 1) / T;                          // tiles of this split
    const int n_my = (n_tiles > warp && !failed) ? (n_tiles - warp + kWarps - 1) / kWarps : 0;   // tiles warp, warp+4, ...

    auto issue = [&](int i) {   // lane 0 only: start the copies of this warp's i-th tile
        const int st = (tiles_done + i) % C::kStages;
        const int tok0 = q_begin + (warp + i * kWarps) * T;                       // multiple of 32: 16-byte aligned sources
        const uint32_t dst = smem_u32(stage_base + st * C::kStageBytes);
        const uint32_t bar = bar0 + 8 * st;
        mbar_expect_tx(bar, C::kStageBytes);
        bulk_g2s(dst, k_codes + (size_t)tok0 * KROW, C::kKTile, bar);
        bulk_g2s(dst + C::kKTile, v_codes + (size_t)tok0 * C::VRAW, C::kVTile, bar);
        bulk_g2s(dst + C::kKTile + C::kVTile, k_meta + (size_t)tok0 * NG * C::kMetaBytes, C::kMetaTile, bar);
        bulk_g2s(dst + C::kKTile + C::kVTile + C::kMetaTile, v_meta + (size_t)tok0 * NG * C::kMetaBytes, C::kMetaTile, bar);
    };
    if (lane == 0) {      // the first copies are in flight while the query is prepared
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the stages held the previous segment's result
        for (int i = 0; i < C::kStages && i < n_my; ++i) issue(i);
    }


    // ---- CTA-wide prologue: permuted query, its fixed-point grid and per-group sums
    float *qs = reinterpret_cast<float *>(smem);                       // [128] q' (exact fp16 values)
    float *sqs = qs + kHeadDim;                                        // [NG] scale * sum_j q'_j
    float *cF = sqs + NG;                                              // scale / F, F = 2^kexp
    int *kexp = reinterpret_cast<int *>(cF + 1);
    float *redmax = reinterpret_cast<float *>(kexp + 1);               // [4]
    {
        const int32_t *idx_k = a.c.reorder_k + (size_t)hk * kHeadDim;
        const int src = idx_k[tid] & (kHeadDim - 1);
        const float qv = __half2float(a.q[((size_t)b * s.Hq + hk) * kHeadDim + src]);
        qs[tid] = qv;
        const float wm = warp_max(fabsf(qv));
        if (lane == 0) redmax[warp] = wm;
    }
    __syncthreads();
    if (tid == 0) {
        // F = 2^k with |q'_j| * F <= 2^30: every q'_j * F / w is then an integer (or rounds at 2^-24 relative)
        float qmax = 0.f;
        for (int w = 0; w < kWarps; ++w) qmax = fmaxf(qmax, redmax[w]);
        int k = 0;
        if (qmax > 0.f) {
            int e;
            const float m = frexpf(qmax, &e);          // qmax = m * 2^e, 0.5 <= m < 1
            k = 30 - ((m == 0.5f) ? e - 1 : e);
        }
        kexp[0] = k;
        cF[0] = ldexpf(a.scale_log2, -k);
    }
    if (tid >= 32 && tid < 32 + NG) {
        const int gg = tid - 32;
        int j0 = gg * G, j1 = (gg + 1) * G;
        if (UNEQ && a.c.bounds_k) {
            j0 = a.c.bounds_k[(size_t)hk * (NG + 1) + gg] & ~(kGranule - 1);
            j1 = a.c.bounds_k[(size_t)hk * (NG + 1) + gg + 1] & ~(kGranule - 1);
        }
        float sq = 0.f;
        for (int j = j0; j < j1 && j < kHeadDim; ++j) sq += qs[j];
        sqs[gg] = sq * a.scale_log2;
    }
    // group of every 32-channel block (two bits each) for keys and values
    const uint32_t kmap = UNEQ ? granule_groups(a.c.bounds_k, hk, G, NG) : 0u, vmap = UNEQ ? granule_groups(a.c.bounds_v, hk, G, NG) : 0u;
    __syncthreads();

    // B operand of the score MMAs (s8).  k-step ks contracts 32 channels; lane t supplies two registers of four
    // bytes each.  2-bit codes: register reg comes from word 2ks+reg under mask t, byte bb = code 4bb+t of that
    // word (weight 4^t).  4-bit codes: register reg comes from word 4ks + 2(t>>1) + reg under mask t&1, byte bb =
    // code 2bb+(t&1) of that word (weight 16^(t&1)).  Column = byte digit of round(q' * F / weight).
    // Thread tid owns channel tid: it writes the four digits of that channel as bytes straight into the
    // register image bimg[digit][ks][reg][t] (byte bb), which the lanes then load word by word (the barrier at the
    // end of a segment keeps the next segment's writes behind these reads).
    uint8_t *bimg0 = smem + C::kQBytes - 512;   // [4][4][2][4] words
    {
        int ks, reg, bb, tt, wlog2;
        if constexpr (KB == 2) {
            ks = tid >> 5; reg = (tid >> 4) & 1; bb = (tid >> 2) & 3; tt = tid & 3; wlog2 = 2 * tt;
        } else {
            const int wi = (tid >> 3) & 3, e = tid & 7;     // word inside the k-step, code inside the word
            ks = tid >> 5; reg = wi & 1; bb = e >> 1; tt = 2 * (wi >> 1) + (e & 1); wlog2 = 4 * (e & 1);
        }
        // q' * 2^(k - wlog2): an exact power-of-two scaling done on the exponent field
        int v = __float2int_rn(qs[tid] * __int_as_float((127 + kexp[0] - wlog2) << 23));
#pragma unroll
        for (int i = 0; i < 4; ++i) {      // balanced base-256 digits, least significant first
            const int di = (i < 3) ? (int)(int8_t)(v & 0xFF) : v;
            v = (v - di) >> 8;
            bimg0[((((i * 4 + ks) * 2 + reg) * 4 + tt) << 2) + bb] = (uint8_t)(di & 0xFF);
        }
    }
    __syncthreads();
    uint32_t bq[4][2];
    {
        const int dig = g & 3;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
#pragma unroll
            for (int reg = 0; reg < 2; ++reg)
                bq[ks][reg] = (g < 4) ? reinterpret_cast<const uint32_t *>(bimg0)[(((dig * 4 + ks) * 2 + reg) * 4 + t)] : 0u;
    }
    const float cFr = cF[0];
    float sqr[NG];
#pragma unroll
    for (int gg = 0; gg < NG; ++gg) sqr[gg] = sqs[gg];

    // ---- per-warp buffers
    float *Sc = reinterpret_cast<float *>(warp_base + C::kStages * C::kStageBytes);      // [T][NG][2]
    uint8_t *Pb = warp_base + C::kStages * C::kStageBytes + C::kScBytes;                 // [k-block][8 columns][4 t][2 halves][4 tokens]

    // online-softmax state (per warp; m is warp-uniform, the sums are per-lane partials)
    float m_run = -CUDART_INF_F, l_part = 0.f, z_part[NG];
#pragma unroll
    for (int gg = 0; gg < NG; ++gg) z_part[gg] = 0.f;
    // int accumulators iacc (exact while the softmax reference and the scale bound stay put) are folded into cv
    // whenever either one moves.  Accumulator f = 16-byte column block f / VCPB, mask f % VCPB.
    float cv[8][4];
    int iacc[8][4];
#pragma unroll
    for (int f = 0; f < 8; ++f)
#pragma unroll
        for (int i = 0; i < 4; ++i) { cv[f][i] = 0.f; iacc[f][i] = 0; }
    float h_bound = 6.103515625e-05f;   // 2^-14: every scale seen so far is below this power of two
    int tiles_since_fold = 0;           // a token adds at most 255 * 240 to an int32 sum: fold at least every 32768 tokens

    const uint32_t kmask = KB == 2 ? (0x03030303u << (2 * t)) : (0x0F0F0F0Fu << (4 * (t & 1)));

    for (int i = 0; i < n_my; ++i) {
        const int st = (tiles_done + i) % C::kStages;
        const uint32_t parity = ((tiles_done + i) / C::kStages) & 1u;
        if (!mbar_wait_bounded(bar0 + 8 * st, parity)) { failed = true; break; }
        const uint8_t *Kc = stage_base + st * C::kStageBytes;
        const uint8_t *Vc = Kc + C::kKTile;
        if constexpr (C::kTern) {
            // Rewrite the tile's V rows (26 bytes of base-3 digits) as rows of 2-bit fields: a lane takes tokens lane and
            // lane + 32; a byte's five digits come from the table as ten bits and are ORed into the row's bit stream.
            uint8_t *Vd = stage_base + C::kWarpBytes - C::kVdBytes;
#pragma unroll
            for (int hf = 0; hf < T / 32; ++hf) {
                const uint16_t *raw = reinterpret_cast<const uint16_t *>(Vc + (lane + 32 * hf) * C::VRAW);      // rows are 2-byte aligned
                uint32_t w[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
#pragma unroll
                for (int n2 = 0; n2 < C::VRAW / 2; ++n2) {
                    const uint32_t two = raw[n2];
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        const int pos = 10 * (2 * n2 + k), wi = pos >> 5, sh = pos & 31;      // ten bits from bit pos of the row on
                        const uint32_t e = digits_sh[k ? (two >> 8) : (two & 255u)];
                        w[wi] |= e << sh;
                        if (sh > 22 && wi + 1 < 8) w[wi + 1] |= e >> (32 - sh);
                    }
                }
                uint4 *o = reinterpret_cast<uint4 *>(Vd + (lane + 32 * hf) * VROW);
                o[0] = make_uint4(w[0], w[1], w[2], w[3]);
                o[1] = make_uint4(w[4], w[5], w[6], w[7]);
            }
            Vc = Vd;      // visible to the other lanes behind the __syncwarp() calls in front of the value MMAs
        }
        const uint8_t *Km = Kc + C::kKTile + C::kVTile;                      // [T][NG] {h, z}
        const uint8_t *Vm = Kc + C::kKTile + C::kVTile + C::kMetaTile;
        // {h, z} of (token, group) as floats: a half2, or two E4M3 bytes (every E4M3 value is an fp16 value)
        auto load_hz = [&](const uint8_t *base, int idx) -> float2 {
            if constexpr (F8) {
                uint32_t r;
                asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(reinterpret_cast<const uint16_t *>(base)[idx]));
                return __half22float2(*reinterpret_cast<const __half2 *>(&r));
            } else {
                return __half22float2(reinterpret_cast<const __half2 *>(base)[idx]);
            }
        };
        const int tok0 = q_begin + (warp + i * kWarps) * T;

        // ---------------- scores: exact integer dot products sum_j q'_j c_j per (token, group)
#pragma unroll
        for (int mt = 0; mt < T / 16; ++mt) {
            uint32_t w0[8], w1[8];      // this lane's words of token rows 16mt+g and 16mt+g+8, two per k-step
            if constexpr (KB == 2) {
                const uint4 *r0 = reinterpret_cast<const uint4 *>(Kc + (16 * mt + g) * KROW);
                const uint4 *r1 = reinterpret_cast<const uint4 *>(Kc + (16 * mt + g + 8) * KROW);
                const uint4 x0a = r0[0], x0b = r0[1], x1a = r1[0], x1b = r1[1];
                w0[0] = x0a.x; w0[1] = x0a.y; w0[2] = x0a.z; w0[3] = x0a.w; w0[4] = x0b.x; w0[5] = x0b.y; w0[6] = x0b.z; w0[7] = x0b.w;
                w1[0] = x1a.x; w1[1] = x1a.y; w1[2] = x1a.z; w1[3] = x1a.w; w1[4] = x1b.x; w1[5] = x1b.y; w1[6] = x1b.z; w1[7] = x1b.w;
            } else {
                // words 4ks + 2(t>>1) and +1 of each k-step: one 8-byte load per k-step and row
                const uint2 *r0 = reinterpret_cast<const uint2 *>(Kc + (16 * mt + g) * KROW) + (t >> 1);
                const uint2 *r1 = reinterpret_cast<const uint2 *>(Kc + (16 * mt + g + 8) * KROW) + (t >> 1);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const uint2 x0 = r0[2 * ks], x1 = r1[2 * ks];
                    w0[2 * ks] = x0.x; w0[2 * ks + 1] = x0.y;
                    w1[2 * ks] = x1.x; w1[2 * ks + 1] = x1.y;
                }
            }
            int acc[NG][4];
#pragma unroll
            for (int gg = 0; gg < NG; ++gg)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[gg][e] = 0;
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                // byte bb of (word & kmask) = weight * code: four channels per AND, no shift
                const uint32_t a0 = w0[2 * ks] & kmask, a1 = w1[2 * ks] & kmask;
                const uint32_t a2 = w0[2 * ks + 1] & kmask, a3 = w1[2 * ks + 1] & kmask;
                if constexpr (UNEQ) {
                    if ((kmap >> (2 * ks)) & 1u) imma16832(acc[1], a0, a1, a2, a3, bq[ks][0], bq[ks][1]);
                    else imma16832(acc[0], a0, a1, a2, a3, bq[ks][0], bq[ks][1]);
                } else {
                    imma16832(acc[(32 * ks) / G], a0, a1, a2, a3, bq[ks][0], bq[ks][1]);
                }
            }
            // lane (g,t) holds columns 2t, 2t+1 = two adjacent digits for tokens 16mt+g and 16mt+g+8
            if (t < 2) {
#pragma unroll
                for (int gg = 0; gg < NG; ++gg) {
                    const float lo = fmaf((float)acc[gg][1], 256.0f, (float)acc[gg][0]);
                    const float hi = fmaf((float)acc[gg][3], 256.0f, (float)acc[gg][2]);
                    Sc[((16 * mt + g) * NG + gg) * 2 + t] = lo;
                    Sc[((16 * mt + g + 8) * NG + gg) * 2 + t] = hi;
                }
            }
        }
        __syncwarp();

        // ---------------- softmax bookkeeping: lane owns tokens lane (and lane+32) of the tile
        float sc[T / 32];
        float hv[T / 32][NG], zv[T / 32][NG];
        // does any score exceed the running maximum, or any scale the running bound (or are the int32 sums getting full)?
        bool moved = ++tiles_since_fold * T >= 32768;
#pragma unroll
        for (int hf = 0; hf < T / 32; ++hf) {
            const int tau = lane + 32 * hf;
            const bool valid = (tok0 + tau) < q_end && (tok0 + tau) >= s.n_sink;      // sinks belong to the merge kernel
            float sv = 0.f;
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) {
                const float2 kz = load_hz(Km, tau * NG + gg);
                const float2 vz = load_hz(Vm, tau * NG + gg);
                hv[hf][gg] = valid ? vz.x : 0.f;      // rows past the end hold unspecified bytes
                zv[hf][gg] = valid ? vz.y : 0.f;
                moved |= (hv[hf][gg] >= h_bound);
                const float2 lh = *reinterpret_cast<const float2 *>(Sc + (tau * NG + gg) * 2);
                const float u = fmaf(lh.y, 65536.0f, lh.x) * cFr;      // scale * sum_j q'_j c_j
                sv = fmaf(kz.x, u, sv);
                sv = fmaf(kz.y, sqr[gg], sv);
            }
            sc[hf] = valid ? sv : -CUDART_INF_F;
            moved |= (sc[hf] > m_run);
        }
        if (__any_sync(0xffffffffu, moved)) {
            // Rare after the first tiles: raise the references and bring every running sum onto them.
            float tmx = sc[0], hm = 0.f;
#pragma unroll
            for (int hf = 0; hf < T / 32; ++hf) {
                tmx = fmaxf(tmx, sc[hf]);
#pragma unroll
                for (int gg = 0; gg < NG; ++gg) hm = fmaxf(hm, hv[hf][gg]);
            }
            const float m_new = fmaxf(m_run, warp_max(tmx));
            // 0 on the first tile (m_run = -inf); nothing to rescale while every token so far was masked
            const float corr = m_new == -CUDART_INF_F ? 1.f : ex2_approx(m_run - m_new);
            m_run = m_new;
            l_part *= corr;
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) z_part[gg] *= corr;
            hm = warp_max(hm);
            // fold the integer sums into cv: value = iacc * 256^digit * h_bound * 2^-32, columns 2t, 2t+1 = digits 2(t&1), +1
            const float f0 = h_bound * ((t & 1) ? 1.52587890625e-05f : 2.3283064365386963e-10f);   // 2^-16 : 2^-32
            const float f1 = f0 * 256.0f;
#pragma unroll
            for (int f = 0; f < 8; ++f) {
                cv[f][0] = fmaf((float)iacc[f][0], f0, cv[f][0]) * corr;
                cv[f][1] = fmaf((float)iacc[f][1], f1, cv[f][1]) * corr;
                cv[f][2] = fmaf((float)iacc[f][2], f0, cv[f][2]) * corr;
                cv[f][3] = fmaf((float)iacc[f][3], f1, cv[f][3]) * corr;
                iacc[f][0] = 0; iacc[f][1] = 0; iacc[f][2] = 0; iacc[f][3] = 0;
                tiles_since_fold = 0;
            }
            if (hm >= h_bound) h_bound = __int_as_float(((__float_as_int(hm) >> 23) + 1) << 23);   // next power of two above hm
        }
        {
            // P operand (u8): p*h on a 32-bit fixed-point grid below h_bound; the four bytes of that integer are
            // the four digit columns of the group.  Token tau is k index (tau & 31) of k-block tau >> 5.
            const float hscale = 4294967296.0f / h_bound;
#pragma unroll
            for (int hf = 0; hf < T / 32; ++hf) {
                // 0 for tokens past the end and for attention sinks (also while m_run is still -inf)
                const float p = sc[hf] == -CUDART_INF_F ? 0.f : ex2_approx(sc[hf] - m_run);
                l_part += p;
                uint8_t *dst = Pb + (hf * 8 * 4 + ((lane >> 2) & 3)) * 8 + (lane >> 4) * 4 + (lane & 3);
#pragma unroll
                for (int gg = 0; gg < NG; ++gg) {
                    uint32_t fx;
                    asm("cvt.rni.sat.u32.f32 %0, %1;" : "=r"(fx) : "f"(p * hv[hf][gg] * hscale));
                    z_part[gg] = fmaf(p, zv[hf][gg], z_part[gg]);
#pragma unroll
                    for (int dg = 0; dg < 4; ++dg) dst[(gg * 4 + dg) * 32] = (uint8_t)(fx >> (8 * dg));
                }
            }
        }
        __syncwarp();

        // ---------------- P.V in int8: rows = byte columns of the V rows, k = 32 tokens per MMA
        {
            const uint32_t vaddr = smem_u32(Vc) + lane * VROW;   // lanes 0-15: tokens 0-15, lanes 16-31: tokens 16-31
#pragma unroll
            for (int kk = 0; kk < T / 32; ++kk) {
                const uint2 pb = *reinterpret_cast<const uint2 *>(Pb + ((kk * 8 + g) * 4 + t) * 8);
#pragma unroll
                for (int hh = 0; hh < VROW / 16; ++hh) {
                    uint32_t rr[4];
                    ldmatrix_b8_trans_x2(rr, vaddr + kk * 32 * VROW + hh * 16);
#pragma unroll
                    for (int j = 0; j < C::VCPB; ++j) {
                        const uint32_t m = VBE == 2 ? (0x03030303u << (2 * j)) : (0x0F0F0F0Fu << (4 * j));
                        imma16832_uu(iacc[hh * C::VCPB + j], rr[0] & m, rr[1] & m, rr[2] & m, rr[3] & m, pb.x, pb.y);
                    }
                }
            }
        }
        __syncwarp();   // every lane is done with this stage, Sc and the P tile
        if (lane == 0 && i + C::kStages < n_my) issue(i + C::kStages);
    }

    if (failed) {
        // Drain (bounded) whatever copies are still in flight into this warp's stages, then report.
        for (int i2 = 0; i2 < n_my; ++i2) {
            const int st = (tiles_done + i2) % C::kStages;
            (void)mbar_wait_bounded(bar0 + 8 * st, ((tiles_done + i2) / C::kStages) & 1u);
        }
        if (lane == 0 && a.c.status) atomicOr(a.c.status, SKVQ_STATUS_COPY_TIMEOUT);
        m_run = -CUDART_INF_F;
        l_part = 0.f;
    }

    // ---- per-warp result: o'[channel] in the (now idle) stage area
    float *Ot = reinterpret_cast<float *>(stage_base);                       // [NG][128]
    float *Ow = Ot + NG * kHeadDim;                                          // [132]: o', m, l
    __syncwarp();
    l_part = warp_sum(l_part);
#pragma unroll
    for (int gg = 0; gg < NG; ++gg) z_part[gg] = warp_sum(z_part[gg]);
    {
        // last fold of the integer sums, then add the four digit columns of each group: a lane pair (t, t^1) holds them
        const float f0 = h_bound * ((t & 1) ? 1.52587890625e-05f : 2.3283064365386963e-10f);
        const float f1 = f0 * 256.0f;
#pragma unroll
        for (int f = 0; f < 8; ++f) {
            float lo = fmaf((float)iacc[f][0], f0, cv[f][0]) + fmaf((float)iacc[f][1], f1, cv[f][1]);   // byte column 16(f/VCPB)+g
            float hi = fmaf((float)iacc[f][2], f0, cv[f][2]) + fmaf((float)iacc[f][3], f1, cv[f][3]);   // byte column +8
            lo += __shfl_xor_sync(0xffffffffu, lo, 1);
            hi += __shfl_xor_sync(0xffffffffu, hi, 1);
            // lanes t = 0,1 carry group 0, lanes t = 2,3 group 1; the even lane of each pair stores
            const int gg = t >> 1;
            if ((t & 1) == 0 && gg < NG) {
                const int bc = (f / C::VCPB) * 16 + g, j = f % C::VCPB;
                Ot[gg * kHeadDim + C::VCPB * bc + j] = lo;
                Ot[gg * kHeadDim + C::VCPB * (bc + 8) + j] = hi;
            }
        }
        __syncwarp();
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
            const int d = lane + 32 * q4;
            const int j = d % C::VCPB;                                 // channel d = VCPB*(byte column) + j carries weight 2^(VB*j)
            const float winv = __int_as_float((127 - VBE * j) << 23);
            const int gd = UNEQ ? (int)((vmap >> (2 * (d >> 5))) & 1u) : d / G;      // group of channel d
            float zg = 0.f;
#pragma unroll
            for (int gg = 0; gg < NG; ++gg)
                if (gd == gg) zg = z_part[gg];
            const float o = Ot[gd * kHeadDim + d] * winv + zg;
            Ow[d] = failed ? 0.f : o;
        }
    }
    if (lane == 0) {
        Ow[kHeadDim] = m_run;
        Ow[kHeadDim + 1] = l_part;
    }
    __syncthreads();

    // ---- merge the four warps and write one partial
    {
        float M = -CUDART_INF_F;
        const float *ow[kWarps];
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            ow[w] = reinterpret_cast<const float *>(smem + C::kQBytes + w * C::kWarpBytes) + NG * kHeadDim;
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
        float *dst = partials + (((size_t)b * s.Hq + hk) * n_parts + part) * kPartialStride;
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

template <int G, int KB, int VB, bool F8, bool UNEQ>
cudaError_t launch_one(const MmaArgs &a, cudaStream_t stream, bool overlap)
{
    using C = Cfg<G, KB, VB, F8>;
    static unsigned long long configured = 0;      // one bit per device
    auto kern = partition_mma_kernel<G, KB, VB, F8, UNEQ>;
    const cudaError_t ec = configure_smem_once(kern, C::kSmemBytes, configured);
    if (ec != cudaSuccess) return ec;
    return launch_dependent(kern, dim3(a.plan.n_slots), dim3(kThreads), C::kSmemBytes, stream, overlap, a);
}

template <int G, bool F8, bool UNEQ>
cudaError_t launch_g(const MmaArgs &a, cudaStream_t stream, bool overlap)
{
    if (a.s.k_bits == 2)
        return a.s.v_bits == 2 ? launch_one<G, 2, 2, F8, UNEQ>(a, stream, overlap)
             : a.s.v_bits == 4 ? launch_one<G, 2, 4, F8, UNEQ>(a, stream, overlap) : launch_one<G, 2, kTernary, F8, UNEQ>(a, stream, overlap);
    return a.s.v_bits == 2 ? launch_one<G, 4, 2, F8, UNEQ>(a, stream, overlap)
         : a.s.v_bits == 4 ? launch_one<G, 4, 4, F8, UNEQ>(a, stream, overlap) : launch_one<G, 4, kTernary, F8, UNEQ>(a, stream, overlap);
}

}  // namespace

// Launches the integer kernel when the configuration is covered (one query head per KV head, 2- or 4-bit codes, G = 64 or
// 128; groups of unequal width with two groups per row); *handled tells the caller whether it did.
cudaError_t launch_partition_mma(const Shape &s, const CachePtrs &c, const __half *q, float scale_log2,
                                 const SplitPlan &plan, float *workspace, cudaStream_t stream, bool overlap, bool *handled)
{
    *handled = false;
    if (s.rep != 1 || (s.G != 64 && s.G != 128) || !plain_width(s.k_bits) || !(plain_width(s.v_bits) || s.v_bits == kTernary)) return cudaSuccess;
    if (s.bounded && s.G != 64) return cudaSuccess;
    MmaArgs a{s, c, q, scale_log2, plan, workspace};
    *handled = true;
    if (s.bounded) return s.meta_fp8 ? launch_g<64, true, true>(a, stream, overlap) : launch_g<64, false, true>(a, stream, overlap);
    if (s.meta_fp8) return s.G == 128 ? launch_g<128, true, false>(a, stream, overlap) : launch_g<64, true, false>(a, stream, overlap);
    return s.G == 128 ? launch_g<128, false, false>(a, stream, overlap) : launch_g<64, false, false>(a, stream, overlap);
}

}  // namespace skvq

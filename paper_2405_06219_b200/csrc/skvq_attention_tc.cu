// Partition kernel of skvq_decode_attention on the fifth-generation tensor cores (tcgen05.mma, accumulators in
// tensor memory) for 2-, 3- or 4-bit K and V in any mix and three-level ("1.5-bit") V, up to 4 query heads per KV head
// per launch, any group size and groups of unequal width (Eq. 1, Algorithm 1); scale and zero point stored as fp16 pairs
// or as E4M3 byte pairs.  It is
// the general tensor-core path: whatever the two mma.sync kernels do not cover runs here.
//
//   q'.K~_t            = sum_g h_{t,g} (sum_{j in g} q'_j c_{t,j}) + sum_g z_{t,g} (sum_{j in g} q'_j)
//   sum_t p_t V~_{t,d} = sum_t (p_t h_{t,g(d)}) c_{t,d} + sum_t p_t z_{t,g(d)}
//
// One CTA = 128 token threads (one tile of 128 tokens at a time, one thread per token) and one control warp; three
// CTAs per SM (128 tensor-memory columns and 69 KB of shared memory each).  The token threads only unpack and do the
// per-(token, head, group) arithmetic; both contractions run asynchronously on the tensor core:
//   * a thread turns its token's packed row into 128 bytes "weight * code" -- one AND per four codes for 2- and 4-bit
//     codes (weights 4^j and 16^j: the codes stay where they are in the word), shifts for the 3-bit stream (weight 1) --
//     and stores them as a row of the A operand of the score MMA (u8, K-major).  The B operand holds the permuted query of every head
//     as four signed byte digits of a 31-bit fixed-point number with the weight 4^j divided out, so the int32
//     accumulators are the exact group dot products: one MMA k-step (32 channels) per 32 channels, a fresh set of
//     16 columns (head, digit) per quantization group.
//   * the thread reads its row of accumulators from tensor memory, combines digits and groups with h and z (fp32),
//     and takes part in a lazy online softmax: the reference of a head moves only when a score exceeds it by 8 in
//     the log2 domain (or the bound on the value scales has to grow), which after the first tiles is rare.
//   * p*h per (head, group) goes onto a 32-bit fixed-point grid; the four bytes of that integer are four columns
//     (group, head, digit) of the B operand of the value MMA (u8, MN-major: one 16-byte store per group and token),
//     whose A operand is the V tile unpacked like K (u8, MN-major): 128 byte columns of V on the M rows x 64 columns
//     of exact int32 sums in tensor memory.  The thread that owns tensor-memory lane c folds the 16 columns of
//     channel c's group into fp32 when the reference moves, every 256 tiles, and at the end of a segment.
//   * the control warp issues every copy and every MMA in the order in which the token threads finish the operands:
//     they arrive on an mbarrier (behind fence.proxy.async), the control lane waits, issues, and commits the MMAs to
//     the mbarrier the token threads wait on.
// K codes are needed one tile before the rest of a tile, so they have a copy ring of their own (cp.async.bulk,
// mbarrier completion); every wait is bounded and reports through the cache's status word; the tensor memory is
// given back on every exit path.
#include "skvq_mma_common.cuh"
#include "skvq_tcgen05.cuh"

namespace skvq {
namespace {

using namespace mmak;
using namespace tc5;

constexpr int kTile = 128;              // tokens per tile = rows of the score MMA = threads per CTA
constexpr int kHeads = 4;               // query heads per KV head served (absent heads carry a zero query)
constexpr int kSlackLog2 = 8;           // the softmax reference moves only when a score exceeds it by this (log2)
constexpr int kRing = 2;                // slots of each of the two copy rings
constexpr int kTmemCols = 128;          // allocation: scores in columns [0, 64), value sums in [64, 128)
constexpr int kScoreCol = 0, kPvCol = 64;
constexpr int kFoldTiles = 256;         // 255 * 240 * 128 * 256 < 2^31: the int32 value sums are folded at least this often
constexpr uint32_t kLbo = 128;          // bytes between core matrices along K (all operands)
constexpr uint32_t kSboK = 1024;        // K-major operands: bytes between groups of 8 rows
constexpr uint32_t kSboMN = 2048;       // MN-major operands: bytes between 16-byte chunks of the M/N extent (128 tokens)

// Shared memory.  The K codes of a tile are needed one tile before everything else of it (its score MMA is issued
// that far ahead), so they travel in a ring of their own.
template <int G, int KB, int VB>
struct TCfg {
    static constexpr int NG = kHeadDim / G;
    static constexpr int kKRow = packed_row_bytes(KB), kVRow = packed_row_bytes(VB);   // bytes per packed token row
    static constexpr int kKTile = kTile * kKRow, kVTile = kTile * kVRow;
    static constexpr int kMetaTile = kTile * NG * 4;                     // room for half2 pairs; E4M3 pairs use half of it
    static constexpr int kVmBytes = kVTile + 2 * kMetaTile;              // V codes, K scale/zero, V scale/zero
    static constexpr int kOffVm = kRing * kKTile;
    static constexpr int kOffKA = kOffVm + kRing * kVmBytes;             // A of the score MMA: [128 tokens][128 bytes]
    static constexpr int kOffQB = kOffKA + kTile * 128;                  // B of the score MMA: [16 (head, digit)][128 bytes]
    // A of the value MMA: [128 tokens][128 byte columns].  Where both operand buffers would leave room for only two CTAs
    // per SM (the wider codes), it lives in the buffer of A of the score MMA: the two are built and consumed in turn (K of
    // tile i+1 in the middle of tile i, V of tile i at its end), each once the MMA that read the other has completed
    // (measured: the third CTA is worth 9-14 %, the extra waits cost 2 %).
    static constexpr bool kShared = tc_shared_operand(G, KB, VB);
    static constexpr int kOffVB = kShared ? kOffKA : kOffQB + 16 * 128;
    static constexpr int kOffPA = kShared ? kOffQB + 16 * 128 : kOffVB + kTile * 128;      // B of the value MMA: [128 tokens][64 (group, head, digit)]
    static constexpr int kOffOs = kOffPA + kTile * 64;                   // folded value sums [4][128] fp32, by byte column
    static constexpr int kOffMisc = kOffOs + kHeads * kHeadDim * 4;      // small arrays, see the kernel
    static constexpr int kSmemBytes = kOffMisc + 1024;
    static constexpr int kCtasPerSm = kTcCtasPerSm;                      // by shared memory (at most 73 KB)
    static_assert(kSmemBytes <= 74752, "three CTAs per SM");
    static_assert(kSmemBytes == tc_smem_bytes(G, KB, VB), "the host sizes the grid from the same figure");
    static_assert(kTile * 128 >= kHeads * kHeadDim * 4, "the V operand buffer doubles as query scratch in the prologue");
    static_assert(kKTile % 16 == 0 && kVTile % 16 == 0, "bulk copies move multiples of 16 bytes");
};

__device__ __forceinline__ uint32_t to_fixed_u32(float x)
{
    uint32_t r;
    asm("cvt.rni.sat.u32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float lo_half(uint32_t w) { return __low2float(*reinterpret_cast<const __half2 *>(&w)); }
__device__ __forceinline__ float hi_half(uint32_t w) { return __high2float(*reinterpret_cast<const __half2 *>(&w)); }

template <int NG>
__device__ __forceinline__ void load_words32(const uint32_t *p, uint32_t (&w)[NG])
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

// The {h, z} words of one token as fp16 pairs, from fp16 pairs or (f8) from E4M3 byte pairs; tile = the token rows as
// they lie in the cache (NG pairs per token).
template <int NG>
__device__ __forceinline__ void load_words(const uint8_t *tile, int tok, bool f8, uint32_t (&w)[NG])
{
    if (f8) {
        const uint8_t *p = tile + tok * NG * 2;
        uint16_t b[NG];
        if constexpr (NG == 4) {
            const uint2 x = *reinterpret_cast<const uint2 *>(p);
            b[0] = (uint16_t)x.x; b[1] = (uint16_t)(x.x >> 16); b[2] = (uint16_t)x.y; b[3] = (uint16_t)(x.y >> 16);
        } else if constexpr (NG == 2) {
            const uint32_t x = *reinterpret_cast<const uint32_t *>(p);
            b[0] = (uint16_t)x; b[1] = (uint16_t)(x >> 16);
        } else {
            b[0] = *reinterpret_cast<const uint16_t *>(p);
        }
#pragma unroll
        for (int i = 0; i < NG; ++i) asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(w[i]) : "h"(b[i]));
    } else {
        load_words32<NG>(reinterpret_cast<const uint32_t *>(tile + tok * NG * 4), w);
    }
}

// One token's packed row -> 128 bytes "weight * code", one per channel, in eight chunks of 16 byte columns; chunk i goes
// to dst + i * chunk_stride.  Which channel and which weight a byte column carries: column_channel / column_shift.
//   2 bits: chunk i = word i under the four masks 0x03030303 << 2j: byte 16i + 4j + b = code j + 4b of the word, times 4^j.
//   4 bits: chunk i = words 2i, 2i+1 under the masks 0x0F0F0F0F, 0xF0F0F0F0: byte 16i + 8v + 4j + b = code 2b + j of word
//           2i + v, times 16^j.
//   3 bits: the row is a bit stream; chunk i = channels 16i .. 16i+15 in order, four 3-bit fields spread into the four
//           bytes of a register (weight 1).
template <int BITS>
__device__ __forceinline__ void unpack_row(const uint8_t *packed, uint8_t *dst, uint32_t chunk_stride)
{
    constexpr int NW = kHeadDim * BITS / 32;
    uint32_t w[NW];
#pragma unroll
    for (int i = 0; i < NW / 4; ++i) {
        const uint4 x = *reinterpret_cast<const uint4 *>(packed + 16 * i);
        w[4 * i] = x.x; w[4 * i + 1] = x.y; w[4 * i + 2] = x.z; w[4 * i + 3] = x.w;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        uint4 o;
        if constexpr (BITS == 2) {
            o = make_uint4(w[i] & 0x03030303u, w[i] & 0x0C0C0C0Cu, w[i] & 0x30303030u, w[i] & 0xC0C0C0C0u);
        } else if constexpr (BITS == 4) {
            o = make_uint4(w[2 * i] & 0x0F0F0F0Fu, w[2 * i] & 0xF0F0F0F0u, w[2 * i + 1] & 0x0F0F0F0Fu, w[2 * i + 1] & 0xF0F0F0F0u);
        } else {
            uint32_t r[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int p = 48 * i + 12 * k, wi = p >> 5, sh = p & 31;      // twelve stream bits from bit p on
                uint32_t f = w[wi] >> sh;
                if (sh > 20) f |= w[wi + 1] << (32 - sh);                      // never past the row: p + 12 <= 384
                f &= 0xFFFu;
                r[k] = (f & 0x7u) | ((f & 0x38u) << 5) | ((f & 0x1C0u) << 10) | ((f & 0xE00u) << 15);
            }
            o = make_uint4(r[0], r[1], r[2], r[3]);
        }
        *reinterpret_cast<uint4 *>(dst + i * chunk_stride) = o;
    }
}

// Three-level codes: one token's 26 bytes (five base-3 digits each; the row is only 2-byte aligned) -> 128 code bytes in
// channel order (weight 1), through a table of the five digits of every byte value: lut[v] = {digits 0-3 in the four
// bytes of .x, digit 4 in the low byte of .y}.  The table's 5-byte pieces are joined into 4-byte registers by byte
// permutes whose selectors are compile-time constants after unrolling.
__device__ __forceinline__ void unpack_row_ternary(const uint8_t *packed, uint8_t *dst, uint32_t chunk_stride, const uint2 *lut)
{
    constexpr int NB = packed_row_bytes(kTernary);      // 26
    uint32_t lo[NB], hi[NB];
    const uint16_t *p = reinterpret_cast<const uint16_t *>(packed);
#pragma unroll
    for (int i = 0; i < NB / 2; ++i) {
        const uint32_t two = p[i];
        const uint2 e0 = lut[two & 255u], e1 = lut[two >> 8];
        lo[2 * i] = e0.x; hi[2 * i] = e0.y;
        lo[2 * i + 1] = e1.x; hi[2 * i + 1] = e1.y;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        uint32_t r[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int pos = 16 * i + 4 * k, n = pos / 5, off = pos % 5;      // channels pos .. pos+3 = digits off .. of byte n, then of byte n+1
            const int n1 = n + 1 < NB ? n + 1 : n;                          // off > 1 implies n + 1 < NB (pos + 3 <= 127)
            r[k] = off == 0 ? lo[n]
                 : off == 1 ? __byte_perm(lo[n], hi[n], 0x4321)
                 : off == 2 ? __byte_perm(__byte_perm(lo[n], hi[n], 0x0432), lo[n1], 0x4210)
                 : off == 3 ? __byte_perm(__byte_perm(lo[n], hi[n], 0x0043), lo[n1], 0x5410)
                            : __byte_perm(hi[n], lo[n1], 0x6540);
        }
        *reinterpret_cast<uint4 *>(dst + i * chunk_stride) = make_uint4(r[0], r[1], r[2], r[3]);
    }
}

// Channel and weight exponent of byte column n of an unpacked row (the K index of the score MMA, the M index of the
// value MMA).  A 32-column block always holds the 32 channels of one granule, whatever the width.
template <int BITS>
__device__ __forceinline__ int column_channel(int n)
{
    if constexpr (BITS == 2) return 16 * (n >> 4) + ((n >> 2) & 3) + 4 * (n & 3);
    else if constexpr (BITS == 4) return 16 * (n >> 4) + 8 * ((n >> 3) & 1) + 2 * (n & 3) + ((n >> 2) & 1);
    else return n;
}
template <int BITS>
__device__ __forceinline__ int column_shift(int n)
{
    if constexpr (BITS == 2) return 2 * ((n >> 2) & 3);
    else if constexpr (BITS == 4) return 4 * ((n >> 2) & 1);
    else return 0;
}

// Barrier 1: the 128 token threads only (the control warp never joins it).
__device__ __forceinline__ void token_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ int token_sync_or(int pred)
{
    int out;
    asm volatile("{\n .reg .pred p, q;\n setp.ne.u32 q, %1, 0;\n bar.red.or.pred p, 1, 128, q;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(out) : "r"(pred) : "memory");
    return out;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

template <int G, int KB, int VB>
__global__ void __launch_bounds__(kTile + 32, TCfg<G, KB, VB>::kCtasPerSm) partition_tc_kernel(MmaArgs a)
{
    using C = TCfg<G, KB, VB>;
    constexpr int NG = C::NG;
    const bool f8 = a.s.meta_fp8 != 0;                    // scale/zero as E4M3 byte pairs
    const int meta_row = NG * (f8 ? 2 : 4);               // bytes of scale/zero per token and tensor
    extern __shared__ __align__(128) uint8_t smem[];
    const Shape &s = a.s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool control = warp == kWarps;      // warp 4 issues every copy and MMA; warps 0-3 own one token each
    const int R = min(kHeads, s.rep - a.head0);      // query heads of every KV head served by this launch
    // Order matters: the merge kernel reads the lengths, the sinks and the window BEFORE its own wait, so it may only be
    // scheduled once everything in front of this grid (append, bookkeeping, plan) has completed and is visible.  Waiting
    // first and triggering afterwards gives exactly that; the merge kernel still runs under this kernel's body.
    asm volatile("griddepcontrol.wait;" ::: "memory");      // the lengths, and the plan kernel's header when there is one
    asm volatile("griddepcontrol.launch_dependents;");      // the merge kernel may start its window part now

    __shared__ __align__(16) Segment seg_sh;
    __shared__ int more_sh;
    __shared__ int fail_sh;
    __shared__ int fresh_sh;         // does the next value MMA overwrite the accumulators?
    __shared__ uint32_t tmem_sh;
    __shared__ SlotWalker walk;      // only thread 0 touches it
    __shared__ __align__(16) int hdr_sh[kPlanSmemInts];
    __shared__ uint2 digits_sh[VB == kTernary ? 256 : 1];      // the five base-3 digits of every byte value
    if constexpr (VB == kTernary) {
        for (int v = tid; v < 256; v += kTile + 32)
            digits_sh[v] = make_uint2((v % 3) | ((v / 3 % 3) << 8) | ((v / 9 % 3) << 16) | ((v / 27 % 3) << 24), v / 81);
    }
    if (a.plan.in_kernel) {
        if (warp == 0) plan_in_warp(a.c.lengths, s.B, s.Hkv, s.W, a.plan.lq_cap, a.plan.n_slots, hdr_sh);
        __syncthreads();
    }
    if (tid == 0) {
        more_sh = walk.start(a.plan.in_kernel ? hdr_sh : reinterpret_cast<const int *>(a.ws), !a.plan.in_kernel, s.B, s.Hkv,
                             blockIdx.x) ? 1 : 0;
        fail_sh = 0;
    }
    __syncthreads();
    if (!more_sh) return;
    float *partials = a.ws + a.plan.hdr_ints;

    // ---- shared memory
    uint8_t *QB = smem + C::kOffQB, *VOp = smem + C::kOffVB;
    float *Os = reinterpret_cast<float *>(smem + C::kOffOs);         // [4][128] by MMA column
    float *qs = reinterpret_cast<float *>(VOp);                      // [4][128] permuted query (prologue only)
    float *sqs_sh = reinterpret_cast<float *>(smem + C::kOffMisc);   // [4][4]  sm_scale*log2(e) * sum_{j in g} q'_j
    float *csc_sh = sqs_sh + 16;                                     // [4]     sm_scale*log2(e) * 2^(e_r - 30)
    int *fexp = reinterpret_cast<int *>(csc_sh + 4);                 // [4]
    float *red = reinterpret_cast<float *>(fexp + 4);                // [4 warps][24] reductions
    uint64_t *bars = reinterpret_cast<uint64_t *>(red + kWarps * 24);
    const uint32_t bar_k = smem_u32(bars);            // [kRing] K codes landed (copy)
    const uint32_t bar_v = bar_k + 8 * kRing;         // [kRing] V codes and scale/zero landed (copy)
    const uint32_t bar_s = bar_v + 8 * kRing;         // score MMA done (tcgen05.commit)
    const uint32_t bar_pv = bar_s + 8;                // value MMA done (tcgen05.commit)
    const uint32_t bar_ka = bar_pv + 8;               // A operand of a score MMA built (128 token threads)
    const uint32_t bar_pa = bar_ka + 8;               // operands of a value MMA built (128 token threads)

    // ---- tensor memory and barriers (once per CTA)
    if (control) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_sh)), "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        if (lane == 0) {
#pragma unroll
            for (int i = 0; i < 2 * kRing + 2; ++i) mbar_init(bar_k + 8 * i, 1);
            mbar_init(bar_ka, kTile);
            mbar_init(bar_pa, kTile);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            proxy_fence();
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_sh;
    const uint32_t tmem_row = tmem + ((uint32_t)((warp & 3) * 32) << 16);      // this warp's 32 lanes

    constexpr uint32_t kIdescS = idesc_i8(128, 16, false, true, false, false);
    constexpr uint32_t kIdescPV = idesc_i8(128, 64, false, false, true, true);

    // kernel-lifetime pipeline counters (every thread counts alike)
    uint32_t tiles_done = 0;           // tiles that went through the rings
    uint32_t s_count = 0;              // score MMAs of finished segments (buffer and barrier phase follow from the index)
    uint32_t pv_count = 0;             // value MMAs of finished segments
    bool failed = false;

    for (;;) {
    if (tid == 0) seg_sh = walk.next(a.c.lengths, s.W, a.plan.lq_cap);
    __syncthreads();
    const int b = seg_sh.b, hk = seg_sh.hk, q_begin = seg_sh.tok_begin, q_end = seg_sh.tok_end, part = seg_sh.part;
    if (!segment_in_bounds(seg_sh, s, a.plan, a.c.status)) break;      // checked build only; uniform: every thread reads the same segment
    const int n_parts = a.plan.s_max;
    const size_t bh = (size_t)b * s.Hkv + hk;
    const int n_tiles = failed ? 0 : (q_end - q_begin + kTile - 1) / kTile;

    // ---- CTA-wide prologue: permuted query per head on a power-of-two scale -> byte digits, group constants.
    // The control warp starts the first copies meanwhile.
    auto rows_of = [&](int i) { return (uint32_t)min(kTile, (q_end - (q_begin + i * kTile) + 63) & ~63); };
    auto issue_k = [&](int i) {       // control lane only (the cache's capacity is a multiple of 64 rows)
        const uint8_t *k_codes = a.c.k_codes + bh * (size_t)s.cap * C::kKRow;
        const uint32_t slot = (tiles_done + i) % kRing, rows = rows_of(i);
        mbar_expect_tx(bar_k + 8 * slot, rows * C::kKRow);
        bulk_g2s(smem_u32(smem + slot * C::kKTile), k_codes + (size_t)(q_begin + i * kTile) * C::kKRow, rows * C::kKRow,
                 bar_k + 8 * slot);
    };
    auto issue_v = [&](int i) {       // control lane only
        const uint8_t *v_codes = a.c.v_codes + bh * (size_t)s.cap * C::kVRow;
        const uint32_t kRowMeta = (uint32_t)meta_row;
        const uint8_t *k_meta = reinterpret_cast<const uint8_t *>(a.c.k_meta) + bh * (size_t)s.cap * kRowMeta;
        const uint8_t *v_meta = reinterpret_cast<const uint8_t *>(a.c.v_meta) + bh * (size_t)s.cap * kRowMeta;
        const uint32_t slot = (tiles_done + i) % kRing, rows = rows_of(i);
        const int tok0 = q_begin + i * kTile;
        const uint32_t dst = smem_u32(smem + C::kOffVm + slot * C::kVmBytes), bar = bar_v + 8 * slot;
        mbar_expect_tx(bar, rows * (C::kVRow + 2 * kRowMeta));
        bulk_g2s(dst, v_codes + (size_t)tok0 * C::kVRow, rows * C::kVRow, bar);
        bulk_g2s(dst + C::kVTile, k_meta + (size_t)tok0 * kRowMeta, rows * kRowMeta, bar);
        bulk_g2s(dst + C::kVTile + C::kMetaTile, v_meta + (size_t)tok0 * kRowMeta, rows * kRowMeta, bar);
    };
    auto wait_ring = [&](uint32_t bar0, int i) {
        const uint32_t t = tiles_done + i;
        if (!mbar_wait_bounded(bar0 + 8 * (t % kRing), (t / kRing) & 1u)) fail_sh = 1;
    };
    if (control) {
        if (lane == 0) {
            proxy_fence();   // the slots were read through the generic proxy by the previous segment
            for (int i = 0; i < kRing && i < n_tiles; ++i) { issue_k(i); issue_v(i); }
        }
    } else {
        const int32_t *idx_k = a.c.reorder_k + (size_t)hk * kHeadDim;
        const int src = idx_k[tid] & (kHeadDim - 1);
#pragma unroll
        for (int r = 0; r < kHeads; ++r) {
            const float qv = r < R ? __half2float(a.q[((size_t)b * s.Hq + hk * s.rep + a.head0 + r) * kHeadDim + src]) : 0.f;
            qs[r * kHeadDim + tid] = qv;
            const float wm = warp_max(fabsf(qv));
            if (lane == 0) red[warp * 24 + r] = wm;
        }
        Os[tid] = 0.f; Os[kHeadDim + tid] = 0.f; Os[2 * kHeadDim + tid] = 0.f; Os[3 * kHeadDim + tid] = 0.f;
    }
    __syncthreads();
    if (tid < kHeads) {
        float qmax = 0.f;
        for (int w = 0; w < kWarps; ++w) qmax = fmaxf(qmax, red[w * 24 + tid]);
        int e = 0;
        if (qmax > 0.f) (void)frexpf(qmax, &e);            // qmax = m * 2^e, 0.5 <= m < 1: |q' * 2^-e| < 1
        fexp[tid] = e;
        csc_sh[tid] = ldexpf(a.scale_log2, e - 30);
    }
    // group of every 32-channel granule (two bits each): position / G, or the cache's boundaries
    const uint32_t kmap = granule_groups(a.c.bounds_k, hk, G, NG), vmap = granule_groups(a.c.bounds_v, hk, G, NG);
    if (tid >= 32 && tid < 32 + kHeads * NG) {
        const int r = (tid - 32) / NG, gg = (tid - 32) % NG;
        float sq = 0.f;
        for (int j = 0; j < kHeadDim; ++j)
            if ((int)((kmap >> (2 * (j >> 5))) & 3u) == gg) sq += qs[r * kHeadDim + j];
        sqs_sh[r * 4 + gg] = sq * a.scale_log2;
    }
    __syncthreads();

    if (control) {
        // ================================================================ control warp: one lane issues, in the order
        // in which the token threads finish the operands
        if (lane == 0 && n_tiles > 0) {
            const uint64_t dKA = smem_desc(smem_u32(smem + C::kOffKA), kLbo, kSboK), dQB = smem_desc(smem_u32(QB), kLbo, kSboK);
            const uint64_t dVB = smem_desc(smem_u32(VOp), kLbo, kSboMN), dPA = smem_desc(smem_u32(smem + C::kOffPA), kLbo, kSboMN);
            bool ok = true;
            auto scores = [&](int j) {      // score MMA of tile j, once its A operand is complete and the old scores are read
                const uint32_t n = s_count + j;
                if (!mbar_wait_bounded(bar_ka, n & 1u)) { ok = false; return; }
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {      // one k-step = one granule; a group's granules are consecutive
                    const uint32_t gk = (kmap >> (2 * ks)) & 3u;
                    const uint32_t acc = (ks > 0 && ((kmap >> (2 * (ks - 1))) & 3u) == gk) ? 1u : 0u;
                    umma_i8(tmem + kScoreCol + 16 * gk, dKA + ((ks * 2 * kLbo) >> 4), dQB + ((ks * 2 * kLbo) >> 4), kIdescS, acc);
                }
                umma_commit(bar_s);
                if (j + kRing < n_tiles) { proxy_fence(); issue_k(j + kRing); }      // the token threads are done with that slot
            };
            scores(0);
            for (int i = 0; i < n_tiles && ok; ++i) {
                if (i + 1 < n_tiles) scores(i + 1);
                if (!ok) break;
                const uint32_t n = pv_count + i;
                if (!mbar_wait_bounded(bar_pa, n & 1u)) { ok = false; break; }
                tc_fence_after();
                const uint32_t fresh = (uint32_t)fresh_sh;
                // channels on the M rows (the V tile as stored is the A operand), (group, head, digit) on the N columns
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    umma_i8(tmem + kPvCol, dVB + ((ks * 4 * kLbo) >> 4), dPA + ((ks * 4 * kLbo) >> 4), kIdescPV,
                            (fresh && ks == 0) ? 0u : 1u);
                umma_commit(bar_pv);
                if (i + kRing < n_tiles) { proxy_fence(); issue_v(i + kRing); }
            }
            if (!ok) fail_sh = 1;
        }
        __syncwarp();
    } else {
        // ================================================================ token threads
        {
            // thread = byte column k of the operand: channel column_channel(k), its weight divided out of the query
            const int ch = column_channel<KB>(tid), sh = column_shift<KB>(tid);
            uint8_t *col = QB + (tid >> 4) * kLbo + (tid & 15);
#pragma unroll
            for (int r = 0; r < kHeads; ++r) {
                int qi = __float2int_rn(ldexpf(qs[r * kHeadDim + ch], 30 - fexp[r] - sh));      // |qi| < 2^30
#pragma unroll
                for (int d = 0; d < 4; ++d) {
                    const int dg = d < 3 ? ((qi + 128) & 255) - 128 : qi;      // balanced digits: qi = sum dg * 256^d
                    qi = (qi - dg) >> 8;
                    const int n = 4 * r + d;
                    col[(n >> 3) * kSboK + (n & 7) * 16] = (uint8_t)(dg & 255);
                }
            }
        }
        float csc[kHeads], sqs[kHeads][NG];
#pragma unroll
        for (int r = 0; r < kHeads; ++r) {
            csc[r] = csc_sh[r];
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) sqs[r][gg] = sqs_sh[r * 4 + gg];
        }
        token_sync();      // the query scratch (in the V operand buffer) is dead from here on

        // running state: this thread's token of every tile, all four heads
        float m_ref[kHeads], l_sum[kHeads], zp[kHeads][NG];
#pragma unroll
        for (int r = 0; r < kHeads; ++r) {
            m_ref[r] = -CUDART_INF_F;
            l_sum[r] = 0.f;
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) zp[r][gg] = 0.f;
        }
        float h_bound = 6.103515625e-05f;      // power of two above every value scale seen so far (2^-14 to start with)
        float hscale = (float)(1u << (32 - kSlackLog2)) / h_bound;
        bool pv_fresh = true;                  // the next value MMA overwrites the accumulators
        int tiles_since_fold = 0;
        uint32_t pv_local = 0;                 // value MMAs of this segment handed to the control warp
        uint32_t pv_waited = 0;

        auto wait_pv = [&]() {                 // every value MMA handed over so far has completed
            if (pv_waited < pv_local) {
                if (!mbar_wait_bounded(bar_pv, (pv_count + pv_local - 1) & 1u)) fail_sh = 1;
                pv_waited = pv_local;
            }
        };
        // every thread: its token's row of tile i -> A operand of the score MMA, then tell the control warp
        auto build_k = [&](int i) {
            if (C::kShared) wait_pv();      // the value MMA of the tile before has read the buffer (as the V operand)
            wait_ring(bar_k, i);
            unpack_row<KB>(smem + ((tiles_done + i) % kRing) * C::kKTile + tid * C::kKRow,
                           smem + C::kOffKA + (tid >> 3) * kSboK + (tid & 7) * 16, kLbo);
            proxy_fence();
            mbar_arrive(bar_ka);
        };
        // Brings the int32 value sums into the fp32 sums in shared memory (relative to the old references and bound).
        // Only this thread touches column tid of Os.
        auto fold_pv = [&]() {
            wait_pv();
            tc_fence_after();
            if (!pv_fresh) {
                // tensor-memory lane tid = byte column tid of the V rows; its group's 16 columns are (head, digit)
                int v[16];
                tmem_ld16(tmem_row + kPvCol + 16 * ((vmap >> (2 * warp)) & 3u), v);      // the 32 byte columns of warp w are granule w
                tmem_wait_ld();
                const float sa = h_bound * (1.0f / (float)(1u << (32 - kSlackLog2)));
#pragma unroll
                for (int r = 0; r < kHeads; ++r) {
                    const float lo = fmaf((float)v[4 * r + 1], 256.0f, (float)v[4 * r]);
                    const float hi = fmaf((float)v[4 * r + 3], 256.0f, (float)v[4 * r + 2]);
                    Os[r * kHeadDim + tid] += fmaf(hi, 65536.0f, lo) * sa;
                }
            }
            tc_fence_before();
            pv_fresh = true;
            tiles_since_fold = 0;
        };

        if (n_tiles > 0) build_k(0);      // the first tile's K operand

        for (int i = 0; i < n_tiles; ++i) {
            const uint32_t n = s_count + i;
            const uint8_t *vm = smem + C::kOffVm + ((tiles_done + i) % kRing) * C::kVmBytes;
            const uint8_t *Km = vm + C::kVTile;                         // [128][NG] {h, z}
            const uint8_t *Vm = vm + C::kVTile + C::kMetaTile;
            uint8_t *PA = smem + C::kOffPA;
            const int tok = q_begin + i * kTile + tid;
            const bool valid = tok < q_end && tok >= s.n_sink;      // sinks belong to the merge kernel

            // ---------------- scores of this thread's token (the MMA was issued one tile ago)
            if (!mbar_wait_bounded(bar_s, n & 1u)) fail_sh = 1;
            tc_fence_after();
            // The accumulators are read in two halves: the second half is in flight while the first is combined, and
            // the next tile's K operand is built as soon as the last read has landed, so that its MMA runs under the rest.
            constexpr int H0 = NG > 1 ? NG / 2 : 1;      // groups in the first half
            int va[H0][16];
#pragma unroll
            for (int gg = 0; gg < H0; ++gg) tmem_ld16(tmem_row + kScoreCol + 16 * gg, va[gg]);
            wait_ring(bar_v, i);
            uint32_t kw[NG], vw[NG];
            load_words<NG>(Km, tid, f8, kw);
            load_words<NG>(Vm, tid, f8, vw);
            tmem_wait_ld();
            int vb[NG - H0 > 0 ? NG - H0 : 1][16];
#pragma unroll
            for (int gg = H0; gg < NG; ++gg) tmem_ld16(tmem_row + kScoreCol + 16 * gg, vb[gg - H0]);
            float sc[kHeads] = {0.f, 0.f, 0.f, 0.f}, zt[kHeads] = {0.f, 0.f, 0.f, 0.f};
            auto combine = [&](const int (&v)[16], int gg) {
                const float hk_ = lo_half(kw[gg]), zk_ = hi_half(kw[gg]);
#pragma unroll
                for (int r = 0; r < kHeads; ++r) {
                    const int lo = v[4 * r] + (v[4 * r + 1] << 8), hi = v[4 * r + 2] + (v[4 * r + 3] << 8);
                    const float u = fmaf((float)hi, 65536.0f, (float)lo);      // 2^30 * sum_j q'_j 2^-e c_j over the group
                    sc[r] = fmaf(hk_, u, sc[r]);
                    zt[r] = fmaf(zk_, sqs[r][gg], zt[r]);
                }
            };
#pragma unroll
            for (int gg = 0; gg < H0; ++gg) combine(va[gg], gg);
            tmem_wait_ld();
            tc_fence_before();
            if (i + 1 < n_tiles) build_k(i + 1);      // the score MMA of this tile has released the A operand and the columns
#pragma unroll
            for (int gg = H0; gg < NG; ++gg) combine(vb[gg - H0], gg);
            float hmax = 0.f;
            float hv[NG], zv[NG];
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) {
                hv[gg] = valid ? lo_half(vw[gg]) : 0.f;      // rows past the end and rows of sinks hold unspecified bytes
                zv[gg] = valid ? hi_half(vw[gg]) : 0.f;
                hmax = fmaxf(hmax, hv[gg]);
            }
            float arg[kHeads];
            bool need = hmax >= h_bound || tiles_since_fold >= kFoldTiles;
#pragma unroll
            for (int r = 0; r < kHeads; ++r) {
                sc[r] = valid ? fmaf(sc[r], csc[r], zt[r]) : -CUDART_INF_F;      // log2 domain
                arg[r] = sc[r] - m_ref[r];                                      // +inf while the head has no reference yet
                need |= valid && arg[r] > (float)kSlackLog2;
            }
            tc_fence_before();
            const int moved = token_sync_or((need ? 1 : 0) | fail_sh);
            if (moved) {
                if (token_sync_or(fail_sh)) { failed = true; break; }      // a uniform decision: every thread leaves, or none
                // Rare after the first tile: raise every head's reference to its running maximum (and the bound on h),
                // fold what was accumulated and bring it onto the new references.
                float hm = warp_max(hmax);
                if (lane == 0) red[warp * 24 + 4] = hm;
#pragma unroll
                for (int r = 0; r < kHeads; ++r) {
                    const float wm = warp_max(sc[r]);
                    if (lane == 0) red[warp * 24 + r] = wm;
                }
                fold_pv();
                token_sync();      // red is complete
#pragma unroll
                for (int r = 0; r < kHeads; ++r) {
                    float mx = m_ref[r];
                    for (int w = 0; w < kWarps; ++w) mx = fmaxf(mx, red[w * 24 + r]);
                    const float corr = mx == -CUDART_INF_F ? 1.f : ex2_approx(m_ref[r] - mx);      // 0 on the first tile with a token
                    m_ref[r] = mx;
                    l_sum[r] *= corr;
#pragma unroll
                    for (int gg = 0; gg < NG; ++gg) zp[r][gg] *= corr;
                    Os[r * kHeadDim + tid] *= corr;
                    arg[r] = sc[r] - m_ref[r];
                }
                hm = 0.f;
                for (int w = 0; w < kWarps; ++w) hm = fmaxf(hm, red[w * 24 + 4]);
                if (hm >= h_bound) {
                    h_bound = __int_as_float(((__float_as_int(hm) >> 23) + 1) << 23);   // next power of two above
                    hscale = (float)(1u << (32 - kSlackLog2)) / h_bound;
                }
                token_sync();      // red is rewritten by the next move
            }

            // ---------------- p and the digits of p*h -> B operand of the value MMA, once the previous one has read it
            wait_pv();
            {
                float ps[kHeads];
#pragma unroll
                for (int r = 0; r < kHeads; ++r) {
                    const float p = sc[r] == -CUDART_INF_F ? 0.f : ex2_approx(arg[r]);      // at most 2^slack
                    l_sum[r] += p;
                    ps[r] = p * hscale;
#pragma unroll
                    for (int gg = 0; gg < NG; ++gg) zp[r][gg] = fmaf(p, zv[gg], zp[r][gg]);
                }
#pragma unroll
                for (int gg = 0; gg < NG; ++gg)
                    *reinterpret_cast<uint4 *>(PA + gg * kSboMN + (tid >> 3) * kLbo + (tid & 7) * 16) =
                        make_uint4(to_fixed_u32(ps[0] * hv[gg]), to_fixed_u32(ps[1] * hv[gg]), to_fixed_u32(ps[2] * hv[gg]),
                                   to_fixed_u32(ps[3] * hv[gg]));
            }

            // ---------------- V tile -> A operand of the value MMA, once the score MMA of the next tile has read the buffer
            // (as its K operand; it was issued when that operand was complete, in the middle of this tile)
            if (C::kShared && i + 1 < n_tiles && !mbar_wait_bounded(bar_s, (n + 1) & 1u)) fail_sh = 1;
            if constexpr (VB == kTernary) unpack_row_ternary(vm + tid * C::kVRow, VOp + (tid >> 3) * kLbo + (tid & 7) * 16, kSboMN, digits_sh);
            else unpack_row<VB>(vm + tid * C::kVRow, VOp + (tid >> 3) * kLbo + (tid & 7) * 16, kSboMN);
            fresh_sh = pv_fresh ? 1 : 0;      // every thread writes the same value
            proxy_fence();
            mbar_arrive(bar_pa);
            ++pv_local;
            pv_fresh = false;
            ++tiles_since_fold;
        }

        // ---- end of the segment: last fold, CTA-wide sums
        if (failed) {
            if (tid == 0 && a.c.status) atomicOr(a.c.status, SKVQ_STATUS_COPY_TIMEOUT);
            pv_waited = pv_local;      // nothing more is waited for
        }
        fold_pv();
#pragma unroll
        for (int r = 0; r < kHeads; ++r) {
            const float ls = warp_sum(l_sum[r]);
            if (lane == 0) red[warp * 24 + r] = ls;
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) {
                const float zs = warp_sum(zp[r][gg]);
                if (lane == 0) red[warp * 24 + 8 + r * 4 + gg] = zs;
            }
        }
        token_sync();
        {
            const int ch = column_channel<VB>(tid);
            const float winv = __int_as_float((127 - column_shift<VB>(tid)) << 23);      // the weight of this byte column, undone
#pragma unroll
            for (int r = 0; r < kHeads; ++r) {
                if (r >= R) break;
                float l = 0.f, z = 0.f;
                for (int w = 0; w < kWarps; ++w) {
                    l += red[w * 24 + r];
                    z += red[w * 24 + 8 + r * 4 + ((vmap >> (2 * (ch >> 5))) & 3u)];
                }
                const bool dead = failed || m_ref[r] == -CUDART_INF_F;
                float *dst = partials + (((size_t)b * s.Hq + hk * s.rep + a.head0 + r) * n_parts + part) * kPartialStride;
                dst[ch] = dead ? 0.f : fmaf(Os[r * kHeadDim + tid], winv, z);
                if (tid == 0) { dst[kHeadDim] = dead ? -CUDART_INF_F : m_ref[r]; dst[kHeadDim + 1] = dead ? 0.f : l; }
            }
        }
    }
    __syncthreads();          // the segment's shared data is dead; thread 0 decides whether there is another one
    if (fail_sh) {
        // bounded drain of whatever copies are still in flight before the slots are reused or the CTA leaves
        if (!failed && tid == 0) for (int i = 0; i < n_tiles; ++i) { wait_ring(bar_k, i); wait_ring(bar_v, i); }
        failed = true;
    }
    tiles_done += (uint32_t)n_tiles;
    s_count += (uint32_t)n_tiles;
    pv_count += (uint32_t)n_tiles;
    if (tid == 0) more_sh = walk.done() ? 0 : 1;
    __syncthreads();
    if (!more_sh) break;
    }

    // ---- give the tensor memory back (every tensor-memory access of this CTA is behind the barriers above)
    tc_fence_before();
    __syncthreads();
    if (control) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

template <int G, int KB, int VB>
cudaError_t launch_one(const MmaArgs &a, cudaStream_t stream, bool overlap)
{
    using C = TCfg<G, KB, VB>;
    static unsigned long long configured = 0;      // one bit per device
    auto kern = partition_tc_kernel<G, KB, VB>;
    const cudaError_t ec = configure_smem_once(kern, C::kSmemBytes, configured);
    if (ec != cudaSuccess) return ec;
    return launch_dependent(kern, dim3(a.plan.n_slots), dim3(kTile + 32), C::kSmemBytes, stream, overlap, a);
}

template <int G>
cudaError_t launch_g(const MmaArgs &a, cudaStream_t stream, bool overlap)
{
    switch (a.s.k_bits * 100 + a.s.v_bits) {
        case 202: return launch_one<G, 2, 2>(a, stream, overlap);
        case 203: return launch_one<G, 2, 3>(a, stream, overlap);
        case 204: return launch_one<G, 2, 4>(a, stream, overlap);
        case 215: return launch_one<G, 2, kTernary>(a, stream, overlap);
        case 302: return launch_one<G, 3, 2>(a, stream, overlap);
        case 303: return launch_one<G, 3, 3>(a, stream, overlap);
        case 304: return launch_one<G, 3, 4>(a, stream, overlap);
        case 315: return launch_one<G, 3, kTernary>(a, stream, overlap);
        case 402: return launch_one<G, 4, 2>(a, stream, overlap);
        case 403: return launch_one<G, 4, 3>(a, stream, overlap);
        case 404: return launch_one<G, 4, 4>(a, stream, overlap);
        case 415: return launch_one<G, 4, kTernary>(a, stream, overlap);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

// Launches the kernel above: every configuration the library accepts is covered (2-, 3- or 4-bit K and V, three-level V, groups of 32,
// 64 or 128 channels or of unequal width, up to 8 query heads per KV head: one launch per four heads); *handled tells the
// caller whether it did.
cudaError_t launch_partition_tc(const Shape &s, const CachePtrs &c, const __half *q, float scale_log2, const SplitPlan &plan,
                                float *workspace, cudaStream_t stream, bool overlap, bool *handled)
{
    *handled = false;
    if (s.rep > 2 * kHeads || (s.G != 128 && s.G != 64 && s.G != 32)) return cudaSuccess;
    *handled = true;
    for (int head0 = 0; head0 < s.rep; head0 += kHeads) {
        MmaArgs a{s, c, q, scale_log2, plan, workspace};
        a.head0 = head0;
        // a second launch reads the same cache again for the next four heads; it starts when the first has finished
        const bool ov = overlap && head0 == 0;
        const cudaError_t e = s.G == 128 ? launch_g<128>(a, stream, ov) : s.G == 64 ? launch_g<64>(a, stream, ov) : launch_g<32>(a, stream, ov);
        if (e != cudaSuccess) return e;
        if (head0 > 0) count_launch(1);
    }
    return cudaSuccess;
}

}  // namespace skvq

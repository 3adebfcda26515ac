// Tile kernel of skvq_quantize_append for bulk appends (prefill): channel reorder on the tensor core, then group-wise
// clipped dynamic asymmetric quantization with two threads per token row (Sec. 3.1 Eq. 1 and Eq. 2, Algorithm 1).
//
// The reorder stored[j] = x[idx[j]] of a tile of 128 tokens is the product X * P^T with the 0/1 matrix
// P[j][k] = (k == idx[j]): every output is one input times 1.0 plus zeros, so fp16 operands with fp32 accumulation give
// the reordered values exactly.  One tcgen05.mma chain (M = 128 tokens, N = 128 stored channels, K = 128 source
// channels, fp16 in, fp32 accumulators in tensor memory) replaces 16384 two-byte gathers, and it lays every token's
// reordered row along one lane of the tensor memory: lane m is token m of the tile.  Group minimum and maximum, scale
// and zero point, the codes and their packing are then register arithmetic without shuffles.
// All code widths: 2- and 4-bit fields as they are, 3-bit codes closed up from 4-bit fields into the row's bit stream,
// three-level codes from 2-bit fields into base-3 bytes.
//
// One CTA = 256 threads = one (sequence, KV head, tensor K or V) and a run of consecutive 128-token tiles.  Warps w and
// w + 4 share the 32 tokens of lane quadrant w & 3: the first takes stored channels 0-63 of each, the second 64-127 (a
// group that spans both halves has its extremes exchanged through shared memory).  Nothing but mbarriers orders copies,
// MMAs and arithmetic:
//   copy      thread 0 brings a tile in with two tensor-map copies (cp.async.bulk.tensor, 64 channels x 128
//             tokens each, 128-byte swizzle: the K-major operand layout of the MMA), two tiles ahead of the arithmetic;
//             rows past the end of the input are filled with zeros by the copy engine;
//   MMA       thread 0 issues 8 k-steps per tile, before it starts on its own share of the tile in front, and commits
//             them to an mbarrier; two accumulators in tensor memory, so the MMAs of tile t+1 run under the arithmetic
//             of tile t;
//   quantize  every thread reads its half row (64 values) from tensor memory into registers once: the
//             extremes of its two 32-channel granules (groups are unions of granules), scale and zero point, the
//             codes, then one 16-byte store of its half of the packed row, and the {scale, zero} words; its arrival on
//             the accumulator's mbarrier lets thread 0 reuse it.
// Every wait is bounded; a wait that ran out is reported through the cache's status word, the threads then run to the end
// of their loops without waiting or storing.  Two CTAs per SM (96 KB of shared memory and 256 tensor-memory columns
// each).  The quantizer arithmetic is that of append_kernel (explicitly rounded fp32 operations), so both kernels
// produce the same bits.
#include <cuda.h>

#include <type_traits>

#include "skvq_append_common.cuh"
#include "skvq_mma_common.cuh"
#include "skvq_tcgen05.cuh"

namespace skvq {
namespace {

using namespace mmak;
using namespace tc5;

constexpr int kTileRows = 128;                       // tokens per tile = rows of the MMA
constexpr int kTileThreads = 2 * kTileRows;          // two threads per token row
constexpr int kOperandBytes = kTileRows * kHeadDim * 2;      // 32 KB: a 128 x 128 fp16 operand
constexpr int kSmemBytes = 3 * kOperandBytes + 1024;      // P and two tiles of X, and room to align them to 1024 bytes
constexpr uint32_t kLboBytes = 128;                  // P (no swizzle): between core matrices along K
constexpr uint32_t kSboBytes = 16 * 128;             // P: between groups of 8 rows: 16 core matrices of 128 bytes
constexpr int kHalfTileBytes = kTileRows * 128;      // X: 64 channels of 128 tokens, 128-byte rows (swizzled)
constexpr int kTmemColumns = 256;                    // two 128 x 128 fp32 accumulators

// Byte offset of the 16-byte piece (row, piece) of a K-major operand without swizzle: piece = 8 consecutive K elements.
__device__ __forceinline__ uint32_t operand_offset(int row, int piece)
{
    return (uint32_t)((row >> 3) * kSboBytes + piece * kLboBytes + (row & 7) * 16);
}

// One box of a three-dimensional tensor map -> shared memory, completion counted in bytes on an mbarrier.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}
// Shared-memory matrix descriptor of a K-major operand in the 128-byte swizzle: rows of 128 bytes, 8-row atoms of 1024
// bytes (stride offset), start address inside the atom for a k-step; descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Barrier 1 + quad: the two warps that share the tokens of lane quadrant quad (64 threads).
__device__ __forceinline__ void pair_sync(int quad) { asm volatile("bar.sync %0, 64;" ::"r"(1 + quad) : "memory"); }

// Stored scale and zero point of a group from its extremes (Eq. 2; both ends clipped by alpha): the words that go to
// the cache, and the values the codes are computed against.
__device__ __forceinline__ void group_parameters(float mn, float mx, float alpha, float qmax, bool meta_fp8, uint32_t &hz_bits,
                                                 float &hf, float &zf)
{
    const float lo = __fadd_rn(__fmul_rn(alpha, mn), 0.0f);      // "+ 0" turns a negative zero into +0
    const float hi = __fadd_rn(__fmul_rn(alpha, mx), 0.0f);
    const float h32 = __fdiv_rn(__fsub_rn(hi, lo), qmax);
    __half2 hz;
    if (meta_fp8) {
        const uint16_t b = to_e4m3x2(h32, lo);
        hz = from_e4m3x2(b);
        hz_bits = b;
    } else {
        hz = __halves2half2(__float2half_rn(h32), __float2half_rn(lo));
        hz_bits = *reinterpret_cast<const uint32_t *>(&hz);
    }
    hf = __low2float(hz);
    zf = __high2float(hz);
}

__device__ __forceinline__ float mul_sat(float a, float b)      // clamp(RN(a * b), 0, 1) in one instruction
{
    float r;
    asm("mul.rn.sat.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}

// Codes of 16 consecutive stored channels against (hf, zf) in fields of FIELD bits (2 or 4; QMAX = the largest code, which
// need not fill the field: 3-bit codes travel in 4-bit fields, three-level codes in 2-bit fields until the row is
// packed): FIELD / 2 words, code j in bits [j*FIELD, (j+1)*FIELD) of the run.
// code = clamp(rint(RN((x - z) / h)), 0, qmax) with IEEE division.  Instead of dividing, u = sat(d * r) with
// r = RN(RN(1/h) / qmax) is the clamped quotient on the scale [0, 1], within 5 * 2^-24 relative of the IEEE quotient / qmax;
// wherever every value within 2^-18 relative of it rounds to the same integer, that integer is the code.  The test is two
// FMAs onto 1.5 * 2^23 (the low mantissa bits of the sum are then the rounded integer, ties to even, like rintf), one with
// the quotient scaled down and one scaled up by 2^-18; both results are packed (four partial sums each, so that no
// addition waits for the one before), and fields in which the two packed runs differ are elements in doubt (a quotient
// next to k + 0.5, exact ties included): doubt[] has their bits set and repair16 redoes them.
template <int BITS, int QMAX>
__device__ __forceinline__ void pack16(const float (&x)[16], float zf, float r, uint32_t (&words)[BITS / 2], uint32_t (&doubt)[BITS / 2])
{
    constexpr int qmax = QMAX, PER_WORD = 32 / BITS, NW = BITS / 2, LANES = 4 / NW;      // BITS = field width; partial sums per word
    constexpr float MAGIC = 12582912.0f;                       // 0x4B400000
    constexpr float UP = (float)qmax * (1.0f + 3.814697265625e-06f), DN = (float)qmax * (1.0f - 3.814697265625e-06f);   // exact products
    uint32_t kconst = 0u;
#pragma unroll
    for (int j = 0; j < PER_WORD; ++j) kconst += 0x4B400000u << (j * BITS);
    uint32_t wa[NW][LANES], wb[NW][LANES];
#pragma unroll
    for (int i = 0; i < NW; ++i)
#pragma unroll
        for (int l = 0; l < LANES; ++l) { wa[i][l] = 0u; wb[i][l] = 0u; }
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const float u = mul_sat(__fsub_rn(x[j], zf), r);
        wa[j / PER_WORD][j % LANES] += __float_as_uint(__fmaf_rn(u, DN, MAGIC)) << ((j % PER_WORD) * BITS);
        wb[j / PER_WORD][j % LANES] += __float_as_uint(__fmaf_rn(u, UP, MAGIC)) << ((j % PER_WORD) * BITS);
    }
#pragma unroll
    for (int i = 0; i < NW; ++i) {
        uint32_t sa = 0u - kconst, sb = 0u - kconst;      // the constant bits of 1.5 * 2^23 come out of the sums (modulo 2^32)
#pragma unroll
        for (int l = 0; l < LANES; ++l) { sa += wa[i][l]; sb += wb[i][l]; }
        words[i] = sa;
        doubt[i] = sa ^ sb;
    }
}

// The elements of a 16-column run that pack16 left in doubt, redone by the defining formula: the warp walks the union of
// its doubtful columns, re-reads each from tensor memory (taddr = this warp's lanes, first column of the run) and the
// lanes concerned patch their field.  Every lane of the warp must call this.
template <int BITS, int QMAX>
__device__ __forceinline__ void repair16(float hf, float zf, uint32_t taddr, uint32_t (&words)[BITS / 2], const uint32_t (&doubt)[BITS / 2])
{
    constexpr int qmax = QMAX, PER_WORD = 32 / BITS, NW = BITS / 2;      // BITS = field width
#pragma unroll
    for (int i = 0; i < NW; ++i) {
        uint32_t todo = __reduce_or_sync(0xffffffffu, doubt[i]);      // the same for every lane: the loop is uniform
        while (todo) {
            const int f = (__ffs(todo) - 1) / BITS;                    // field of this word = column i * PER_WORD + f of the run
            const uint32_t field = ((1u << BITS) - 1u) << (f * BITS);
            todo &= ~field;
            float xv;
            tmem_ld1(taddr + i * PER_WORD + f, xv);
            tmem_wait_ld();
            if (doubt[i] & field) {
                float c = hf != 0.0f ? rintf(__fdiv_rn(__fsub_rn(xv, zf), hf)) : 0.0f;
                c = fminf(fmaxf(c, 0.0f), (float)qmax);
                words[i] = (words[i] & ~field) | ((uint32_t)(int)c << (f * BITS));
            }
        }
    }
}

// Minimum and maximum of 16 values.
__device__ __forceinline__ void extremes16(const float (&x)[16], float &lo, float &hi)
{
    lo = x[0];
    hi = x[0];
#pragma unroll
    for (int j = 1; j < 16; ++j) {
        lo = fminf(lo, x[j]);
        hi = fmaxf(hi, x[j]);
    }
}

template <int G>
__global__ void __launch_bounds__(kTileThreads, 2)
append_tile_kernel(AppendArgs a, int tiles_per_cta, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v)
{
    constexpr int NG = kHeadDim / G;
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ __align__(8) uint64_t bar_sh[6];
    __shared__ uint32_t tmem_sh;
    __shared__ int fail_sh;
    __shared__ uint32_t tern_sh[2][kTileRows];                 // [tile & 1][token]: code 64 of a three-level row, for the thread of the first half
    __shared__ __align__(16) float4 ext_sh[2][2][kTileRows];   // [tile & 1][half][token]: {min, max} of a half row's two granules, for the thread of the other half
    const Shape &s = a.s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool control = tid == 0;      // thread 0 also copies and issues the MMAs
    const int quad = warp & 3, half = (warp >> 2) & 1;         // tensor-memory lanes 32*quad .. +31; stored channels 64*half .. +63
    const int row = 32 * quad + lane;                          // this thread's token of every tile
    const int b = blockIdx.z, tensor = blockIdx.x & 1, h = blockIdx.y;
    const int L0 = a.c.lengths[b];
    const int n_b = seq_new_count(a, b);
    const int L1 = L0 + n_b;
    if (n_b == 0 || L1 > s.max_tokens) return;       // uniform over the CTA; overflow is reported by the bookkeeping kernel
    int f0, f1;
    bulk_range(L0, s.n_sink, max(L1 - s.W, 0), f0, f1);
    const int n_tiles = (f1 - f0 + kTileRows - 1) / kTileRows;
    const int t_begin = (blockIdx.x >> 1) * tiles_per_cta, t_end = min(n_tiles, t_begin + tiles_per_cta);      // this CTA's run of tiles
    if (t_begin >= t_end) return;
    if (!SKVQ_IN_BOUNDS(f0 >= L0 && f1 <= s.cap && f1 - L0 <= a.n_new, a.c.status)) return;
    const int T = t_end - t_begin;

    uint8_t *base = smem + ((1024u - (smem_u32(smem) & 1023u)) & 1023u);      // the swizzle pattern repeats every 1024 bytes
    uint8_t *P = base, *X = base + kOperandBytes;      // X: two tile buffers of two half tiles each
    const uint32_t bar_full = smem_u32(&bar_sh[0]);    // + 8 * (t & 1): the copies of tile t have landed
    const uint32_t bar_mma = bar_full + 16;            // + 8 * (t & 1): the MMAs of tile t have completed
    const uint32_t bar_free = bar_full + 32;           // + 8 * (t & 1): every arithmetic thread is done with the accumulator of tile t

    // ---- once per CTA: the permutation operand, the tensor memory, the barriers
    {
        uint4 *p4 = reinterpret_cast<uint4 *>(P);
#pragma unroll
        for (int i = 0; i < kOperandBytes / 16 / kTileThreads; ++i) p4[tid + i * kTileThreads] = make_uint4(0u, 0u, 0u, 0u);
    }
    if (warp == 0) tmem_alloc(smem_u32(&tmem_sh), kTmemColumns);
    if (control) {
#pragma unroll
        for (int i = 0; i < 4; ++i) mbar_init(bar_full + 8 * i, 1);
        mbar_init(bar_free, kTileThreads);
        mbar_init(bar_free + 8, kTileThreads);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fail_sh = 0;
    }
    __syncthreads();
    if (tid < kHeadDim) {
        const int32_t *idx = (tensor ? a.c.reorder_v : a.c.reorder_k) + (size_t)h * kHeadDim;
        const int k = idx[tid] & (kHeadDim - 1);      // stored channel tid takes source channel k: P[tid][k] = 1
        *reinterpret_cast<__half *>(P + operand_offset(tid, k >> 3) + (k & 7) * 2) = __float2half(1.0f);
    }
    proxy_fence();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_sh;
    volatile int *fail = &fail_sh;

    // ---- thread 0's second job: copies and MMAs, one tile ahead of the arithmetic
    const CUtensorMap *map = tensor ? &map_v : &map_k;
    const uint64_t dP = smem_desc(smem_u32(P), kLboBytes, kSboBytes);
    constexpr uint32_t kIdesc = idesc_f16_f32(kTileRows, kHeadDim);
    bool alive = true;
    auto copy_tile = [&](int t) {      // both halves of tile t into buffer t & 1
        const uint32_t dst = smem_u32(X) + (t & 1) * kOperandBytes, bar = bar_full + 8 * (t & 1);
        const int tok = f0 + (t_begin + t) * kTileRows - L0;      // row of the input
        mbar_expect_tx(bar, kOperandBytes);
        tma_load_3d(dst, map, h * kHeadDim, tok, b, bar);
        tma_load_3d(dst + kHalfTileBytes, map, h * kHeadDim + 64, tok, b, bar);
    };
    auto issue_mmas = [&](int t) {     // once tile t has landed and the arithmetic is done with tile t-2, which had the same accumulator
        const uint32_t ph = (uint32_t)(t >> 1) & 1u;
        if (alive && !mbar_wait_bounded(bar_full + 8 * (t & 1), ph)) { alive = false; *fail = 1; }
        if (t >= 2 && alive && !mbar_wait_bounded(bar_free + 8 * (t & 1), ph ^ 1u)) { alive = false; *fail = 1; }
        tc_fence_after();
        const uint32_t xb = smem_u32(X) + (t & 1) * kOperandBytes;
#pragma unroll
        for (int ks = 0; ks < kHeadDim / 16; ++ks) {      // 16 source channels = 32 bytes of a swizzled row per k-step
            const uint64_t dX = smem_desc_sw128(xb + (ks >> 2) * kHalfTileBytes + (ks & 3) * 32);
            umma_f16(tmem + (uint32_t)(t & 1) * kHeadDim, dX, dP + ((ks * 2 * kLboBytes) >> 4), kIdesc, ks > 0 ? 1u : 0u);
        }
        umma_commit(bar_mma + 8 * (t & 1));
    };
    auto refill = [&](int t) {         // the buffer of tile t takes tile t+2 once the MMAs of tile t have read it
        if (t + 2 >= T) return;
        if (alive && !mbar_wait_bounded(bar_mma + 8 * (t & 1), (uint32_t)(t >> 1) & 1u)) { alive = false; *fail = 1; }
        copy_tile(t + 2);
    };
    if (control) {
        copy_tile(0);
        if (T > 1) copy_tile(1);
        issue_mmas(0);
        refill(0);
    }
    __syncwarp();

    {
        // ================================================================ the arithmetic
        const int bits = tensor ? s.v_bits : s.k_bits;
        const bool f8 = s.meta_fp8 != 0;
        const size_t bh = (size_t)b * s.Hkv + h;
        const float *alpha = (tensor ? a.c.alpha_v : a.c.alpha_k) + (size_t)h * NG;
        const uint32_t gmap = granule_groups(tensor ? a.c.bounds_v : a.c.bounds_k, h, G, NG);      // group of every 32-channel granule
        auto group_of = [&](int granule) { return (gmap >> (2 * granule)) & 3u; };
        // Does a group reach into both halves of the row?  Then the two threads of a token exchange their extremes.
        const bool spans = group_of(1) == group_of(2);
        // This thread's two granules belong to one or two groups: parameter set 0 is the group of its first granule, set 1
        // that of its second when it is another one.  The other half's granules feed a set only when their group spans.
        const uint32_t g0 = group_of(2 * half), g1 = group_of(2 * half + 1);
        const bool two_sets = g1 != g0;
        const float alpha0 = alpha[g0], alpha1 = alpha[g1];
        const uint32_t p0 = group_of(2 * (half ^ 1)), p1 = group_of(2 * (half ^ 1) + 1);      // the partner's granules
        const bool p0_in0 = spans && p0 == g0, p1_in0 = spans && p1 == g0, p0_in1 = spans && two_sets && p0 == g1,
                   p1_in1 = spans && two_sets && p1 == g1;
        // {scale, zero} of a group are written by the thread that holds its first granule
        const bool writes0 = half == 0 || group_of(1) != g0;
        uint8_t *codes = (tensor ? a.c.v_codes : a.c.k_codes) + bh * (size_t)s.cap * packed_row_bytes(bits);
        uint8_t *meta = reinterpret_cast<uint8_t *>(tensor ? a.c.v_meta : a.c.k_meta) + bh * (size_t)s.cap * NG * (f8 ? 2 : 4);
        const uint32_t tmem_half = tmem + ((uint32_t)(quad * 32) << 16) + 64 * half;      // this thread's lane, its first column
        const float qmaxf = (float)code_max(bits);
        const float qmax_inv = bits == 2 ? 1.0f / 3.0f : (bits == 4 ? 1.0f / 15.0f : (bits == 3 ? 1.0f / 7.0f : 0.5f));
        for (int t = 0; t < T; ++t) {
            if (*fail) alive = false;
            if (control && t + 1 < T) issue_mmas(t + 1);      // they run under this tile's arithmetic
            __syncwarp();
            if (alive && !mbar_wait_bounded(bar_mma + 8 * (t & 1), (uint32_t)(t >> 1) & 1u)) { alive = false; *fail = 1; }
            tc_fence_after();
            const uint32_t trow = tmem_half + (uint32_t)(t & 1) * kHeadDim;
            const int tok = f0 + (t_begin + t) * kTileRows + row;
            const bool valid = alive && tok < f1;

            // ---- the thread's half row into registers, the extremes of its two 32-channel granules
            float x0[16], x1[16], x2[16], x3[16];
            tmem_ld16f(trow, x0);
            tmem_ld16f(trow + 16, x1);
            tmem_ld16f(trow + 32, x2);
            tmem_ld16f(trow + 48, x3);
            tmem_wait_ld16f(x0);
            tmem_wait_ld16f(x1);
            tmem_wait_ld16f(x2);
            tmem_wait_ld16f(x3);
            float lo[2], hi[2];
            {
                float lo0, hi0, lo1, hi1;
                extremes16(x0, lo0, hi0);
                extremes16(x1, lo1, hi1);
                lo[0] = fminf(lo0, lo1);
                hi[0] = fmaxf(hi0, hi1);
                extremes16(x2, lo0, hi0);
                extremes16(x3, lo1, hi1);
                lo[1] = fminf(lo0, lo1);
                hi[1] = fmaxf(hi0, hi1);
            }
            float slo[2] = {lo[0], lo[1]}, shi[2] = {hi[0], hi[1]};      // extremes of the two parameter sets
            if (!two_sets) {
                slo[0] = fminf(lo[0], lo[1]);
                shi[0] = fmaxf(hi[0], hi[1]);
            }
            if (spans) {      // uniform: a property of the KV head
                // Two buffers and one barrier per tile: a thread rewrites the entry of tile t when it works on tile t+2, behind
                // the barrier of tile t+1, which its partner reaches only after it has read the entry of tile t.
                ext_sh[t & 1][half][row] = make_float4(lo[0], hi[0], lo[1], hi[1]);
                pair_sync(quad);
                const float4 o = ext_sh[t & 1][half ^ 1][row];
                if (p0_in0) { slo[0] = fminf(slo[0], o.x); shi[0] = fmaxf(shi[0], o.y); }
                if (p1_in0) { slo[0] = fminf(slo[0], o.z); shi[0] = fmaxf(shi[0], o.w); }
                if (p0_in1) { slo[1] = fminf(slo[1], o.x); shi[1] = fmaxf(shi[1], o.y); }
                if (p1_in1) { slo[1] = fminf(slo[1], o.z); shi[1] = fmaxf(shi[1], o.w); }
            }

            // ---- scale and zero point of the thread's one or two groups
            float hf[2], zf[2], rq[2];
            uint32_t hz[2];
            group_parameters(slo[0], shi[0], alpha0, qmaxf, f8, hz[0], hf[0], zf[0]);
            // degenerate group (h == 0): every quotient is taken as 0.  1/qmax is a rounded constant: see pack16
            rq[0] = hf[0] != 0.0f ? __fmul_rn(__frcp_rn(hf[0]), qmax_inv) : 0.0f;
            hz[1] = hz[0]; hf[1] = hf[0]; zf[1] = zf[0]; rq[1] = rq[0];
            if (two_sets) {      // uniform over the warp
                group_parameters(slo[1], shi[1], alpha1, qmaxf, f8, hz[1], hf[1], zf[1]);
                rq[1] = hf[1] != 0.0f ? __fmul_rn(__frcp_rn(hf[1]), qmax_inv) : 0.0f;
            }

            // ---- the codes of the thread's two granules, then its half of the packed row.  WIDTH is the cache's code width
            // (2, 3, 4, or kTernary); the codes are formed in fields of 2 or 4 bits.
            auto quantize_half = [&](auto width_tag) {
                constexpr int WIDTH = decltype(width_tag)::value;      // a compile-time constant inside
                constexpr int FIELD = (WIDTH == 2 || WIDTH == kTernary) ? 2 : 4, QMAX = code_max(WIDTH), NW = FIELD / 2;
                uint32_t cw[2][2][NW];                                 // [granule][chunk][word]
#pragma unroll
                for (int gr = 0; gr < 2; ++gr) {
                    const float hg = hf[gr], zg = zf[gr], rg = rq[gr];      // set 1 equals set 0 when both granules share a group
                    uint32_t d0[NW], d1[NW];
                    pack16<FIELD, QMAX>(gr == 0 ? x0 : x2, zg, rg, cw[gr][0], d0);
                    pack16<FIELD, QMAX>(gr == 0 ? x1 : x3, zg, rg, cw[gr][1], d1);
                    uint32_t any = 0u;
#pragma unroll
                    for (int i = 0; i < NW; ++i) any |= d0[i] | d1[i];
                    if (__any_sync(0xffffffffu, any != 0u)) {      // rare: some quotient of the warp lies next to a rounding boundary
                        repair16<FIELD, QMAX>(hg, zg, trow + 32 * gr, cw[gr][0], d0);
                        repair16<FIELD, QMAX>(hg, zg, trow + 32 * gr + 16, cw[gr][1], d1);
                    }
                }
                uint8_t *crow = codes + (size_t)tok * packed_row_bytes(WIDTH);
                if constexpr (WIDTH == 2) {
                    if (valid) *reinterpret_cast<uint4 *>(crow + 16 * half) = make_uint4(cw[0][0][0], cw[0][1][0], cw[1][0][0], cw[1][1][0]);
                } else if constexpr (WIDTH == 4) {
                    if (valid) {
                        *reinterpret_cast<uint4 *>(crow + 32 * half) = make_uint4(cw[0][0][0], cw[0][0][1], cw[0][1][0], cw[0][1][1]);
                        *reinterpret_cast<uint4 *>(crow + 32 * half + 16) = make_uint4(cw[1][0][0], cw[1][0][1], cw[1][1][0], cw[1][1][1]);
                    }
                } else if constexpr (WIDTH == 3) {
                    // eight 4-bit fields of a word -> 24 bits of the row's bit stream (code j in bits [3j, 3j+3)): pairs of
                    // fields close up inside their byte, then the four bytes close up; 64 codes = 24 bytes per half row
                    uint32_t r[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const uint32_t w = cw[i >> 2][(i >> 1) & 1][i & 1];
                        const uint32_t p = (w & 0x07070707u) | ((w >> 1) & 0x38383838u);
                        r[i] = (p & 0x3Fu) | ((p >> 2) & 0xFC0u) | ((p >> 4) & 0x3F000u) | ((p >> 6) & 0xFC0000u);
                    }
                    if (valid) {
                        uint2 *o = reinterpret_cast<uint2 *>(crow + 24 * half);
                        o[0] = make_uint2(r[0] | (r[1] << 24), (r[1] >> 8) | (r[2] << 16));
                        o[1] = make_uint2((r[2] >> 16) | (r[3] << 8), r[4] | (r[5] << 24));
                        o[2] = make_uint2((r[5] >> 8) | (r[6] << 16), (r[6] >> 16) | (r[7] << 8));
                    }
                } else {
                    // three-level codes: byte n of the row = codes 5n .. 5n+4 as base-3 digits.  Bytes 0-12 belong to the
                    // first half of the row, which needs code 64 from the second (handed over through shared memory);
                    // bytes 13-25 to the second half (local codes 1 .. 63, then nothing: the last digits are 0).
                    auto code = [&](int j) -> uint32_t {      // j: compile-time index into the thread's 64 codes
                        return j < 64 ? (cw[j >> 5][(j >> 4) & 1][0] >> (2 * (j & 15))) & 3u : 0u;
                    };
                    if (half == 1) tern_sh[t & 1][row] = code(0);
                    pair_sync(quad);      // two buffers, one barrier per tile: as for the extremes
                    const uint32_t c64 = half == 0 ? tern_sh[t & 1][row] : 0u;
                    uint32_t by[13];
                    if (half == 0) {
#pragma unroll
                        for (int n = 0; n < 13; ++n) {
                            const uint32_t last = 5 * n + 4 < 64 ? code(5 * n + 4) : c64;
                            by[n] = code(5 * n) + 3u * code(5 * n + 1) + 9u * code(5 * n + 2) + 27u * code(5 * n + 3) + 81u * last;
                        }
                    } else {
#pragma unroll
                        for (int n = 0; n < 13; ++n)
                            by[n] = code(5 * n + 1) + 3u * code(5 * n + 2) + 9u * code(5 * n + 3) + 27u * code(5 * n + 4) + 81u * code(5 * n + 5);
                    }
                    if (valid) {      // rows of 26 bytes are 2-byte aligned; the second half starts at an odd byte
                        uint8_t *o = crow + 13 * half;
                        if (half == 0) {
#pragma unroll
                            for (int n = 0; n < 6; ++n) *reinterpret_cast<uint16_t *>(o + 2 * n) = (uint16_t)(by[2 * n] | (by[2 * n + 1] << 8));
                            o[12] = (uint8_t)by[12];
                        } else {
                            o[0] = (uint8_t)by[0];
#pragma unroll
                            for (int n = 0; n < 6; ++n) *reinterpret_cast<uint16_t *>(o + 1 + 2 * n) = (uint16_t)(by[2 * n + 1] | (by[2 * n + 2] << 8));
                        }
                    }
                }
            };
            if (bits == 2) quantize_half(std::integral_constant<int, 2>{});
            else if (bits == 4) quantize_half(std::integral_constant<int, 4>{});
            else if (bits == 3) quantize_half(std::integral_constant<int, 3>{});
            else quantize_half(std::integral_constant<int, kTernary>{});
            // the accumulator may be overwritten: the last tensor-memory read of this tile (a repair) is behind us
            tc_fence_before();
            mbar_arrive(bar_free + 8 * (t & 1));
            if (valid) {
                const size_t mrow = (size_t)tok * NG;
                if (writes0) {
                    if (f8) reinterpret_cast<uint16_t *>(meta)[mrow + g0] = (uint16_t)hz[0];
                    else reinterpret_cast<uint32_t *>(meta)[mrow + g0] = hz[0];
                }
                if (two_sets) {
                    if (f8) reinterpret_cast<uint16_t *>(meta)[mrow + g1] = (uint16_t)hz[1];
                    else reinterpret_cast<uint32_t *>(meta)[mrow + g1] = hz[1];
                }
            }
            if (control) refill(t + 1);
            __syncwarp();
        }
    }

    // ---- leave: nothing of this CTA is in flight any more
    tc_fence_before();
    __syncthreads();
    if (tid == 0 && fail_sh && a.c.status) atomicOr(a.c.status, SKVQ_STATUS_COPY_TIMEOUT);
    if (warp == 0) tmem_dealloc(tmem, kTmemColumns);
}

}  // namespace

namespace {

// cuTensorMapEncodeTiled through the runtime's driver entry point (the library does not link against the driver).
using EncodeTiled = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                 const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiled encode_tiled()
{
    static EncodeTiled fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiled>(p);
    }();
    return fn;
}

// The input [B][n_new][Hkv][D] as a tensor of (channel of the token row, token, sequence); a box is 64 channels of 128
// tokens of one sequence, stored in the 128-byte swizzle.  Tokens past n_new read as zeros.
cudaError_t make_input_map(CUtensorMap *map, const __half *x, const Shape &s, int n_new)
{
    const EncodeTiled enc = encode_tiled();
    if (!enc) return cudaErrorNotSupported;
    const cuuint64_t row_elems = (cuuint64_t)s.Hkv * kHeadDim;
    const cuuint64_t dims[3] = {row_elems, (cuuint64_t)n_new, (cuuint64_t)s.B};
    const cuuint64_t strides[2] = {row_elems * 2, row_elems * 2 * (cuuint64_t)n_new};      // bytes: token, sequence
    const cuuint32_t box[3] = {64, (cuuint32_t)kTileRows, 1};
    const cuuint32_t elem[3] = {1, 1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<__half *>(x), dims, strides, box, elem,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int G>
cudaError_t launch_g(const AppendArgs &a, int tiles_per_cta, const CUtensorMap &mk, const CUtensorMap &mv, dim3 grid, cudaStream_t stream)
{
    static unsigned long long configured = 0;      // one bit per device
    if (!(configured & (1ull << (current_device() & (kMaxDevices - 1))))) {
        // two CTAs of 97 KB each only fit the largest shared-memory carveout
        const cudaError_t ec = cudaFuncSetAttribute(append_tile_kernel<G>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                                    (int)cudaSharedmemCarveoutMaxShared);
        if (ec != cudaSuccess) return ec;
    }
    const cudaError_t e = configure_smem_once(append_tile_kernel<G>, kSmemBytes, configured);
    if (e != cudaSuccess) return e;
    append_tile_kernel<G><<<grid, kTileThreads, kSmemBytes, stream>>>(a, tiles_per_cta, mk, mv);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_append_tiles(const AppendArgs &a, cudaStream_t stream)
{
    const Shape &s = a.s;
    alignas(64) CUtensorMap mk, mv;
    cudaError_t e = make_input_map(&mk, a.k, s, a.n_new);
    if (e != cudaSuccess) return e;
    e = make_input_map(&mv, a.v, s, a.n_new);
    if (e != cudaSuccess) return e;
    const int max_tiles = (a.n_new + kTileRows - 1) / kTileRows;
    // A CTA's set-up (the permutation operand, the tensor memory, the first copies) costs about two tiles' time: long runs
    // of tiles per CTA, as long as the grid still has several waves of the two CTAs an SM holds.
    const long total_tiles = (long)max_tiles * 2 * s.Hkv * s.B;
    const long want_ctas = 8L * 2 * sm_count();      // measured: 32 tiles per CTA 3.55, 16: 3.49, 8: 3.37, 4: 3.10 TB/s on a 1 GiB chunk
    int tiles_per_cta = (int)(total_tiles / want_ctas);
    tiles_per_cta = tiles_per_cta < 4 ? 4 : (tiles_per_cta > 32 ? 32 : tiles_per_cta);
    dim3 grid(2 * ((max_tiles + tiles_per_cta - 1) / tiles_per_cta), s.Hkv, s.B);      // x: (run of tiles, tensor)
    if (s.G == 128) return launch_g<128>(a, tiles_per_cta, mk, mv, grid, stream);
    if (s.G == 64) return launch_g<64>(a, tiles_per_cta, mk, mv, grid, stream);
    return launch_g<32>(a, tiles_per_cta, mk, mv, grid, stream);
}

}  // namespace skvq

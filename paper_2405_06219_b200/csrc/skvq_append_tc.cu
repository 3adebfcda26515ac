// Tile kernel of skvq_quantize_append for bulk appends (prefill): channel reorder on the tensor core, then group-wise
// clipped dynamic asymmetric quantization with one thread per token row (Sec. 3.1 Eq. 1 and Eq. 2, Algorithm 1).
//
// The reorder stored[j] = x[idx[j]] of a tile of 128 tokens is the product X * P^T with the 0/1 matrix
// P[j][k] = (k == idx[j]): every output is one input times 1.0 plus zeros, so fp16 operands with fp32 accumulation give
// the reordered values exactly.  One tcgen05.mma chain (M = 128 tokens, N = 128 stored channels, K = 128 source
// channels, fp16 in, fp32 accumulators in tensor memory) replaces 16384 two-byte gathers, and it hands every thread
// its token's whole reordered row: lane m of the tensor memory is token m of the tile.  Group minimum and maximum,
// scale and zero point, the codes and their packing are then register arithmetic of one thread, without shuffles.
//
// One CTA = 128 threads = one (sequence, KV head, tensor K or V) and a run of consecutive 128-token tiles:
//   copy      16-byte cp.async pieces of the next tile straight into the canonical K-major operand layout
//             (8-row x 16-byte core matrices), issued as soon as the MMAs of the current tile have read the buffer;
//   MMA       thread 0 issues 8 k-steps, commits them to an mbarrier (bounded wait);
//   quantize  every thread reads its row from tensor memory 32 channels at a time: one pass for the extremes of every
//             32-channel granule (groups are unions of granules), one pass that quantizes, then 16-byte stores of the
//             packed row and of the {scale, zero} words.
// Three CTAs per SM (64 KB of shared memory and 128 tensor-memory columns each) keep copies, MMAs and arithmetic of
// different tiles in flight.  The quantizer arithmetic is that of append_kernel (explicitly rounded fp32 operations),
// so both kernels produce the same bits.
#include <type_traits>

#include "skvq_append_common.cuh"
#include "skvq_mma_common.cuh"
#include "skvq_tcgen05.cuh"

namespace skvq {
namespace {

using namespace mmak;
using namespace tc5;

constexpr int kTileRows = 128;                       // tokens per tile = rows of the MMA = threads per CTA
constexpr int kTilesPerCta = 8;                      // consecutive tiles one CTA works through
constexpr int kOperandBytes = kTileRows * kHeadDim * 2;      // 32 KB: a 128 x 128 fp16 operand
constexpr int kSmemBytes = 2 * kOperandBytes;        // P and one tile of X
constexpr uint32_t kLboBytes = 128;                  // between core matrices along K
constexpr uint32_t kSboBytes = 16 * 128;             // between groups of 8 rows: 16 core matrices of 128 bytes
constexpr int kTmemColumns = 128;                    // one 128 x 128 fp32 accumulator

// Byte offset of the 16-byte piece (row, piece) of a K-major operand without swizzle: piece = 8 consecutive K elements.
__device__ __forceinline__ uint32_t operand_offset(int row, int piece)
{
    return (uint32_t)((row >> 3) * kSboBytes + piece * kLboBytes + (row & 7) * 16);
}

__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void *gsrc)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gsrc) : "memory");
}

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

// Codes of 32 consecutive stored channels against (hf, zf): BITS words, code j in bits [j*BITS, (j+1)*BITS) of the run.
// code = clamp(rint(RN((x - z) / h)), 0, qmax) with IEEE division.  Instead of dividing, u = sat(d * RN(RN(1/h) / qmax))
// is the clamped quotient on the scale [0, 1], within 5 * 2^-24 relative of the IEEE quotient / qmax; wherever every
// value within 2^-18 relative of it rounds to the same integer, that integer is the code.  The test is two FMAs onto
// 1.5 * 2^23 (the low mantissa bits of the sum are then the rounded integer, ties to even, like rintf), one with the
// quotient scaled down and one scaled up by 2^-18; both results are packed, and fields in which the two packed rows
// differ are elements in doubt (a quotient next to k + 0.5, exact ties included).  Those are redone by the defining
// formula: the warp walks the union of its doubtful columns, re-reads each from tensor memory (taddr = this warp's
// lanes, first column of the run) and the lanes concerned patch their field.  Every lane of the warp must call this.
template <int BITS>
__device__ __forceinline__ void quantize32(const float (&x)[32], float hf, float zf, uint32_t taddr, uint32_t (&words)[BITS])
{
    constexpr int qmax = (1 << BITS) - 1, PER_WORD = 32 / BITS;
    constexpr float MAGIC = 12582912.0f;                       // 0x4B400000
    constexpr float UP = (float)qmax * (1.0f + 3.814697265625e-06f), DN = (float)qmax * (1.0f - 3.814697265625e-06f);   // exact products
    uint32_t kconst = 0u;
#pragma unroll
    for (int j = 0; j < PER_WORD; ++j) kconst += 0x4B400000u << (j * BITS);
    const float r = hf != 0.0f ? __fmul_rn(__frcp_rn(hf), 1.0f / (float)qmax) : 0.0f;      // degenerate group (h == 0): every code is 0
    uint32_t wb[BITS];
#pragma unroll
    for (int i = 0; i < BITS; ++i) {
        words[i] = 0u - kconst;      // the constant bits of 1.5 * 2^23 come out of the sums (modulo 2^32)
        wb[i] = 0u - kconst;
    }
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const float u = mul_sat(__fsub_rn(x[j], zf), r);
        words[j / PER_WORD] += __float_as_uint(__fmaf_rn(u, DN, MAGIC)) << ((j % PER_WORD) * BITS);
        wb[j / PER_WORD] += __float_as_uint(__fmaf_rn(u, UP, MAGIC)) << ((j % PER_WORD) * BITS);
    }
    uint32_t any = 0u;
#pragma unroll
    for (int i = 0; i < BITS; ++i) {
        wb[i] ^= words[i];           // non-zero fields: elements in doubt
        any |= wb[i];
    }
    if (__any_sync(0xffffffffu, any != 0u)) {
#pragma unroll
        for (int i = 0; i < BITS; ++i) {
            uint32_t todo = __reduce_or_sync(0xffffffffu, wb[i]);      // the same for every lane: the loop is uniform
            while (todo) {
                const int f = (__ffs(todo) - 1) / BITS;                // field of this word = column i * PER_WORD + f of the run
                const uint32_t field = (uint32_t)qmax << (f * BITS);
                todo &= ~field;
                float xv;
                tmem_ld1(taddr + i * PER_WORD + f, xv);
                tmem_wait_ld();
                if (wb[i] & field) {
                    float c = hf != 0.0f ? rintf(__fdiv_rn(__fsub_rn(xv, zf), hf)) : 0.0f;
                    c = fminf(fmaxf(c, 0.0f), (float)qmax);
                    words[i] = (words[i] & ~field) | ((uint32_t)(int)c << (f * BITS));
                }
            }
        }
    }
}

template <int G>
__global__ void __launch_bounds__(kTileRows, 3) append_tile_kernel(AppendArgs a)
{
    constexpr int NG = kHeadDim / G;
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ __align__(8) uint64_t bar_sh;
    __shared__ uint32_t tmem_sh;
    __shared__ int fail_sh;
    const Shape &s = a.s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.z, tensor = blockIdx.x & 1, h = blockIdx.y;
    const int L0 = a.c.lengths[b];
    const int n_b = seq_new_count(a, b);
    const int L1 = L0 + n_b;
    if (n_b == 0 || L1 > s.max_tokens) return;       // uniform over the CTA; overflow is reported by the bookkeeping kernel
    int f0, f1;
    bulk_range(L0, s.n_sink, max(L1 - s.W, 0), f0, f1);
    const int n_tiles = (f1 - f0 + kTileRows - 1) / kTileRows;
    const int t_begin = (blockIdx.x >> 1) * kTilesPerCta, t_end = min(n_tiles, t_begin + kTilesPerCta);
    if (t_begin >= t_end) return;
    if (!SKVQ_IN_BOUNDS(f0 >= L0 && f1 <= s.cap && f1 - L0 <= a.n_new, a.c.status)) return;

    const int bits = tensor ? s.v_bits : s.k_bits;
    const bool f8 = s.meta_fp8 != 0;
    const size_t bh = (size_t)b * s.Hkv + h;
    const size_t tok_stride = (size_t)s.Hkv * kHeadDim;
    const __half *src = (tensor ? a.v : a.k) + ((size_t)b * a.n_new * s.Hkv + h) * kHeadDim;      // token L0 of this sequence and head
    const int32_t *idx = (tensor ? a.c.reorder_v : a.c.reorder_k) + (size_t)h * kHeadDim;
    const float *alpha = (tensor ? a.c.alpha_v : a.c.alpha_k) + (size_t)h * NG;
    const uint32_t gmap = granule_groups(tensor ? a.c.bounds_v : a.c.bounds_k, h, G, NG);      // group of every 32-channel granule
    uint8_t *codes = (tensor ? a.c.v_codes : a.c.k_codes) + bh * (size_t)s.cap * packed_row_bytes(bits);
    uint8_t *meta = reinterpret_cast<uint8_t *>(tensor ? a.c.v_meta : a.c.k_meta) + bh * (size_t)s.cap * NG * (f8 ? 2 : 4);

    uint8_t *P = smem, *X = smem + kOperandBytes;
    const uint32_t bar = smem_u32(&bar_sh);

    // ---- once per CTA: the permutation operand, the tensor memory, the barrier
    {
        uint4 *p4 = reinterpret_cast<uint4 *>(P);
#pragma unroll
        for (int i = 0; i < kOperandBytes / 16 / kTileRows; ++i) p4[tid + i * kTileRows] = make_uint4(0u, 0u, 0u, 0u);
    }
    if (warp == 0) tmem_alloc(smem_u32(&tmem_sh), kTmemColumns);
    if (tid == 0) {
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fail_sh = 0;
    }
    __syncthreads();
    {
        const int k = idx[tid] & (kHeadDim - 1);      // stored channel tid takes source channel k: P[tid][k] = 1
        *reinterpret_cast<__half *>(P + operand_offset(tid, k >> 3) + (k & 7) * 2) = __float2half(1.0f);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_sh;
    const uint32_t tmem_row = tmem + ((uint32_t)(warp * 32) << 16);      // this warp's 32 lanes

    // Copies of tile t: warp w moves pieces 4w .. 4w+3 (64 consecutive bytes) of every row; a warp instruction covers 8
    // rows x 4 pieces = four whole core matrices in shared memory.  Rows past the end of the range are left as they are
    // (their products only reach their own accumulator rows, which nobody stores).
    auto issue_copies = [&](int t) {
        const int tok0 = f0 + (t_begin + t) * kTileRows;
        const int rows = min(kTileRows, f1 - tok0);
        const int piece = 4 * warp + (lane >> 3);
        const __half *g = src + (size_t)(tok0 - L0 + (lane & 7)) * tok_stride + piece * 8;
        const uint32_t dst = smem_u32(X) + operand_offset(lane & 7, piece);
#pragma unroll
        for (int i = 0; i < kTileRows / 8; ++i)
            if (8 * i < rows) cp_async16(dst + i * kSboBytes, g + (size_t)(8 * i) * tok_stride);      // rows is a multiple of 64
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    const int T = t_end - t_begin;
    const uint64_t dX = smem_desc(smem_u32(X), kLboBytes, kSboBytes), dP = smem_desc(smem_u32(P), kLboBytes, kSboBytes);
    constexpr uint32_t kIdesc = idesc_f16_f32(kTileRows, kHeadDim);
    issue_copies(0);

    for (int t = 0; t < T; ++t) {
        // ---- tile t has landed: make it visible to the tensor core, which also has finished with the accumulators'
        // previous contents once every thread is here
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        proxy_fence();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < kHeadDim / 16; ++ks)      // 16 source channels = two core matrices per k-step
                umma_f16(tmem, dX + ((ks * 2 * kLboBytes) >> 4), dP + ((ks * 2 * kLboBytes) >> 4), kIdesc, ks > 0 ? 1u : 0u);
            umma_commit(bar);
        }
        if (!mbar_wait_bounded(bar, (uint32_t)t & 1u)) fail_sh = 1;
        tc_fence_after();
        if (__syncthreads_or(fail_sh)) break;                 // a uniform decision; also: every thread knows the buffer is free
        if (t + 1 < T) issue_copies(t + 1);                   // in flight while this tile is quantized

        // ---- this thread's token
        const int tok = f0 + (t_begin + t) * kTileRows + tid;
        const bool valid = tok < f1;
        float x[32];
        float mn[kGranules], mx[kGranules];
#pragma unroll
        for (int gr = 0; gr < kGranules; ++gr) {
            tmem_ld32(tmem_row + 32 * gr, x);
            tmem_wait_ld();
            float lo = x[0], hi = x[0];
#pragma unroll
            for (int j = 1; j < 32; ++j) {
                lo = fminf(lo, x[j]);
                hi = fmaxf(hi, x[j]);
            }
            mn[gr] = lo;
            mx[gr] = hi;
        }
        float hf[NG], zf[NG];
        uint32_t hz[NG];
#pragma unroll
        for (int g = 0; g < NG; ++g) {
            float lo = CUDART_INF_F, hi = -CUDART_INF_F;
#pragma unroll
            for (int gr = 0; gr < kGranules; ++gr)
                if (((gmap >> (2 * gr)) & 3u) == (uint32_t)g) {
                    lo = fminf(lo, mn[gr]);
                    hi = fmaxf(hi, mx[gr]);
                }
            group_parameters(lo, hi, alpha[g], (float)code_max(bits), f8, hz[g], hf[g], zf[g]);
        }
        // second pass: the codes, 32 channels at a time, and the packed row (the code width is a compile-time constant
        // inside, so that the row stays in registers)
        auto quantize_row = [&](auto bits_tag) {
            constexpr int BITS = decltype(bits_tag)::value;
            uint32_t *crow = reinterpret_cast<uint32_t *>(codes + (size_t)tok * packed_row_bytes(BITS));
#pragma unroll 1      // rolled on purpose: one copy of the arithmetic in the instruction cache
            for (int gr = 0; gr < kGranules; ++gr) {
                tmem_ld32(tmem_row + 32 * gr, x);
                tmem_wait_ld();
                const uint32_t g = (gmap >> (2 * gr)) & 3u;
                float hg = hf[0], zg = zf[0];
#pragma unroll
                for (int i = 1; i < NG; ++i)
                    if (g == (uint32_t)i) { hg = hf[i]; zg = zf[i]; }
                uint32_t cw[BITS];
                quantize32<BITS>(x, hg, zg, tmem_row + 32 * gr, cw);
                if (valid) {
                    if constexpr (BITS == 2) *reinterpret_cast<uint2 *>(crow + 2 * gr) = make_uint2(cw[0], cw[1]);
                    else *reinterpret_cast<uint4 *>(crow + 4 * gr) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
                }
            }
        };
        if (bits == 2) quantize_row(std::integral_constant<int, 2>{});
        else quantize_row(std::integral_constant<int, 4>{});
        tc_fence_before();
        if (valid) {
            if (f8) {
                uint16_t *m = reinterpret_cast<uint16_t *>(meta + (size_t)tok * NG * 2);
#pragma unroll
                for (int g = 0; g < NG; ++g) m[g] = (uint16_t)hz[g];
            } else {
                uint32_t *m = reinterpret_cast<uint32_t *>(meta + (size_t)tok * NG * 4);
                if constexpr (NG == 4) *reinterpret_cast<uint4 *>(m) = make_uint4(hz[0], hz[1], hz[2], hz[3]);
                else if constexpr (NG == 2) *reinterpret_cast<uint2 *>(m) = make_uint2(hz[0], hz[1]);
                else m[0] = hz[0];
            }
        }
    }

    // ---- leave: nothing of this CTA is in flight any more (a failed wait still drains its own copies)
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (fail_sh && tid == 0 && a.c.status) atomicOr(a.c.status, SKVQ_STATUS_COPY_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemColumns);
}

}  // namespace

cudaError_t launch_append_tiles(const AppendArgs &a, cudaStream_t stream)
{
    const Shape &s = a.s;
    const int max_tiles = (a.n_new + kTileRows - 1) / kTileRows;
    dim3 grid(2 * ((max_tiles + kTilesPerCta - 1) / kTilesPerCta), s.Hkv, s.B);      // x: (run of tiles, tensor)
    static unsigned long long configured[3] = {0, 0, 0};      // one bit per device, per instantiation
    cudaError_t e;
    if (s.G == 128) {
        e = configure_smem_once(append_tile_kernel<128>, kSmemBytes, configured[0]);
        if (e != cudaSuccess) return e;
        append_tile_kernel<128><<<grid, kTileRows, kSmemBytes, stream>>>(a);
    } else if (s.G == 64) {
        e = configure_smem_once(append_tile_kernel<64>, kSmemBytes, configured[1]);
        if (e != cudaSuccess) return e;
        append_tile_kernel<64><<<grid, kTileRows, kSmemBytes, stream>>>(a);
    } else {
        e = configure_smem_once(append_tile_kernel<32>, kSmemBytes, configured[2]);
        if (e != cudaSuccess) return e;
        append_tile_kernel<32><<<grid, kTileRows, kSmemBytes, stream>>>(a);
    }
    return cudaGetLastError();
}

}  // namespace skvq

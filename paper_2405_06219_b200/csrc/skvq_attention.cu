// skvq_decode_attention: softmax(q K~^T) V~ of one query per sequence over
// [packed quantized prefix || fp16 window] (Eq. 1, Algorithm 1), split along the sequence
// (flash-decoding) with a log-sum-exp merge.  Dequantization happens in registers.
//
// Per (sequence, KV head, split) one CTA serves all rep = Hq/Hkv query heads that share the
// KV head.  It never forms h*code+z per element for the scores: with q' the permuted query,
//   q'.K~_t = sum_g h_{t,g} (sum_{j in g} q'_j c_{t,j}) + sum_g z_{t,g} (sum_{j in g} q'_j)
// so the zero points cost one multiply-add per group.  Scores live in the log2 domain
// (sm_scale*log2(e) folded into q').  Partials (o'[128], m, l) of the quantized prefix go to the
// caller's workspace; merge_kernel walks the fp16 window itself, combines everything, divides by
// the softmax denominator, undoes the value permutation and writes fp16.
#include <math_constants.h>

#include <type_traits>

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

// Field j (BITS wide) of a row held as 32-bit words of a little-endian bit stream; a 3-bit field may span two words.
template <int BITS>
__device__ __forceinline__ uint32_t stream_field(const uint32_t *w, int j)
{
    const int bit = j * BITS, i = bit >> 5, sh = bit & 31;
    uint32_t v = w[i] >> sh;
    if (sh + BITS > 32) v |= w[i + 1] << (32 - sh);      // never past the row: 128 * BITS is a multiple of 32
    return v & ((1u << BITS) - 1u);
}

// Scalar partition kernel (what the tensor-core kernels do not cover: 3-bit codes, groups of unequal width, 4-bit
// codes with several query heads per KV head or groups of 32): one thread per token for the scores, one per channel
// for P.V.  Scale and zero point are applied per 32-channel granule, whose group comes from a small map, so equal and
// unequal groups take the same path.
template <int KBITS, int VBITS>
__global__ void __launch_bounds__(kThreads) partition_kernel(AttnArgs a)
{
    const Shape &s = a.s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rep = s.rep, ng = s.ng;
    // Order matters: the merge kernel reads the lengths, the sinks and the window BEFORE its own wait, so it may only be
    // scheduled once everything in front of this grid (append, bookkeeping, plan) has completed and is visible.  Waiting
    // first and triggering afterwards gives exactly that; the merge kernel still runs under this kernel's body.
    asm volatile("griddepcontrol.wait;" ::: "memory");      // the lengths, and the plan kernel's header when there is one
    asm volatile("griddepcontrol.launch_dependents;");      // the merge kernel may start its window part now

    __shared__ __align__(16) Segment seg_sh;
    __shared__ int more_sh;
    __shared__ SlotWalker walk;      // only thread 0 touches it; shared memory keeps it out of everybody's registers
    __shared__ __align__(16) int hdr_sh[kPlanSmemInts];
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

    __shared__ float sq[kMaxRep][kHeadDim];        // permuted query, times sm_scale*log2(e)
    __shared__ float sqsum[kMaxRep][kGranules];    // per-granule sums of the above
    __shared__ float sp[kMaxRep][kTile];           // probabilities of the current tile
    __shared__ float sred[kMaxRep][kThreads / 32];

    for (;;) {
    if (tid == 0) seg_sh = walk.next(a.c.lengths, s.W, a.plan.lq_cap);
    __syncthreads();
    const int b = seg_sh.b, hk = seg_sh.hk, q_begin = seg_sh.tok_begin, q_end = seg_sh.tok_end, part_idx = seg_sh.part;
    if (!segment_in_bounds(seg_sh, s, a.plan, a.c.status)) break;      // checked build only; uniform: every thread reads the same segment
    const size_t bh = (size_t)b * s.Hkv + hk;
    const int32_t *idx_k = a.c.reorder_k + (size_t)hk * kHeadDim;
    for (int r = 0; r < rep; ++r) {
        const __half *qrow = a.q + ((size_t)b * s.Hq + hk * rep + r) * kHeadDim;
        sq[r][tid] = __half2float(qrow[idx_k[tid] & (kHeadDim - 1)]) * a.scale_log2;
    }
    __syncthreads();
    if (tid < rep * kGranules) {
        const int r = tid / kGranules, gr = tid % kGranules;
        float acc = 0.f;
        for (int j = gr * kGranule; j < (gr + 1) * kGranule; ++j) acc += sq[r][j];
        sqsum[r][gr] = acc;
    }
    const uint32_t kmap = granule_groups(a.c.bounds_k, hk, s.G, ng), vmap = granule_groups(a.c.bounds_v, hk, s.G, ng);
    __syncthreads();

    constexpr int KROW = kHeadDim * KBITS / 8, VROW = kHeadDim * VBITS / 8;
    const uint8_t *k_codes = a.c.k_codes + bh * (size_t)s.cap * KROW;
    const uint8_t *v_codes = a.c.v_codes + bh * (size_t)s.cap * VROW;
    // {h, z} of row r, group g: a half2, or two E4M3 bytes (every E4M3 value is an fp16 value)
    const bool f8 = s.meta_fp8 != 0;
    auto load_hz = [&](const __half2 *base, size_t idx) -> float2 {
        if (!f8) return __half22float2(base[idx]);
        const uint16_t b = reinterpret_cast<const uint16_t *>(base)[idx];
        uint32_t r;
        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(b));
        return __half22float2(*reinterpret_cast<const __half2 *>(&r));
    };
    const size_t meta0 = bh * (size_t)s.cap * ng;
    const __half2 *k_meta = a.c.k_meta, *v_meta = a.c.v_meta;

    float m_run[kMaxRep], l_thread[kMaxRep], acc[kMaxRep];
#pragma unroll
    for (int r = 0; r < kMaxRep; ++r) { m_run[r] = -CUDART_INF_F; l_thread[r] = 0.f; acc[r] = 0.f; }

    {
        const int t_begin = q_begin, t_end = q_end;
        for (int tile0 = t_begin; tile0 < t_end; tile0 += kTile) {
            const int t = tile0 + tid;
            const bool valid = t < t_end && t >= s.n_sink;      // sinks belong to the merge kernel
            float sc[kMaxRep];
#pragma unroll
            for (int r = 0; r < kMaxRep; ++r) sc[r] = -CUDART_INF_F;
            if (valid) {
#pragma unroll
                for (int r = 0; r < kMaxRep; ++r) sc[r] = 0.f;
                const uint4 *row4 = reinterpret_cast<const uint4 *>(k_codes + (size_t)t * KROW);      // rows are multiples of 16 bytes
                constexpr int GW = kGranule * KBITS / 32;      // words per granule: its 32 fields start on a word boundary
#pragma unroll
                for (int gr = 0; gr < kGranules; ++gr) {
                    uint32_t w[GW];
#pragma unroll
                    for (int i = 0; i < GW; ++i) {
                        const int wi = gr * GW + i;
                        const uint4 x = __ldg(row4 + (wi >> 2));
                        w[i] = (wi & 3) == 0 ? x.x : (wi & 3) == 1 ? x.y : (wi & 3) == 2 ? x.z : x.w;
                    }
                    float part[kMaxRep];
#pragma unroll
                    for (int r = 0; r < kMaxRep; ++r) part[r] = 0.f;
#pragma unroll
                    for (int jj = 0; jj < kGranule; ++jj) {
                        const float code = (float)stream_field<KBITS>(w, jj);
#pragma unroll
                        for (int r = 0; r < kMaxRep; ++r)
                            if (r < rep) part[r] = fmaf(sq[r][gr * kGranule + jj], code, part[r]);
                    }
                    const float2 hz = load_hz(k_meta, meta0 + (size_t)t * ng + ((kmap >> (2 * gr)) & 3u));
#pragma unroll
                    for (int r = 0; r < kMaxRep; ++r)
                        if (r < rep) sc[r] += hz.x * part[r] + hz.y * sqsum[r][gr];
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
                    corr[r] = m_new == -CUDART_INF_F ? 1.f : exp2f(m_run[r] - m_new);   // 0 on the first tile with a token
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
            {
                const int g = (vmap >> (2 * (tid >> 5))) & 3u;
                const int bit = tid * VBITS, wi = bit >> 5, sh = bit & 31;
                const bool two = sh + VBITS > 32;      // a 3-bit field that runs into the next word of its row
                for (int tt = max(s.n_sink - tile0, 0); tt < n_tok; ++tt) {      // rows of sinks hold unspecified bytes
                    const size_t row = (size_t)(tile0 + tt);
                    const uint32_t *rw = reinterpret_cast<const uint32_t *>(v_codes + row * VROW);
                    uint32_t word = __ldg(rw + wi) >> sh;
                    if (two) word |= __ldg(rw + wi + 1) << (32 - sh);
                    const float2 hz = load_hz(v_meta, meta0 + row * ng + g);
                    const float val = fmaf(hz.x, (float)(word & ((1u << VBITS) - 1u)), hz.y);
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
            float *part = partials + (((size_t)b * s.Hq + hk * rep + r) * a.plan.s_max + part_idx) * kPartialStride;
            part[tid] = acc[r];
            if (tid == 0) {
                float l = 0.f;
                for (int w = 0; w < kThreads / 32; ++w) l += sred[r][w];
                part[kHeadDim] = m_run[r];
                part[kHeadDim + 1] = l;
            }
        }
    }
    __syncthreads();          // the segment's shared data is dead; thread 0 decides whether there is another one
    if (tid == 0) more_sh = walk.done() ? 0 : 1;
    __syncthreads();
    if (!more_sh) break;
    }
}

// Writes the workspace header of the flat partition: units (256 quantized tokens) per sequence as an exclusive
// prefix array, their total over all KV heads, and the units per slot.  One warp; B is small next to the cache.
__global__ void plan_kernel(AttnArgs a)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");      // whatever wrote the lengths (the append kernels, typically)
    asm volatile("griddepcontrol.launch_dependents;");      // the partition kernel may be scheduled; it waits for this grid before it reads the header
    int *hdr = reinterpret_cast<int *>(a.ws);
    int *pre = hdr + kPlanHdrInts;
    const int lane = threadIdx.x & 31;
    __shared__ int ups_sh;
    if (threadIdx.x < 32) {
    int run = 0;
    for (int base = 0; base < a.s.B; base += 32) {
        const int b = base + lane;
        int nu = 0;
        if (b < a.s.B) nu = (min(max(a.c.lengths[b] - a.s.W, 0), a.plan.lq_cap) + kUnitTok - 1) / kUnitTok;
        int incl = nu;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += v;
        }
        if (b < a.s.B) pre[b] = run + incl - nu;
        run += __shfl_sync(0xffffffffu, incl, 31);
    }
    const long long total = (long long)run * a.s.Hkv;
    const int ups = (int)max((total + a.plan.n_slots - 1) / a.plan.n_slots, 1LL);
    if (lane == 0) {
        pre[a.s.B] = run;
        hdr[0] = (int)total;
        hdr[1] = ups;
        ups_sh = ups;
    }
    }
    __syncthreads();
    // first sequence of every slot: the largest b with Hkv * pre[b] <= w * ups (for slots past the end: unused)
    int *slot_b = pre + a.s.B + 1;
    for (int w = threadIdx.x; w < a.plan.n_slots; w += blockDim.x) {
        const long long f = (long long)w * ups_sh;
        int lo = 0, hi = a.s.B - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if ((long long)a.s.Hkv * pre[mid] <= f) lo = mid; else hi = mid - 1;
        }
        slot_b[w] = lo;
    }
}

// One CTA per (query head, sequence): walks the fp16 rows -- the attention sinks that have left the window, then
// the window -- and then combines that with the split partials of the quantized prefix.  Every row is read with
// coalesced 16-byte loads (16 lanes per 256-byte row, two rows per warp instruction), keys and values alike; a lane
// keeps its eight channels of the permuted query and of the running value sums in registers.
constexpr int kMergeTile = 64;      // rows per pass: 4 warps x 8 row pairs, all 16 loads of a lane in flight at once
__global__ void __launch_bounds__(kHeadDim) merge_kernel(AttnArgs a)
{
    const int hq = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const Shape &s = a.s;
    const int hk = hq / s.rep;
    const int W = s.W;
    // Read before this kernel's own griddepcontrol.wait: safe because every partition kernel (and the plan kernel) waits for
    // its predecessors BEFORE it lets its dependents be scheduled, so by the time a CTA of this grid runs, the append and
    // bookkeeping kernels in front of the partition kernel have completed and their writes (lengths, ring, sinks) are visible.
    const int L = a.c.lengths[b];
    const int Lq = max(L - W, 0);
    __shared__ __align__(16) float sq[kHeadDim];
    __shared__ float sp[kMergeTile];
    __shared__ float sred[kThreads / 32];
    __shared__ __align__(16) int hdr_sh[kPlanSmemInts];
    if (a.plan.in_kernel && warp == 0)      // the same header the partition CTAs derived; published by the barriers below
        plan_in_warp(a.c.lengths, s.B, s.Hkv, s.W, a.plan.lq_cap, a.plan.n_slots, hdr_sh);
    const size_t bh = (size_t)b * s.Hkv + hk;
    sq[tid] = __half2float(a.q[((size_t)b * s.Hq + hq) * kHeadDim + (a.c.reorder_k[(size_t)hk * kHeadDim + tid] & (kHeadDim - 1))]) *
              a.scale_log2;
    __syncthreads();
    __shared__ __align__(16) float sacc[kThreads / 32][kHeadDim];      // written with 16-byte stores
    const int vsub = lane >> 4, vchunk = lane & 15;                    // row of the pair, 16-byte piece of the row
    float q8[8];
    {
        const float4 qa = *reinterpret_cast<const float4 *>(&sq[8 * vchunk]), qb = *reinterpret_cast<const float4 *>(&sq[8 * vchunk + 4]);
        q8[0] = qa.x; q8[1] = qa.y; q8[2] = qa.z; q8[3] = qa.w; q8[4] = qb.x; q8[5] = qb.y; q8[6] = qb.z; q8[7] = qb.w;
    }
    float m_run = -CUDART_INF_F, l_thread = 0.f;
    float a8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    // Online softmax over the fp16 rows of tokens [t_begin, t_end): row of token t = t % ring (ring > 0) or t.
    auto walk = [&](const __half *k_rows, const __half *v_rows, int t_begin, int t_end, int ring) {
    for (int tile0 = t_begin; tile0 < t_end; tile0 += kMergeTile) {
        // this lane's rows of the tile: tt = 2 * (warp + 4 i) + vsub, i = 0..7
        const int tt0 = 2 * warp + vsub;
        int r0 = tile0 + tt0;
        if (ring) r0 %= ring;
        uint4 ku[kMergeTile / 8], vu[kMergeTile / 8];
        int rows[kMergeTile / 8];
#pragma unroll
        for (int i = 0; i < kMergeTile / 8; ++i) {
            int r = r0 + 8 * i;
            if (ring) r = ring >= kMergeTile ? (r >= ring ? r - ring : r) : r % ring;
            rows[i] = r;
            ku[i] = make_uint4(0u, 0u, 0u, 0u);
            if (tile0 + tt0 + 8 * i < t_end) ku[i] = __ldg(reinterpret_cast<const uint4 *>(k_rows + (size_t)r * kHeadDim) + vchunk);
        }
        // the value rows do not depend on the scores: fetch them behind the key rows
#pragma unroll
        for (int i = 0; i < kMergeTile / 8; ++i) {
            vu[i] = make_uint4(0u, 0u, 0u, 0u);
            if (tile0 + tt0 + 8 * i < t_end) vu[i] = __ldg(reinterpret_cast<const uint4 *>(v_rows + (size_t)rows[i] * kHeadDim) + vchunk);
        }
#pragma unroll
        for (int i = 0; i < kMergeTile / 8; ++i) {
            const __half2 *h2 = reinterpret_cast<const __half2 *>(&ku[i]);
            float d = 0.f;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 kv = __half22float2(h2[e]);
                d = fmaf(q8[2 * e], kv.x, fmaf(q8[2 * e + 1], kv.y, d));
            }
#pragma unroll
            for (int msk = 8; msk > 0; msk >>= 1) d += __shfl_xor_sync(0xffffffffu, d, msk);      // over the 16 lanes of the row
            if (vchunk == 0) sp[tt0 + 8 * i] = (tile0 + tt0 + 8 * i < t_end) ? d : -CUDART_INF_F;
        }
        __syncthreads();
        const float tm = warp_max(fmaxf(sp[lane], sp[lane + 32]));      // every warp finds the same tile maximum
        const float m_new = fmaxf(m_run, tm);               // finite: the tile has a valid token
        const float corr = exp2f(m_run - m_new);            // exp2(-inf) = 0 on the first tile
        l_thread *= corr;
        m_run = m_new;
#pragma unroll
        for (int e = 0; e < 8; ++e) a8[e] *= corr;
#pragma unroll
        for (int i = 0; i < kMergeTile / 8; ++i) {
            const float pt = exp2f(sp[tt0 + 8 * i] - m_new);      // 0 past the end (score -inf); the 16 lanes of a row agree
            if (vchunk == 0) l_thread += pt;                      // once per row
            const __half2 *h2 = reinterpret_cast<const __half2 *>(&vu[i]);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 vv = __half22float2(h2[e]);
                a8[2 * e] = fmaf(pt, vv.x, a8[2 * e]);
                a8[2 * e + 1] = fmaf(pt, vv.y, a8[2 * e + 1]);
            }
        }
        __syncthreads();   // sp is rewritten by the next tile
    }
    };
    // attention sinks that have left the window (fp16 copies), then the window itself
    const int n_s = min(s.n_sink, Lq);
    if (n_s > 0) walk(a.c.k_sink + bh * (size_t)s.n_sink * kHeadDim, a.c.v_sink + bh * (size_t)s.n_sink * kHeadDim, 0, n_s, 0);
    if (W > 0) walk(a.c.k_win + bh * (size_t)W * kHeadDim, a.c.v_win + bh * (size_t)W * kHeadDim, Lq, L, W);
#pragma unroll
    for (int i = 0; i < 8; ++i) a8[i] += __shfl_xor_sync(0xffffffffu, a8[i], 16);
    if (vsub == 0) {
        *reinterpret_cast<float4 *>(&sacc[warp][8 * vchunk]) = make_float4(a8[0], a8[1], a8[2], a8[3]);
        *reinterpret_cast<float4 *>(&sacc[warp][8 * vchunk + 4]) = make_float4(a8[4], a8[5], a8[6], a8[7]);
    }
    const float lw = warp_sum(l_thread);
    if (lane == 0) sred[warp] = lw;
    __syncthreads();
    float l_win = 0.f, acc = 0.f;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) { l_win += sred[w]; acc += sacc[w][tid]; }

    // The window above does not depend on the partition kernel; its partials do: wait for that grid here
    // (a no-op unless this kernel was launched with programmatic stream serialization).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // log-sum-exp merge: the window and the S split partials; thread d owns reordered channel d
    int S = pair_partials(a.plan.in_kernel ? hdr_sh : reinterpret_cast<const int *>(a.ws), s.Hkv, b, hk);
    if (!SKVQ_IN_BOUNDS(S >= 0 && S <= a.plan.s_max, a.c.status)) S = 0;
    const float *part = a.ws + a.plan.hdr_ints + ((size_t)b * s.Hq + hq) * a.plan.s_max * kPartialStride;
    float M = m_run;
    for (int i = 0; i < S; ++i) M = fmaxf(M, part[(size_t)i * kPartialStride + kHeadDim]);
    float o = 0.f, l = 0.f;
    if (M > -CUDART_INF_F) {
        const float ww = exp2f(m_run - M);
        o = acc * ww;
        l = l_win * ww;
        for (int i = 0; i < S; ++i) {
            const float *p = part + (size_t)i * kPartialStride;
            const float w = exp2f(p[kHeadDim] - M);
            o = fmaf(p[tid], w, o);
            l = fmaf(p[kHeadDim + 1], w, l);
        }
    }
    const float res = l > 0.f ? o / l : 0.f;
    const int dst = a.c.reorder_v[(size_t)hk * kHeadDim + tid] & (kHeadDim - 1);
    a.out[((size_t)b * s.Hq + hq) * kHeadDim + dst] = __float2half_rn(res);
}

}  // namespace

// Resident CTAs per SM of the partition kernel that serves this shape (sets how many CTAs make one wave).
// Resident CTAs per SM of the partition kernel that serves this shape (sets how many CTAs make one wave).  It must not
// depend on whether group boundaries are given: the workspace is sized from the configuration alone.
static int partition_ctas_per_sm(const Shape &s)
{
    if (s.k_bits == 3 || s.v_bits == 3) return 8;                              // scalar kernel
    if (s.rep == 1 && s.G >= 64) return s.k_bits == s.v_bits ? 4 : 3;           // integer kernel
    if (s.k_bits == 2 && s.v_bits == 2 && (s.rep == 3 || (s.rep > 4 && s.rep <= 8)) && (s.G == 128 || s.G == 64 || s.G == 32))
        return 3;                                                              // tcgen05 kernel: 128 tensor-memory columns, 69 KB
    if (s.k_bits == 2 && s.v_bits == 2 && s.rep <= 4) return 2;                // grouped-query kernel, 244 registers
    return 8;                                                                  // scalar kernel
}

int current_device()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) {
        (void)cudaGetLastError();
        dev = 0;
    }
    return dev;
}

int sm_count()
{
    static int n[kMaxDevices] = {};        // per device: a process may drive GPUs of different sizes
    const int dev = current_device() & (kMaxDevices - 1);
    if (n[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
            n[dev] = v;
        else
            n[dev] = 148;
        (void)cudaGetLastError();
    }
    return n[dev];
}

SplitPlan plan_splits(const Shape &s, int max_len, int requested_splits)
{
    SplitPlan p;
    p.lq_cap = max_len - s.W > 0 ? max_len - s.W : 0;
    const long units = ((long)p.lq_cap + kUnitTok - 1) / kUnitTok;     // per (sequence, KV head), at most
    const long pairs = (long)s.B * s.Hkv;
    const long total = units * pairs > 0 ? units * pairs : 1;
    long n;
    if (requested_splits > 0) {
        n = (long)requested_splits * pairs;
    } else {
        // every slot gets the same work, so one full wave is enough (a second wave costs a second prologue,
        // pipeline fill and epilogue: about 8 us measured)
        const long slots = (long)sm_count() * partition_ctas_per_sm(s);
        n = slots;
    }
    if (n > total) n = total;
    if (n > (1L << 20)) n = 1L << 20;
    p.n_slots = (int)n;
    // A pair of nu units spreads over at most floor(nu / ups) + 2 slots, and ups >= total / n_slots >= Hkv * nu / n_slots.
    long s_max = n / s.Hkv + 2;
    if (s_max > units) s_max = units > 0 ? units : 1;
    p.s_max = (int)s_max;
    p.in_kernel = s.B <= 32 ? 1 : 0;
    p.hdr_ints = p.in_kernel ? 0 : (kPlanHdrInts + s.B + 1 + p.n_slots + 63) / 64 * 64;
    return p;
}

// A launch that may start before the kernel in front of it on the stream has finished; the kernel itself waits
// (griddepcontrol.wait) where it first needs that kernel's results.
template <typename Kern, typename Args>
static cudaError_t launch_dependent(Kern kern, dim3 grid, dim3 block, size_t smem, cudaStream_t stream, bool overlap,
                                    const Args &args)
{
    cudaLaunchConfig_t lc = {};
    lc.gridDim = grid;
    lc.blockDim = block;
    lc.dynamicSmemBytes = smem;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = overlap ? 1 : 0;
    lc.attrs = attr;
    lc.numAttrs = 1;
    return cudaLaunchKernelEx(&lc, kern, args);
}

cudaError_t launch_attention(const Shape &s, const CachePtrs &c, const __half *q, __half *out, float sm_scale,
                             const SplitPlan &plan, float *workspace, cudaEvent_t ev_begin, cudaEvent_t ev_end,
                             cudaStream_t stream)
{
    AttnArgs a{s, c, q, out, sm_scale * 1.4426950408889634f, plan, workspace};
    cudaError_t e = cudaSuccess;
    if (!plan.in_kernel) {
        e = launch_dependent(plan_kernel, dim3(1), dim3(256), 0, stream, true, a);
        if (e != cudaSuccess) return e;
    }
    if (ev_begin) cudaEventRecord(ev_begin, stream);
    const bool overlap = !ev_begin;      // an event between two kernels serialises them anyway
    dim3 grid(plan.n_slots);
    bool handled = false;
    cudaError_t em = cudaSuccess;
    // the tensor-core kernels serve 2- and 4-bit codes; groups of unequal width when there are two per row (the integer
    // and the grouped-query kernel).  3-bit streams and the other unequal-group shapes take the scalar kernel.
    if (s.k_bits != 3 && s.v_bits != 3) {
        em = launch_partition_mma(s, c, q, a.scale_log2, plan, workspace, stream, overlap, &handled);
        if (em != cudaSuccess) return em;
        if (!handled) {
            em = launch_partition_gqa(s, c, q, a.scale_log2, plan, workspace, stream, overlap, &handled);
            if (em != cudaSuccess) return em;
        }
        if (!handled && !s.bounded) {
            em = launch_partition_tc(s, c, q, a.scale_log2, plan, workspace, stream, overlap, &handled);
            if (em != cudaSuccess) return em;
        }
    }
    if (!handled) {
        auto launch_scalar = [&](auto kb, auto vb) {
            return launch_dependent(partition_kernel<decltype(kb)::value, decltype(vb)::value>, grid, dim3(kThreads), 0, stream,
                                    overlap, a);
        };
        auto with_k = [&](auto kb) {
            switch (s.v_bits) {
                case 2: return launch_scalar(kb, std::integral_constant<int, 2>{});
                case 3: return launch_scalar(kb, std::integral_constant<int, 3>{});
                default: return launch_scalar(kb, std::integral_constant<int, 4>{});
            }
        };
        switch (s.k_bits) {
            case 2: em = with_k(std::integral_constant<int, 2>{}); break;
            case 3: em = with_k(std::integral_constant<int, 3>{}); break;
            default: em = with_k(std::integral_constant<int, 4>{}); break;
        }
    }
    if (em != cudaSuccess) return em;
    if (ev_end) cudaEventRecord(ev_end, stream);
    // merge CTAs may be scheduled while the last partition CTAs still run: they do the window part first and
    // wait before they read the partials
    e = launch_dependent(merge_kernel, dim3(s.Hq, s.B), dim3(kHeadDim), 0, stream, !ev_end, a);
    if (e != cudaSuccess) return e;
    count_launch(plan.in_kernel ? 2 : 3);
    return cudaGetLastError();
}

}  // namespace skvq

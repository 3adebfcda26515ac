// skvq_decode_attention: softmax(q K~^T) V~ of one query per sequence over
// [packed quantized prefix || fp16 window] (Eq. 1, Algorithm 1), split along the sequence
// (flash-decoding) with a log-sum-exp merge.  Dequantization happens in registers.
//
// This file holds what all partition kernels share -- the host side of the flat partition (plan_splits), the plan
// kernel, the dispatch -- and the merge kernel.  The partition kernels themselves (skvq_attention_mma.cu, _gqa.cu,
// _tc.cu) write partials (o'[128], m, l) of the quantized prefix to the caller's workspace; they never form
// h*code+z per element for the scores: with q' the permuted query,
//   q'.K~_t = sum_g h_{t,g} (sum_{j in g} q'_j c_{t,j}) + sum_g z_{t,g} (sum_{j in g} q'_j)
// so the zero points cost one multiply-add per group.  Scores live in the log2 domain (sm_scale*log2(e) folded into
// q').  merge_kernel walks the fp16 window itself, combines everything, divides by the softmax denominator, undoes
// the value permutation and writes fp16.
#include <math_constants.h>

#include "skvq_internal.cuh"

namespace skvq {
namespace {

constexpr int kThreads = 128;

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
    const bool integer = plain_width(s.k_bits) && (plain_width(s.v_bits) || s.v_bits == kTernary) && s.rep == 1 && s.G >= 64;
    if (integer) return s.k_bits == s.v_bits ? 4 : 3;           // integer kernel (three-level values are rewritten as 2-bit rows)
    if (s.k_bits == 2 && (s.v_bits == 2 || s.v_bits == kTernary) && (s.rep == 1 || s.rep == 2 || s.rep == 4)) return 2;   // grouped-query kernel, 244 registers
    return kTcCtasPerSm;      // tcgen05 kernel: 128 tensor-memory columns, at most 73 KB of shared memory
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
    // the integer and the grouped-query kernel serve 2- and 4-bit codes in equal groups, or in two groups of unequal
    // width per row; everything else (3-bit streams, three-level values, 4-bit with several query heads or groups of 32,
    // other unequal groups, 3 and 5-8 query heads per KV head) goes to the tcgen05 kernel
    if (plain_width(s.k_bits) && (plain_width(s.v_bits) || s.v_bits == kTernary)) {
        em = launch_partition_mma(s, c, q, a.scale_log2, plan, workspace, stream, overlap, &handled);
        if (em != cudaSuccess) return em;
        if (!handled) {
            em = launch_partition_gqa(s, c, q, a.scale_log2, plan, workspace, stream, overlap, &handled);
            if (em != cudaSuccess) return em;
        }
    }
    if (!handled) {
        em = launch_partition_tc(s, c, q, a.scale_log2, plan, workspace, stream, overlap, &handled);
        if (em != cudaSuccess) return em;
    }
    if (!handled) return cudaErrorInvalidValue;      // every configuration skvq_check_config accepts has a kernel above
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

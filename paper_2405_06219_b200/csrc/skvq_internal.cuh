// Private declarations shared by the translation units of libskvq (not installed).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "skvq.h"

namespace skvq {

constexpr int kHeadDim = 128;
constexpr int kMaxRep = 8;            // query heads per KV head supported by the kernels
constexpr int kPartialStride = 132;   // floats per split partial: o'[128], m (log2 domain), l, 2 pad
constexpr int kGranule = SKVQ_GROUP_GRANULE;          // group boundaries are multiples of this many channels
constexpr int kGranules = kHeadDim / kGranule;
constexpr int kTernary = SKVQ_BITS_TERNARY;           // the width value of the three-level code

// Bytes of one packed row of kHeadDim codes; largest code; is the width one of the plain power-of-two fields (2, 4)?
__host__ __device__ constexpr int packed_row_bytes(int bits) { return bits == kTernary ? (kHeadDim + 4) / 5 : kHeadDim * bits / 8; }
__host__ __device__ constexpr int code_max(int bits) { return bits == kTernary ? 2 : (1 << bits) - 1; }
__host__ __device__ constexpr bool plain_width(int bits) { return bits == 2 || bits == 4; }

// Dynamic shared memory of the tcgen05 partition kernel (two-slot rings of K codes and of V codes with both tensors'
// scale/zero, the MMA operands, folded sums, small arrays) for 128-token tiles.  Three CTAs of it fit an SM (3 x (73 KB +
// 1 KB reserved + statics) is what 227 KB hold); where the K and the V operand would not both fit beside the rings, they
// share one buffer (tc_shared_operand).
__host__ __device__ constexpr int tc_ring_bytes(int G, int k_bits, int v_bits)
{
    return 2 * 128 * packed_row_bytes(k_bits) + 2 * (128 * packed_row_bytes(v_bits) + 2 * 128 * (kHeadDim / G) * 4);
}
__host__ __device__ constexpr bool tc_shared_operand(int G, int k_bits, int v_bits)
{
    return tc_ring_bytes(G, k_bits, v_bits) + 2 * 128 * 128 + 16 * 128 + 128 * 64 + 4 * kHeadDim * 4 + 1024 > 74752;
}
__host__ __device__ constexpr int tc_smem_bytes(int G, int k_bits, int v_bits)
{
    return tc_ring_bytes(G, k_bits, v_bits) + (tc_shared_operand(G, k_bits, v_bits) ? 1 : 2) * 128 * 128 + 16 * 128 + 128 * 64 +
           4 * kHeadDim * 4 + 1024;
}
constexpr int kTcCtasPerSm = 3;

// Everything the kernels need, by value.
struct Shape {
    int B, Hq, Hkv, rep;   // rep = Hq / Hkv
    int k_bits, v_bits, G, ng;
    int W, cap, max_tokens;
    int n_sink;            // positions below this are kept fp16 in the sink store when they leave the window
    int meta_fp8;          // scale/zero stored as two E4M3 bytes per (token, group) instead of a half2
    int bounded;           // group boundaries of unequal width are given (CachePtrs::bounds_k / bounds_v)
};

struct CachePtrs {
    uint8_t *k_codes, *v_codes;
    __half2 *k_meta, *v_meta;
    __half *k_win, *v_win;
    int32_t *lengths;
    const int32_t *reorder_k, *reorder_v;
    const float *alpha_k, *alpha_v;
    int32_t *status;
    __half *k_sink, *v_sink;
    const int32_t *bounds_k, *bounds_v;      // [Hkv][ng+1] or NULL
};

// Flat partition of the quantized prefixes.  The unit is 256 tokens of one (sequence, KV head); all units of a
// call are laid end to end, ordered by (sequence, KV head, position), and cut into n_slots equal runs, one
// per CTA of the partition kernel.  A run may cross into the next KV head or sequence: each piece is a segment
// with its own partial.  Every CTA therefore does the same amount of work whatever the batch shape is.
constexpr int kUnitTok = 256;
constexpr int kPlanHdrInts = 4;    // workspace header: [0] total units, [1] units per slot, then the prefix array [B+1]
                                   // and the first sequence of every slot [n_slots]

struct SplitPlan {
    int n_slots;     // CTAs of the partition kernel
    int s_max;       // partial slots per (sequence, query head) in the workspace
    int hdr_ints;    // ints in front of the partials: header + prefix [B+1] + first sequence per slot [n_slots], padded to 64
    int lq_cap;      // quantized tokens per sequence the call looks at (from max_len_hint)
    int in_kernel;   // batch <= 32: every CTA derives the header itself from the lengths (one warp scan), no plan kernel
};
constexpr int kPlanSmemInts = 40;   // header (4) + prefix [33] of a batch of up to 32 in shared memory, padded

// Chooses the partition for lengths up to max_len (host).  requested_splits > 0 asks for about that many
// pieces per (sequence, KV head).
SplitPlan plan_splits(const Shape &s, int max_len, int requested_splits);

struct Segment {
    int b, hk;                 // sequence, KV head
    int tok_begin, tok_end;    // quantized tokens of that pair this segment covers
    int part;                  // index of its partial among the pair's partials
};

// Checked build (-DSKVQ_CHECKED, a debugging aid where no memory checker can be run): every row, slot and partial index
// is compared with the size of the buffer it addresses before it is used; a violation ORs SKVQ_STATUS_BOUNDS into the
// status word and the access is skipped.  In the normal build the macro is the constant true and costs nothing.
#ifdef SKVQ_CHECKED
#define SKVQ_IN_BOUNDS(cond, status) ((cond) ? true : (((status) != nullptr ? (void)atomicOr((status), SKVQ_STATUS_BOUNDS) : (void)0), false))
#else
#define SKVQ_IN_BOUNDS(cond, status) (true)
#endif

#ifdef __CUDACC__
// What a partition kernel is about to work on lies inside the cache and the workspace (checked build only).
__device__ inline bool segment_in_bounds(const Segment &sg, const Shape &s, const SplitPlan &p, int32_t *status)
{
    return SKVQ_IN_BOUNDS(sg.b >= 0 && sg.b < s.B && sg.hk >= 0 && sg.hk < s.Hkv && sg.tok_begin >= 0 && sg.tok_begin <= sg.tok_end &&
                          ((sg.tok_end + SKVQ_TOKEN_ALIGN - 1) & ~(SKVQ_TOKEN_ALIGN - 1)) <= s.cap && sg.part >= 0 && sg.part < p.s_max, status);
}

// Group of every 32-channel granule of KV head hk, packed two bits per granule: equal groups of G channels, or the
// boundaries in bounds[hk][0..ng] (multiples of 32; an entry that is not is treated as the next multiple below).
__device__ inline uint32_t granule_groups(const int32_t *bounds, int hk, int G, int ng)
{
    uint32_t map = 0;
#pragma unroll
    for (int gr = 0; gr < kGranules; ++gr) {
        int g = (gr * kGranule) / G;
        if (bounds) {
            g = 0;
            for (int i = 1; i < ng; ++i) g += (gr * kGranule >= bounds[(size_t)hk * (ng + 1) + i]) ? 1 : 0;
        }
        map |= (uint32_t)g << (2 * gr);
    }
    return map;
}

// One thread walks the segments of slot w.  hdr is the workspace header written by the plan kernel.
struct SlotWalker {
    const int *pre;     // units (per KV head) of the sequences before b, [B+1]
    int Hkv, B, ups;    // ups = units per slot
    int f, f1, b, w;

    // hdr: the header in the workspace (with the per-slot table behind the prefix) or a copy made by plan_in_warp
    // (no table: the first sequence is found by bisection).
    __device__ bool start(const int *hdr, bool has_table, int B_, int Hkv_, int w_)
    {
        pre = hdr + kPlanHdrInts; Hkv = Hkv_; B = B_; w = w_;
        const int total = hdr[0];
        ups = hdr[1];
        f = w * ups;
        f1 = min(f + ups, total);
        if (f >= f1) return false;
        if (has_table) {
            b = pre[B + 1 + w];             // found by the plan kernel
        } else {
            int lo = 0, hi = B - 1;         // the largest b with Hkv * pre[b] <= f
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if (Hkv * pre[mid] <= f) lo = mid; else hi = mid - 1;
            }
            b = lo;
        }
        return true;
    }
    __device__ bool done() const { return f >= f1; }
    // The next segment; lq_b = quantized tokens of sequence b that the call looks at.
    __device__ Segment next(const int32_t *lengths, int W, int lq_cap)
    {
        while (pre[b + 1] == pre[b]) ++b;   // sequences without quantized tokens own no unit
        const int nu = pre[b + 1] - pre[b];
        const int base = Hkv * pre[b];
        const int hk = (f - base) / nu, u0 = (f - base) - hk * nu;
        const int take = min(nu - u0, f1 - f);
        const int lq = min(max(lengths[b] - W, 0), lq_cap);
        Segment sg;
        sg.b = b; sg.hk = hk;
        sg.tok_begin = u0 * kUnitTok;
        sg.tok_end = min((u0 + take) * kUnitTok, lq);
        sg.part = w - (base + hk * nu) / ups;
        f += take;
        if (f == base + Hkv * nu) ++b;
        return sg;
    }
};

// The header for a batch of at most 32 sequences, computed by one full warp into hdr_s[kPlanSmemInts]: units per
// sequence (256 quantized tokens each) as an exclusive prefix, their total over all KV heads, units per slot.
__device__ inline void plan_in_warp(const int32_t *lengths, int B, int Hkv, int W, int lq_cap, int n_slots, int *hdr_s)
{
    const int lane = threadIdx.x & 31;
    int nu = 0;
    if (lane < B) nu = (min(max(lengths[lane] - W, 0), lq_cap) + kUnitTok - 1) / kUnitTok;
    int incl = nu;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += v;
    }
    hdr_s[kPlanHdrInts + lane] = incl - nu;
    const int run = __shfl_sync(0xffffffffu, incl, 31);
    if (lane == 0) {
        const int total = run * Hkv;
        hdr_s[kPlanHdrInts + 32] = run;     // also pre[B] when B == 32; for B < 32 pre[B] = incl - nu of lane B = run already
        hdr_s[0] = total;
        hdr_s[1] = max((total + n_slots - 1) / n_slots, 1);
    }
}

// Number of partials of pair (b, hk) and the slot that wrote the first one (merge kernel).
__device__ inline int pair_partials(const int *hdr, int Hkv, int b, int hk)
{
    const int *pre = hdr + kPlanHdrInts;
    const int nu = pre[b + 1] - pre[b];
    if (nu == 0) return 0;
    const int start = Hkv * pre[b] + hk * nu, ups = hdr[1];
    return (start + nu - 1) / ups - start / ups + 1;
}
#endif

// Kernel launchers (host).  Each returns a cudaError_t from the launch and bumps the launch counter.
cudaError_t launch_append(const Shape &s, const CachePtrs &c, const __half *k, const __half *v,
                          const int32_t *n_new_per_seq, int n_new, cudaStream_t stream);
cudaError_t launch_attention(const Shape &s, const CachePtrs &c, const __half *q, __half *out, float sm_scale,
                             const SplitPlan &plan, float *workspace, cudaEvent_t ev_begin, cudaEvent_t ev_end,
                             cudaStream_t stream);

cudaError_t launch_partition_mma(const Shape &s, const CachePtrs &c, const __half *q, float scale_log2,
                                 const SplitPlan &plan, float *workspace, cudaStream_t stream, bool overlap, bool *handled);

cudaError_t launch_partition_gqa(const Shape &s, const CachePtrs &c, const __half *q, float scale_log2,
                                 const SplitPlan &plan, float *workspace, cudaStream_t stream, bool overlap, bool *handled);

cudaError_t launch_partition_tc(const Shape &s, const CachePtrs &c, const __half *q, float scale_log2,
                                const SplitPlan &plan, float *workspace, cudaStream_t stream, bool overlap, bool *handled);

void count_launch(int n = 1);

// Per-device state of the host side: function attributes (the dynamic shared-memory opt-in) belong to a device, so a
// process that drives several GPUs has to set them once on each.
constexpr int kMaxDevices = 64;
int current_device();                      // cudaGetDevice, or 0 when that fails
int sm_count();                            // multiprocessors of the current device

// Sets the dynamic shared-memory limit of `kern` once per device.  `done` is a bit mask owned by the caller (one per kernel).
template <typename Kern>
inline cudaError_t configure_smem_once(Kern kern, int bytes, unsigned long long &done)
{
    const int dev = current_device();
    const unsigned long long bit = 1ull << (dev & (kMaxDevices - 1));
    if (done & bit) return cudaSuccess;
    const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) done |= bit;     // racing host threads set the same attribute twice: harmless
    return e;
}

}  // namespace skvq

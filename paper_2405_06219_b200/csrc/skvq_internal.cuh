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

// Everything the kernels need, by value.
struct Shape {
    int B, Hq, Hkv, rep;   // rep = Hq / Hkv
    int k_bits, v_bits, G, ng;
    int W, cap, max_tokens;
};

struct CachePtrs {
    uint8_t *k_codes, *v_codes;
    __half2 *k_meta, *v_meta;
    __half *k_win, *v_win;
    int32_t *lengths;
    const int32_t *reorder_k, *reorder_v;
    const float *alpha_k, *alpha_v;
    int32_t *status;
};

struct SplitPlan {
    int split_len;   // quantized tokens per split (multiple of SKVQ_TOKEN_ALIGN)
    int n_splits;    // splits of the quantized prefix per (sequence, KV head); the fp16 window belongs to the merge kernel
};

// Chooses the sequence partition for lengths up to max_len (host).
SplitPlan plan_splits(const Shape &s, int max_len, int requested_splits);

// Kernel launchers (host).  Each returns a cudaError_t from the launch and bumps the launch counter.
cudaError_t launch_append(const Shape &s, const CachePtrs &c, const __half *k, const __half *v,
                          const int32_t *n_new_per_seq, int n_new, cudaStream_t stream);
cudaError_t launch_attention(const Shape &s, const CachePtrs &c, const __half *q, __half *out, float sm_scale,
                             const SplitPlan &plan, float *workspace, cudaEvent_t ev_begin, cudaEvent_t ev_end,
                             cudaStream_t stream);

cudaError_t launch_partition_mma(const Shape &s, const CachePtrs &c, const __half *q, float scale_log2,
                                 const SplitPlan &plan, float *workspace, cudaStream_t stream, bool *handled);

cudaError_t launch_partition_gqa(const Shape &s, const CachePtrs &c, const __half *q, float scale_log2,
                                 const SplitPlan &plan, float *workspace, cudaStream_t stream, bool *handled);

void count_launch(int n = 1);

}  // namespace skvq

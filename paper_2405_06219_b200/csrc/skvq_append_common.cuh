// Pieces shared by the kernels of skvq_quantize_append: launch arguments, which tokens the tile kernel takes, the
// FP8 (E4M3) conversions of the stored scale and zero point.
#pragma once
#include "skvq_internal.cuh"

namespace skvq {

struct AppendArgs {
    Shape s;
    CachePtrs c;
    const __half *k, *v;
    const int32_t *n_new_per_seq;
    int n_new;
    int use_bulk;   // the tile kernel runs alongside and takes the bulk_range() tokens
};

__device__ __forceinline__ int seq_new_count(const AppendArgs &a, int b)
{
    int n = a.n_new_per_seq ? a.n_new_per_seq[b] : a.n_new;
    return min(max(n, 0), a.n_new);
}

// Tokens [f0, f1) of a sequence (multiples of 64, possibly empty) are quantized by the tile kernel: they are
// new, they end up below the window, and they form whole aligned tiles.
__device__ __forceinline__ void bulk_range(int L0, int n_sink, int q_end, int &f0, int &f1)
{
    f0 = (max(L0, n_sink) + 63) & ~63;      // attention sinks are not quantized: they stay with append_kernel
    f1 = q_end & ~63;
    if (f1 < f0) f1 = f0;
}

// fp32 scale and zero point -> the two E4M3 bytes {h, z} (round to nearest even, saturating at 448) ...
__device__ __forceinline__ uint16_t to_e4m3x2(float h, float z)
{
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(z), "f"(h));      // first operand -> upper byte
    return r;
}
// ... and back: {h, z} as a half2 (every E4M3 value is an fp16 value)
__device__ __forceinline__ __half2 from_e4m3x2(uint16_t b)
{
    uint32_t r;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(b));
    return *reinterpret_cast<const __half2 *>(&r);
}


// The tensor-core tile kernel (skvq_append_tc.cu): quantizes the bulk_range() tokens of every sequence and KV head.
cudaError_t launch_append_tiles(const AppendArgs &a, cudaStream_t stream);

}  // namespace skvq

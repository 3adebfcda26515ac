// C-ABI entry points of libskvq: argument validation, sizing helpers and the host-buffer decode step.
#include <atomic>

#include "skvq_internal.cuh"

// Profiler ranges around the entry points (header-only NVTX 3), compiled in with -DSKVQ_NVTX: a timeline then shows
// which kernels belong to which call.  Without the define the macro is empty.
#ifdef SKVQ_NVTX
#include <nvtx3/nvToolsExt.h>
namespace {
struct NvtxRange {
    explicit NvtxRange(const char *name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
};
}  // namespace
#define SKVQ_RANGE(name) NvtxRange skvq_nvtx_range_(name)
#else
#define SKVQ_RANGE(name) do {} while (0)
#endif

namespace skvq {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

static int check_cfg(const skvq_config *c)
{
    if (!c) return SKVQ_ERR_INVALID_ARG;
    if (c->batch < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->window < 0 || c->max_tokens < 1)
        return SKVQ_ERR_INVALID_ARG;
    if (c->batch > 65535 || c->n_kv_heads > 65535) return SKVQ_ERR_UNSUPPORTED;
    if (c->head_dim != kHeadDim) return SKVQ_ERR_UNSUPPORTED;
    if (c->k_bits < 2 || c->k_bits > 4 || ((c->v_bits < 2 || c->v_bits > 4) && c->v_bits != kTernary)) return SKVQ_ERR_UNSUPPORTED;
    if (c->group_size != 32 && c->group_size != 64 && c->group_size != 128) return SKVQ_ERR_UNSUPPORTED;
    if (c->n_q_heads % c->n_kv_heads != 0) return SKVQ_ERR_UNSUPPORTED;
    if (c->n_q_heads / c->n_kv_heads > kMaxRep) return SKVQ_ERR_UNSUPPORTED;
    if (c->n_sink < 0) return SKVQ_ERR_INVALID_ARG;
    if (c->n_sink > 64) return SKVQ_ERR_UNSUPPORTED;
    if (c->meta_fp8 != 0 && c->meta_fp8 != 1) return SKVQ_ERR_INVALID_ARG;
    return SKVQ_OK;
}

static int quant_capacity(const skvq_config *c)
{
    long rows = (long)c->max_tokens - c->window;
    if (rows < 0) rows = 0;
    rows = (rows + SKVQ_TOKEN_ALIGN - 1) / SKVQ_TOKEN_ALIGN * SKVQ_TOKEN_ALIGN;
    if (rows < SKVQ_TOKEN_ALIGN) rows = SKVQ_TOKEN_ALIGN;
    return (int)rows;
}

static Shape make_shape(const skvq_config *c)
{
    Shape s;
    s.B = c->batch;
    s.Hq = c->n_q_heads;
    s.Hkv = c->n_kv_heads;
    s.rep = s.Hq / s.Hkv;
    s.k_bits = c->k_bits;
    s.v_bits = c->v_bits;
    s.G = c->group_size;
    s.ng = kHeadDim / s.G;
    s.W = c->window;
    s.cap = quant_capacity(c);
    s.max_tokens = c->max_tokens;
    s.n_sink = c->n_sink;
    s.meta_fp8 = c->meta_fp8;
    s.bounded = 0;      // set by check_cache when the cache carries group boundaries
    return s;
}

static bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

static int check_cache(const skvq_config *cfg, const skvq_cache *c, CachePtrs *out)
{
    if (!c) return SKVQ_ERR_INVALID_ARG;
    if (!c->k_codes || !c->v_codes || !c->k_meta || !c->v_meta || !c->lengths || !c->reorder_k || !c->reorder_v ||
        !c->alpha_k || !c->alpha_v)
        return SKVQ_ERR_INVALID_ARG;
    if (cfg->window > 0 && (!c->k_win || !c->v_win)) return SKVQ_ERR_INVALID_ARG;
    if (cfg->n_sink > 0 && (!c->k_sink || !c->v_sink)) return SKVQ_ERR_INVALID_ARG;
    const void *ptrs[] = {c->k_codes, c->v_codes, c->k_meta, c->v_meta, c->k_win, c->v_win,
                          c->lengths, c->reorder_k, c->reorder_v, c->alpha_k, c->alpha_v, c->k_sink, c->v_sink};
    if ((reinterpret_cast<uintptr_t>(c->group_bounds_k) | reinterpret_cast<uintptr_t>(c->group_bounds_v)) & 3u) return SKVQ_ERR_MISALIGNED;
    for (const void *p : ptrs)
        if (p && misaligned(p)) return SKVQ_ERR_MISALIGNED;
    out->k_codes = static_cast<uint8_t *>(c->k_codes);
    out->v_codes = static_cast<uint8_t *>(c->v_codes);
    out->k_meta = static_cast<__half2 *>(c->k_meta);
    out->v_meta = static_cast<__half2 *>(c->v_meta);
    out->k_win = static_cast<__half *>(c->k_win);
    out->v_win = static_cast<__half *>(c->v_win);
    out->lengths = c->lengths;
    out->reorder_k = c->reorder_k;
    out->reorder_v = c->reorder_v;
    out->alpha_k = c->alpha_k;
    out->alpha_v = c->alpha_v;
    out->status = c->status;
    out->k_sink = static_cast<__half *>(c->k_sink);
    out->v_sink = static_cast<__half *>(c->v_sink);
    out->bounds_k = c->group_bounds_k;
    out->bounds_v = c->group_bounds_v;
    return SKVQ_OK;
}

static size_t workspace_bytes(const Shape &s, const SplitPlan &p)
{
    return ((size_t)p.hdr_ints + (size_t)s.B * s.Hq * p.s_max * kPartialStride) * sizeof(float);
}

}  // namespace skvq

using namespace skvq;

extern "C" {

int skvq_version(void) { return 100; }

const char *skvq_strerror(int code)
{
    switch (code) {
        case SKVQ_OK: return "ok";
        case SKVQ_ERR_INVALID_ARG: return "invalid argument";
        case SKVQ_ERR_UNSUPPORTED: return "unsupported configuration";
        case SKVQ_ERR_MISALIGNED: return "device buffer is not 16-byte aligned";
        case SKVQ_ERR_CAPACITY: return "token count exceeds the cache capacity";
        case SKVQ_ERR_WORKSPACE: return "workspace missing or too small";
        case SKVQ_ERR_CUDA: return "CUDA runtime error at launch";
        case SKVQ_ERR_SCRATCH_LIMIT: return "split partials exceed the library's built-in scratch array";
        default: return "unknown error code";
    }
}

uint64_t skvq_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int skvq_check_config(const skvq_config *cfg) { return check_cfg(cfg); }

int skvq_check_group_bounds(const skvq_config *cfg, const int32_t *bounds_host)
{
    const int rc = check_cfg(cfg);
    if (rc != SKVQ_OK) return rc;
    if (!bounds_host) return SKVQ_ERR_INVALID_ARG;
    const int ng = kHeadDim / cfg->group_size;
    for (int h = 0; h < cfg->n_kv_heads; ++h) {
        const int32_t *b = bounds_host + (size_t)h * (ng + 1);
        if (b[0] != 0 || b[ng] != kHeadDim) return SKVQ_ERR_INVALID_ARG;
        for (int g = 0; g < ng; ++g)
            if (b[g + 1] <= b[g] || b[g + 1] % SKVQ_GROUP_GRANULE != 0) return SKVQ_ERR_INVALID_ARG;
    }
    return SKVQ_OK;
}

int32_t skvq_quant_capacity(const skvq_config *cfg)
{
    const int rc = check_cfg(cfg);
    return rc != SKVQ_OK ? rc : quant_capacity(cfg);
}

int skvq_cache_sizes(const skvq_config *cfg, size_t bytes_out[6])
{
    const int rc = check_cfg(cfg);
    if (rc != SKVQ_OK) return rc;
    if (!bytes_out) return SKVQ_ERR_INVALID_ARG;
    const Shape s = make_shape(cfg);
    const size_t rows = (size_t)s.B * s.Hkv * s.cap;
    bytes_out[0] = rows * packed_row_bytes(s.k_bits);
    bytes_out[1] = rows * packed_row_bytes(s.v_bits);
    bytes_out[2] = rows * s.ng * (s.meta_fp8 ? 2 : sizeof(__half2));
    bytes_out[3] = bytes_out[2];
    bytes_out[4] = (size_t)s.B * s.Hkv * s.W * kHeadDim * sizeof(__half);
    bytes_out[5] = bytes_out[4];
    return SKVQ_OK;
}

size_t skvq_sink_bytes(const skvq_config *cfg)
{
    if (check_cfg(cfg) != SKVQ_OK) return 0;
    return (size_t)cfg->batch * cfg->n_kv_heads * cfg->n_sink * kHeadDim * sizeof(__half);
}

int skvq_quantize_append(const skvq_config *cfg, const skvq_cache *cache, const void *k, const void *v,
                         const int32_t *n_new_per_seq, int32_t n_new, void *cuda_stream)
{
    SKVQ_RANGE("skvq_quantize_append");
    int rc = check_cfg(cfg);
    if (rc != SKVQ_OK) return rc;
    CachePtrs c;
    rc = check_cache(cfg, cache, &c);
    if (rc != SKVQ_OK) return rc;
    if (n_new < 0) return SKVQ_ERR_INVALID_ARG;
    if (n_new == 0) return SKVQ_OK;
    if (!k || !v) return SKVQ_ERR_INVALID_ARG;
    if (misaligned(k) || misaligned(v) || (n_new_per_seq && (reinterpret_cast<uintptr_t>(n_new_per_seq) & 3u)))
        return SKVQ_ERR_MISALIGNED;
    if (n_new > cfg->max_tokens) return SKVQ_ERR_CAPACITY;
    Shape s = make_shape(cfg);
    s.bounded = (c.bounds_k || c.bounds_v) ? 1 : 0;
    const cudaError_t e = launch_append(s, c, static_cast<const __half *>(k), static_cast<const __half *>(v),
                                        n_new_per_seq, n_new, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? SKVQ_OK : SKVQ_ERR_CUDA;
}

size_t skvq_workspace_size(const skvq_config *cfg, int32_t max_len_hint, int32_t n_splits)
{
    if (check_cfg(cfg) != SKVQ_OK || max_len_hint < 0 || n_splits < 0) return 0;
    const Shape s = make_shape(cfg);
    if (max_len_hint > s.max_tokens) max_len_hint = s.max_tokens;
    return workspace_bytes(s, plan_splits(s, max_len_hint, n_splits));
}

int skvq_decode_attention(const skvq_config *cfg, const skvq_cache *cache, const void *q, void *out,
                          const skvq_attn_args *args, void *cuda_stream)
{
    SKVQ_RANGE("skvq_decode_attention");
    int rc = check_cfg(cfg);
    if (rc != SKVQ_OK) return rc;
    CachePtrs c;
    rc = check_cache(cfg, cache, &c);
    if (rc != SKVQ_OK) return rc;
    if (!q || !out || !args) return SKVQ_ERR_INVALID_ARG;
    if (misaligned(q) || misaligned(out)) return SKVQ_ERR_MISALIGNED;
    if (args->max_len_hint < 0 || args->n_splits < 0) return SKVQ_ERR_INVALID_ARG;
    if (args->max_len_hint > cfg->max_tokens) return SKVQ_ERR_CAPACITY;
    Shape s = make_shape(cfg);
    s.bounded = (c.bounds_k || c.bounds_v) ? 1 : 0;
    const SplitPlan plan = plan_splits(s, args->max_len_hint, args->n_splits);
    if (!args->workspace || args->workspace_bytes < workspace_bytes(s, plan)) return SKVQ_ERR_WORKSPACE;
    if (misaligned(args->workspace)) return SKVQ_ERR_MISALIGNED;
    const cudaError_t e = launch_attention(s, c, static_cast<const __half *>(q), static_cast<__half *>(out),
                                           args->sm_scale, plan, static_cast<float *>(args->workspace),
                                           static_cast<cudaEvent_t>(args->ev_begin),
                                           static_cast<cudaEvent_t>(args->ev_end),
                                           static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? SKVQ_OK : SKVQ_ERR_CUDA;
}

size_t skvq_step_staging_size(const skvq_config *cfg)
{
    if (check_cfg(cfg) != SKVQ_OK) return 0;
    const size_t kv = (size_t)cfg->batch * cfg->n_kv_heads * kHeadDim * sizeof(__half);
    const size_t qo = (size_t)cfg->batch * cfg->n_q_heads * kHeadDim * sizeof(__half);
    return 2 * kv + 2 * qo;
}

int skvq_decode_step_host(const skvq_config *cfg, const skvq_cache *cache, const void *k_new_host,
                          const void *v_new_host, const void *q_host, void *out_host, void *staging,
                          const skvq_attn_args *args, void *cuda_stream)
{
    SKVQ_RANGE("skvq_decode_step_host");
    int rc = check_cfg(cfg);
    if (rc != SKVQ_OK) return rc;
    if (!k_new_host || !v_new_host || !q_host || !out_host || !staging || !args) return SKVQ_ERR_INVALID_ARG;
    if (misaligned(staging)) return SKVQ_ERR_MISALIGNED;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t kv = (size_t)cfg->batch * cfg->n_kv_heads * kHeadDim * sizeof(__half);
    const size_t qo = (size_t)cfg->batch * cfg->n_q_heads * kHeadDim * sizeof(__half);
    char *base = static_cast<char *>(staging);
    void *d_k = base, *d_v = base + kv, *d_q = base + 2 * kv, *d_out = base + 2 * kv + qo;
    const char *hk = static_cast<const char *>(k_new_host);
    if (static_cast<const char *>(v_new_host) == hk + kv && static_cast<const char *>(q_host) == hk + 2 * kv) {
        // the three inputs lie back to back in host memory, in the order they have in `staging`: one copy
        if (cudaMemcpyAsync(d_k, k_new_host, 2 * kv + qo, cudaMemcpyHostToDevice, stream) != cudaSuccess) return SKVQ_ERR_CUDA;
    } else {
        if (cudaMemcpyAsync(d_k, k_new_host, kv, cudaMemcpyHostToDevice, stream) != cudaSuccess) return SKVQ_ERR_CUDA;
        if (cudaMemcpyAsync(d_v, v_new_host, kv, cudaMemcpyHostToDevice, stream) != cudaSuccess) return SKVQ_ERR_CUDA;
        if (cudaMemcpyAsync(d_q, q_host, qo, cudaMemcpyHostToDevice, stream) != cudaSuccess) return SKVQ_ERR_CUDA;
    }
    rc = skvq_quantize_append(cfg, cache, d_k, d_v, nullptr, 1, cuda_stream);
    if (rc != SKVQ_OK) return rc;
    rc = skvq_decode_attention(cfg, cache, d_q, d_out, args, cuda_stream);
    if (rc != SKVQ_OK) return rc;
    if (cudaMemcpyAsync(out_host, d_out, qo, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return SKVQ_ERR_CUDA;
    return SKVQ_OK;
}

// ---------------------------------------------------------------- decode attention without a caller workspace
// Split partials of skvq_decode_attention_noalloc live in this array instead of caller memory.  Every GPU that
// loads the library carries it until the process exits.  In host code the name below is only a handle for
// cudaGetSymbolAddress; the kernels are given the device address that call returns.
static __device__ __align__(256) unsigned char g_noalloc_scratch[SKVQ_NOALLOC_SCRATCH_BYTES];

namespace {
std::atomic<float *> g_noalloc_ptr[kMaxDevices];

// Device address of the array on the current device, looked up once per device.  With CUDA's lazy module loading
// this lookup is also what places the library's image -- and with it the array -- on that device, so it can fail
// on a device whose memory is already full; callers make their first call at start-up.  The address is kept for
// the life of the process: a cudaDeviceReset() invalidates it (documented in skvq.h).
int noalloc_scratch(float **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SKVQ_ERR_CUDA;
    float *p = g_noalloc_ptr[dev].load(std::memory_order_acquire);
    if (!p) {
        void *sym = nullptr;
        if (cudaGetSymbolAddress(&sym, g_noalloc_scratch) != cudaSuccess || !sym) return SKVQ_ERR_CUDA;
        p = static_cast<float *>(sym);
        g_noalloc_ptr[dev].store(p, std::memory_order_release);   // racing threads store the same address
    }
    *out = p;
    return SKVQ_OK;
}
}  // namespace

int skvq_decode_attention_noalloc(const skvq_config *cfg, const skvq_cache *cache, const void *q, void *out,
                                  float sm_scale, int32_t max_len_hint, int32_t n_splits, void *cuda_stream)
{
    SKVQ_RANGE("skvq_decode_attention_noalloc");
    int rc = check_cfg(cfg);
    if (rc != SKVQ_OK) return rc;
    CachePtrs c;
    rc = check_cache(cfg, cache, &c);
    if (rc != SKVQ_OK) return rc;
    if (!q || !out) return SKVQ_ERR_INVALID_ARG;
    if (misaligned(q) || misaligned(out)) return SKVQ_ERR_MISALIGNED;
    if (max_len_hint < 0 || n_splits < 0) return SKVQ_ERR_INVALID_ARG;
    if (max_len_hint > cfg->max_tokens) return SKVQ_ERR_CAPACITY;
    Shape s = make_shape(cfg);
    s.bounded = (c.bounds_k || c.bounds_v) ? 1 : 0;
    const SplitPlan plan = plan_splits(s, max_len_hint, n_splits);
    if (workspace_bytes(s, plan) > (size_t)SKVQ_NOALLOC_SCRATCH_BYTES) return SKVQ_ERR_SCRATCH_LIMIT;
    float *scratch = nullptr;
    rc = noalloc_scratch(&scratch);
    if (rc != SKVQ_OK) return rc;
    // Nothing in the array has to start at zero: every partial the merge reads is written by this call first.
    const cudaError_t e = launch_attention(s, c, static_cast<const __half *>(q), static_cast<__half *>(out), sm_scale,
                                           plan, scratch, nullptr, nullptr, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? SKVQ_OK : SKVQ_ERR_CUDA;
}

}  // extern "C"
